"""Helpers shared by the GPU parity tests: the same seeded bits go to the CUDA
library (as device tensors) and to the CPU oracle (as raw uint16 arrays)."""
import numpy as np
import torch

from oracle import aweq_oracle as orc
from paper_2311_01305_b200 import synth


def odt(t: torch.Tensor) -> int:
    return orc.F16 if t.dtype == torch.float16 else orc.BF16


def bits(t: torch.Tensor) -> np.ndarray:
    return synth.raw_bits(t)


def rand16(shape, dtype, seed, scale=1.0, offset=0.0, outlier_cols=0, outlier_scale=40.0):
    """Seeded CPU tensor with a few outlier columns and an optional per-column offset."""
    g = torch.Generator().manual_seed(seed)
    v = torch.randn(shape, generator=g) * scale
    if outlier_cols:
        idx = torch.randperm(shape[1], generator=g)[:outlier_cols]
        v[:, idx] *= outlier_scale
    if isinstance(offset, float) and offset != 0.0:
        v = v + (torch.rand(shape[1], generator=g) - 0.5) * 2 * offset
    if dtype == torch.float16:
        v = v.clamp(-65504, 65504)
    return v.to(dtype)


def guarded(shape, dtype, device="cuda", pad=1024, fill=0x5A):
    """An output tensor with sentinel-filled bands before and after it."""
    n = int(np.prod(shape))
    esz = torch.empty(0, dtype=dtype).element_size()
    pad_elems = (pad + esz - 1) // esz
    pad_elems = (pad_elems * esz + 255) // 256 * 256 // esz
    buf = torch.empty(n + 2 * pad_elems, dtype=dtype, device=device)
    buf.view(torch.uint8).fill_(fill)
    view = buf[pad_elems:pad_elems + n].view(shape)

    def check():
        raw = buf.view(torch.uint8)
        lo = raw[:pad_elems * esz]
        hi = raw[(pad_elems + n) * esz:]
        assert bool((lo == fill).all()) and bool((hi == fill).all()), "write outside the output buffer"
    return view, check


def mean_tolerance(ref_mean, mean_abs):
    """|delta| <= 1e-6 * max(|ref|, 1e-3 * mean|x|): 1e-6 relative, with a floor
    for channels whose mean cancels to (nearly) zero."""
    return 1e-6 * np.maximum(np.abs(ref_mean.astype(np.float64)), 1e-3 * mean_abs)


def assert_same_values(a, b, what=""):
    """Equality of values (+0 == -0), for results that must be exact."""
    a = np.asarray(a)
    b = np.asarray(b)
    assert a.shape == b.shape, (what, a.shape, b.shape)
    bad = ~((a == b) | (np.isnan(a.astype(np.float64)) & np.isnan(b.astype(np.float64))))
    assert not bad.any(), "%s: %d mismatches, first at %s: %s vs %s" % (
        what, int(bad.sum()), np.argwhere(bad)[0], a[bad][0], b[bad][0])


def oracle_layer(Xc, Wcs, bits, gran, group, biases=None, act_quant=True, equalize=True, bias_correct=True,
                 criterion=0):
    """The six steps through the CPU oracle for one input and the matrices it feeds."""
    dt = odt(Xc)
    xs = orc.stats(bits_of(Xc), dt)
    wr = None
    for Wc in Wcs:
        wr = orc.wrange(bits_of(Wc), dt, prev=wr)
    f = orc.factors(xs[0], xs[1], xs[2], wr[0], wr[1], criterion)
    s = f["s"] if equalize else None
    rinv = f["rinv"] if equalize else None
    mu = f["mu_hat"] if equalize else xs[2]
    res = {"stats": xs, "wrange": wr, "factors": f, "linears": []}
    for i, Wc in enumerate(Wcs):
        codes, step, zp, delta = orc.equalize_quantize(bits_of(Wc), dt, s, mu if bias_correct else None, bits, gran, group)
        lin = {"codes": codes, "step": step, "zp": zp, "delta": delta}
        if bias_correct:
            b = None if biases is None or biases[i] is None else bits_of(biases[i])
            lin["bias_f32"], lin["bias_16"] = orc.bias_correct(delta, b, dt)
        res["linears"].append(lin)
    if act_quant:
        res["act"] = orc.quant_act(bits_of(Xc), dt, rinv, orc.PER_ROW)
    return res


def bits_of(t):
    return bits(t)


def check_bias16(bias16: torch.Tensor, bias32: torch.Tensor, ref16_bits) -> None:
    """The 16-bit corrected bias is the library's own binary32 bias rounded once to the 16-bit
    type (exactly), and agrees with the oracle's 16-bit bias to 1e-3 absolute for fp16; a bf16
    value (8 significant bits: one ulp is 2e-3 already at 0.25) may sit one ulp from the
    oracle's when the two binary32 values straddle a rounding boundary."""
    tag = odt(bias16)
    b32 = bias32.detach().cpu().numpy()
    assert_same_values(bits(bias16), orc.encode16(b32, tag), "16-bit bias = round16(binary32 bias)")
    got = orc.decode16(bits(bias16), tag).astype(np.float64)
    want = orc.decode16(np.asarray(ref16_bits), tag).astype(np.float64)
    tol = np.full(want.shape, 1e-3)
    if tag == orc.BF16:
        a = np.maximum(np.abs(want), 2.0 ** -126)
        tol = np.maximum(tol, 2.0 ** (np.floor(np.log2(a)) - 7))
    assert np.all(np.abs(got - want) <= tol)
