"""Folding 1/s into the producers and the decoder walk, against the CPU oracle.

``aweq_fold_scale`` is bit-exact (binary32 product, one rounding to 16 bits).  The walk is a
fixed order of library calls; the oracle takes the same steps in the same order, so every
code, Step, zero-point and folded parameter must be identical.
"""
import numpy as np
import pytest
import torch

from oracle import aweq_oracle as orc
from paper_2311_01305_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("shape", [(768, 768), (1000, 24), (333, 1), (64, 13), (5, 4104)])
def test_fold_scale_matrix(dtype, shape):
    from paper_2311_01305_b200 import aweq
    P = util.rand16(shape, dtype, 51 + shape[0], scale=2.0)
    g = torch.Generator().manual_seed(52)
    rinv = torch.exp(torch.randn(shape[0], generator=g)).float()
    ref = orc.fold_scale(util.bits(P), util.odt(P), rinv.numpy())
    out, check = util.guarded(shape, dtype)
    aweq.aweq_fold_scale(P.to(DEV), rinv.to(DEV), out)
    torch.cuda.synchronize()
    check()
    assert np.array_equal(util.bits(out), ref)
    # in place, and a vector
    Pg = P.to(DEV)
    aweq.aweq_fold_scale(Pg, rinv.to(DEV))
    v = P[:, 0].contiguous().to(DEV)
    aweq.aweq_fold_scale(v, rinv.to(DEV))
    torch.cuda.synchronize()
    assert np.array_equal(util.bits(Pg), ref)
    assert np.array_equal(util.bits(v), ref[:, 0])


def test_fold_scale_pitched_rows():
    from paper_2311_01305_b200 import aweq
    big = util.rand16((40, 64), torch.float16, 53).to(DEV)
    view = big[:, :48]                                   # pitch 64, 48 columns
    rinv = torch.linspace(0.5, 2.0, 40)
    ref = orc.fold_scale(util.bits(view.contiguous()), orc.F16, rinv.numpy())
    keep = big[:, 48:].clone()
    aweq.aweq_fold_scale(view, rinv.to(DEV))
    torch.cuda.synchronize()
    assert np.array_equal(util.bits(big[:, :48].contiguous()), ref)
    assert torch.equal(big[:, 48:], keep)                # columns beyond the view untouched


def _small_decoder(kind, dtype, act_quant, bits, gran, group):
    n, h, f = 300, 64, 160
    if kind == "llama":
        inputs, linears = synth._llama_layer(n, h, f, "normal", 0, lambda c: 2, 30.0, 0.05)
    else:
        spec = lambda name, c: synth.ActSpec(name, n, c, "normal", 0, 2, 30.0)
        inputs = (spec("attn_in", h), spec("o_in", h), spec("fc1_in", h), spec("fc2_in", f))
        L = synth.LinearSpec
        linears = (L("q", h, h, "attn_in", 0.05), L("k", h, h, "attn_in", 0.05), L("v", h, h, "attn_in", 0.05),
                   L("o", h, h, "o_in", 0.05), L("fc1", f, h, "fc1_in", 0.05), L("fc2", h, f, "fc2_in", 0.05))
    return synth.Workload("small_" + kind, dtype, 77, inputs, linears, (bits,), gran, group, act_quant)


@pytest.mark.parametrize("kind,dtype,act_quant,bits,gran,group", [
    ("llama", "bf16", False, 4, "group", 32), ("llama", "f16", True, 8, "row", 0), ("opt", "f16", True, 8, "row", 0)])
def test_decoder_walk_matches_oracle_in_the_same_order(kind, dtype, act_quant, bits, gran, group):
    from paper_2311_01305_b200 import calibrate
    wl = _small_decoder(kind, dtype, act_quant, bits, gran, group)
    td = synth.torch_dtype(dtype)
    Xc = {i.name: synth.make_activations(i, dtype, synth.tensor_seed(wl.seed, 0, k), "cpu",
                                         channel_offset=torch.linspace(-1, 1, i.c_in))
          for k, i in enumerate(wl.inputs)}
    Wc = {l.name: synth.make_weight(l, dtype, synth.tensor_seed(wl.seed, 0, 100 + k), "cpu")
          for k, l in enumerate(wl.linears)}
    Bc = {l.name: util.rand16((1, l.c_out), td, 200 + k, scale=0.1)[0].contiguous() for k, l in enumerate(wl.linears)}
    prod = synth.producers(wl)
    norm_names = sorted({p for kd, p in prod.values() if kd == "norm"})
    Nc = {nm: synth.make_norm(wl.inputs[0].c_in, dtype, 300 + k, "cpu", shift=(kind == "opt"))
          for k, nm in enumerate(norm_names)}
    walk = calibrate.DecoderWalk(wl, bits, {k: v.to(DEV) for k, v in Xc.items()}, {k: v.to(DEV) for k, v in Wc.items()},
                                 {k: v.to(DEV) for k, v in Bc.items()},
                                 {k: tuple(None if t is None else t.to(DEV) for t in v) for k, v in Nc.items()})
    walk.run()
    torch.cuda.synchronize()
    art = walk.artifacts()

    # the oracle, same order: factors of linear-produced inputs, fold, then every input
    dt = orc.F16 if dtype == "f16" else orc.BF16
    ogran = orc.PER_ROW if gran == "row" else orc.PER_GROUP
    Wb = {k: util.bits(v) for k, v in Wc.items()}
    Bb = {k: util.bits(v) for k, v in Bc.items()}
    for inp in wl.inputs:
        kd, p = prod[inp.name]
        if kd != "linear":
            continue
        xs = orc.stats(util.bits(Xc[inp.name]), dt)
        wr = None
        for l in wl.linears:
            if l.input == inp.name:
                wr = orc.wrange(Wb[l.name], dt, prev=wr)
        f = orc.factors(xs[0], xs[1], xs[2], wr[0], wr[1])
        Wb[p] = orc.fold_scale(Wb[p], dt, f["rinv"])
        Bb[p] = orc.fold_scale(Bb[p], dt, f["rinv"])
    assert sorted(x[2] for x in art["folded"] if x[1] == "linear") == sorted(p for kd, p in prod.values() if kd == "linear")
    for inp in wl.inputs:
        lins = [l for l in wl.linears if l.input == inp.name]
        xb = util.bits(Xc[inp.name])
        xs = orc.stats(xb, dt)
        wr = None
        for l in lins:
            wr = orc.wrange(Wb[l.name], dt, prev=wr)
        f = orc.factors(xs[0], xs[1], xs[2], wr[0], wr[1])
        o = art["inputs"][inp.name]
        util.assert_same_values(o["s"].cpu().numpy(), f["s"], "s " + inp.name)
        for l in lins:
            codes, step, zp, delta = orc.equalize_quantize(Wb[l.name], dt, f["s"], f["mu_hat"], bits, ogran, group)
            lo = art["linears"][l.name]
            util.assert_same_values(lo["codes"].cpu().numpy(), codes, "codes " + l.name)
            util.assert_same_values(lo["step"].cpu().numpy(), step, "Step " + l.name)
            util.assert_same_values(lo["zp"].cpu().numpy(), zp, "Z " + l.name)
            bf, _ = orc.bias_correct(delta, Bb[l.name], dt)
            assert np.allclose(lo["bias_f32"].cpu().numpy(), bf, rtol=0, atol=1e-5)
        if act_quant:
            xq, st, z = orc.quant_act(xb, dt, f["rinv"], orc.PER_ROW)
            util.assert_same_values(o["Xq"].cpu().numpy(), xq, "Xq " + inp.name)
        kd, p = prod[inp.name]
        if kd == "norm":
            for t_gpu, t_cpu in zip(art["norms"][p], Nc[p]):
                if t_cpu is not None:
                    assert np.array_equal(util.bits(t_gpu), orc.fold_scale(util.bits(t_cpu), dt, f["rinv"]))
    # the folded producers differ from the originals, the other matrices do not
    for l in wl.linears:
        changed = not torch.equal(walk.W[l.name].cpu(), Wc[l.name])
        assert changed == (l.name in {p for kd, p in prod.values() if kd == "linear"})
        assert np.array_equal(util.bits(walk.W[l.name]), Wb[l.name])


@pytest.mark.parametrize("shape", [(300, 768), (7, 13), (1, 1)])
def test_relabel_signed_matches_the_oracle(shape):
    """q' = q - 128, Z' = Z - 128 against the oracle's routine, zero-points at the int32 edge
    included (Z' saturates); the de-quantised values Step (q' - Z') are those of the unsigned codes."""
    from paper_2311_01305_b200 import aweq
    rng = np.random.default_rng(shape[0])
    q = rng.integers(0, 256, shape).astype(np.uint8)
    zp = rng.integers(-300, 600, shape[0]).astype(np.int32)
    zp[0] = -2147483648 + 5                      # saturates
    if shape[0] > 2:
        zp[1], zp[2] = -2147483648 + 128, 2147483647
    o_q, o_z = orc.relabel_signed(q, zp)
    out, check = util.guarded(shape, torch.uint8)
    zp_out, check_z = util.guarded((shape[0],), torch.int32)
    aweq.aweq_relabel_signed(torch.from_numpy(q).to(DEV), out, torch.from_numpy(zp).to(DEV), zp_out)
    torch.cuda.synchronize()
    check()
    check_z()
    qs = out.cpu().numpy().view(np.int8)
    assert np.array_equal(qs, o_q)
    assert np.array_equal(zp_out.cpu().numpy(), o_z)
    assert zp_out.cpu().numpy()[0] == -2147483648
    keep = zp.astype(np.int64) - 128 >= -2147483648
    assert np.array_equal((qs.astype(np.int64) - zp_out.cpu().numpy().astype(np.int64)[:, None])[keep],
                          (q.astype(np.int64) - zp.astype(np.int64)[:, None])[keep])
    # in place, codes only
    t = torch.from_numpy(q).to(DEV)
    aweq.aweq_relabel_signed(t)
    torch.cuda.synchronize()
    assert np.array_equal(t.cpu().numpy().view(np.int8), orc.relabel_signed(q)[0])
