"""Pins of the CPU oracle against things other than itself.

Every test here checks ``oracle/`` against what the paper (arXiv 2311.01305)
or the mathematics fixes: hand-worked quantiser cases (Eq. 1-2), closed forms,
the invariants the paper states (Eq. 3 output preservation, equal channel
ranges after equalisation, zero mean output error after bias correction), the
closed-form minimum of Eq. 8, NumPy/PyTorch library routines on the special
cases that reduce to them, and brute force on tiny tensors.  No GPU needed.
"""
import os

import numpy as np
import pytest
import torch

from oracle import aweq_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "quantizer_handworked.txt")


def f16_bits(a):
    return np.asarray(a, dtype=np.float16).view(np.uint16)


def bf16_bits(a):
    return torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def bits_to_f64(bits, dtype):
    """Library decode (NumPy / PyTorch), independent of the oracle's decoder."""
    if dtype == orc.F16:
        return bits.view(np.float16).astype(np.float64)
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()


# ---------------------------------------------------------------- 16-bit formats
def test_decode_f16_exhaustive_against_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    got = orc.decode16(bits, orc.F16)
    ref = bits.view(np.float16).astype(np.float32)
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.array_equal(got[ok].view(np.uint32), ref[ok].view(np.uint32))


def test_decode_bf16_exhaustive_against_torch():
    bits = np.arange(65536, dtype=np.uint16)
    got = orc.decode16(bits, orc.BF16)
    ref = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32).numpy()
    ok = ~np.isnan(ref)
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    assert np.array_equal(got[ok].view(np.uint32), ref[ok].view(np.uint32))


def test_encode_f16_against_numpy_rounding():
    rng = np.random.default_rng(1)
    x = np.concatenate([
        rng.standard_normal(20000) * 10.0 ** rng.uniform(-9, 5, 20000),
        np.array([0.0, -0.0, 65504.0, 65519.99, 65520.0, 1e9, -1e9, 2.0 ** -24, 2.0 ** -25, 3 * 2.0 ** -26,
                  2.0 ** -14, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, np.inf, -np.inf]),
    ])
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    got = orc.encode16(x, orc.F16)
    assert np.array_equal(got, ref)
    # every finite binary16 value survives a round trip
    allbits = np.arange(65536, dtype=np.uint16)
    vals = allbits.view(np.float16).astype(np.float64)
    fin = np.isfinite(vals)
    assert np.array_equal(orc.encode16(vals[fin], orc.F16), allbits[fin])


def test_encode_bf16_against_torch_rounding():
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(20000) * 10.0 ** rng.uniform(-30, 30, 20000)).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = orc.encode16(x.astype(np.float64), orc.BF16)
    assert np.array_equal(got, ref)


# ---------------------------------------------------------------- quantiser, Eq. 1-2
def _golden_cases():
    cases = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        b, v, st, z, q = [p.strip() for p in line.split("|")]
        cases.append((int(b), [float(t) for t in v.split()], float(st), int(z), [int(t) for t in q.split()]))
    return cases


@pytest.mark.parametrize("bits,vec,step,zp,codes", _golden_cases())
def test_quantizer_handworked(bits, vec, step, zp, codes):
    st, z, q = orc.quantize_vector(np.array(vec, np.float32), bits)
    assert st == np.float32(step)
    assert z == zp
    assert q.tolist() == codes


def test_quantizer_endpoints_error_bound_monotone():
    rng = np.random.default_rng(3)
    for bits in (2, 3, 4, 8):
        qmax = 2 ** bits - 1
        for trial in range(200):
            n = int(rng.integers(2, 300))
            v = (rng.standard_normal(n) * 10.0 ** rng.uniform(-3, 3) + rng.uniform(-5, 5)).astype(np.float32)
            st, z, q = orc.quantize_vector(v, bits)
            assert q[np.argmin(v)] == 0 and q[np.argmax(v)] == qmax
            assert q.min() >= 0 and q.max() <= qmax
            # Eq. 2: Step is the range over the number of steps
            assert st == pytest.approx((float(v.max()) - float(v.min())) / qmax, rel=3e-7)
            # reconstruction error of round-to-nearest is at most half a step
            deq = st * (q.astype(np.float64) - z)
            unclamped = q < qmax
            err = np.abs(deq - v.astype(np.float64))
            assert np.all(err[unclamped] <= st * 0.5 * (1 + 1e-5) + np.abs(v[unclamped]) * 2.0 ** -21)
            # the top clamp can cost at most one extra half step
            assert np.all(err <= st * (1 + 1e-5))
            order = np.argsort(v, kind="stable")
            assert np.all(np.diff(q[order]) >= 0)


def test_quantizer_bruteforce_nearest_grid_point():
    """On tiny vectors the code is the grid point Step*(k - Z) nearest to v."""
    rng = np.random.default_rng(4)
    for bits in (2, 3, 4):
        for _ in range(300):
            v = rng.standard_normal(8).astype(np.float32)
            st, z, q = orc.quantize_vector(v, bits)
            ks = np.arange(2 ** bits)
            grid = st * (ks.astype(np.float64) - z)
            dist = np.abs(grid[None, :] - v.astype(np.float64)[:, None])
            best = dist.min(axis=1)
            mine = dist[np.arange(8), q]
            # equal to the optimum up to the width of a rounding tie
            assert np.all(mine <= best + st * 1e-5)


def test_quantizer_literal_division_rarely_differs():
    """Reading of Eq. 1: v/Step evaluated as v*(1/Step).  Dividing instead changes
    a code only at a rounding tie, and then by one."""
    rng = np.random.default_rng(5)
    diff = total = 0
    for _ in range(200):
        v = rng.standard_normal(512).astype(np.float32)
        _, z1, q1 = orc.quantize_vector(v, 8, literal_division=False)
        _, z2, q2 = orc.quantize_vector(v, 8, literal_division=True)
        d = np.abs((q1 - z1) - (q2 - z2))
        assert d.max() <= 1
        diff += int((d != 0).sum())
        total += v.size
    assert diff / total < 1e-3


def test_quantizer_against_float64_textbook_rtn():
    """AWE off and BC off is the plain min-max round-to-nearest baseline of the
    paper's Section 4.2; evaluated in float64 it agrees except at near-ties."""
    rng = np.random.default_rng(6)
    bad = total = 0
    for bits in (3, 4, 8):
        qmax = 2 ** bits - 1
        for _ in range(100):
            v = (rng.standard_normal(256) * 3).astype(np.float32)
            st, z, q = orc.quantize_vector(v, bits)
            v64 = v.astype(np.float64)
            st64 = (v64.max() - v64.min()) / qmax
            q64 = np.clip(np.rint(v64 / st64) - np.rint(v64.min() / st64), 0, qmax)
            d = np.abs(q64 - q)
            assert d.max() <= 1
            bad += int((d != 0).sum())
            total += v.size
    assert bad / total < 2e-3


def test_pack_layouts_against_numpy_bitstream():
    rng = np.random.default_rng(7)
    for bits in (3, 4, 8):
        q = rng.integers(0, 2 ** bits, size=(5, 64)).astype(np.int32)
        packed = orc.pack(q, bits)
        # dense little-endian bit stream, code i at bits [i*b, (i+1)*b)
        bitsarr = ((q[:, :, None] >> np.arange(bits)) & 1).astype(np.uint8).reshape(5, -1)
        ref = np.packbits(bitsarr, axis=1, bitorder="little")
        assert np.array_equal(packed, ref)
        assert np.array_equal(orc.unpack(packed, 64, bits), q)
    q = rng.integers(0, 16, size=(3, 16)).astype(np.int32)
    assert np.array_equal(orc.pack(q, 4), (q[:, 0::2] | (q[:, 1::2] << 4)).astype(np.uint8))


# ---------------------------------------------------------------- statistics
@pytest.mark.parametrize("dtype", [orc.F16, orc.BF16])
def test_stats_closed_forms(dtype):
    N, C = 257, 24
    n = np.arange(N, dtype=np.float64)[:, None]
    a = np.arange(C, dtype=np.float64)[None, :] - 7
    b = (np.arange(C, dtype=np.float64)[None, :] % 5) - 2          # slopes -2..2
    if dtype == orc.BF16:
        n_eff = n % 64                                           # keep values bf16-exact (|v| < 256)
        Xv = a + b * n_eff
    else:
        Xv = a + b * n                                           # |v| <= 16+512, fp16-exact integers
    X = f16_bits(Xv) if dtype == orc.F16 else bf16_bits(Xv)
    xmin, xmax, xmean, xsum = orc.stats(X, dtype)
    assert np.array_equal(xmin, Xv.min(axis=0).astype(np.float32))
    assert np.array_equal(xmax, Xv.max(axis=0).astype(np.float32))
    if dtype == orc.F16:   # arithmetic series: mean = a + b (N-1)/2
        assert np.allclose(xmean, (a + b * (N - 1) / 2).ravel(), rtol=0, atol=1e-5)
    assert np.array_equal(xsum, Xv.sum(axis=0))                  # integer sums are exact in fp64
    # alternating +c / -c over an even number of rows has mean exactly 0
    alt = np.where(np.arange(256)[:, None] % 2 == 0, 1.0, -1.0) * (np.arange(C)[None, :] + 0.5)
    bits = f16_bits(alt) if dtype == orc.F16 else bf16_bits(alt)
    _, _, m, _ = orc.stats(bits, dtype)
    assert np.all(m == 0)


@pytest.mark.parametrize("dtype", [orc.F16, orc.BF16])
def test_stats_and_wrange_against_numpy(dtype):
    rng = np.random.default_rng(8)
    Xv = rng.standard_normal((300, 40)) * rng.uniform(0.1, 30, 40)[None, :] + rng.uniform(-3, 3, 40)[None, :]
    X = f16_bits(Xv) if dtype == orc.F16 else bf16_bits(Xv)
    ref = bits_to_f64(X, dtype)
    xmin, xmax, xmean, xsum = orc.stats(X, dtype)
    assert np.array_equal(xmin, ref.min(axis=0).astype(np.float32))
    assert np.array_equal(xmax, ref.max(axis=0).astype(np.float32))
    assert np.allclose(xmean, ref.mean(axis=0), rtol=1e-6, atol=1e-9)
    assert np.allclose(xsum, ref.sum(axis=0), rtol=1e-13)
    # a weight matrix is reduced over its rows (output channels), per input channel
    W = X[:37]
    wmin, wmax = orc.wrange(W, dtype)
    assert np.array_equal(wmin, ref[:37].min(axis=0).astype(np.float32))
    assert np.array_equal(wmax, ref[:37].max(axis=0).astype(np.float32))
    # merging two matrices that share the input = range of their row concatenation
    wmin2, wmax2 = orc.wrange(X[37:90], dtype, prev=(wmin, wmax))
    assert np.array_equal(wmin2, ref[:90].min(axis=0).astype(np.float32))
    assert np.array_equal(wmax2, ref[:90].max(axis=0).astype(np.float32))


# ---------------------------------------------------------------- factors, Eq. 3-10
def _layer(rng, N=64, C_in=32, C_out=16, offset=True):
    Xv = rng.standard_normal((N, C_in)) * rng.uniform(0.2, 40, C_in)[None, :]
    if offset:
        Xv = Xv + rng.uniform(-4, 4, C_in)[None, :]
    Wv = rng.standard_normal((C_out, C_in)) * 0.02
    X, W = f16_bits(Xv), f16_bits(Wv)
    return X, W, bits_to_f64(X, orc.F16), bits_to_f64(W, orc.F16)


def _factors_for(X, W):
    xmin, xmax, xmean, _ = orc.stats(X, orc.F16)
    wmin, wmax = orc.wrange(W, orc.F16)
    return (xmin, xmax, xmean, wmin, wmax), orc.factors(xmin, xmax, xmean, wmin, wmax)


def test_factors_eq10_and_equal_ranges():
    rng = np.random.default_rng(9)
    X, W, Xd, Wd = _layer(rng)
    (xmin, xmax, xmean, wmin, wmax), f = _factors_for(X, W)
    rx = (xmax - xmin).astype(np.float64)
    rw = (wmax - wmin).astype(np.float64)
    s = f["s"].astype(np.float64)
    # Eq. 10 and its simplification sqrt(rX / rW)
    assert np.allclose(s, np.sqrt(rx * rw) / rw, rtol=1e-7)
    assert np.allclose(s, np.sqrt(rx / rw), rtol=1e-7)
    # the assumption that leads to Eq. 10: equalised channel ranges coincide
    assert np.allclose(rx / s, s * rw, rtol=3e-7)
    assert np.allclose(f["rinv"].astype(np.float64) * s, 1.0, rtol=1.5e-7)
    assert np.allclose(f["mu_hat"], xmean.astype(np.float64) / s, rtol=3e-7, atol=1e-12)
    assert f["dead"] == 0


def test_equalization_preserves_layer_output_eq3():
    rng = np.random.default_rng(10)
    X, W, Xd, Wd = _layer(rng)
    _, f = _factors_for(X, W)
    s = f["s"].astype(np.float64)
    Y = Xd @ Wd.T
    Yhat = (Xd / s[None, :]) @ (Wd * s[None, :]).T
    assert np.allclose(Yhat, Y, rtol=1e-12, atol=1e-12 * np.abs(Y).max())
    # exact when s is a power of two
    s2 = 2.0 ** rng.integers(-3, 4, s.size)
    assert np.array_equal(((Xd / s2) * (Wd[3] * s2)), Xd * Wd[3])


def test_factors_attain_closed_form_minimum_of_eq8():
    """For any s > 0, max_j(rX_j/s_j) * max_k(s_k rW_k) >= max_j rX_j rW_j, and
    Eq. 10 attains it."""
    rng = np.random.default_rng(11)
    X, W, Xd, Wd = _layer(rng, C_in=24)
    (xmin, xmax, xmean, wmin, wmax), f = _factors_for(X, W)
    rx = (xmax - xmin).astype(np.float64)
    rw = (wmax - wmin).astype(np.float64)
    bound = (rx * rw).max()
    assert f["scalars"][7] == pytest.approx(bound, rel=1e-6)
    assert f["scalars"][6] == pytest.approx(rx.max() * rw.max(), rel=1e-12)
    assert f["scalars"][7] <= f["scalars"][6] * (1 + 1e-9)
    cand = np.exp(rng.uniform(-6, 6, (20000, rx.size)))
    vals = (rx[None, :] / cand).max(axis=1) * (cand * rw[None, :]).max(axis=1)
    assert vals.min() >= bound * (1 - 1e-12)
    # perturbing the solution never does better either
    s = f["s"].astype(np.float64)
    cand = s[None, :] * np.exp(rng.uniform(-0.3, 0.3, (20000, rx.size)))
    vals = (rx[None, :] / cand).max(axis=1) * (cand * rw[None, :]).max(axis=1)
    assert vals.min() >= bound * (1 - 1e-12)


def test_precision_and_objective_from_equalized_tensors():
    """Eq. 4-5 evaluated directly on the equalised tensors X^ and W^."""
    rng = np.random.default_rng(12)
    X, W, Xd, Wd = _layer(rng)
    (xmin, xmax, xmean, wmin, wmax), f = _factors_for(X, W)
    def rng_of(T):
        return T.max(axis=0) - T.min(axis=0), T.max() - T.min()
    rx, RX = rng_of(Xd)
    rw, RW = rng_of(Wd)
    assert f["scalars"][0] == pytest.approx(RX, rel=1e-12)
    assert f["scalars"][1] == pytest.approx(RW, rel=1e-12)
    assert np.allclose(f["pX"], rx / RX, rtol=1e-6)
    assert np.allclose(f["pW"], rw / RW, rtol=1e-6)
    assert f["scalars"][4] == pytest.approx(((rx / RX) * (rw / RW)).sum(), rel=1e-9)
    s = f["s"].astype(np.float64)
    Xh = (Xd.astype(np.float32) * f["rinv"][None, :]).astype(np.float64)
    Wh = (Wd.astype(np.float32) * f["s"][None, :]).astype(np.float64)
    erx, ERX = rng_of(Xh)
    erw, ERW = rng_of(Wh)
    assert f["scalars"][2] == pytest.approx(ERX, rel=1e-9)
    assert f["scalars"][3] == pytest.approx(ERW, rel=1e-9)
    assert f["scalars"][5] == pytest.approx(((erx / ERX) * (erw / ERW)).sum(), rel=1e-9)
    # the point of the method: total precision goes up
    assert f["scalars"][5] > f["scalars"][4]


def test_factors_dead_channels_get_unit_factor():
    xmin = np.array([0.0, 1.0, -1.0, 0.0], np.float32)
    xmax = np.array([1.0, 1.0, 1.0, np.inf], np.float32)
    wmin = np.array([-1.0, -1.0, 0.5, -1.0], np.float32)
    wmax = np.array([1.0, 1.0, 0.5, 1.0], np.float32)
    f = orc.factors(xmin, xmax, np.zeros(4, np.float32), wmin, wmax)
    assert f["s"][0] == pytest.approx(np.sqrt(0.5))
    assert f["s"][1:].tolist() == [1.0, 1.0, 1.0]
    assert f["dead"] == 3


# ---------------------------------------------------------------- weights: fold + quantise
@pytest.mark.parametrize("bits,gran,group", [(8, orc.PER_ROW, 0), (4, orc.PER_GROUP, 8), (3, orc.PER_GROUP, 16),
                                             (4, orc.PER_TENSOR, 0)])
def test_equalize_quantize_is_rowwise_quantizer_of_scaled_weights(bits, gran, group):
    rng = np.random.default_rng(13)
    X, W, Xd, Wd = _layer(rng)
    _, f = _factors_for(X, W)
    codes, step, zp, delta = orc.equalize_quantize(W, orc.F16, f["s"], f["mu_hat"], bits, gran, group)
    C_out, C_in = Wd.shape
    What = Wd.astype(np.float32) * f["s"][None, :]          # binary32 product, input channel j scaled by s_j
    q = orc.unpack(codes, C_in, bits)
    if gran == orc.PER_TENSOR:
        st, z, qq = orc.quantize_vector(What.ravel(), bits)
        assert step[0] == np.float32(st) and zp[0] == z
        assert np.array_equal(q, qq.reshape(C_out, C_in))
    else:
        glen = group if gran == orc.PER_GROUP else C_in
        ng = C_in // glen
        for o in range(C_out):
            for g in range(ng):
                st, z, qq = orc.quantize_vector(What[o, g * glen:(g + 1) * glen], bits)
                assert step[o * ng + g] == np.float32(st) and zp[o * ng + g] == z
                assert np.array_equal(q[o, g * glen:(g + 1) * glen], qq)
    # eps . E[x^] in float64 from the dequantised weights
    Wq = orc.dequantize(codes, step, zp, C_in, bits, gran, group)
    ref = ((Wq - What.astype(np.float64)) * f["mu_hat"].astype(np.float64)[None, :]).sum(axis=1)
    assert np.allclose(delta, ref, rtol=1e-10, atol=1e-14)
    # second route (from stored codes) gives the same
    d2 = orc.bias_delta_from_codes(W, orc.F16, f["s"], codes, step, zp, f["mu_hat"], bits, gran, group)
    assert np.allclose(d2, delta, rtol=1e-12, atol=1e-15)


def test_no_equalization_is_plain_rtn():
    rng = np.random.default_rng(14)
    X, W, Xd, Wd = _layer(rng)
    codes, step, zp, _ = orc.equalize_quantize(W, orc.F16, None, None, 4, orc.PER_ROW)
    q = orc.unpack(codes, Wd.shape[1], 4)
    for o in range(Wd.shape[0]):
        st, z, qq = orc.quantize_vector(Wd[o].astype(np.float32), 4)
        assert (step[o], zp[o]) == (np.float32(st), z) and np.array_equal(q[o], qq)


# ---------------------------------------------------------------- bias correction, Eq. 11-15
@pytest.mark.parametrize("bits,gran,group", [(8, orc.PER_ROW, 0), (4, orc.PER_GROUP, 8), (3, orc.PER_ROW, 0)])
def test_bias_correction_zeroes_the_mean_output_error(bits, gran, group):
    """Eq. 11 by brute force: after the correction the mean over the calibration
    set of (quantised-layer output - original output) vanishes."""
    rng = np.random.default_rng(15)
    X, W, Xd, Wd = _layer(rng, N=200, C_in=32, C_out=12, offset=True)
    _, f = _factors_for(X, W)
    codes, step, zp, delta = orc.equalize_quantize(W, orc.F16, f["s"], f["mu_hat"], bits, gran, group)
    bias = rng.standard_normal(Wd.shape[0]) * 0.1
    bias_bits = f16_bits(bias)
    bias64 = bits_to_f64(bias_bits, orc.F16)
    bf, b16 = orc.bias_correct(delta, bias_bits, orc.F16)
    Xh = (Xd.astype(np.float32) * f["rinv"][None, :]).astype(np.float64)      # the input the layer sees
    Wh = (Wd.astype(np.float32) * f["s"][None, :]).astype(np.float64)
    Wq = orc.dequantize(codes, step, zp, Wd.shape[1], bits, gran, group)
    y = Xh @ Wh.T + bias64[None, :]
    y_q = Xh @ Wq.T + bias64[None, :]
    y_c = Xh @ Wq.T + bf.astype(np.float64)[None, :]
    raw = (y_q - y).mean(axis=0)
    fixed = (y_c - y).mean(axis=0)
    scale = (np.abs(Wq - Wh) * np.abs(Xh).mean(axis=0)[None, :]).sum(axis=1)
    assert np.all(np.abs(fixed) <= 2e-6 * scale + 1e-9)
    assert np.abs(raw).max() > 50 * np.abs(fixed).max()      # the correction is what removed it
    # sign and placement: bias' = bias - eps.E[x^]
    assert np.allclose(bf, bias64 - delta, rtol=0, atol=1e-7)
    assert np.allclose(bits_to_f64(b16, orc.F16), bias64 - delta, rtol=0, atol=1e-3)
    # a layer without bias gets one
    bf0, _ = orc.bias_correct(delta, None, orc.F16)
    assert np.allclose(bf0, -delta, rtol=1e-6, atol=1e-12)


# ---------------------------------------------------------------- activations
def test_quant_act_is_rowwise_quantizer_of_scaled_inputs():
    rng = np.random.default_rng(16)
    X, W, Xd, Wd = _layer(rng, N=40, C_in=48)
    (xmin, xmax, xmean, wmin, wmax), f = _factors_for(X, W)
    Xq, step, zp = orc.quant_act(X, orc.F16, f["rinv"], orc.PER_ROW)
    Xh = Xd.astype(np.float32) * f["rinv"][None, :]
    for n in range(Xd.shape[0]):
        st, z, qq = orc.quantize_vector(Xh[n], 8)
        assert (step[n], zp[n]) == (np.float32(st), z) and np.array_equal(Xq[n], qq)
    # static per-tensor range taken from the per-channel statistics
    lo_hi = np.array([(xmin * f["rinv"]).min(), (xmax * f["rinv"]).max()], np.float32)
    assert lo_hi[0] == Xh.min() and lo_hi[1] == Xh.max()
    Xq2, st2, zp2 = orc.quant_act(X, orc.F16, f["rinv"], orc.PER_TENSOR, lo_hi)
    st, z, qq = orc.quantize_vector(Xh.ravel(), 8)
    assert (st2[0], zp2[0]) == (np.float32(st), z) and np.array_equal(Xq2.ravel(), qq)
    # without factors it is the plain per-token quantiser
    Xq3, st3, zp3 = orc.quant_act(X, orc.F16, None, orc.PER_ROW)
    st, z, qq = orc.quantize_vector(Xd[5].astype(np.float32), 8)
    assert (st3[5], zp3[5]) == (np.float32(st), z) and np.array_equal(Xq3[5], qq)


def test_equalization_reduces_activation_quantization_error():
    """What Section 3.2 is for: with outlier channels, per-tensor 8-bit activation
    error after equalisation is far below the error without it."""
    rng = np.random.default_rng(17)
    Xv = rng.standard_normal((256, 64))
    Xv[:, [3, 40]] *= 60.0
    Wv = rng.standard_normal((32, 64)) * 0.02
    X, W = f16_bits(Xv), f16_bits(Wv)
    Xd, Wd = bits_to_f64(X, orc.F16), bits_to_f64(W, orc.F16)
    (xmin, xmax, xmean, wmin, wmax), f = _factors_for(X, W)
    def out_err(rinv, s):
        r = np.ones(64, np.float32) if rinv is None else rinv
        lo_hi = np.array([(xmin * r).min(), (xmax * r).max()], np.float32)
        Xq, st, z = orc.quant_act(X, orc.F16, rinv, orc.PER_TENSOR, lo_hi)
        Xdq = st[0] * (Xq.astype(np.float64) - z[0])
        sv = np.ones(64) if s is None else s.astype(np.float64)
        Wh = Wd * sv[None, :]
        return np.mean((Xdq @ Wh.T - Xd @ Wd.T) ** 2)
    assert out_err(f["rinv"], f["s"]) < 0.2 * out_err(None, None)


# ---------------------------------------------------------------- forward check, Eq. 11 on data
def test_forward_check_hand_worked():
    """A 2-token, 2-input, 3-output layer worked by hand (all values exact in binary):
    X~ = Step^x (Xq - Z^x) = [[1, 0], [0, 4]],  W~ = Step^w (Wq - Z^w) = [[0, 4], [1, 0], [-2, 1]],
    y~ = X~ W~^T + bias_q = [[0, 1, -2], [16, 0, 4]] + [0.5, -1, 0] = [[0.5, 0, -2], [16.5, -1, 4]],
    y  = X W^T + bias with X = [[1, .5], [0, 4]], W = [[.5, 4], [1, .25], [-2, 1]], bias = [0, 1, 0]
       = [[2.5, 2.125, -1.5], [16, 2, 4]],
    d  = y~ - y = [[-2, -2.125, -0.5], [0.5, -3, 0]]."""
    Xq = np.array([[3, 1], [2, 6]], np.uint8)
    act_step, act_zp = [0.5, 1.0], [1, 2]
    Wq = np.array([[2, 4], [5, 1], [0, 3]], np.uint8)
    w_step, w_zp = [2.0, 0.25, 1.0], [2, 1, 2]
    bias_q = np.array([0.5, -1.0, 0.0], np.float32)
    X = f16_bits([[1, 0.5], [0, 4]])
    W = f16_bits([[0.5, 4], [1, 0.25], [-2, 1]])
    bias = f16_bits([0, 1, 0])
    mean_err, sums = orc.forward_check(Xq, act_step, act_zp, Wq, w_step, w_zp, bias_q, X, W, orc.F16, bias)
    assert mean_err.tolist() == [-0.75, -2.5625, -0.25]
    assert sums.tolist() == [4 + 4.515625 + 0.25 + 0.25 + 9 + 0,
                             6.25 + 4.515625 + 2.25 + 256 + 4 + 16,
                             0.5625 + 6.56640625 + 0.0625, 6.0]
    # without biases the products alone are compared; an uncorrected layer (bias_q None) keeps its bias,
    # which cancels in y~ - y but counts in sum y^2
    mean_err0, sums0 = orc.forward_check(Xq, act_step, act_zp, Wq, w_step, w_zp, None, X, W, orc.F16, None)
    assert mean_err0.tolist() == [-0.75 - 0.5, -2.5625 + 1 + 1, -0.25]
    mean_err1, sums1 = orc.forward_check(Xq, act_step, act_zp, Wq, w_step, w_zp, None, X, W, orc.F16, bias)
    assert mean_err1.tolist() == mean_err0.tolist() and sums1[0] == sums0[0]
    assert sums0[1] == 6.25 + 1.265625 + 2.25 + 256 + 1 + 16 and sums1[1] == sums[1]


def test_forward_check_against_numpy_matmul_and_bf16():
    rng = np.random.default_rng(31)
    N, C_in, C_out = 37, 48, 20
    Xq = rng.integers(0, 256, (N, C_in)).astype(np.uint8)
    Wq = rng.integers(0, 256, (C_out, C_in)).astype(np.uint8)
    act_step = rng.uniform(0.01, 0.05, N).astype(np.float32)
    act_zp = rng.integers(0, 256, N).astype(np.int32)
    w_step = rng.uniform(0.001, 0.01, C_out).astype(np.float32)
    w_zp = rng.integers(-40, 300, C_out).astype(np.int32)          # a zero-point may lie outside the code range
    bias_q = rng.standard_normal(C_out).astype(np.float32)
    for dt, to_bits in ((orc.F16, f16_bits), (orc.BF16, bf16_bits)):
        X, W, b = to_bits(rng.standard_normal((N, C_in))), to_bits(rng.standard_normal((C_out, C_in)) * 0.1), \
            to_bits(rng.standard_normal(C_out))
        mean_err, sums = orc.forward_check(Xq, act_step, act_zp, Wq, w_step, w_zp, bias_q, X, W, dt, b)
        Xt = act_step.astype(np.float64)[:, None] * (Xq.astype(np.float64) - act_zp[:, None])
        Wt = w_step.astype(np.float64)[:, None] * (Wq.astype(np.float64) - w_zp[:, None])
        yq = Xt @ Wt.T + bias_q.astype(np.float64)[None, :]
        y = bits_to_f64(X, dt) @ bits_to_f64(W, dt).T + bits_to_f64(b, dt)[None, :]
        d = yq - y
        assert np.allclose(mean_err, d.mean(axis=0), rtol=1e-12, atol=1e-12)
        assert np.allclose(sums, [(d * d).sum(), (y * y).sum(), (d.mean(axis=0) ** 2).sum(), N * C_out], rtol=1e-12)


def test_forward_check_sees_what_bias_correction_removes():
    """Eq. 11-15 tie three oracle routines together.  With activations that the 8-bit grid holds
    exactly, the mean output error of the quantised layer is eps . E[x^] (the step-4 sums), and
    it vanishes once the step-5 bias is used."""
    rng = np.random.default_rng(32)
    N, C_in, C_out = 120, 32, 10
    Xq = rng.integers(0, 256, (N, C_in)).astype(np.uint8)
    Xq[:, 0], Xq[:, 1] = 0, 255                                    # every token spans the whole code range
    act_zp = rng.integers(100, 140, N).astype(np.int32)
    act_step = np.full(N, 2.0 ** -6, np.float32)
    Xhat = (Xq.astype(np.float64) - act_zp[:, None]) * 2.0 ** -6   # |x^| < 4, multiples of 1/64: exact in fp16
    s = np.ones(C_in, np.float32)                                  # identity equalisation: X = X^
    mu_hat = Xhat.mean(axis=0).astype(np.float32)
    Wd = (rng.standard_normal((C_out, C_in)) * 0.05).astype(np.float16)
    codes, w_step, w_zp, delta = orc.equalize_quantize(Wd.view(np.uint16), orc.F16, s, mu_hat, 8, orc.PER_ROW)
    bias = f16_bits(rng.standard_normal(C_out) * 0.1)
    bf, _ = orc.bias_correct(delta, bias, orc.F16)
    X = f16_bits(Xhat)
    assert np.array_equal(bits_to_f64(X, orc.F16), Xhat)
    # the activation quantiser reproduces these codes, so step 6 and the check agree on the grid
    q_codes, q_step, q_zp = orc.quant_act(X, orc.F16, None)
    assert np.array_equal(q_codes, Xq) and np.array_equal(q_zp, act_zp) and np.array_equal(q_step, act_step)
    raw, _ = orc.forward_check(Xq, act_step, act_zp, codes, w_step, w_zp, None, X, Wd.view(np.uint16), orc.F16, bias)
    fixed, sums = orc.forward_check(Xq, act_step, act_zp, codes, w_step, w_zp, bf, X, Wd.view(np.uint16), orc.F16, bias)
    mu64 = mu_hat.astype(np.float64)
    scale = np.abs(delta).max()
    assert np.allclose(raw, delta + (Xhat.mean(axis=0) - mu64) @ (orc.dequantize(codes, w_step, w_zp, C_in, 8, orc.PER_ROW)
                                                                     - Wd.astype(np.float64)).T, rtol=0, atol=1e-9 * scale)
    # what is left: binary32 rounding of mu_hat (relative 2^-24 of the sums) and of bias' (half an ulp)
    assert np.abs(fixed).max() <= 1e-6 * scale + 2.0 ** -24 * np.abs(bf).max()
    assert np.abs(raw).max() > 1000 * np.abs(fixed).max()
    assert sums[3] == N * C_out and sums[2] == pytest.approx((fixed ** 2).sum(), rel=1e-12)


# ---------------------------------------------------------------- folding 1/s into the producer (after Eq. 3)
def test_fold_scale_against_library_casts_and_exact_cases():
    rng = np.random.default_rng(41)
    P = rng.standard_normal((9, 13)) * 3
    rinv = np.exp(rng.standard_normal(9)).astype(np.float32)
    # fp16: NumPy's float32 -> float16 cast rounds to nearest even
    Pb = f16_bits(P)
    got = orc.fold_scale(Pb, orc.F16, rinv)
    ref = (Pb.view(np.float16).astype(np.float32) * rinv[:, None]).astype(np.float16).view(np.uint16)
    assert np.array_equal(got, ref)
    # bf16: PyTorch's cast
    Pb = bf16_bits(P)
    got = orc.fold_scale(Pb, orc.BF16, rinv)
    prod = torch.from_numpy(bits_to_f64(Pb, orc.BF16).astype(np.float32) * rinv[:, None])
    assert np.array_equal(got, prod.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))
    # powers of two are exact; a vector is a one-column matrix
    v = f16_bits([1.5, -3.0, 0.125, 7.0])
    out = orc.fold_scale(v, orc.F16, np.array([2.0, 0.5, 4.0, 0.25], np.float32))
    assert bits_to_f64(out, orc.F16).tolist() == [3.0, -1.5, 0.5, 1.75]
    # the scale belongs to the ROW (a transposed fold fails here)
    M = f16_bits([[1, 2], [3, 4]])
    out = orc.fold_scale(M, orc.F16, np.array([2.0, 0.5], np.float32))
    assert bits_to_f64(out, orc.F16).tolist() == [[2.0, 4.0], [1.5, 2.0]]


def test_folds_leave_a_decoder_block_unchanged():
    """Eq. 3 through the producers: scaling the gain / shift of a normalisation layer, the value
    projection (seen through the attention weights), ``up`` (seen through the gate) and ``fc1``
    (seen through ReLU) by 1/s gives exactly the equalised input X diag(s)^-1 of the next layer,
    up to the 16-bit rounding of the folded parameters."""
    rng = np.random.default_rng(42)
    T, h, f = 24, 16, 40
    x = rng.standard_normal((T, h))
    s = np.exp(rng.standard_normal(h) * 0.5).astype(np.float32)
    sf = np.exp(rng.standard_normal(f) * 0.5).astype(np.float32)
    rinv, rinvf = (1.0 / s).astype(np.float32), (1.0 / sf).astype(np.float32)
    dec = lambda b: bits_to_f64(b, orc.F16)
    fold = lambda a, r: dec(orc.fold_scale(f16_bits(a), orc.F16, r))
    q16 = lambda a: dec(f16_bits(a))
    tol = 2.0 ** -10                                           # one 16-bit rounding of each folded parameter

    # normalisation layer: (x - mean) / std * gain + shift
    gain, shift = q16(1 + 0.1 * rng.standard_normal(h)), q16(0.1 * rng.standard_normal(h))
    z = (x - x.mean(axis=1, keepdims=True)) / x.std(axis=1, keepdims=True)
    ln = z * gain + shift
    ln_f = z * fold(gain, rinv) + fold(shift, rinv)
    assert np.allclose(ln_f, ln * rinv, rtol=0, atol=tol * (np.abs(z) * np.abs(gain) + np.abs(shift)).max() * rinv.max())

    # value projection through softmax attention: o_in = A (x Wv^T + bv)
    Wv, bv = q16(rng.standard_normal((h, h)) * 0.2), q16(rng.standard_normal(h) * 0.1)
    A = np.exp(rng.standard_normal((T, T)))
    A /= A.sum(axis=1, keepdims=True)
    o_in = A @ (x @ Wv.T + bv)
    o_in_f = A @ (x @ fold(Wv, rinv).T + fold(bv, rinv))
    scale = (np.abs(A) @ (np.abs(x) @ np.abs(Wv).T + np.abs(bv))) * rinv
    assert np.all(np.abs(o_in_f - o_in * rinv) <= tol * scale)

    # gated MLP: down_in = silu(x Wg^T) * (x Wu^T)
    Wg, Wu = q16(rng.standard_normal((f, h)) * 0.2), q16(rng.standard_normal((f, h)) * 0.2)
    g = x @ Wg.T
    act = g / (1 + np.exp(-g))
    down_in = act * (x @ Wu.T)
    down_in_f = act * (x @ fold(Wu, rinvf).T)
    assert np.all(np.abs(down_in_f - down_in * rinvf) <= tol * np.abs(act) * (np.abs(x) @ np.abs(Wu).T) * rinvf)

    # ReLU MLP: fc2_in = relu(x W1^T + b1); needs s > 0
    W1, b1 = q16(rng.standard_normal((f, h)) * 0.2), q16(rng.standard_normal(f) * 0.1)
    fc2_in = np.maximum(x @ W1.T + b1, 0)
    fc2_in_f = np.maximum(x @ fold(W1, rinvf).T + fold(b1, rinvf), 0)
    assert np.all(np.abs(fc2_in_f - fc2_in * rinvf) <= tol * (np.abs(x) @ np.abs(W1).T + np.abs(b1)) * rinvf)


# ---------------------------------------------------------------- weight-only forward check
def test_forward_check_weights_hand_worked():
    """2 tokens, 4 inputs, 2 outputs, 4-bit codes, groups of 2 (values exact in binary).
    rinv = [1, .5, 2, 1];  X = [[1, 2, .5, -1], [0, 4, 1, 2]]  ->  x^ = [[1, 1, 1, -1], [0, 2, 2, 2]]
    row 0: codes [3, 5 | 9, 1], Step [.5, .25], Z [3, 1]  ->  W~ = [0, 1, 2, 0]
    row 1: codes [0, 15 | 4, 4], Step [1, 2],  Z [8, 4]   ->  W~ = [-8, 7, 0, 0]
    y~ = x^ W~^T = [[3, -1], [6, 14]];  W = [[.5, .5, 1, 0], [-8, 3, 0, .5]]  ->  y = [[2, -2.5], [3, 13]]
    d = [[1, 1.5], [3, 1]]  (no biases)."""
    q = np.array([[3, 5, 9, 1], [0, 15, 4, 4]], np.int32)
    codes = orc.pack(q, 4)
    step, zp = np.array([0.5, 0.25, 1.0, 2.0], np.float32), np.array([3, 1, 8, 4], np.int32)
    rinv = np.array([1, 0.5, 2, 1], np.float32)
    X = f16_bits([[1, 2, 0.5, -1], [0, 4, 1, 2]])
    W = f16_bits([[0.5, 0.5, 1, 0], [-8, 3, 0, 0.5]])
    me, sums = orc.forward_check_weights(codes, step, zp, 4, orc.PER_GROUP, 2, rinv, None, X, W, orc.F16)
    assert me.tolist() == [2.0, 1.25]
    assert sums.tolist() == [1 + 2.25 + 9 + 1, 4 + 6.25 + 9 + 169, 4 + 1.5625, 4.0]
    # biases: bias' - bias shifts every d of the channel; an uncorrected layer keeps its bias
    bias = f16_bits([1.0, -2.0])
    me_b, _ = orc.forward_check_weights(codes, step, zp, 4, orc.PER_GROUP, 2, rinv, np.array([0.5, -2.0], np.float32), X, W,
                                        orc.F16, bias)
    assert me_b.tolist() == [1.5, 1.25]
    me_k, _ = orc.forward_check_weights(codes, step, zp, 4, orc.PER_GROUP, 2, rinv, None, X, W, orc.F16, bias)
    assert me_k.tolist() == [2.0, 1.25]


@pytest.mark.parametrize("bits,gran,group", [(8, orc.PER_ROW, 0), (4, orc.PER_GROUP, 8), (3, orc.PER_GROUP, 16),
                                             (5, orc.PER_TENSOR, 0)])
def test_forward_check_weights_against_numpy_and_bias_correction(bits, gran, group):
    """NumPy matmul on the de-quantised weights; and Eq. 11-15 for a weight-only layer: after the
    step-5 correction the mean output error vanishes (down to the binary32 rounding of mu_hat and
    bias'), before it it is the step-4 sum eps . E[x^]."""
    rng = np.random.default_rng(51 + bits)
    X, W, Xd, Wd = _layer(rng, N=150, C_in=32, C_out=11, offset=True)
    _, f = _factors_for(X, W)
    codes, step, zp, delta = orc.equalize_quantize(W, orc.F16, f["s"], f["mu_hat"], bits, gran, group)
    bias = f16_bits(rng.standard_normal(11) * 0.1)
    bf, _ = orc.bias_correct(delta, bias, orc.F16)
    raw, sums_raw = orc.forward_check_weights(codes, step, zp, bits, gran, group, f["rinv"], None, X, W, orc.F16, bias)
    fixed, _ = orc.forward_check_weights(codes, step, zp, bits, gran, group, f["rinv"], bf, X, W, orc.F16, bias)
    Wq = orc.dequantize(codes, step, zp, 32, bits, gran, group)
    Xh = Xd.astype(np.float64) * f["rinv"].astype(np.float64)[None, :]
    b64 = bits_to_f64(bias, orc.F16)
    y = Xd.astype(np.float64) @ Wd.astype(np.float64).T + b64
    d = (Xh @ Wq.T + b64) - y
    assert np.allclose(raw, d.mean(axis=0), rtol=1e-10, atol=1e-12)
    assert np.allclose(sums_raw, [(d * d).sum(), (y * y).sum(), (d.mean(axis=0) ** 2).sum(), d.size], rtol=1e-10)
    # eps is taken against W^ = fl(W s) and E[x^] = fl(mean x * rinv): binary32 roundings of the equalised
    # operands separate the two routes by parts in 1e-6 of the terms
    scale = (np.abs(Wq) * np.abs(Xh).mean(axis=0)[None, :]).sum(axis=1)
    assert np.all(np.abs(raw - delta) <= 3e-6 * scale)
    assert np.all(np.abs(fixed) <= 3e-6 * scale + 2.0 ** -24 * np.abs(bf))
    assert np.abs(raw).max() > 20 * np.abs(fixed).max()


# ---------------------------------------------------------------- the comparison criterion (Section 3.1)
def test_absmax_criterion_closed_form_and_what_it_balances():
    """Fed with the largest magnitudes, Eq. 10 is s = sqrt(max|x| / max|w|) and makes the largest
    magnitudes of the equalised activations and weights equal per channel (what the per-channel
    equalisation the paper starts from does); the range criterion makes the RANGES equal instead.
    On channels with an offset the two differ; on symmetric channels they coincide."""
    rng = np.random.default_rng(61)
    C = 40
    xmin = -rng.uniform(0.5, 3, C).astype(np.float32)
    xmax = rng.uniform(0.5, 3, C).astype(np.float32)
    xmin[:10] += 4.0                                        # offset channels: all positive
    xmax[:10] += 4.0
    xmean = ((xmin + xmax) / 2).astype(np.float32)
    wmin = -rng.uniform(0.01, 0.1, C).astype(np.float32)
    wmax = rng.uniform(0.01, 0.1, C).astype(np.float32)
    xmin[20:30], wmin[20:30] = -xmax[20:30], -wmax[20:30]   # symmetric channels
    f = orc.factors(xmin, xmax, xmean, wmin, wmax, orc.ABSMAX)
    ax = np.maximum(np.abs(xmin), np.abs(xmax)).astype(np.float64)
    aw = np.maximum(np.abs(wmin), np.abs(wmax)).astype(np.float64)
    assert np.allclose(f["s"], np.sqrt(ax / aw), rtol=2e-7)
    assert np.allclose(f["rinv"], 1.0 / f["s"], rtol=1e-7) and np.allclose(f["mu_hat"], xmean * f["rinv"], rtol=1e-7)
    assert np.allclose(ax / f["s"], f["s"] * aw, rtol=3e-7)                      # equal largest magnitudes
    g = orc.factors(xmin, xmax, xmean, wmin, wmax, orc.RANGE)
    rx, rw = (xmax - xmin).astype(np.float64), (wmax - wmin).astype(np.float64)
    assert np.allclose(rx / g["s"], g["s"] * rw, rtol=3e-7)                      # equal ranges
    assert np.allclose(f["s"][20:30], g["s"][20:30], rtol=3e-7)                  # symmetric: the same factor
    assert np.all(f["s"][:10] > 1.1 * g["s"][:10])                               # offset: abs-max overstates x
    assert np.array_equal(g["s"], orc.factors(xmin, xmax, xmean, wmin, wmax)["s"])   # the default is the paper's
    # the diagnostics stay range-based under either criterion
    assert np.array_equal(f["pX"], g["pX"]) and np.array_equal(f["pW"], g["pW"])


# ---------------------------------------------------------------- signed relabelling of 8-bit codes
def test_relabel_signed_keeps_dequantised_values_and_saturates():
    """q' = q - 128 and Z' = Z - 128 leave Step (q - Z) unchanged (Eq. 1 de-quantised, with the
    code range moved); checked on all 256 codes with integers typed here, by the two's-complement
    identity (subtracting 128 modulo 256 flips the top bit), and at the int32 edge, where Z'
    saturates instead of wrapping."""
    q = np.arange(256, dtype=np.uint8)
    zp = np.array([0, 128, -7, 300, 2147483647, -2147483648 + 128, -2147483648 + 127, -2147483648], np.int32)
    qs, zs = orc.relabel_signed(q, zp)
    assert qs.dtype == np.int8 and qs[0] == -128 and qs[128] == 0 and qs[255] == 127
    assert np.array_equal(qs.astype(np.int64), np.arange(256) - 128)
    assert np.array_equal(qs.view(np.uint8), q ^ 0x80)
    assert zs.tolist() == [-128, 0, -135, 172, 2147483519, -2147483648, -2147483648, -2147483648]
    ok = zp.astype(np.int64) - 128 >= -2147483648           # where nothing saturates the values are kept
    step = 0.37
    for k in np.flatnonzero(ok):
        assert np.array_equal(step * (qs.astype(np.int64) - int(zs[k])), step * (q.astype(np.int64) - int(zp[k])))
    only_codes, none = orc.relabel_signed(q.reshape(16, 16))
    assert none is None and only_codes.shape == (16, 16)
