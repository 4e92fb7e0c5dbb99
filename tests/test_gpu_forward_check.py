"""Forward check (tensor-core GEMMs + comparison kernels) against the CPU oracle.

The oracle evaluates both layers in binary64 straight from the definitions.  The GPU takes
the integer product exactly and folds the zero-points in 64-bit integers, so the quantised
side agrees to binary64 rounding; the 16-bit product is accumulated in binary32 by the
tensor cores, so that side agrees exactly only where binary32 accumulation is exact
(small-integer operands) and otherwise within the accumulation bound

    |Y_gpu - Y| <= K * 2^-23 * sum_k |x_k w_k|      (K additions, each off by at most one
                                                      unit in the last place of a partial sum)

which the realistic case asserts element-wise through the means.  All oracle inputs are
seeded or come from the oracle itself, never from the GPU.
"""
import numpy as np
import pytest
import torch

from oracle import aweq_oracle as orc
from paper_2311_01305_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _run(Xq, act_step, act_zp, Wq, w_step, w_zp, bias_q, X, W, bias):
    from paper_2311_01305_b200 import aweq
    t = lambda a, dt=None: None if a is None else torch.as_tensor(np.ascontiguousarray(a), dtype=dt).to(DEV)
    C_out = W.shape[0]
    mean_err, check_me = util.guarded((C_out,), torch.float64)
    sums, check_s = util.guarded((4,), torch.float64)
    aweq.aweq_forward_check(t(Xq), t(act_step, torch.float32), t(act_zp, torch.int32), t(Wq), t(w_step, torch.float32),
                            t(w_zp, torch.int32), t(bias_q, torch.float32), X.to(DEV), W.to(DEV),
                            None if bias is None else bias.to(DEV), mean_err, sums)
    torch.cuda.synchronize()
    check_me()
    check_s()
    return mean_err.cpu().numpy(), sums.cpu().numpy()


def _int_valued(shape, dtype, seed, lim):
    g = torch.Generator().manual_seed(seed)
    return torch.randint(-lim, lim + 1, shape, generator=g).to(dtype)


def _codes(shape, seed, lo=0, hi=256):
    return np.random.default_rng(seed).integers(lo, hi, shape).astype(np.uint8)


# N, C_in, C_out: ragged token blocks and tiles; two token chunks; a K wide enough for the split product
EXACT_SHAPES = [(1000, 768, 200), (77, 16, 8), (16384 + 300, 256, 64), (300, 32768 + 128, 16), (129, 4096, 136)]


@pytest.mark.parametrize("N,C_in,C_out", EXACT_SHAPES)
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_forward_check_exact_operands(N, C_in, C_out, dtype):
    """Operands whose binary32 accumulation is exact (|x|, |w| <= 3, integers): every output
    must agree with the oracle to binary64 rounding, whatever the tile, chunk or K split."""
    seed = N + C_in + C_out
    rng = np.random.default_rng(seed)
    Xq, Wq = _codes((N, C_in), seed), _codes((C_out, C_in), seed + 1)
    act_step = rng.uniform(0.01, 0.05, N).astype(np.float32)
    act_zp = rng.integers(0, 256, N).astype(np.int32)
    w_step = rng.uniform(0.001, 0.01, C_out).astype(np.float32)
    w_zp = rng.integers(-40, 300, C_out).astype(np.int32)
    bias_q = rng.standard_normal(C_out).astype(np.float32)
    X = _int_valued((N, C_in), dtype, seed + 2, 3)
    W = _int_valued((C_out, C_in), dtype, seed + 3, 3)
    bias = _int_valued((C_out,), dtype, seed + 4, 5)
    got_me, got_s = _run(Xq, act_step, act_zp, Wq, w_step, w_zp, bias_q, X, W, bias)
    dt = util.odt(X)
    ref_me, ref_s = orc.forward_check(Xq, act_step, act_zp, Wq, w_step, w_zp, bias_q, util.bits(X), util.bits(W), dt,
                                      util.bits(bias))
    rms = np.sqrt(ref_s[0] / ref_s[3])
    assert np.all(np.abs(got_me - ref_me) <= 1e-11 * rms)
    assert np.allclose(got_s, ref_s, rtol=1e-11, atol=0)


def test_forward_check_extreme_codes_do_not_overflow():
    """All codes 255 at the widest unsplit K and across the split: the int32 partial products
    stay below 2^31 and the 64-bit fold is exact."""
    for C_in in (32768, 32768 + 4096):
        N, C_out = 40, 8
        Xq = np.full((N, C_in), 255, np.uint8)
        Wq = np.full((C_out, C_in), 255, np.uint8)
        one_n, one_o = np.ones(N, np.float32), np.ones(C_out, np.float32)
        zero_n, zero_o = np.zeros(N, np.int32), np.zeros(C_out, np.int32)
        X = torch.zeros((N, C_in), dtype=torch.float16)
        W = torch.zeros((C_out, C_in), dtype=torch.float16)
        got_me, got_s = _run(Xq, one_n, zero_n, Wq, one_o, zero_o, None, X, W, None)
        assert np.all(got_me == 255.0 * 255.0 * C_in)
        assert got_s[1] == 0.0 and got_s[3] == N * C_out
        # and with the largest zero-points: every term cancels
        got_me, _ = _run(Xq, one_n, zero_n + 255, Wq, one_o, zero_o + 255, None, X, W, None)
        assert np.all(got_me == 0.0)


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("correct", [True, False])
def test_forward_check_of_a_calibrated_layer(dtype, correct):
    """The whole chain on a realistic layer: oracle calibration (steps 1-6) feeds both sides."""
    N, C_in, C_out = 1536 + 40, 768, 1024 + 8
    Xc = util.rand16((N, C_in), dtype, 41, scale=1.0, offset=0.5, outlier_cols=4)
    Wc = util.rand16((C_out, C_in), dtype, 42, scale=0.03)
    bias = util.rand16((1, C_out), dtype, 43, scale=0.1)[0].contiguous()
    cal = util.oracle_layer(Xc, [Wc], 8, orc.PER_ROW, 0, biases=[bias], bias_correct=True)
    lin, (Xq, act_step, act_zp) = cal["linears"][0], cal["act"]
    dt = util.odt(Xc)
    bias_q = lin["bias_f32"] if correct else None
    got_me, got_s = _run(Xq, act_step, act_zp, lin["codes"], lin["step"], lin["zp"], bias_q, Xc, Wc, bias)
    ref_me, ref_s = orc.forward_check(Xq, act_step, act_zp, lin["codes"], lin["step"], lin["zp"], bias_q,
                                      util.bits(Xc), util.bits(Wc), dt, util.bits(bias))
    Xa, Wa = np.abs(Xc.double().numpy()), np.abs(Wc.double().numpy())
    bound = C_in * 2.0 ** -23 * (Xa @ Wa.T)                       # per-output accumulation bound
    assert np.all(np.abs(got_me - ref_me) <= bound.mean(axis=0))
    # sum d^2: |sum (d+e)^2 - sum d^2| <= 2 sqrt(sum d^2 sum e^2) + sum e^2
    e2 = (bound ** 2).sum()
    assert abs(got_s[0] - ref_s[0]) <= 2 * np.sqrt(ref_s[0] * e2) + e2
    assert abs(got_s[1] - ref_s[1]) <= 2 * np.sqrt(ref_s[1] * e2) + e2
    assert got_s[3] == ref_s[3]
    # in practice the accumulation error is far inside the bound: the means agree to 1e-5 of the output scale
    y_rms = np.sqrt(ref_s[1] / ref_s[3])
    assert np.abs(got_me - ref_me).max() <= 1e-5 * y_rms
    if correct:
        # activation rounding is the only source of mean error left (Eq. 11-15 remove the weights' part)
        raw = cal["linears"][0]["delta"]
        assert np.abs(ref_me).max() < np.abs(raw).max()


def test_forward_check_rejects_bad_arguments():
    from paper_2311_01305_b200 import aweq
    N, C_in, C_out = 32, 24, 8                                     # C_in not a multiple of 16
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=DEV)
    with pytest.raises(aweq.AweqError) as e:
        aweq.aweq_forward_check(z((N, C_in), torch.uint8), z(N, torch.float32), z(N, torch.int32),
                                z((C_out, C_in), torch.uint8), z(C_out, torch.float32), z(C_out, torch.int32), None,
                                z((N, C_in), torch.float16), z((C_out, C_in), torch.float16), None,
                                z(C_out, torch.float64), z(4, torch.float64), ws=aweq.workspace(1 << 22))
    assert e.value.code == 2          # AWEQ_ERR_SHAPE
    C_in = 32
    with pytest.raises(aweq.AweqError) as e:
        aweq.aweq_forward_check(z((N, C_in), torch.uint8), z(N, torch.float32), z(N, torch.int32),
                                z((C_out, C_in), torch.uint8), z(C_out, torch.float32), z(C_out, torch.int32), None,
                                z((N, C_in), torch.float16), z((C_out, C_in), torch.float16), None,
                                z(C_out, torch.float64), z(4, torch.float64), ws=aweq.workspace(4096))
    assert e.value.code == 7          # AWEQ_ERR_WORKSPACE


# ------------------------------------------------------------------ weight-only forward check
def _run_weights(codes, step, zp, bits, gran, group, rinv, bias_q, X, W, bias):
    from paper_2311_01305_b200 import aweq
    t = lambda a, dt=None: None if a is None else torch.as_tensor(np.ascontiguousarray(a), dtype=dt).to(DEV)
    C_out = W.shape[0]
    mean_err, check_me = util.guarded((C_out,), torch.float64)
    sums, check_s = util.guarded((4,), torch.float64)
    aweq.aweq_forward_check_weights(t(codes), t(step, torch.float32), t(zp, torch.int32), bits, gran, group,
                                    t(rinv, torch.float32), t(bias_q, torch.float32), X.to(DEV), W.to(DEV),
                                    None if bias is None else bias.to(DEV), mean_err, sums)
    torch.cuda.synchronize()
    check_me()
    check_s()
    return mean_err.cpu().numpy(), sums.cpu().numpy()


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("N,C_in,C_out,bits,gran,group", [
    (1000, 256, 72, 4, orc.PER_GROUP, 128), (16384 + 77, 64, 40, 3, orc.PER_GROUP, 16),
    (130, 4096, 136, 8, orc.PER_ROW, 0), (77, 48, 8, 5, orc.PER_TENSOR, 0), (90, 160, 24, 2, orc.PER_GROUP, 32)])
def test_forward_check_weights_exact_operands(N, C_in, C_out, bits, gran, group, dtype):
    """Power-of-two Step and 1/s and small-integer operands: dW = W~/s - W is exact in 16 bits and both
    GEMMs are exact in binary32, so every output must agree with the oracle to binary64 rounding for
    every bit-width, granularity, tile and chunk shape."""
    seed = N + C_in + bits
    rng = np.random.default_rng(seed)
    glen = {orc.PER_ROW: C_in, orc.PER_TENSOR: C_out * C_in, orc.PER_GROUP: group}[gran]
    npairs = C_out * C_in // glen
    step = (2.0 ** rng.integers(-1, 1, npairs)).astype(np.float32)                # 0.5 or 1
    zp = rng.integers(0, 1 << bits, npairs).astype(np.int32)
    # codes within 12 of their zero-point: |W~ / s - W| <= 15 in quarters, exact even in bf16
    q = np.clip(np.repeat(zp, glen).reshape(C_out, C_in) + rng.integers(-12, 13, (C_out, C_in)), 0, (1 << bits) - 1)
    codes = orc.pack(q.astype(np.int32), bits)
    rinv = (2.0 ** rng.integers(-1, 1, C_in)).astype(np.float32)                  # 0.5 or 1
    X = _int_valued((N, C_in), dtype, seed + 2, 3)
    W = _int_valued((C_out, C_in), dtype, seed + 3, 3)
    bias = _int_valued((C_out,), dtype, seed + 4, 5)
    bias_q = rng.standard_normal(C_out).astype(np.float32)
    got_me, got_s = _run_weights(codes, step, zp, bits, gran, group, rinv, bias_q, X, W, bias)
    ref_me, ref_s = orc.forward_check_weights(codes, step, zp, bits, gran, group, rinv, bias_q, util.bits(X), util.bits(W),
                                              util.odt(X), util.bits(bias))
    rms = np.sqrt(ref_s[0] / ref_s[3])
    assert np.all(np.abs(got_me - ref_me) <= 1e-11 * rms)
    assert np.allclose(got_s, ref_s, rtol=1e-11, atol=0)


@pytest.mark.parametrize("dtype,bits,gran,group", [(torch.bfloat16, 4, orc.PER_GROUP, 128), (torch.bfloat16, 3, orc.PER_GROUP, 128),
                                                   (torch.float16, 8, orc.PER_ROW, 0)])
@pytest.mark.parametrize("correct", [True, False])
def test_forward_check_weights_of_a_calibrated_layer(dtype, bits, gran, group, correct):
    """Oracle calibration (steps 1-5) feeds both sides.  The mean error is E[x] . dW with dW = W~/s - W
    in binary32 (three roundings) and binary64 column sums: tight.  For the sums of squares the GPU
    rounds dW to 16 bits (relative 2^-m, m = 9 for bf16 and 12 for fp16) and accumulates both GEMMs
    in binary32 (K 2^-23 of the absolute sum): the bound below, per output."""
    N, C_in, C_out = 1536 + 40, 768, 512 + 8
    Xc = util.rand16((N, C_in), dtype, 61, scale=1.0, offset=0.5, outlier_cols=4)
    Wc = util.rand16((C_out, C_in), dtype, 62, scale=0.03)
    bias = util.rand16((1, C_out), dtype, 63, scale=0.1)[0].contiguous()
    cal = util.oracle_layer(Xc, [Wc], bits, gran, group, biases=[bias], act_quant=False)
    lin, f = cal["linears"][0], cal["factors"]
    dt = util.odt(Xc)
    bias_q = lin["bias_f32"] if correct else None
    got_me, got_s = _run_weights(lin["codes"], lin["step"], lin["zp"], bits, gran, group, f["rinv"], bias_q, Xc, Wc, bias)
    ref_me, ref_s = orc.forward_check_weights(lin["codes"], lin["step"], lin["zp"], bits, gran, group, f["rinv"], bias_q,
                                              util.bits(Xc), util.bits(Wc), dt, util.bits(bias))
    Wq = orc.dequantize(lin["codes"], lin["step"], lin["zp"], C_in, bits, gran, group) * f["rinv"].astype(np.float64)[None, :]
    W64 = Wc.double().numpy()
    Xa = np.abs(Xc.double().numpy())
    m = 9 if dtype == torch.bfloat16 else 12
    e_w = 2.0 ** -m * np.abs(Wq - W64) + 3 * 2.0 ** -24 * (np.abs(Wq) + np.abs(W64))      # rounding of dW
    bound = Xa @ e_w.T + C_in * 2.0 ** -23 * (Xa @ (np.abs(Wq - W64) + e_w).T)           # d, per output
    mu = np.abs(Xc.double().numpy().mean(axis=0))
    me_tol = mu @ (3 * 2.0 ** -24 * (np.abs(Wq) + np.abs(W64)) + 1e-8 * np.abs(Wq - W64)).T + 1e-12
    assert np.all(np.abs(got_me - ref_me) <= me_tol)
    e2 = (bound ** 2).sum()
    assert abs(got_s[0] - ref_s[0]) <= 2 * np.sqrt(ref_s[0] * e2) + e2
    ybound = C_in * 2.0 ** -23 * (Xa @ np.abs(W64).T)
    y2 = (ybound ** 2).sum()
    assert abs(got_s[1] - ref_s[1]) <= 2 * np.sqrt(ref_s[1] * y2) + y2
    assert got_s[3] == ref_s[3]
    # in practice: the means agree to 1e-5 of the error's RMS, the mean squared error to 1e-3
    d_rms = np.sqrt(ref_s[0] / ref_s[3])
    assert np.abs(got_me - ref_me).max() <= 1e-5 * d_rms
    assert abs(got_s[0] - ref_s[0]) <= 1e-3 * ref_s[0]
    if correct:
        assert np.abs(ref_me).max() < 1e-3 * np.abs(lin["delta"]).max() + 1e-7      # Eq. 15 removed the mean error


def test_forward_check_layer_sized_sampled_channels():
    """A LLaMA-13B-sized projection (5120 x 5120) on four token chunks, calibrated by the oracle; the
    oracle then evaluates a sample of output channels (a forward check of those rows of W alone),
    which must match the same channels of the full GPU check."""
    N, C = 3 * 16384 + 24, 5120
    Xc = util.rand16((N, C), torch.float16, 71, scale=1.0, offset=0.5, outlier_cols=26, outlier_scale=80.0)
    Wc = util.rand16((C, C), torch.float16, 72, scale=0.015)
    cal = util.oracle_layer(Xc, [Wc], 8, orc.PER_ROW, 0)
    lin, (Xq, act_step, act_zp) = cal["linears"][0], cal["act"]
    got_me, got_s = _run(Xq, act_step, act_zp, lin["codes"], lin["step"], lin["zp"], lin["bias_f32"], Xc, Wc, None)
    rows = np.array([0, 1234, 2559, 5119])
    ref_me, ref_s = orc.forward_check(Xq, act_step, act_zp, lin["codes"][rows], lin["step"][rows], lin["zp"][rows],
                                      lin["bias_f32"][rows], util.bits(Xc), util.bits(Wc[rows].contiguous()), orc.F16)
    y_rms = np.sqrt(ref_s[1] / ref_s[3])
    assert np.abs(got_me[rows] - ref_me).max() <= 1e-5 * y_rms
    assert got_s[3] == N * C
    # the sampled channels carry their share of the sums (the layer is statistically uniform over channels)
    assert 0.5 < (got_s[0] / C) / (ref_s[0] / len(rows)) < 2.0
    # weight-only check of the same layer at 4 bits, same sample
    cal4 = util.oracle_layer(Xc, [Wc], 4, orc.PER_GROUP, 128, act_quant=False)
    l4, f4 = cal4["linears"][0], cal4["factors"]
    got4, s4 = _run_weights(l4["codes"], l4["step"], l4["zp"], 4, orc.PER_GROUP, 128, f4["rinv"], l4["bias_f32"], Xc, Wc, None)
    ng = C // 128
    pick = (rows[:, None] * ng + np.arange(ng)[None, :]).reshape(-1)
    ref4, r4 = orc.forward_check_weights(l4["codes"][rows], l4["step"][pick], l4["zp"][pick], 4, orc.PER_GROUP, 128, f4["rinv"],
                                         l4["bias_f32"][rows], util.bits(Xc), util.bits(Wc[rows].contiguous()), orc.F16)
    d_rms = np.sqrt(r4[0] / r4[3])
    assert np.abs(got4[rows] - ref4).max() <= 1e-5 * d_rms
    assert 0.5 < (s4[0] / C) / (r4[0] / len(rows)) < 2.0
