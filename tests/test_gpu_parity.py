"""Element-by-element parity of the CUDA library (through its C ABI) with the
CPU oracle on the same seeded inputs.  Integer outputs (codes, zero-points,
packed bytes) and exact statistics (min / max, Step) must be identical; means,
factors and corrected biases must agree within the stated tolerances."""
import numpy as np
import pytest
import torch

from oracle import aweq_oracle as orc
from tests import util

pytestmark = pytest.mark.gpu

aweq = None


@pytest.fixture(scope="module", autouse=True)
def _lib():
    global aweq
    from paper_2311_01305_b200 import aweq as _a
    aweq = _a
    yield


DEV = "cuda"


def dev_stats(X, N=None):
    C = X.shape[1]
    n = X.shape[0] if N is None else N
    xmin, g1 = util.guarded((C,), torch.float32)
    xmax, g2 = util.guarded((C,), torch.float32)
    xmean, g3 = util.guarded((C,), torch.float32)
    xsum, g4 = util.guarded((C,), torch.float64)
    ws = aweq.workspace(aweq.workspace_bytes(aweq.OP_STATS, n, C))
    st = aweq.new_status()
    aweq.aweq_stats(X, xmin, xmax, xmean, xsum=xsum, ws=ws, st=st, N=N)
    torch.cuda.synchronize()
    for g in (g1, g2, g3, g4):
        g()
    return xmin.cpu().numpy(), xmax.cpu().numpy(), xmean.cpu().numpy(), xsum.cpu().numpy(), aweq.read_status(st)


# ------------------------------------------------------------------ step 1
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("shape", [(1, 8), (7, 8), (257, 24), (1000, 768), (2048, 768), (4099, 2056),
                                   (333, 11008), (9000, 4096), (70, 36864),
                                   # the wider CTAs (320 / 384 consumer threads): exact fits and ragged slabs, and rows of
                                   # three or more slabs (three stages)
                                   (3001, 3072), (1777, 5120), (1500, 2824), (700, 4808), (900, 5608), (600, 9216),
                                   (650, 13824)])
def test_stats_matches_oracle(shape, dtype):
    Xc = util.rand16(shape, dtype, seed=shape[0] * 31 + shape[1], offset=2.0, outlier_cols=min(6, shape[1] // 4))
    o_min, o_max, o_mean, o_sum = orc.stats(util.bits(Xc), util.odt(Xc))
    xmin, xmax, xmean, xsum, st = dev_stats(Xc.to(DEV))
    util.assert_same_values(xmin, o_min, "xmin")
    util.assert_same_values(xmax, o_max, "xmax")
    mean_abs = np.abs(Xc.double().numpy()).mean(axis=0)
    assert np.all(np.abs(xmean.astype(np.float64) - o_mean) <= util.mean_tolerance(o_mean, mean_abs))
    assert np.allclose(xsum, o_sum, rtol=0, atol=1e-6 * 1e-3 * mean_abs.max() * shape[0])
    assert st == {"nonfinite": 0, "zero_range": 0, "wait_timeout": 0}


def test_stats_row_pitch_and_determinism():
    big = util.rand16((3000, 1024 + 64), torch.float16, seed=5, offset=1.0).to(DEV)
    X = big[:, 32:32 + 1024][:, :1016]          # pitch 1088, 1016 columns, base offset 64 bytes
    assert X.data_ptr() % 16 == 0
    o = orc.stats(util.bits(X), orc.F16)
    a = dev_stats(X)
    b = dev_stats(X)
    util.assert_same_values(a[0], o[0])
    util.assert_same_values(a[1], o[1])
    for u, v in zip(a[:4], b[:4]):
        assert np.array_equal(u.view(np.uint8), v.view(np.uint8))    # bit-reproducible


def test_stats_streamed_in_chunks_equals_one_shot():
    Xc = util.rand16((5000, 520), torch.bfloat16, seed=11, offset=3.0)
    X = Xc.to(DEV)
    C = X.shape[1]
    xmin = torch.empty(C, device=DEV); xmax = torch.empty(C, device=DEV); xmean = torch.empty(C, device=DEV)
    xsum = torch.empty(C, dtype=torch.float64, device=DEV)
    count = torch.zeros(1, dtype=torch.int64, device=DEV)
    ws = aweq.workspace(aweq.workspace_bytes(aweq.OP_STATS, 5000, C))
    cuts = [0, 1203, 1203, 4000, 5000]           # includes an empty chunk
    for i in range(len(cuts) - 1):
        chunk = X[cuts[i]:cuts[i + 1]]
        if chunk.shape[0] == 0:
            aweq.aweq_stats(X[:1], xmin, xmax, xmean, xsum=xsum, count=count, accumulate=i > 0, ws=ws, N=0)
        else:
            aweq.aweq_stats(chunk, xmin, xmax, xmean, xsum=xsum, count=count, accumulate=i > 0, ws=ws)
    torch.cuda.synchronize()
    o_min, o_max, o_mean, o_sum = orc.stats(util.bits(Xc), orc.BF16)
    assert int(count.item()) == 5000
    util.assert_same_values(xmin.cpu().numpy(), o_min)
    util.assert_same_values(xmax.cpu().numpy(), o_max)
    mean_abs = np.abs(Xc.double().numpy()).mean(axis=0)
    assert np.all(np.abs(xmean.cpu().numpy().astype(np.float64) - o_mean) <= util.mean_tolerance(o_mean, mean_abs))


def test_stats_extreme_values():
    # largest finite values, subnormals, signed zeros, constant and one-sided columns
    N, C = 64, 16
    v = torch.zeros((N, C), dtype=torch.float16)
    v[:, 0] = 65504.0
    v[::2, 1] = -65504.0
    v[:, 2] = 6e-8          # subnormal
    v[::3, 3] = -0.0
    v[:, 4] = torch.linspace(1, 64, N)
    v[:, 5] = -torch.linspace(1, 64, N)
    o = orc.stats(util.bits(v), orc.F16)
    d = dev_stats(v.to(DEV))
    util.assert_same_values(d[0], o[0])
    util.assert_same_values(d[1], o[1])
    assert np.allclose(d[2], o[2], rtol=1e-6, atol=0)
    assert d[4]["nonfinite"] == 0


def test_stats_counts_nonfinite_channels():
    v = util.rand16((100, 32), torch.float16, seed=3)
    v[17, 5] = float("nan")
    v[3, 9] = float("inf")
    d = dev_stats(v.to(DEV))
    assert d[4]["nonfinite"] == 2


# ------------------------------------------------------------------ step 2
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("shape", [(768, 768), (3072, 768), (100, 4104), (4096, 11008), (5120, 5120), (64, 5608), (777, 3072)])
def test_wrange_matches_oracle_and_merges(shape, dtype):
    Wc = util.rand16(shape, dtype, seed=shape[0] + 7 * shape[1], scale=0.02)
    W = Wc.to(DEV)
    C = shape[1]
    wmin, g1 = util.guarded((C,), torch.float32)
    wmax, g2 = util.guarded((C,), torch.float32)
    ws = aweq.workspace(aweq.workspace_bytes(aweq.OP_WRANGE, shape[0], C))
    aweq.aweq_wrange(W, wmin, wmax, ws=ws)
    torch.cuda.synchronize()
    g1(); g2()
    o_min, o_max = orc.wrange(util.bits(Wc), util.odt(Wc))
    util.assert_same_values(wmin.cpu().numpy(), o_min)
    util.assert_same_values(wmax.cpu().numpy(), o_max)
    W2c = util.rand16((shape[0] // 2 + 1, C), dtype, seed=99, scale=0.03)
    ws2 = aweq.workspace(aweq.workspace_bytes(aweq.OP_WRANGE, W2c.shape[0], C))
    aweq.aweq_wrange(W2c.to(DEV), wmin, wmax, accumulate=True, ws=ws2)
    torch.cuda.synchronize()
    o2 = orc.wrange(util.bits(W2c), util.odt(W2c), prev=(o_min, o_max))
    util.assert_same_values(wmin.cpu().numpy(), o2[0])
    util.assert_same_values(wmax.cpu().numpy(), o2[1])


# ------------------------------------------------------------------ step 3
def _oracle_front(Xc, Wcs):
    xs = orc.stats(util.bits(Xc), util.odt(Xc))
    wr = None
    for Wc in Wcs:
        wr = orc.wrange(util.bits(Wc), util.odt(Wc), prev=wr)
    f = orc.factors(xs[0], xs[1], xs[2], wr[0], wr[1])
    return xs, wr, f


def dev_factors(xmin, xmax, xmean, wmin, wmax):
    C = xmin.size
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    outs = {k: torch.empty(C, device=DEV) for k in ("s", "rinv", "mu_hat", "pX", "pW")}
    scalars = torch.empty(8, dtype=torch.float64, device=DEV)
    st = aweq.new_status()
    aweq.aweq_factors(t(xmin), t(xmax), t(xmean), t(wmin), t(wmax), outs["s"], outs["rinv"], outs["mu_hat"],
                      outs["pX"], outs["pW"], scalars, st=st)
    torch.cuda.synchronize()
    r = {k: v.cpu().numpy() for k, v in outs.items()}
    r["scalars"] = scalars.cpu().numpy()
    r["status"] = aweq.read_status(st)
    return r


@pytest.mark.parametrize("C_in", [8, 768, 4096, 36864])
def test_factors_match_oracle(C_in):
    Xc = util.rand16((200, C_in), torch.float16, seed=C_in, offset=2.0, outlier_cols=min(8, C_in // 4))
    Wc = util.rand16((64, C_in), torch.float16, seed=C_in + 1, scale=0.02)
    xs, wr, f = _oracle_front(Xc, [Wc])
    d = dev_factors(xs[0], xs[1], xs[2], wr[0], wr[1])
    # Eq. 10 is evaluated in binary64 and rounded once on both sides: identical factors
    util.assert_same_values(d["s"], f["s"], "s")
    util.assert_same_values(d["rinv"], f["rinv"], "rinv")
    for k in ("pX", "pW"):
        assert np.allclose(d[k], f[k], rtol=1e-6, atol=0), k
    assert np.allclose(d["mu_hat"], f["mu_hat"], rtol=1e-6, atol=1e-12)
    assert np.allclose(d["scalars"], f["scalars"], rtol=1e-6, atol=0)
    assert d["status"]["zero_range"] == f["dead"] == 0


def test_factors_dead_channels():
    xmin = np.array([0, 1, -1, 0, -2, 0, 0, 0], np.float32)
    xmax = np.array([1, 1, 1, np.inf, 2, 1, 1, 1], np.float32)
    wmin = np.array([-1, -1, .5, -1, -1, -1, -1, -1], np.float32)
    wmax = np.array([1, 1, .5, 1, 1, 1, 1, 1], np.float32)
    f = orc.factors(xmin, xmax, np.zeros(8, np.float32), wmin, wmax)
    d = dev_factors(xmin, xmax, np.zeros(8, np.float32), wmin, wmax)
    util.assert_same_values(d["s"], f["s"])
    assert d["status"]["zero_range"] == f["dead"] == 3


# ------------------------------------------------------------------ step 4
def dev_equalize_quantize(W, s, mu, bits, gran, group):
    C_out, C_in = W.shape
    ns = 1 if gran == aweq.PER_TENSOR else (C_out if gran == aweq.PER_ROW else C_out * (C_in // group))
    codes, g1 = util.guarded((C_out, C_in * bits // 8), torch.uint8)
    step, g2 = util.guarded((ns,), torch.float32)
    zp, g3 = util.guarded((ns,), torch.int32)
    epsmu, g4 = util.guarded((C_out,), torch.float32)
    ws = aweq.workspace(aweq.workspace_bytes(aweq.OP_EQUALIZE_QUANTIZE, C_out, C_in, bits, gran, group))
    st = aweq.new_status()
    t = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    aweq.aweq_equalize_quantize(W, t(s), t(mu), bits, gran, group, codes, step, zp,
                                epsmu if mu is not None else None, ws=ws, st=st)
    torch.cuda.synchronize()
    g1(); g2(); g3()
    if mu is not None:
        g4()
    assert aweq.read_status(st)["wait_timeout"] == 0
    return codes.cpu().numpy(), step.cpu().numpy(), zp.cpu().numpy(), epsmu.cpu().numpy()


def check_weights(Xc, Wc, bits, gran, group, equalize=True):
    xs, wr, f = _oracle_front(Xc, [Wc])
    s = f["s"] if equalize else None
    mu = f["mu_hat"] if equalize else xs[2]
    o_codes, o_step, o_zp, o_delta = orc.equalize_quantize(util.bits(Wc), util.odt(Wc), s, mu, bits, gran, group)
    codes, step, zp, epsmu = dev_equalize_quantize(Wc.to(DEV), s, mu, bits, gran, group)
    util.assert_same_values(zp, o_zp, "zero-points")
    util.assert_same_values(step, o_step, "Step")
    util.assert_same_values(codes, o_codes, "packed codes")
    # eps . E[x^]: binary32 accumulation against the oracle's binary64
    Wq = orc.dequantize(o_codes, o_step, o_zp, Wc.shape[1], bits, gran, group)
    What = Wc.float().numpy() * (s[None, :] if s is not None else 1.0)
    scale = (np.abs(Wq - What) * np.abs(mu)[None, :]).sum(axis=1)
    assert np.all(np.abs(epsmu - o_delta) <= 1e-5 * scale + 1e-30)
    return (codes, step, zp, epsmu), (o_codes, o_step, o_zp, o_delta), f


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("C_out,C_in,bits", [(4, 8, 8), (33, 24, 8), (768, 768, 8), (100, 3072, 8), (300, 4096, 8),
                                             (40, 5120, 8), (20, 9216, 8), (12, 13824, 8), (9, 36864, 8), (6, 24576, 8), (5, 30720, 8), (3, 40960, 8),
                                             (64, 1032, 4), (64, 776, 3), (50, 512, 2), (31, 264, 5), (17, 520, 6),
                                             (23, 2056, 7)])
def test_equalize_quantize_per_row(C_out, C_in, bits, dtype):
    Xc = util.rand16((128, C_in), dtype, seed=C_in + bits, offset=2.0, outlier_cols=min(6, C_in // 4))
    Wc = util.rand16((C_out, C_in), dtype, seed=C_out * 3 + C_in, scale=0.02)
    check_weights(Xc, Wc, bits, aweq.PER_ROW, 0)


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("C_out,C_in,bits,group", [(300, 4096, 4, 128), (300, 4096, 3, 128), (64, 11008, 4, 128),
                                                   (64, 11008, 3, 128), (37, 768, 4, 8), (37, 776, 3, 8),
                                                   (37, 784, 3, 16), (19, 1056, 4, 32), (19, 1088, 8, 64),
                                                   (19, 2304, 2, 256), (21, 640, 5, 128), (21, 1024, 3, 256),
                                                   (1, 128, 4, 128), (7, 384, 3, 128), (9, 640, 8, 128),
                                                   (301, 4224, 4, 128), (8, 256, 3, 128), (40, 1152, 8, 128)])
def test_equalize_quantize_per_group(C_out, C_in, bits, group, dtype):
    Xc = util.rand16((128, C_in), dtype, seed=C_in + bits, offset=2.0, outlier_cols=6)
    Wc = util.rand16((C_out, C_in), dtype, seed=C_out * 3 + C_in, scale=0.02)
    check_weights(Xc, Wc, bits, aweq.PER_GROUP, group)


@pytest.mark.parametrize("bits", [8, 4, 3])
def test_equalize_quantize_per_tensor_and_rtn(bits):
    Xc = util.rand16((128, 1032), torch.float16, seed=1, offset=2.0, outlier_cols=6)
    Wc = util.rand16((77, 1032), torch.float16, seed=2, scale=0.02)
    check_weights(Xc, Wc, bits, aweq.PER_TENSOR, 0)
    check_weights(Xc, Wc, bits, aweq.PER_ROW, 0, equalize=False)
    check_weights(Xc, Wc, bits, aweq.PER_GROUP, 8, equalize=False)
    W2 = util.rand16((45, 1408), torch.bfloat16, seed=3, scale=0.02)
    X2 = util.rand16((64, 1408), torch.bfloat16, seed=4, offset=2.0, outlier_cols=6)
    check_weights(X2, W2, bits, aweq.PER_GROUP, 128, equalize=False)


@pytest.mark.parametrize("bits,gran,group", [(4, 2, 128), (3, 2, 128), (8, 1, 0), (4, 2, 32)])
def test_equalize_quantize_row_pitch(bits, gran, group):
    """W as a column slice of a wider matrix (row pitch larger than C_in)."""
    big = util.rand16((70, 1160), torch.bfloat16, seed=31, scale=0.02).to(DEV)
    W = big[:, 8:8 + 1024]
    s = (torch.rand(1024, generator=torch.Generator().manual_seed(2)) + 0.5).numpy()
    mu = (torch.randn(1024, generator=torch.Generator().manual_seed(3)) * 0.2).numpy()
    o = orc.equalize_quantize(util.bits(W), orc.BF16, s, mu, bits, gran, group)
    d = dev_equalize_quantize(W, s, mu, bits, gran, group)
    util.assert_same_values(d[2], o[2], "zero-points")
    util.assert_same_values(d[1], o[1], "Step")
    util.assert_same_values(d[0], o[0], "codes")


def test_equalize_quantize_degenerate_rows():
    C_in = 256
    W = torch.randn((12, C_in), generator=torch.Generator().manual_seed(4)) * 0.02
    W[0] = 0.25                       # constant row
    W[1] = 0.0                        # all zero
    W[2] = W[2].abs() + 1.0           # all positive: negative zero-point
    W[3] = -W[3].abs() - 1.0          # all negative: zero-point above qmax
    W[4] = 65504.0
    W[4, ::2] = -65504.0              # full fp16 range
    W[5] = 6e-8                       # subnormal constant
    W[6, :128] = 1000.0               # tiny spread on a large offset: huge zero-point
    W[6, 128:] = 1000.5
    W[7, 0] = 30000.0                 # one outlier
    Wc = W.to(torch.float16)
    Xc = util.rand16((64, C_in), torch.float16, seed=8, offset=1.0)
    for bits, gran, group in [(8, aweq.PER_ROW, 0), (4, aweq.PER_GROUP, 128), (3, aweq.PER_GROUP, 32)]:
        check_weights(Xc, Wc, bits, gran, group, equalize=False)
        check_weights(Xc, Wc, bits, gran, group, equalize=True)


def test_equalize_quantize_int32_saturation():
    """The hand-worked saturation cases of the quantiser (a tiny spread on a huge offset; the
    zero-point or the rounded values leave the int32 range) through step 4: 16-bit ones times
    factors that carry the values, so that W^ = s exactly."""
    cases = [([8421504.0, 8421505.0], -2147483392, [0, 255]), ([8421505.0, 8421506.0], -2147483648, [0, 0]),
             ([2.0 ** 41 - 2.0 ** 17, 2.0 ** 41], -2147483648, [0, 0])]
    for dtype in (torch.float16, torch.bfloat16):
        for C_in in (8, 264, 384):
            Wc = torch.ones((2, C_in), dtype=dtype)
            Wc[1] = -1.0                                       # the mirrored row: Z above the range
            for vals, zp_want, codes_want in cases:
                s = np.array([vals[j % 2] for j in range(C_in)], np.float32)
                mu = np.zeros(C_in, np.float32)
                o = orc.equalize_quantize(util.bits(Wc), util.odt(Wc), s, mu, 8, orc.PER_ROW)
                d = dev_equalize_quantize(Wc.to(DEV), s, mu, 8, aweq.PER_ROW, 0)
                util.assert_same_values(d[2], o[2], "zero-points")
                util.assert_same_values(d[1], o[1], "Step")
                util.assert_same_values(d[0], o[0], "codes")
                assert d[2][0] == zp_want and d[0][0, :2].tolist() == codes_want
                if vals[0] == 8421505.0:
                    assert d[2][1] == 2147483647 and not d[0][1].any()
                if C_in % 128 == 0:                            # the same through the group quantiser
                    o = orc.equalize_quantize(util.bits(Wc), util.odt(Wc), s, mu, 8, orc.PER_GROUP, 128)
                    d = dev_equalize_quantize(Wc.to(DEV), s, mu, 8, aweq.PER_GROUP, 128)
                    util.assert_same_values(d[2], o[2], "zero-points")
                    util.assert_same_values(d[1], o[1], "Step")
                    util.assert_same_values(d[0], o[0], "codes")
                    assert d[2][0] == zp_want and d[0][0, :2].tolist() == codes_want


def _nan_vector_mask(t16: torch.Tensor, bits: int) -> np.ndarray:
    """True for the packed bytes that hold codes of a 16-byte input vector containing a NaN
    (eight columns = `bits` bytes); rows must be whole vectors."""
    nan = torch.isnan(t16.float()).numpy()
    vec = nan.reshape(nan.shape[0], -1, 8).any(axis=2)
    return np.repeat(vec, bits, axis=1)


@pytest.mark.parametrize("gran,group,bits", [(1, 0, 8), (2, 128, 4), (2, 128, 3), (2, 32, 4)])
def test_equalize_quantize_nonfinite_inputs(gran, group, bits):
    """Inf / NaN elements injected on the host.  Infinite elements: every code, Step and
    zero-point equals the oracle's.  NaN elements: the extremes ignore them on both sides, so
    Step, Z and all codes outside the NaN's own 16-byte vector equal the oracle's."""
    C_out, C_in = 24, 512
    W = torch.randn((C_out, C_in), generator=torch.Generator().manual_seed(77)) * 0.02
    W[1, 5] = float("inf")
    W[2, 130] = float("-inf")
    W[4, 0] = float("inf"); W[4, 300] = float("-inf")
    W[6, 128:256] = float("inf")
    s = (torch.rand(C_in, generator=torch.Generator().manual_seed(78)) + 0.5).numpy()
    for with_nan in (False, True):
        if with_nan:
            W[3, 7] = float("nan")
            W[5, 511] = float("nan"); W[5, 256] = float("inf")
        Wc = W.to(torch.float16)
        o = orc.equalize_quantize(util.bits(Wc), orc.F16, s, None, bits, gran, group)
        d = dev_equalize_quantize(Wc.to(DEV), s, None, bits, gran, group)
        util.assert_same_values(d[2], o[2], "zero-points")
        util.assert_same_values(d[1], o[1], "Step")
        keep = ~_nan_vector_mask(Wc, bits)
        assert keep.all() != with_nan
        util.assert_same_values(d[0][keep], o[0][keep], "codes")


# ------------------------------------------------------------------ step 5
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("bits,gran,group", [(8, 1, 0), (4, 2, 128), (3, 2, 128), (4, 0, 0)])
def test_bias_correct_both_routes(bits, gran, group, dtype):
    C_out, C_in = 96, 1024
    Xc = util.rand16((256, C_in), dtype, seed=21, offset=3.0, outlier_cols=6)
    Wc = util.rand16((C_out, C_in), dtype, seed=22, scale=0.02)
    bias_c = util.rand16((1, C_out), dtype, seed=23, scale=0.1)[0]
    (codes, step, zp, epsmu), (o_codes, o_step, o_zp, o_delta), f = check_weights(Xc, Wc, bits, gran, group)
    o_f32, o_16 = orc.bias_correct(o_delta, util.bits(bias_c), util.odt(bias_c))
    dt = aweq.F16 if dtype == torch.float16 else aweq.BF16
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    for route in ("fused", "standalone"):
        for with_bias in (True, False):
            b16, g1 = util.guarded((C_out,), dtype)
            b32, g2 = util.guarded((C_out,), torch.float32)
            bin_ = bias_c.to(DEV) if with_bias else None
            if route == "fused":
                aweq.aweq_bias_correct(t(epsmu), None, None, None, None, None, None, bits, gran, group, bin_, b16,
                                       b32, dt)
            else:
                aweq.aweq_bias_correct(None, Wc.to(DEV), t(f["s"]), t(o_codes), t(o_step), t(o_zp), t(f["mu_hat"]),
                                       bits, gran, group, bin_, b16, b32, dt)
            torch.cuda.synchronize()
            g1(); g2()
            ref32 = o_f32 if with_bias else orc.bias_correct(o_delta, None, util.odt(bias_c))[0]
            ref16 = o_16 if with_bias else orc.bias_correct(o_delta, None, util.odt(bias_c))[1]
            assert np.allclose(b32.cpu().numpy(), ref32, rtol=0, atol=1e-5)
            util.check_bias16(b16, b32, ref16)


# ------------------------------------------------------------------ step 6
def dev_quant_act(X, rinv, bits, gran, lo_hi=None):
    N, C = X.shape
    Xq, g1 = util.guarded((N, C), torch.uint8)
    ns = N if gran == aweq.PER_ROW else 1
    step, g2 = util.guarded((ns,), torch.float32)
    zp, g3 = util.guarded((ns,), torch.int32)
    st = aweq.new_status()
    t = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    aweq.aweq_quant_act(X, t(rinv), bits, gran, t(lo_hi), Xq, step, zp, st=st)
    torch.cuda.synchronize()
    g1(); g2(); g3()
    assert aweq.read_status(st)["wait_timeout"] == 0
    return Xq.cpu().numpy(), step.cpu().numpy(), zp.cpu().numpy()


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("N,C_in", [(1, 8), (5, 24), (2048, 768), (1000, 3072), (777, 4096), (300, 5120),
                                    (130, 9216), (129, 11008), (65, 13824), (33, 36864), (20, 40960),
                                    (70, 10248), (41, 20488), (1, 13824), (23, 24576), (9, 24568), (7, 36872), (5, 24584), (14, 32768), (1, 36864),
                                    # plain-load teams with the next row in flight: every team size at its widest and just past it,
                                    # a row count below the number of teams, a width just past the eight-warp teams
                                    (3000, 1536), (2500, 1544), (3, 768), (600, 3080), (400, 6144), (350, 6152),
                                    (200, 12288), (2, 12288), (100, 12296)])
def test_quant_act_per_token(N, C_in, dtype):
    Xc = util.rand16((N, C_in), dtype, seed=N + C_in, offset=1.0, outlier_cols=min(6, C_in // 4))
    Wc = util.rand16((16, C_in), dtype, seed=5, scale=0.02)
    _, _, f = _oracle_front(Xc, [Wc])
    for rinv in (f["rinv"], None):
        o = orc.quant_act(util.bits(Xc), util.odt(Xc), rinv, orc.PER_ROW)
        d = dev_quant_act(Xc.to(DEV), rinv, 8, aweq.PER_ROW)
        util.assert_same_values(d[2], o[2], "zero-points")
        util.assert_same_values(d[1], o[1], "Step")
        util.assert_same_values(d[0], o[0], "codes")


def test_quant_act_row_pitch_and_low_bits():
    big = util.rand16((500, 1104), torch.float16, seed=9, offset=1.0).to(DEV)
    X = big[:, 8:8 + 1024]
    rinv = (torch.rand(1024, generator=torch.Generator().manual_seed(1)) + 0.5).numpy()
    for bits in (8, 4):
        o = orc.quant_act(util.bits(X), orc.F16, rinv, orc.PER_ROW, bits=bits)
        d = dev_quant_act(X, rinv, bits, aweq.PER_ROW)
        for a, b in zip(d, o):
            util.assert_same_values(a, b)


def test_quant_act_static_per_tensor_range():
    Xc = util.rand16((300, 1032), torch.float16, seed=13, offset=1.0, outlier_cols=4)
    Wc = util.rand16((16, 1032), torch.float16, seed=14, scale=0.02)
    xs, _, f = _oracle_front(Xc, [Wc])
    lo_hi = np.array([(xs[0] * f["rinv"]).min(), (xs[1] * f["rinv"]).max()], np.float32)
    o = orc.quant_act(util.bits(Xc), orc.F16, f["rinv"], orc.PER_TENSOR, lo_hi)
    d = dev_quant_act(Xc.to(DEV), f["rinv"], 8, aweq.PER_TENSOR, lo_hi)
    for a, b in zip(d, o):
        util.assert_same_values(a, b)
    # a static range narrower than the data: both clamps fire
    lo_hi2 = (lo_hi * 0.25).astype(np.float32)
    o = orc.quant_act(util.bits(Xc), orc.F16, f["rinv"], orc.PER_TENSOR, lo_hi2)
    d = dev_quant_act(Xc.to(DEV), f["rinv"], 8, aweq.PER_TENSOR, lo_hi2)
    for a, b in zip(d, o):
        util.assert_same_values(a, b)
    assert (o[0] == 0).sum() > 10 and (o[0] == 255).sum() > 10


def test_quant_act_degenerate_rows():
    C = 512
    X = torch.randn((8, C), generator=torch.Generator().manual_seed(3))
    X[0] = 3.0
    X[1] = 0.0
    X[2] = X[2].abs() + 5
    X[3] = -X[3].abs() - 5
    X[4, :256] = 2000.0
    X[4, 256:] = 2001.0
    X[5] = 65504.0
    X[5, 1::2] = -65504.0
    Xc = X.to(torch.float16)
    o = orc.quant_act(util.bits(Xc), orc.F16, None, orc.PER_ROW)
    d = dev_quant_act(Xc.to(DEV), None, 8, aweq.PER_ROW)
    for a, b in zip(d, o):
        util.assert_same_values(a, b)


@pytest.mark.parametrize("C", [2304, 5120, 13824, 36864, 40960])
def test_quant_act_wide_degenerate_rows_and_pitch(C):
    """The degenerate rows of the narrow test at the widths of the larger teams (one warp with nine
    vectors, four, eight and sixteen warps, the cluster pair), inside a wider allocation (row pitch
    C + 64), with a factor vector: constant and zero rows, one-sided rows, a row whose top rounds past
    2^b - 1 (the literal path), the largest finite values, and rows with Inf."""
    g = torch.Generator().manual_seed(17)
    X = torch.randn((11, C + 64), generator=g)
    X[0] = 3.0
    X[1] = 0.0
    X[2] = X[2].abs() + 5
    X[3] = -X[3].abs() - 5
    X[4, :C // 2] = 2000.0
    X[4, C // 2:] = 2001.0
    X[5] = 65504.0
    X[5, 1::2] = -65504.0
    X[6, C - 1] = 300.0                       # the extreme sits in the last vector of the row
    X[7, 0] = -300.0                          # ... and in the first
    X[8, C // 2 + 3] = float("inf")
    X[9, 5] = float("-inf")
    big = X.to(torch.float16).to(DEV)
    Xv = big[:, :C]
    assert Xv.stride(0) == C + 64
    rinv = (torch.rand(C, generator=g) + 0.5).numpy()
    o = orc.quant_act(util.bits(Xv), orc.F16, rinv, orc.PER_ROW)
    d = dev_quant_act(Xv, rinv, 8, aweq.PER_ROW)
    util.assert_same_values(d[2], o[2], "zero-points")
    util.assert_same_values(d[1], o[1], "Step")
    util.assert_same_values(d[0], o[0], "codes")


def test_quant_act_int32_saturation_and_nonfinite():
    """Step 6 on the hand-worked saturation cases (ones times 1/s values that carry the data)
    and on rows with Inf / NaN elements: the oracle's numbers, element by element."""
    C = 520
    Xc = torch.ones((4, C), dtype=torch.float16)
    Xc[3] = -1.0
    for vals, zp_want, codes_want in [([8421504.0, 8421505.0], -2147483392, [0, 255]),
                                      ([8421505.0, 8421506.0], -2147483648, [0, 0])]:
        rinv = np.array([vals[j % 2] for j in range(C)], np.float32)
        o = orc.quant_act(util.bits(Xc), orc.F16, rinv, orc.PER_ROW)
        d = dev_quant_act(Xc.to(DEV), rinv, 8, aweq.PER_ROW)
        for a, b in zip(d, o):
            util.assert_same_values(a, b)
        assert d[2][0] == zp_want and d[0][0, :2].tolist() == codes_want
    assert d[2][3] == 2147483647 and not d[0][3].any()
    X = torch.randn((6, C), generator=torch.Generator().manual_seed(5))
    X[1, 9] = float("inf")
    X[2, 100] = float("-inf")
    X[5, 0] = float("inf"); X[5, 519] = float("-inf")
    for with_nan in (False, True):
        if with_nan:
            X[3, 3] = float("nan")
            X[4, 0] = float("inf"); X[4, 519] = float("nan")
        Xc = X.to(torch.float16)
        o = orc.quant_act(util.bits(Xc), orc.F16, None, orc.PER_ROW)
        d = dev_quant_act(Xc.to(DEV), None, 8, aweq.PER_ROW)
        util.assert_same_values(d[2], o[2], "zero-points")
        util.assert_same_values(d[1], o[1], "Step")
        keep = ~_nan_vector_mask(Xc, 8)
        util.assert_same_values(d[0][keep], o[0][keep], "codes")


# ------------------------------------------------------------------ host-side validation (no fault, an error code)
def test_bad_arguments_are_error_codes():
    X = torch.zeros((16, 64), dtype=torch.float16, device=DEV)
    out = torch.empty(64, device=DEV)
    ws = aweq.workspace(aweq.workspace_bytes(aweq.OP_STATS, 16, 64))
    with pytest.raises(aweq.AweqError) as e:
        aweq.aweq_stats(X, out, out, out, ws=None)
    assert e.value.code == 7
    with pytest.raises(aweq.AweqError) as e:
        aweq.aweq_stats(X[:, :60], out, out, out, ws=ws)        # 60 columns: not a multiple of 8
    assert e.value.code == 2
    with pytest.raises(aweq.AweqError) as e:
        aweq.aweq_stats(X[:, 4:12], out, out, out, ws=ws)       # base pointer 8-byte aligned only
    assert e.value.code == 3
    codes = torch.empty((16, 64), dtype=torch.uint8, device=DEV)
    step = torch.empty(16, device=DEV); zp = torch.empty(16, dtype=torch.int32, device=DEV)
    with pytest.raises(aweq.AweqError) as e:
        aweq.aweq_equalize_quantize(X, None, None, 9, aweq.PER_ROW, 0, codes, step, zp)
    assert e.value.code == 5
    with pytest.raises(aweq.AweqError) as e:
        aweq.aweq_equalize_quantize(X, None, None, 4, aweq.PER_GROUP, 48, codes, step, zp)
    assert e.value.code == 6
    with pytest.raises(aweq.AweqError) as e:
        aweq.aweq_quant_act(X, None, 8, aweq.PER_TENSOR, None, codes, step, zp)
    assert e.value.code == 1


def test_factors_absmax_criterion_matches_oracle():
    Xc = util.rand16((300, 1032), torch.float16, seed=21, offset=2.0, outlier_cols=5)
    Wc = util.rand16((64, 1032), torch.float16, seed=22, scale=0.02)
    xs = orc.stats(util.bits(Xc), orc.F16)
    wr = orc.wrange(util.bits(Wc), orc.F16)
    f = orc.factors(xs[0], xs[1], xs[2], wr[0], wr[1], orc.ABSMAX)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    C = 1032
    o = {k: torch.empty(C, device=DEV) for k in ("s", "rinv", "mu", "pX", "pW")}
    sc = torch.empty(8, dtype=torch.float64, device=DEV)
    aweq.aweq_factors_absmax(t(xs[0]), t(xs[1]), t(xs[2]), t(wr[0]), t(wr[1]), o["s"], o["rinv"], o["mu"], o["pX"], o["pW"], sc)
    torch.cuda.synchronize()
    util.assert_same_values(o["s"].cpu().numpy(), f["s"], "s")
    util.assert_same_values(o["rinv"].cpu().numpy(), f["rinv"], "rinv")
    assert np.allclose(o["mu"].cpu().numpy(), f["mu_hat"], rtol=1e-6, atol=1e-12)
    assert np.allclose(o["pX"].cpu().numpy(), f["pX"], rtol=1e-6) and np.allclose(sc.cpu().numpy(), f["scalars"], rtol=1e-6)
    g = orc.factors(xs[0], xs[1], xs[2], wr[0], wr[1])
    assert not np.array_equal(f["s"], g["s"])                 # offset data: the two criteria differ
