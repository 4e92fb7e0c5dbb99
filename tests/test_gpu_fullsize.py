"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The inputs are drawn on the GPU with the seeded generators (the 16-bit values
are the canonical input); the oracle cannot sweep 10^9 elements in seconds, so
it recomputes sampled outputs one by one from the same bits:
  * statistics: every output of a sample of channels (whole columns of X are
    copied back), including the outlier channels;
  * factors: Eq. 10 for the sampled channels from oracle statistics and oracle
    weight ranges of those channels;
  * weight and activation quantisers: whole sampled rows, with a seeded factor
    vector handed to both sides (codes, Step and zero-points are functions of
    one row and the factors only).
"""
import numpy as np
import pytest
import torch

from oracle import aweq_oracle as orc
from paper_2311_01305_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _dt(wl):
    return orc.F16 if wl.dtype == "f16" else orc.BF16


def _sample_channels(inp, seed, n=48):
    g = torch.Generator().manual_seed(seed)
    cols = torch.randperm(inp.c_in, generator=g)[:n]
    if inp.n_outliers:
        idx, _ = synth.outlier_columns(inp.c_in, inp.n_outliers, inp.outlier_scale, seed)
        cols = torch.cat([cols, idx[:8]])
    return torch.unique(cols)


def _seeded_factors(c_in, seed):
    g = torch.Generator().manual_seed(seed)
    s = torch.exp(torch.randn(c_in, generator=g) * 0.7).float()
    mu = (torch.randn(c_in, generator=g) * 0.3).float()
    return s, (1.0 / s).float(), mu


def check_stats_and_factors(wl, inp_index, X, Ws, lins):
    from paper_2311_01305_b200 import aweq
    inp = wl.inputs[inp_index]
    C = inp.c_in
    o = {k: torch.empty(C, device=DEV) for k in ("xmin", "xmax", "xmean", "wmin", "wmax", "s", "rinv", "mu")}
    ws = aweq.workspace(max(aweq.workspace_bytes(aweq.OP_STATS, X.shape[0], C),
                            max(aweq.workspace_bytes(aweq.OP_WRANGE, W.shape[0], C) for W in Ws)))
    st = aweq.new_status()
    aweq.aweq_stats(X, o["xmin"], o["xmax"], o["xmean"], ws=ws, st=st)
    for i, W in enumerate(Ws):
        aweq.aweq_wrange(W, o["wmin"], o["wmax"], accumulate=i > 0, ws=ws, st=st)
    aweq.aweq_factors(o["xmin"], o["xmax"], o["xmean"], o["wmin"], o["wmax"], o["s"], o["rinv"], o["mu"], st=st)
    torch.cuda.synchronize()
    assert aweq.read_status(st) == {"nonfinite": 0, "zero_range": 0, "wait_timeout": 0}
    cols = _sample_channels(inp, synth.tensor_seed(wl.seed, 0, inp_index)).to(DEV)
    Xs = X[:, cols].contiguous().cpu()
    xs = orc.stats(util.bits(Xs), _dt(wl))
    wr = None
    for W in Ws:
        wr = orc.wrange(util.bits(W[:, cols].contiguous().cpu()), _dt(wl), prev=wr)
    f = orc.factors(xs[0], xs[1], xs[2], wr[0], wr[1])
    got = {k: v[cols].cpu().numpy() for k, v in o.items()}
    util.assert_same_values(got["xmin"], xs[0], "xmin")
    util.assert_same_values(got["xmax"], xs[1], "xmax")
    mean_abs = np.abs(Xs.double().numpy()).mean(axis=0)
    assert np.all(np.abs(got["xmean"].astype(np.float64) - xs[2]) <= util.mean_tolerance(xs[2], mean_abs))
    util.assert_same_values(got["wmin"], wr[0], "wmin")
    util.assert_same_values(got["wmax"], wr[1], "wmax")
    util.assert_same_values(got["s"], f["s"], "s")
    util.assert_same_values(got["rinv"], f["rinv"], "rinv")
    assert np.allclose(got["mu"], f["mu_hat"], rtol=1e-6, atol=1e-9 * mean_abs.max())
    # properties that hold for every channel: ordering, finiteness, equal equalised ranges
    xmin, xmax, s = o["xmin"], o["xmax"], o["s"]
    assert bool((xmin <= o["xmean"]).all()) and bool((o["xmean"] <= xmax).all())
    rx, rw = (xmax - xmin).double(), (o["wmax"] - o["wmin"]).double()
    assert bool(torch.isfinite(s).all()) and bool((s > 0).all())
    assert torch.allclose(rx / s.double(), s.double() * rw, rtol=3e-7)


def check_weight_rows(wl, W, bits, gran, group, seed, nrows=24):
    from paper_2311_01305_b200 import aweq
    C_out, C_in = W.shape
    s, _, mu = _seeded_factors(C_in, seed)
    pairs = C_out if gran == aweq.PER_ROW else C_out * (C_in // group)
    codes = torch.empty((C_out, C_in * bits // 8), dtype=torch.uint8, device=DEV)
    step = torch.empty(pairs, device=DEV)
    zp = torch.empty(pairs, dtype=torch.int32, device=DEV)
    epsmu = torch.empty(C_out, device=DEV)
    st = aweq.new_status()
    ws = aweq.workspace(aweq.workspace_bytes(aweq.OP_EQUALIZE_QUANTIZE, C_out, C_in, bits, gran, group))
    aweq.aweq_equalize_quantize(W, s.to(DEV), mu.to(DEV), bits, gran, group, codes, step, zp, epsmu, ws=ws, st=st)
    torch.cuda.synchronize()
    assert aweq.read_status(st)["wait_timeout"] == 0
    rows = torch.randperm(C_out, generator=torch.Generator().manual_seed(seed))[:nrows].sort().values
    rows = torch.unique(torch.cat([rows, torch.tensor([0, C_out - 1])]))
    Wr = W[rows.to(DEV)].cpu()
    o_codes, o_step, o_zp, o_delta = orc.equalize_quantize(util.bits(Wr), _dt(wl), s.numpy(), mu.numpy(), bits,
                                                           orc.PER_ROW if gran == aweq.PER_ROW else orc.PER_GROUP, group)
    ng = 1 if gran == aweq.PER_ROW else C_in // group
    pick = (rows[:, None] * ng + torch.arange(ng)[None, :]).reshape(-1)
    util.assert_same_values(zp.cpu()[pick].numpy(), o_zp, "zero-points")
    util.assert_same_values(step.cpu()[pick].numpy(), o_step, "Step")
    util.assert_same_values(codes[rows.to(DEV)].cpu().numpy(), o_codes, "packed codes")
    Wq = orc.dequantize(o_codes, o_step, o_zp, C_in, bits, orc.PER_ROW if gran == aweq.PER_ROW else orc.PER_GROUP, group)
    What = Wr.float().numpy() * s.numpy()[None, :]
    scale = (np.abs(Wq - What) * np.abs(mu.numpy())[None, :]).sum(axis=1)
    assert np.all(np.abs(epsmu.cpu()[rows].numpy() - o_delta) <= 1e-5 * scale + 1e-30)
    # any size: codes use the whole range of every row
    assert int(zp.min()) > -(1 << 20) and int(zp.max()) < (1 << 20)


def check_act_rows(wl, X, seed, nrows=32):
    from paper_2311_01305_b200 import aweq
    N, C = X.shape
    _, rinv, _ = _seeded_factors(C, seed)
    Xq = torch.empty((N, C), dtype=torch.uint8, device=DEV)
    step = torch.empty(N, device=DEV)
    zp = torch.empty(N, dtype=torch.int32, device=DEV)
    st = aweq.new_status()
    aweq.aweq_quant_act(X, rinv.to(DEV), 8, aweq.PER_ROW, None, Xq, step, zp, st=st)
    torch.cuda.synchronize()
    assert aweq.read_status(st)["wait_timeout"] == 0
    rows = torch.randperm(N, generator=torch.Generator().manual_seed(seed))[:nrows].sort().values
    rows = torch.unique(torch.cat([rows, torch.tensor([0, N - 1])]))
    o = orc.quant_act(util.bits(X[rows.to(DEV)].cpu()), _dt(wl), rinv.numpy(), orc.PER_ROW)
    util.assert_same_values(zp.cpu()[rows].numpy(), o[2], "zero-points")
    util.assert_same_values(step.cpu()[rows].numpy(), o[1], "Step")
    util.assert_same_values(Xq[rows.to(DEV)].cpu().numpy(), o[0], "codes")
    # any size: the minimum of every token maps to code 0 and its maximum to the top code
    # (254 when the two roundings fall on opposite sides of a tie)
    assert bool((Xq.min(dim=1).values == 0).all()) and bool((Xq.max(dim=1).values >= 254).all())


def _gen(wl, which_inputs):
    X = {i: synth.make_activations(wl.inputs[i], wl.dtype, synth.tensor_seed(wl.seed, 0, i), DEV) for i in which_inputs}
    W = {l.name: synth.make_weight(l, wl.dtype, synth.tensor_seed(wl.seed, 0, 100 + k), DEV)
         for k, l in enumerate(wl.linears)}
    return X, W


def test_llama7b_layer_full_size():
    from paper_2311_01305_b200 import aweq
    wl = synth.workloads()["llama7b_layer_w4w3_g128"]
    for i in (0, 3):                                     # attention input (q, k, v share it) and the 11008-wide input
        X, W = _gen(wl, [i])
        lins = [l for l in wl.linears if l.input == wl.inputs[i].name]
        check_stats_and_factors(wl, i, X[i], [W[l.name] for l in lins], lins)
        del X
        for bits in wl.w_bits:
            check_weight_rows(wl, W[lins[0].name], bits, aweq.PER_GROUP, wl.group, seed=7 + bits)
        del W
        torch.cuda.empty_cache()


def test_llama13b_layer_full_size():
    from paper_2311_01305_b200 import aweq
    wl = synth.workloads()["llama13b_layer_w8a8"]
    for i in (0, 3):
        X, W = _gen(wl, [i])
        lins = [l for l in wl.linears if l.input == wl.inputs[i].name]
        check_stats_and_factors(wl, i, X[i], [W[l.name] for l in lins], lins)
        check_act_rows(wl, X[i], seed=11 + i)
        del X
        check_weight_rows(wl, W[lins[0].name], 8, aweq.PER_ROW, 0, seed=13 + i)
        del W
        torch.cuda.empty_cache()


def test_opt66b_ffn_full_size():
    from paper_2311_01305_b200 import aweq
    wl = synth.workloads()["opt66b_ffn_w8a8"]
    X, W = _gen(wl, [1])                                 # the 36864-wide input: the largest rows
    lins = [l for l in wl.linears if l.input == wl.inputs[1].name]
    check_stats_and_factors(wl, 1, X[1], [W[l.name] for l in lins], lins)
    check_act_rows(wl, X[1], seed=17)
    del X
    check_weight_rows(wl, W["fc2"], 8, aweq.PER_ROW, 0, seed=19, nrows=8)
    check_weight_rows(wl, W["fc1"], 8, aweq.PER_ROW, 0, seed=23, nrows=8)
    torch.cuda.empty_cache()


def test_opt125m_model_layer_full_size():
    from paper_2311_01305_b200 import aweq
    wl = synth.workloads()["opt125m_model_w8a8"]
    for i in (0, 3):
        X, W = _gen(wl, [i])
        lins = [l for l in wl.linears if l.input == wl.inputs[i].name]
        check_stats_and_factors(wl, i, X[i], [W[l.name] for l in lins], lins)
        check_act_rows(wl, X[i], seed=29 + i)
        check_weight_rows(wl, W[lins[0].name], 8, aweq.PER_ROW, 0, seed=31 + i)
        del X, W
        torch.cuda.empty_cache()
