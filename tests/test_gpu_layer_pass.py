"""The fused layer pass (all six steps through one C-ABI call per input)
against the oracle chain: the single OPT-125M-shaped W8A8 linear at full size,
matrices that share one input, and the AWE / BC switches of the paper's
ablation (Table 4)."""
import numpy as np
import pytest
import torch

from oracle import aweq_oracle as orc
from paper_2311_01305_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make_workload_tensors(wl, device="cpu", layer=0, offset=None):
    X, W = {}, {}
    for i, inp in enumerate(wl.inputs):
        off = None if offset is None else torch.linspace(-offset, offset, inp.c_in)
        X[inp.name] = synth.make_activations(inp, wl.dtype, synth.tensor_seed(wl.seed, layer, i), device,
                                             channel_offset=off)
    for i, lin in enumerate(wl.linears):
        W[lin.name] = synth.make_weight(lin, wl.dtype, synth.tensor_seed(wl.seed, layer, 100 + i), device)
    return X, W


def compare_layer(wl, bits, Xc, Wc, bias_c=None, flags=0):
    from paper_2311_01305_b200 import aweq, calibrate
    Xd = {k: v.to(DEV) for k, v in Xc.items()}
    Wd = {k: v.to(DEV) for k, v in Wc.items()}
    bd = None if bias_c is None else {k: v.to(DEV) for k, v in bias_c.items()}
    cal = calibrate.LayerCalibrator(wl, bits, Xd, Wd, bd, flags=flags)
    n0 = aweq.launch_count()
    cal.run()
    torch.cuda.synchronize()
    assert aweq.launch_count() > n0
    assert aweq.read_status(cal.status) == {"nonfinite": 0, "zero_range": 0, "wait_timeout": 0}
    gran = orc.PER_ROW if wl.w_gran == "row" else orc.PER_GROUP
    eq = not (flags & aweq.FLAG_NO_EQUALIZE)
    bc = not (flags & aweq.FLAG_NO_BIAS_CORRECT)
    for inp in wl.inputs:
        lins = [l for l in wl.linears if l.input == inp.name]
        ref = util.oracle_layer(Xc[inp.name], [Wc[l.name] for l in lins], bits, gran, wl.group,
                                None if bias_c is None else [bias_c.get(l.name) for l in lins],
                                act_quant=wl.act_quant, equalize=eq, bias_correct=bc,
                                criterion=1 if flags & aweq.FLAG_ABSMAX_CRITERION else 0)
        o = {k: v.cpu().numpy() for k, v in cal.out[inp.name].items()}
        util.assert_same_values(o["xmin"], ref["stats"][0])
        util.assert_same_values(o["xmax"], ref["stats"][1])
        mean_abs = np.abs(Xc[inp.name].double().numpy()).mean(axis=0)
        assert np.all(np.abs(o["xmean"].astype(np.float64) - ref["stats"][2]) <= util.mean_tolerance(ref["stats"][2], mean_abs))
        util.assert_same_values(o["wmin"], ref["wrange"][0])
        util.assert_same_values(o["wmax"], ref["wrange"][1])
        f = ref["factors"]
        # Eq. 10 is evaluated in binary64 on both sides: identical factors
        util.assert_same_values(o["s"], f["s"], "s")
        util.assert_same_values(o["rinv"], f["rinv"], "rinv")
        assert np.allclose(o["mu_hat"], f["mu_hat"], rtol=1e-6, atol=1e-9 * mean_abs.max())
        assert np.allclose(o["pX"], f["pX"], rtol=1e-6) and np.allclose(o["pW"], f["pW"], rtol=1e-6)
        assert np.allclose(o["scalars"], f["scalars"], rtol=1e-6)
        for l, r in zip(lins, ref["linears"]):
            lo = {k: v.cpu() for k, v in cal.out[l.name].items()}
            util.assert_same_values(lo["zp"].numpy(), r["zp"], l.name + " zp")
            util.assert_same_values(lo["step"].numpy(), r["step"], l.name + " step")
            util.assert_same_values(lo["codes"].numpy(), r["codes"], l.name + " codes")
            if bc:
                assert np.allclose(lo["bias_f32"].numpy(), r["bias_f32"], rtol=0, atol=1e-5)
                util.check_bias16(lo["bias"], lo["bias_f32"], r["bias_16"])
        if wl.act_quant:
            util.assert_same_values(o["act_zp"], ref["act"][2], "act zp")
            util.assert_same_values(o["act_step"], ref["act"][1], "act step")
            util.assert_same_values(o["Xq"], ref["act"][0], "act codes")
    return cal


def test_opt125m_single_linear_w8a8_full_size():
    wl = synth.workloads()["opt125m_linear_w8a8"]
    Xc, Wc = make_workload_tensors(wl)
    bias = {"linear": torch.zeros(768, dtype=torch.float16)}
    compare_layer(wl, 8, Xc, Wc, bias)


def test_opt125m_single_linear_with_channel_offsets_makes_a_bias():
    wl = synth.workloads()["opt125m_linear_w8a8"]
    Xc, Wc = make_workload_tensors(wl, offset=3.0)
    cal = compare_layer(wl, 8, Xc, Wc, None)
    assert float(cal.out["linear"]["bias_f32"].abs().max()) > 1e-4


@pytest.mark.parametrize("name,bits", [("opt125m_model_w8a8", 8), ("llama7b_layer_w4w3_g128", 4),
                                       ("llama7b_layer_w4w3_g128", 3), ("llama13b_layer_w8a8", 8)])
def test_decoder_layer_shapes_with_shared_inputs_few_tokens(name, bits):
    wl = synth.workloads(n_tokens_scale=1.0 / 1024)[name]       # 256 tokens, full channel counts
    Xc, Wc = make_workload_tensors(wl, offset=1.0)
    compare_layer(wl, bits, Xc, Wc, None)


@pytest.mark.parametrize("n_w,c_in,tokens", [(5, 1032, 300), (3, 776, 37), (1, 4096, 3000), (4, 264, 1000),
                                             # the 384- and 320-thread sweeps with ragged slabs, and a three-stage ring
                                             (2, 2824, 1500), (3, 4808, 900), (2, 5608, 333), (1, 9224, 400)])
def test_matrices_sharing_one_input_fused_and_separate_ranges(n_w, c_in, tokens):
    """Up to three matrices on one input have their ranges taken inside the statistics sweep (one
    launch, the matrices as further segments of the row stack); four or more go through launches of
    their own in stacks of four.  Odd sizes: rows that are no multiple of eight, a ragged last slab."""
    from paper_2311_01305_b200 import aweq
    inputs = (synth.ActSpec("x", tokens, c_in, "normal", 0, 3, 30.0),)
    linears = tuple(synth.LinearSpec("w%d" % k, 40 + 27 * k, c_in, "x", 0.02) for k in range(n_w))
    wl = synth.Workload("custom", "bf16", 11, inputs, linears, (8,), "row", 0, True)
    Xc, Wc = make_workload_tensors(wl, offset=0.5)
    cal = compare_layer(wl, 8, Xc, Wc, None)
    assert cal.passes[0].fused_ranges == (n_w <= 3)


def test_ablation_switches():
    from paper_2311_01305_b200 import aweq
    wl = synth.workloads(n_tokens_scale=1.0 / 8)["opt125m_linear_w8a8"]
    Xc, Wc = make_workload_tensors(wl, offset=2.0)
    for flags in (aweq.FLAG_NO_EQUALIZE, aweq.FLAG_NO_BIAS_CORRECT, aweq.FLAG_NO_EQUALIZE | aweq.FLAG_NO_BIAS_CORRECT,
                  aweq.FLAG_ABSMAX_CRITERION):
        compare_layer(wl, 8, Xc, Wc, None, flags=flags)


@pytest.mark.parametrize("overlap", [False, True])
def test_sharded_path_with_one_rank_equals_fused_layer_pass(overlap):
    """The token-sharded route (the same pass with the statistics leaving the REDUCE part in
    exchange form, merged by two all-reduces and re-formed inside the QUANT part) on a one-rank
    NCCL group gives exactly what the fused layer pass gives, on one stream and on two."""
    import socket
    import torch.distributed as dist
    from paper_2311_01305_b200 import calibrate
    wl = synth.workloads(n_tokens_scale=1.0 / 256)["opt125m_model_w8a8"]
    Xc, Wc = make_workload_tensors(wl, offset=1.0)
    Xd = {k: v.to(DEV) for k, v in Xc.items()}
    Wd = {k: v.to(DEV) for k, v in Wc.items()}
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % port, rank=0, world_size=1,
                            device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        a = calibrate.LayerCalibrator(wl, 8, Xd, Wd, None)
        b = calibrate.ShardedLayerCalibrator(wl, 8, Xd, Wd, None, overlap=overlap)
        a.run(); b.run()
        torch.cuda.synchronize()
        # the exchange buffers hold what the statistics say
        C = wl.inputs[0].c_in
        o = b.out[wl.inputs[0].name]
        assert torch.equal(b.stat_negmin_max[:C], -o["xmin"]) and torch.equal(b.stat_negmin_max[C:2 * C], o["xmax"])
        assert float(b.stat_sum_count[C]) == Xd[wl.inputs[0].name].shape[0]
    finally:
        dist.destroy_process_group()
    for name, outs in a.out.items():
        for k, v in outs.items():
            assert torch.equal(v, b.out[name][k]), (name, k)


@pytest.mark.parametrize("name,scale,bits", [("opt125m_model_w8a8", 1.0 / 64, 8), ("llama7b_layer_w4w3_g128", 1.0 / 256, 4)])
def test_two_stream_schedule_equals_single_stream(name, scale, bits):
    """The pass split into its parts (column reductions and step 6 on one stream, factors and the
    weight quantiser on another, ordered by events) writes exactly what the single-stream pass writes, run after run."""
    from paper_2311_01305_b200 import aweq, calibrate
    wl = synth.workloads(n_tokens_scale=scale)[name]
    Xc, Wc = make_workload_tensors(wl, offset=1.0)
    Xd = {k: v.to(DEV) for k, v in Xc.items()}
    Wd = {k: v.to(DEV) for k, v in Wc.items()}
    a = calibrate.LayerCalibrator(wl, bits, Xd, Wd, None)
    b = calibrate.LayerCalibrator(wl, bits, Xd, Wd, None, overlap=True)
    assert b.overlap
    a.run()
    for _ in range(3):
        for outs in b.out.values():                      # poison: a stale output must not pass
            for v in outs.values():
                v.view(torch.uint8).fill_(0x5A)
        b.run()
    torch.cuda.synchronize()
    assert aweq.read_status(b.status)["wait_timeout"] == 0
    for nm, outs in a.out.items():
        for k, v in outs.items():
            assert torch.equal(v.view(torch.uint8), b.out[nm][k].view(torch.uint8)), (nm, k)
    # a single part on its own: the reduction phase leaves the other outputs alone
    lp = b.passes[0]
    first = wl.inputs[0].name
    b.out[first]["s"].fill_(-1.0)
    lp(b.ws, b.status, aweq.FLAG_PHASE_REDUCE)
    torch.cuda.synchronize()
    assert bool((b.out[first]["s"] == -1.0).all()) and torch.equal(b.out[first]["xmin"], a.out[first]["xmin"])


@pytest.mark.parametrize("overlap", [False, True])
def test_graph_replay_equals_eager(overlap):
    """One pass captured into a CUDA graph (with both streams when the two-stream schedule is on)
    writes, on replay, exactly what the eager pass writes."""
    from paper_2311_01305_b200 import aweq, calibrate
    wl = synth.workloads(n_tokens_scale=1.0 / 64)["opt125m_model_w8a8"]
    Xc, Wc = make_workload_tensors(wl, offset=1.0)
    Xd = {k: v.to(DEV) for k, v in Xc.items()}
    Wd = {k: v.to(DEV) for k, v in Wc.items()}
    a = calibrate.LayerCalibrator(wl, 8, Xd, Wd, None)
    b = calibrate.LayerCalibrator(wl, 8, Xd, Wd, None, overlap=overlap)
    a.run()
    E = lambda: torch.cuda.Event(enable_timing=True)
    hooks = []
    for _ in b.passes:
        pairs = ((E(), E()), (E(), E()))
        for pr in pairs:
            for e in pr:
                e.record()                                # create the handles
        hooks.append(pairs)
    graph = b.capture(hooks)
    n0 = aweq.launch_count()
    for _ in range(2):
        for outs in b.out.values():
            for v in outs.values():
                v.view(torch.uint8).fill_(0x5A)
        graph.replay()
    torch.cuda.synchronize()
    assert aweq.launch_count() == n0                      # replays go through no library call
    # the profiling hooks were recorded by the replay itself and can be read back
    for stats_pair, act_pair in hooks:
        assert 0.0 < stats_pair[0].elapsed_time(stats_pair[1]) < 50.0
        assert 0.0 < act_pair[0].elapsed_time(act_pair[1]) < 50.0
    assert aweq.read_status(b.status)["wait_timeout"] == 0
    for nm, outs in a.out.items():
        for k, v in outs.items():
            assert torch.equal(v.view(torch.uint8), b.out[nm][k].view(torch.uint8)), (nm, k)
    # the trial of both launch modes times real passes and leaves the results as they were
    trial = b.launch_trial(graph, steps=2)
    assert 0.0 < trial["eager_ms"] < 50.0 and 0.0 < trial["graph_ms"] < 50.0
    for nm, outs in a.out.items():
        for k, v in outs.items():
            assert torch.equal(v.view(torch.uint8), b.out[nm][k].view(torch.uint8)), (nm, k)
