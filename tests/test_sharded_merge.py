"""The multi-rank path on CPU: two gloo ranks each hold a token shard of two layer inputs,
compute their own statistics, put them into the exchange form the library's REDUCE part writes
({-xmin, xmax} as binary32, {column sums, token count} as binary64, all inputs in one flat
buffer each), merge them with ``calibrate.exchange_stats`` -- the one exchange of a
token-sharded calibration pass -- and must arrive at the statistics of the whole calibration
set, as the oracle computes them from all tokens."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import aweq_oracle as orc
from tests import util

SHAPES = ((900, 64), (900, 200))           # two inputs of one layer
CUTS = [0, 350, 900]                       # uneven shards


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _inputs():
    return [util.rand16(shape, torch.float16, seed=42 + k, offset=2.0, outlier_cols=4) for k, shape in enumerate(SHAPES)]


def _workload():
    from paper_2311_01305_b200 import synth
    ins = tuple(synth.ActSpec("in%d" % k, n, c, "normal") for k, (n, c) in enumerate(SHAPES))
    lins = tuple(synth.LinearSpec("lin%d" % k, 8, c, "in%d" % k, 0.02) for k, (n, c) in enumerate(SHAPES))
    return synth.Workload("two_inputs", "f16", 0, ins, lins, (8,), "row", 0, False)


def _rank(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2311_01305_b200 import calibrate
    layout, n_mm, n_sc = calibrate.exchange_layout(_workload())
    mm, sc = np.zeros(n_mm, np.float32), np.zeros(n_sc, np.float64)
    for k, X in enumerate(_inputs()):
        shard = X[CUTS[rank]:CUTS[rank + 1]]
        C = X.shape[1]
        xmin, xmax, _, xsum = orc.stats(util.bits(shard), orc.F16)
        mo, so = layout["in%d" % k]
        mm[mo:mo + C], mm[mo + C:mo + 2 * C] = -xmin, xmax
        sc[so:so + C], sc[so + C] = xsum, shard.shape[0]
    mm, sc = torch.from_numpy(mm), torch.from_numpy(sc)
    calibrate.exchange_stats(mm, sc)
    q.put((rank, mm.numpy(), sc.numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_statistics_exchange_equals_whole_set():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in range(2)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert np.array_equal(results[0][1], results[1][1]) and np.array_equal(results[0][2], results[1][2])
    _, mm, sc = results[0]
    from paper_2311_01305_b200 import calibrate
    layout, _, _ = calibrate.exchange_layout(_workload())
    for k, X in enumerate(_inputs()):
        C = X.shape[1]
        mo, so = layout["in%d" % k]
        xmin, xmax, xmean, xsum = orc.stats(util.bits(X), orc.F16)
        gmin, gmax = -mm[mo:mo + C], mm[mo + C:mo + 2 * C]
        gsum, cnt = sc[so:so + C], sc[so + C]
        assert cnt == X.shape[0]
        assert np.array_equal(gmin, xmin) and np.array_equal(gmax, xmax)
        assert np.allclose(gsum, xsum, rtol=1e-13, atol=1e-12)
        assert np.allclose((gsum / cnt).astype(np.float32), xmean, rtol=1e-6, atol=1e-9)


def test_exchange_layout_of_a_decoder_layer():
    """Host logic of the sharded calibrator: slices in input order, none overlapping, each on a
    16-byte boundary, inputs that feed no linear left out."""
    import dataclasses
    from paper_2311_01305_b200 import calibrate, synth
    wl = synth.workloads(1.0 / 1024)["opt125m_model_w8a8"]
    wl = dataclasses.replace(wl, linears=tuple(l for l in wl.linears if l.input != "o_in"))
    layout, n_mm, n_sc = calibrate.exchange_layout(wl)
    assert list(layout) == ["attn_in", "fc1_in", "fc2_in"]
    widths = {i.name: i.c_in for i in wl.inputs}
    end_mm = end_sc = 0
    for name, (mm, sc) in layout.items():
        assert mm >= end_mm and sc >= end_sc and (mm * 4) % 16 == 0 and (sc * 8) % 16 == 0
        end_mm, end_sc = mm + 2 * widths[name], sc + widths[name] + 1
    assert n_mm >= end_mm and n_sc >= end_sc
