"""The multi-rank path on CPU: two gloo ranks each hold a token shard, compute
their own statistics, merge them with ``calibrate.allreduce_stats`` (the one
exchange of a token-sharded calibration pass) and must arrive at the
statistics of the whole calibration set."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import aweq_oracle as orc
from tests import util


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2311_01305_b200 import calibrate
    X = util.rand16((900, 64), torch.float16, seed=42, offset=2.0, outlier_cols=4)
    cuts = [0, 350, 900]                                   # uneven shards
    shard = X[cuts[rank]:cuts[rank + 1]]
    xmin, xmax, _, xsum = orc.stats(util.bits(shard), orc.F16)
    t = [torch.from_numpy(a.copy()) for a in (xmin, xmax, xsum)]
    count = torch.tensor([shard.shape[0]], dtype=torch.int64)
    calibrate.allreduce_stats(t[0], t[1], t[2], count)
    q.put((rank, t[0].numpy(), t[1].numpy(), t[2].numpy(), int(count.item())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_statistics_merge_equals_whole_set():
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
    X = util.rand16((900, 64), torch.float16, seed=42, offset=2.0, outlier_cols=4)
    xmin, xmax, xmean, xsum = orc.stats(util.bits(X), orc.F16)
    for _, gmin, gmax, gsum, cnt in results:
        assert cnt == 900
        assert np.array_equal(gmin, xmin) and np.array_equal(gmax, xmax)
        assert np.allclose(gsum, xsum, rtol=1e-13, atol=1e-12)
        assert np.allclose((gsum / cnt).astype(np.float32), xmean, rtol=1e-6, atol=1e-9)
