"""aweq_stats_static: the statistics step for callers that cannot hand the
library any scratch memory (they may not allocate on the device: code inside a
host framework's memory pool, plug-ins that only receive tensors, sections
where cudaMalloc's device-wide synchronisation is not acceptable).  The scratch
is an array built into the library.  The test drives the entry point through
the C ABI twice in a row, on different shapes so that the second call runs over
what the first one left in the shared array, and compares each result with the
ordinary aweq_stats entry point, which takes caller scratch, and with the CPU
oracle.  The shapes include the widths at which the built-in array is exactly
full (2048 columns), the widest accepted row (16384) and the narrow layout that
keeps two sets of partials per row split (768).  This file is collected last on
purpose."""
import numpy as np
import pytest
import torch

from oracle import aweq_oracle as orc
from tests import util

pytestmark = pytest.mark.gpu


def _both(aweq, X):
    C = X.shape[1]
    ref = [torch.empty(C, device="cuda") for _ in range(3)]
    got = [util.guarded((C,), torch.float32) for _ in range(3)]
    ws = aweq.workspace(aweq.workspace_bytes(aweq.OP_STATS, X.shape[0], C))
    st = aweq.new_status()
    aweq.aweq_stats(X, ref[0], ref[1], ref[2], ws=ws, st=st)
    aweq.aweq_stats_static(X, got[0][0], got[1][0], got[2][0], st=st)
    torch.cuda.synchronize()
    for _, check in got:
        check()
    assert aweq.read_status(st) == {"nonfinite": 0, "zero_range": 0, "wait_timeout": 0}
    return [r.cpu().numpy() for r in ref], [g[0].cpu().numpy() for g in got]


def test_static_scratch_entry_matches_stats_twice_in_a_row():
    from paper_2311_01305_b200 import aweq
    shapes = [((6000, 4096), torch.bfloat16), ((777, 1032), torch.float16), ((1500, 2048), torch.float16),
              ((24, 16384), torch.bfloat16), ((5000, 768), torch.float16)]
    for shape, dtype in shapes:
        Xc = util.rand16(shape, dtype, seed=shape[0], offset=2.0, outlier_cols=6)
        ref, got = _both(aweq, Xc.cuda())
        util.assert_same_values(got[0], ref[0], "xmin")
        util.assert_same_values(got[1], ref[1], "xmax")
        mean_abs = np.abs(Xc.double().numpy()).mean(axis=0)
        assert np.all(np.abs(got[2].astype(np.float64) - ref[2]) <= util.mean_tolerance(ref[2], mean_abs))
        o = orc.stats(util.bits(Xc), util.odt(Xc))
        util.assert_same_values(got[0], o[0], "xmin against the oracle")
        util.assert_same_values(got[1], o[1], "xmax against the oracle")
        assert np.all(np.abs(got[2].astype(np.float64) - o[2]) <= util.mean_tolerance(o[2], mean_abs))


def test_static_scratch_entry_rejects_sizes_beyond_its_limit():
    from paper_2311_01305_b200 import aweq
    X = torch.zeros((8, 16392), dtype=torch.float16, device="cuda")
    out = torch.empty(16392, device="cuda")
    with pytest.raises(aweq.AweqError) as e:
        aweq.aweq_stats_static(X, out, out, out)
    assert e.value.code == 10
