"""The C-ABI library loads without a GPU, exports every symbol the public
header declares, and its host-only helpers behave (no compute is launched)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "aweq.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2311_01305_b200 import build
    return ctypes.CDLL(build.build())


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(aweq_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_header_declares_the_six_steps():
    names = declared_functions()
    for f in ("aweq_stats", "aweq_wrange", "aweq_factors", "aweq_equalize_quantize", "aweq_bias_correct",
              "aweq_quant_act", "aweq_layer_pass", "aweq_workspace_bytes"):
        assert f in names


def test_every_declared_symbol_is_exported(lib):
    for name in declared_functions():
        assert hasattr(lib, name), "libaweq.so does not export %s" % name


def test_host_helpers(lib):
    lib.aweq_strerror.restype = ctypes.c_char_p
    assert lib.aweq_strerror(0) == b"ok"
    for code in range(1, 10):
        assert len(lib.aweq_strerror(code)) > 3
    assert lib.aweq_version() >= 100
    lib.aweq_workspace_bytes.restype = ctypes.c_size_t
    lib.aweq_workspace_bytes.argtypes = [ctypes.c_int] + [ctypes.c_longlong] * 2 + [ctypes.c_int] * 3
    small = lib.aweq_workspace_bytes(1, 2048, 768, 0, 0, 0)
    big = lib.aweq_workspace_bytes(1, 262144, 11008, 0, 0, 0)
    assert 0 < small < big < 64 << 20
    assert lib.aweq_workspace_bytes(6, 262144, 4096, 8, 1, 0) == 0
    # groups of 128 at 3 / 4 / 8 bits: one float per (256-column window, row) for the eps . E[x^] partials
    assert lib.aweq_workspace_bytes(4, 4096, 4096, 4, 2, 128) == 16 * 4096 * 4
    assert lib.aweq_workspace_bytes(4, 4101, 11008, 3, 2, 128) == (43 * 4104 * 4 + 255) // 256 * 256
    assert lib.aweq_workspace_bytes(4, 4096, 4096, 4, 2, 64) == 0
    assert lib.aweq_workspace_bytes(4, 4096, 4096, 4, 0, 0) > 0


def test_validation_rejects_null_before_any_cuda_call(lib):
    vp, ll, i, sz = ctypes.c_void_p, ctypes.c_longlong, ctypes.c_int, ctypes.c_size_t
    lib.aweq_stats.argtypes = [vp, i, ll, ll, ll, vp, vp, vp, vp, vp, i, vp, sz, vp, vp]
    assert lib.aweq_stats(None, 0, 16, 64, 64, None, None, None, None, None, 0, None, 0, None, None) == 1
    lib.aweq_factors.argtypes = [vp] * 5 + [ll] + [vp] * 8
    assert lib.aweq_factors(None, None, None, None, None, 8, None, None, None, None, None, None, None, None) == 1
    lib.aweq_factors_absmax.argtypes = [vp] * 5 + [ll] + [vp] * 8
    assert lib.aweq_factors_absmax(None, None, None, None, None, 8, None, None, None, None, None, None, None, None) == 1
    lib.aweq_layer_pass.argtypes = [vp, vp, sz, vp, vp]
    assert lib.aweq_layer_pass(None, None, 0, None, None) == 1
    lib.aweq_fold_scale.argtypes = [vp, i, ll, ll, ll, vp, vp, ll, vp]
    assert lib.aweq_fold_scale(None, 0, 8, 8, 8, None, None, 8, None) == 1
    lib.aweq_relabel_signed.argtypes = [vp, ll, vp, vp, ll, vp, vp]
    assert lib.aweq_relabel_signed(None, 16, None, None, 0, None, None) == 1
    lib.aweq_forward_check.argtypes = [vp] * 9 + [i, vp, ll, ll, ll, vp, vp, vp, sz, vp]
    assert lib.aweq_forward_check(*([None] * 9), 0, None, 64, 64, 64, None, None, None, 0, None) == 1
    lib.aweq_forward_check_workspace_bytes.restype = sz
    lib.aweq_forward_check_workspace_bytes.argtypes = [ll, ll, ll]
    small = lib.aweq_forward_check_workspace_bytes(100, 768, 768)
    assert 0 < small < 8 << 20
    # bounded by the token chunk: the intermediates do not grow with N
    assert lib.aweq_forward_check_workspace_bytes(1 << 20, 4096, 4096) < 1 << 30
    assert lib.aweq_forward_check_workspace_bytes(0, 64, 64) == 0


def test_binding_imports_and_names_match_header():
    from paper_2311_01305_b200 import aweq
    for name in declared_functions():
        if name in ("aweq_strerror", "aweq_last_cuda_error", "aweq_version", "aweq_launch_count",
                    "aweq_workspace_bytes", "aweq_layer_pass_workspace_bytes", "aweq_layer_pass_fuses_ranges",
                    "aweq_forward_check_workspace_bytes",
                    "aweq_forward_check_weights_workspace_bytes"):
            continue
        assert hasattr(aweq, name), name


# ---------------------------------------------------------------- launch planners (host logic)
SMEM_LIMIT = 227 * 1024           # opt-in shared memory per CTA on sm_100
WIDTHS = sorted(set(list(range(8, 2049, 8)) + list(range(2048, 40961, 248)) +
                    [768, 3072, 4096, 5120, 9216, 10240, 10248, 11008, 13824, 20480, 20488, 36864, 40960]))


def _plan(lib, op, rows, cols):
    arr = (ctypes.c_longlong * 8)()
    lib.aweq_plan_query.argtypes = [ctypes.c_int, ctypes.c_longlong, ctypes.c_longlong, ctypes.POINTER(ctypes.c_longlong * 8)]
    rc = lib.aweq_plan_query(op, rows, cols, ctypes.byref(arr))
    return rc, tuple(arr)


def test_column_reduction_plans_fit_the_hardware(lib):
    lib.aweq_workspace_bytes.restype = ctypes.c_size_t
    lib.aweq_workspace_bytes.argtypes = [ctypes.c_int] + [ctypes.c_longlong] * 2 + [ctypes.c_int] * 3
    for cols in WIDTHS:
        for rows in (1, 7, 100, 4096, 262144):
            rc, (ctas, threads, smem, nslab, slab_w, nsplit, phases, stage_rows) = _plan(lib, 1, rows, cols)
            assert rc == 0
            nvec = cols // 8
            # 256, 320 or 384 consumer threads and the producer warp
            assert 1 <= ctas <= 148 and ctas == nslab * nsplit and threads in (288, 352, 416)
            consumers = threads - 32
            stages, rem = divmod(smem - 128, stage_rows * slab_w * 16)        # the ring: two to four stages
            assert smem <= SMEM_LIMIT and rem == 0 and stages in (2, 3, 4)
            assert nslab * slab_w >= nvec and slab_w <= consumers           # every column has an owner
            assert phases in (1, 2) and stage_rows % (8 * phases) == 0      # whole eight-row groups per phase
            assert phases * ((slab_w + 31) // 32 * 32) <= consumers         # phases fit the consumer threads
            base_slabs = -(-nvec // 256)
            if consumers > 256:
                # a wider CTA only where it brings the row into one or two slabs that 256 threads cut into more
                assert nslab <= 2 and nslab < base_slabs and phases == 1 and stages == (4 if consumers == 320 else 3)
            else:
                assert stages == (3 if nslab >= 3 else 2)
            assert stage_rows * slab_w * 16 <= (1 << 20) - 1                # one mbarrier transaction count
            # the partials of the largest split count fit the advertised workspace
            assert nsplit * phases * cols * 16 + 256 <= lib.aweq_workspace_bytes(1, rows, cols, 0, 0, 0)


def test_row_quantiser_plans_fit_the_hardware(lib):
    for op in (4, 6):
        for cols in WIDTHS:
            for rows in (1, 5, 300, 65536):
                rc, (ctas, threads, smem, team, V, R, S, wide) = _plan(lib, op, rows, cols)
                assert rc == 0, (op, rows, cols)
                nvec = cols // 8
                assert 1 <= ctas <= 444 and threads in (256, 512, 1024) and smem <= SMEM_LIMIT
                assert team % 32 == 0 and (threads % team == 0 or team == 2 * threads) and team * V >= nvec      # the row is covered
                if wide == 2:                                   # plain loads: no stages, a row per team
                    assert V >= 1 and team * (V - 1) < nvec
                    assert R == 0 and S == 0 and smem <= 1024
                    if op == 4:
                        assert (threads == 256 and team <= 256 and V <= 10) or (threads == team == 1024 and V <= 5)
                    else:
                        # step 6 has two rows of a team in flight: at most nine vectors per thread, teams of up to 16 warps
                        assert cols <= 36864 and V <= 9 and ((threads == 256 and team <= 256) or threads == team == 512)
                    # three CTAs per SM while the registers allow it, else two; one when the team is a whole large CTA
                    assert ctas <= 148 * (1 if team > 256 else 3 if V <= (3 if op == 6 else 4) else 2)
                    assert ctas <= max(1, -(-rows // (threads // team)))
                    continue
                # a row per cluster of two CTAs, half a row each, in shared-memory stages
                half = (nvec + 1) // 2
                assert wide == 3 and op == 6 and cols > 36864 and threads == 512 and team == 1024 and V == 5 and R <= 4
                assert S >= 2 and R >= 1
                assert ctas % 2 == 0 and ctas <= 148 and 512 * V >= half and smem == 4096 + S * R * half * 16
    # beyond the supported width the query says so instead of planning something that cannot launch
    assert _plan(lib, 6, 100, 40968)[0] == 2 and _plan(lib, 4, 100, 81920)[0] == 2
    assert _plan(lib, 6, 100, 36)[0] == 2 and _plan(lib, 5, 100, 64)[0] == 9


def test_reference_arm_of_the_bench_loads_only_the_oracle():
    """`bench.py --impl reference` times the oracle alone: the process must map the oracle's shared
    object and never the CUDA library (checked from /proc/<pid>/maps at exit of a tiny run)."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = ("import sys, runpy, atexit\n"
            "def report():\n"
            "    maps = open('/proc/self/maps').read()\n"
            "    sys.stderr.write('MAPS libaweq.so=%d libaweq_oracle.so=%d\\n' % ('libaweq.so' in maps, 'libaweq_oracle.so' in maps))\n"
            "atexit.register(report)\n"
            "sys.argv = ['bench.py', '--impl', 'reference', '--steps', '1', '--warmup', '0', '--cpu-sample-tokens', '64',\n"
            "            '--workload', 'opt125m_linear_w8a8']\n"
            "runpy.run_path('bench.py', run_name='__main__')\n")
    r = subprocess.run([sys.executable, "-c", code], cwd=root, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    assert "MAPS libaweq.so=0 libaweq_oracle.so=1" in r.stderr, r.stderr[-500:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["gpu_launches"] == 0
    assert set(line["config"]) >= {"workload", "w_bits", "w_gran", "group", "act_quant", "storage"}
