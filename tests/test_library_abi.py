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
    assert lib.aweq_workspace_bytes(4, 4096, 4096, 4, 2, 128) == 0
    assert lib.aweq_workspace_bytes(4, 4096, 4096, 4, 0, 0) > 0


def test_validation_rejects_null_before_any_cuda_call(lib):
    vp, ll, i, sz = ctypes.c_void_p, ctypes.c_longlong, ctypes.c_int, ctypes.c_size_t
    lib.aweq_stats.argtypes = [vp, i, ll, ll, ll, vp, vp, vp, vp, vp, i, vp, sz, vp, vp]
    assert lib.aweq_stats(None, 0, 16, 64, 64, None, None, None, None, None, 0, None, 0, None, None) == 1
    lib.aweq_factors.argtypes = [vp] * 5 + [ll] + [vp] * 8
    assert lib.aweq_factors(None, None, None, None, None, 8, None, None, None, None, None, None, None, None) == 1
    lib.aweq_layer_pass.argtypes = [vp, vp, sz, vp, vp]
    assert lib.aweq_layer_pass(None, None, 0, None, None) == 1
    lib.aweq_fold_scale.argtypes = [vp, i, ll, ll, ll, vp, vp, ll, vp]
    assert lib.aweq_fold_scale(None, 0, 8, 8, 8, None, None, 8, None) == 1
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
                    "aweq_workspace_bytes", "aweq_layer_pass_workspace_bytes", "aweq_forward_check_workspace_bytes"):
            continue
        assert hasattr(aweq, name), name
