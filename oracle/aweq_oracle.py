"""NumPy-facing wrapper of the plain-C AWEQ oracle.  TEST INFRASTRUCTURE ONLY.

The arithmetic lives in ``aweq_oracle.c`` (scalar loops written from the paper,
arXiv 2311.01305: Eq. 1-2 quantiser, Eq. 3 equalisation, Eq. 10 factors,
Eq. 11-15 bias correction).  This module only compiles that file with gcc,
loads it with ctypes and moves NumPy arrays in and out.  It imports nothing
from the CUDA package and the CUDA package imports nothing from here; only
tests, the smoke check and the benchmark's CPU-baseline leg use it.

16-bit tensors are passed as ``uint16`` arrays of raw bits plus a dtype tag
(``F16`` / ``BF16``) so that both sides of a parity test see identical inputs.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

F16, BF16 = 0, 1
PER_TENSOR, PER_ROW, PER_GROUP = 0, 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "aweq_oracle.c")
_LIB = os.path.join(_HERE, "libaweq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-frounding-math", "-Wall", "-Wextra", _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_threads.restype = ctypes.c_int
        _lib.oracle_factors.restype = ctypes.c_int64
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "16-bit tensors are passed as raw uint16 bits"
    return a


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


i64 = ctypes.c_int64
ci = ctypes.c_int


def threads() -> int:
    return int(_load().oracle_threads())


def set_threads(n: int) -> None:
    _load().oracle_set_threads(ci(n))


def decode16(bits: np.ndarray, dtype: int) -> np.ndarray:
    bits = _u16(bits)
    out = np.empty(bits.shape, np.float32)
    _load().oracle_decode16(_p(bits), ci(dtype), i64(bits.size), _p(out))
    return out


def encode16(x: np.ndarray, dtype: int) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, np.uint16)
    _load().oracle_encode16(_p(x), ci(dtype), i64(x.size), _p(out))
    return out


def stats(X: np.ndarray, dtype: int):
    """Step 1 -> (xmin, xmax, xmean, xsum[f64]) per channel of X[N, C]."""
    X = _u16(X)
    N, C = X.shape
    xmin = np.empty(C, np.float32)
    xmax = np.empty(C, np.float32)
    xmean = np.empty(C, np.float32)
    xsum = np.empty(C, np.float64)
    _load().oracle_stats(_p(X), ci(dtype), i64(N), i64(C), i64(C), _p(xmin), _p(xmax), _p(xmean), _p(xsum))
    return xmin, xmax, xmean, xsum


def wrange(W: np.ndarray, dtype: int, prev=None):
    """Step 2 -> (wmin, wmax) per input channel of W[C_out, C_in]; ``prev`` merges."""
    W = _u16(W)
    C_out, C_in = W.shape
    if prev is None:
        wmin = np.empty(C_in, np.float32)
        wmax = np.empty(C_in, np.float32)
    else:
        wmin, wmax = (np.array(prev[0], np.float32), np.array(prev[1], np.float32))
    _load().oracle_wrange(_p(W), ci(dtype), i64(C_out), i64(C_in), i64(C_in), _p(wmin), _p(wmax),
                          ci(0 if prev is None else 1))
    return wmin, wmax


RANGE, ABSMAX = 0, 1


def factors(xmin, xmax, xmean, wmin, wmax, criterion=RANGE):
    """Step 3 -> dict(s, rinv, mu_hat, pX, pW, scalars[8], dead).  ``criterion``: RANGE is the paper's
    (Eq. 4-10); ABSMAX feeds Eq. 10 with the largest magnitudes instead (the comparison criterion)."""
    xmin, xmax, xmean, wmin, wmax = map(_f32, (xmin, xmax, xmean, wmin, wmax))
    C = xmin.size
    out = {k: np.empty(C, np.float32) for k in ("s", "rinv", "mu_hat", "pX", "pW")}
    scalars = np.empty(8, np.float64)
    dead = _load().oracle_factors(_p(xmin), _p(xmax), _p(xmean), _p(wmin), _p(wmax), i64(C),
                                  _p(out["s"]), _p(out["rinv"]), _p(out["mu_hat"]), _p(out["pX"]),
                                  _p(out["pW"]), _p(scalars), ci(criterion))
    out["scalars"] = scalars
    out["dead"] = int(dead)
    return out


def quantize_vector(v, bits: int, literal_division: bool = False):
    """Eq. 1-2 on one binary32 vector -> (Step, Z, codes[int32])."""
    v = _f32(v).ravel()
    step = ctypes.c_float()
    zp = ctypes.c_int32()
    q = np.empty(v.size, np.int32)
    _load().oracle_quantize_vector(_p(v), i64(v.size), ci(bits), ci(int(literal_division)),
                                   ctypes.byref(step), ctypes.byref(zp), _p(q))
    return float(step.value), int(zp.value), q


def pack(q: np.ndarray, bits: int) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int32)
    rows, cols = q.shape
    out = np.empty((rows, cols * bits // 8), np.uint8)
    _load().oracle_pack(_p(q), i64(rows), i64(cols), ci(bits), _p(out))
    return out


def unpack(codes: np.ndarray, cols: int, bits: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    rows = codes.shape[0]
    q = np.empty((rows, cols), np.int32)
    _load().oracle_unpack(_p(codes), i64(rows), i64(cols), ci(bits), _p(q))
    return q


def _n_scales(rows, cols, gran, group):
    if gran == PER_TENSOR:
        return 1
    if gran == PER_ROW:
        return rows
    return rows * (cols // group)


def equalize_quantize(W, dtype, s, mu_hat, bits, gran, group=0, literal_division=False):
    """Step 4 -> (codes[u8, packed], step, zp, delta[f64] or None)."""
    W = _u16(W)
    C_out, C_in = W.shape
    s, mu_hat = _f32(s), _f32(mu_hat)
    ns = _n_scales(C_out, C_in, gran, group)
    codes = np.empty((C_out, C_in * bits // 8), np.uint8)
    step = np.empty(ns, np.float32)
    zp = np.empty(ns, np.int32)
    delta = np.empty(C_out, np.float64)
    _load().oracle_equalize_quantize(_p(W), ci(dtype), i64(C_out), i64(C_in), i64(C_in), _p(s), _p(mu_hat),
                                     ci(bits), ci(gran), i64(group), ci(int(literal_division)),
                                     _p(codes), _p(step), _p(zp), _p(delta))
    return codes, step, zp, (delta if mu_hat is not None else None)


def dequantize(codes, step, zp, cols, bits, gran, group=0) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    rows = codes.shape[0]
    out = np.empty((rows, cols), np.float64)
    _load().oracle_dequantize(_p(codes), _p(_f32(step)), _p(np.ascontiguousarray(zp, dtype=np.int32)),
                              i64(rows), i64(cols), ci(bits), ci(gran), i64(group), _p(out))
    return out


def bias_correct(delta, bias_in, bias_dtype):
    """Step 5 -> (bias_f32, bias_16[raw bits])."""
    delta = np.ascontiguousarray(delta, dtype=np.float64)
    C_out = delta.size
    bias_in = None if bias_in is None else _u16(bias_in)
    bf = np.empty(C_out, np.float32)
    b16 = np.empty(C_out, np.uint16)
    _load().oracle_bias_correct(_p(delta), _p(bias_in), ci(bias_dtype), i64(C_out), _p(bf), _p(b16))
    return bf, b16


def bias_delta_from_codes(W, dtype, s, codes, step, zp, mu_hat, bits, gran, group=0):
    W = _u16(W)
    C_out, C_in = W.shape
    delta = np.empty(C_out, np.float64)
    _load().oracle_bias_delta_from_codes(_p(W), ci(dtype), i64(C_out), i64(C_in), i64(C_in), _p(_f32(s)),
                                         _p(np.ascontiguousarray(codes, dtype=np.uint8)), _p(_f32(step)),
                                         _p(np.ascontiguousarray(zp, dtype=np.int32)), _p(_f32(mu_hat)),
                                         ci(bits), ci(gran), i64(group), _p(delta))
    return delta


def quant_act(X, dtype, rinv, gran=PER_ROW, lo_hi=None, bits=8, literal_division=False):
    """Step 6 -> (Xq[u8, one code per byte], step, zp)."""
    X = _u16(X)
    N, C = X.shape
    rinv = _f32(rinv)
    lo_hi = _f32(lo_hi)
    ns = 1 if gran == PER_TENSOR else N
    Xq = np.empty((N, C), np.uint8)
    step = np.empty(ns, np.float32)
    zp = np.empty(ns, np.int32)
    _load().oracle_quant_act(_p(X), ci(dtype), i64(N), i64(C), i64(C), _p(rinv), ci(gran), _p(lo_hi),
                             ci(bits), ci(int(literal_division)), _p(Xq), _p(step), _p(zp))
    return Xq, step, zp


def forward_check(Xq, act_step, act_zp, Wq, w_step, w_zp, bias_q, X, W, dtype, bias=None):
    """Eq. 11 evaluated on data -> (mean_err[C_out] f64, sums[4] f64): quantised layer against
    the 16-bit layer (one byte per code; ``bias_q`` binary32 or None; ``bias`` raw 16-bit or None)."""
    X, W = _u16(X), _u16(W)
    N, C_in = X.shape
    C_out = W.shape[0]
    Xq = np.ascontiguousarray(Xq, dtype=np.uint8)
    Wq = np.ascontiguousarray(Wq, dtype=np.uint8)
    assert Xq.shape == (N, C_in) and Wq.shape == (C_out, C_in)
    mean_err = np.empty(C_out, np.float64)
    sums = np.empty(4, np.float64)
    bias = None if bias is None else _u16(bias)
    _load().oracle_forward_check(_p(Xq), _p(_f32(act_step)), _p(np.ascontiguousarray(act_zp, dtype=np.int32)),
                                 _p(Wq), _p(_f32(w_step)), _p(np.ascontiguousarray(w_zp, dtype=np.int32)),
                                 _p(_f32(bias_q)), _p(X), _p(W), ci(dtype), _p(bias), i64(N), i64(C_in), i64(C_out),
                                 _p(mean_err), _p(sums))
    return mean_err, sums


def fold_scale(P, dtype, rinv):
    """Row r of the 16-bit matrix (or element r of the vector) P times rinv[r], as raw 16-bit bits."""
    P = _u16(P)
    rows = P.shape[0]
    cols = 1 if P.ndim == 1 else P.shape[1]
    out = np.empty_like(P)
    _load().oracle_fold_scale(_p(P), ci(dtype), i64(rows), i64(cols), _p(_f32(rinv)), _p(out))
    return out


def relabel_signed(codes, zp=None):
    """8-bit codes q -> q - 128 (int8), zero-points Z -> Z - 128 (saturating) -> (codes_signed, zp_signed or None)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.empty(codes.shape, np.int8)
    zp_in = None if zp is None else np.ascontiguousarray(zp, dtype=np.int32)
    zp_out = None if zp is None else np.empty(zp_in.shape, np.int32)
    _load().oracle_relabel_signed(_p(codes), i64(codes.size), _p(out), _p(zp_in), i64(0 if zp is None else zp_in.size),
                                  _p(zp_out))
    return out, zp_out


def forward_check_weights(codes, step, zp, bits, gran, group, rinv, bias_q, X, W, dtype, bias=None):
    """Eq. 11 on data for a weight-only layer -> (mean_err[C_out] f64, sums[4] f64); packed codes as
    ``equalize_quantize`` returns them, ``rinv`` binary32 or None."""
    X, W = _u16(X), _u16(W)
    N, C_in = X.shape
    C_out = W.shape[0]
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    assert codes.shape == (C_out, C_in * bits // 8)
    mean_err = np.empty(C_out, np.float64)
    sums = np.empty(4, np.float64)
    bias = None if bias is None else _u16(bias)
    _load().oracle_forward_check_weights(_p(codes), _p(_f32(step)), _p(np.ascontiguousarray(zp, dtype=np.int32)),
                                         ci(bits), ci(gran), i64(group), _p(_f32(rinv)), _p(_f32(bias_q)), _p(X), _p(W),
                                         ci(dtype), _p(bias), i64(N), i64(C_in), i64(C_out), _p(mean_err), _p(sums))
    return mean_err, sums
