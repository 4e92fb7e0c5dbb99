"""Thin Python binding of the C-ABI CUDA library ``libaweq.so``.

Every function here has the name and the argument order of the C entry point
declared in ``include/aweq.h`` and does argument marshalling only: tensors
become device pointers, the current PyTorch CUDA stream becomes the ``stream``
argument, scratch memory is a ``torch.uint8`` tensor.  All arithmetic of the
AWEQ calibration pass (arXiv 2311.01305) runs in the library's kernels; there
is no Python or CPU fallback, and importing this module fails loudly when the
library has not been built (``python -m paper_2311_01305_b200.build``).
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libaweq.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(
        "libaweq.so is missing: build the CUDA library first with "
        "`python -m paper_2311_01305_b200.build` (needs nvcc; no GPU required to build)")
_lib = ctypes.CDLL(LIB_PATH)

OK = 0
F16, BF16 = 0, 1
PER_TENSOR, PER_ROW, PER_GROUP = 0, 1, 2
OP_STATS, OP_WRANGE, OP_EQUALIZE_QUANTIZE, OP_BIAS_CORRECT, OP_QUANT_ACT = 1, 2, 4, 5, 6
FLAG_NO_EQUALIZE, FLAG_NO_BIAS_CORRECT = 1, 2
FLAG_PHASE_REDUCE, FLAG_PHASE_QUANT, FLAG_PHASE_ACT = 4, 8, 16
FLAG_ABSMAX_CRITERION = 32
FLAG_MERGED_STATS = 64

_vp, _ll, _i, _sz = ctypes.c_void_p, ctypes.c_longlong, ctypes.c_int, ctypes.c_size_t


class DevStatus(ctypes.Structure):
    _fields_ = [("nonfinite", ctypes.c_ulonglong), ("zero_range", ctypes.c_ulonglong),
                ("wait_timeout", ctypes.c_ulonglong), ("reserved", ctypes.c_ulonglong)]


class LayerArgs(ctypes.Structure):
    _fields_ = [
        ("X", _vp), ("dt", _i), ("N", _ll), ("C_in", _ll), ("ldx", _ll),
        ("n_w", _i), ("W", ctypes.POINTER(_vp)), ("C_out", ctypes.POINTER(_ll)), ("ldw", ctypes.POINTER(_ll)),
        ("bits", _i), ("gran", _i), ("group", _i),
        ("bias_in", ctypes.POINTER(_vp)), ("bias_out", ctypes.POINTER(_vp)), ("bias_out_f32", ctypes.POINTER(_vp)),
        ("codes", ctypes.POINTER(_vp)), ("step", ctypes.POINTER(_vp)), ("zp", ctypes.POINTER(_vp)),
        ("epsmu", ctypes.POINTER(_vp)),
        ("xmin", _vp), ("xmax", _vp), ("xmean", _vp), ("wmin", _vp), ("wmax", _vp), ("s", _vp), ("rinv", _vp),
        ("mu_hat", _vp), ("pX", _vp), ("pW", _vp), ("scalars", _vp),
        ("Xq", _vp), ("act_step", _vp), ("act_zp", _vp), ("act_bits", _i), ("flags", _i),
        ("ev_stats_begin", _vp), ("ev_stats_end", _vp), ("ev_act_begin", _vp), ("ev_act_end", _vp),
        ("stat_negmin_max", _vp), ("stat_sum_count", _vp),
    ]


_lib.aweq_strerror.restype = ctypes.c_char_p
_lib.aweq_strerror.argtypes = [_i]
_lib.aweq_last_cuda_error.restype = ctypes.c_char_p
_lib.aweq_version.restype = _i
_lib.aweq_launch_count.restype = ctypes.c_ulonglong
_lib.aweq_workspace_bytes.restype = _sz
_lib.aweq_workspace_bytes.argtypes = [_i, _ll, _ll, _i, _i, _i]
_lib.aweq_stats.argtypes = [_vp, _i, _ll, _ll, _ll, _vp, _vp, _vp, _vp, _vp, _i, _vp, _sz, _vp, _vp]
_lib.aweq_stats_static.argtypes = [_vp, _i, _ll, _ll, _ll, _vp, _vp, _vp, _vp, _vp]
_lib.aweq_stats_static.restype = _i
_lib.aweq_wrange.argtypes = [_vp, _i, _ll, _ll, _ll, _vp, _vp, _i, _vp, _sz, _vp, _vp]
_lib.aweq_factors.argtypes = [_vp, _vp, _vp, _vp, _vp, _ll, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.aweq_factors_absmax.argtypes = [_vp, _vp, _vp, _vp, _vp, _ll, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.aweq_factors_absmax.restype = _i
_lib.aweq_equalize_quantize.argtypes = [_vp, _i, _ll, _ll, _ll, _vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _sz,
                                        _vp, _vp]
_lib.aweq_bias_correct.argtypes = [_vp, _vp, _i, _vp, _vp, _vp, _vp, _vp, _ll, _ll, _ll, _i, _i, _i, _vp, _vp, _vp,
                                   _i, _vp, _vp]
_lib.aweq_quant_act.argtypes = [_vp, _i, _ll, _ll, _ll, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.aweq_layer_pass_workspace_bytes.restype = _sz
_lib.aweq_layer_pass_workspace_bytes.argtypes = [ctypes.POINTER(LayerArgs)]
_lib.aweq_layer_pass_fuses_ranges.restype = ctypes.c_int
_lib.aweq_layer_pass_fuses_ranges.argtypes = [ctypes.POINTER(LayerArgs)]
_lib.aweq_layer_pass.argtypes = [ctypes.POINTER(LayerArgs), _vp, _sz, _vp, _vp]
_lib.aweq_plan_query.argtypes = [_i, _ll, _ll, ctypes.POINTER(_ll * 8)]
_lib.aweq_plan_query.restype = _i
_lib.aweq_relabel_signed.argtypes = [_vp, _ll, _vp, _vp, _ll, _vp, _vp]
_lib.aweq_relabel_signed.restype = _i
_lib.aweq_fold_scale.argtypes = [_vp, _i, _ll, _ll, _ll, _vp, _vp, _ll, _vp]
_lib.aweq_fold_scale.restype = _i
_lib.aweq_forward_check_workspace_bytes.restype = _sz
_lib.aweq_forward_check_workspace_bytes.argtypes = [_ll, _ll, _ll]
_lib.aweq_forward_check.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _vp, _ll, _ll, _ll, _vp, _vp, _vp,
                                    _sz, _vp]
_lib.aweq_forward_check_weights_workspace_bytes.restype = _sz
_lib.aweq_forward_check_weights_workspace_bytes.argtypes = [_ll, _ll, _ll]
_lib.aweq_forward_check_weights.argtypes = [_vp, _vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _i, _vp, _ll, _ll, _ll, _vp, _vp,
                                            _vp, _sz, _vp]
_lib.aweq_forward_check_weights.restype = _i
for _f in ("aweq_stats", "aweq_wrange", "aweq_factors", "aweq_equalize_quantize", "aweq_bias_correct",
           "aweq_quant_act", "aweq_layer_pass", "aweq_forward_check"):
    getattr(_lib, _f).restype = _i


class AweqError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        msg = _lib.aweq_strerror(code).decode()
        if code == 8:
            msg += ": " + _lib.aweq_last_cuda_error().decode()
        super().__init__("aweq status %d: %s" % (code, msg))


def _check(code: int) -> None:
    if code != OK:
        raise AweqError(code)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("device tensors only (there is no CPU path)")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def dtype_tag(t: torch.Tensor) -> int:
    if t.dtype == torch.float16:
        return F16
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("16-bit tensors must be float16 or bfloat16, got %s" % t.dtype)


def _ld(t: torch.Tensor) -> int:
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError("matrices must be 2-D with a contiguous innermost dimension")
    return t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def strerror(code: int) -> str:
    return _lib.aweq_strerror(code).decode()


def version() -> int:
    return int(_lib.aweq_version())


def launch_count() -> int:
    return int(_lib.aweq_launch_count())


def workspace_bytes(op: int, rows: int, cols: int, bits: int = 0, gran: int = 0, group: int = 0) -> int:
    return int(_lib.aweq_workspace_bytes(op, rows, cols, bits, gran, group))


def workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A 256-byte aligned scratch tensor of at least ``nbytes`` bytes."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def new_status(device="cuda") -> torch.Tensor:
    """A zeroed device status block (4 x uint64 viewed as int64)."""
    return torch.zeros(4, dtype=torch.int64, device=device)


def read_status(st: torch.Tensor) -> dict:
    v = st.cpu().tolist()
    return {"nonfinite": v[0], "zero_range": v[1], "wait_timeout": v[2]}


def aweq_stats(X, xmin, xmax, xmean, xsum=None, count=None, accumulate=False, ws=None, st=None, N=None):
    n = X.shape[0] if N is None else N
    _check(_lib.aweq_stats(_ptr(X), dtype_tag(X), n, X.shape[1], _ld(X), _ptr(xmin), _ptr(xmax), _ptr(xmean),
                           _ptr(xsum), _ptr(count), int(accumulate), _ptr(ws), 0 if ws is None else ws.numel(),
                           _ptr(st), _stream()))


def aweq_stats_static(X, xmin, xmax, xmean, st=None):
    """Step 1 with the library's built-in scratch: for callers that cannot allocate
    device memory (no ``ws`` argument; C_in <= 16384).  Same results as aweq_stats."""
    _check(_lib.aweq_stats_static(_ptr(X), dtype_tag(X), X.shape[0], X.shape[1], _ld(X), _ptr(xmin), _ptr(xmax),
                                  _ptr(xmean), _ptr(st), _stream()))


def aweq_wrange(W, wmin, wmax, accumulate=False, ws=None, st=None):
    _check(_lib.aweq_wrange(_ptr(W), dtype_tag(W), W.shape[0], W.shape[1], _ld(W), _ptr(wmin), _ptr(wmax),
                            int(accumulate), _ptr(ws), 0 if ws is None else ws.numel(), _ptr(st), _stream()))


def aweq_factors(xmin, xmax, xmean, wmin, wmax, s, rinv, mu_hat, pX=None, pW=None, scalars=None, st=None):
    _check(_lib.aweq_factors(_ptr(xmin), _ptr(xmax), _ptr(xmean), _ptr(wmin), _ptr(wmax), xmin.numel(), _ptr(s),
                             _ptr(rinv), _ptr(mu_hat), _ptr(pX), _ptr(pW), _ptr(scalars), _ptr(st), _stream()))


def aweq_factors_absmax(xmin, xmax, xmean, wmin, wmax, s, rinv, mu_hat, pX=None, pW=None, scalars=None, st=None):
    _check(_lib.aweq_factors_absmax(_ptr(xmin), _ptr(xmax), _ptr(xmean), _ptr(wmin), _ptr(wmax), xmin.numel(), _ptr(s),
                                    _ptr(rinv), _ptr(mu_hat), _ptr(pX), _ptr(pW), _ptr(scalars), _ptr(st), _stream()))


def aweq_equalize_quantize(W, s, mu_hat, bits, gran, group, codes, step, zp, epsmu=None, ws=None, st=None):
    _check(_lib.aweq_equalize_quantize(_ptr(W), dtype_tag(W), W.shape[0], W.shape[1], _ld(W), _ptr(s), _ptr(mu_hat),
                                       bits, gran, group, _ptr(codes), _ptr(step), _ptr(zp), _ptr(epsmu), _ptr(ws),
                                       0 if ws is None else ws.numel(), _ptr(st), _stream()))


def aweq_bias_correct(epsmu, W, s, codes, step, zp, mu_hat, bits, gran, group, bias_in, bias_out, bias_out_f32,
                      bias_dt, C_out=None, st=None):
    if W is not None:
        c_out, c_in, ld, dt = W.shape[0], W.shape[1], _ld(W), dtype_tag(W)
    else:
        c_out, c_in, ld, dt = (epsmu.numel() if C_out is None else C_out), 8, 8, bias_dt
    _check(_lib.aweq_bias_correct(_ptr(epsmu), _ptr(W), dt, _ptr(s), _ptr(codes), _ptr(step), _ptr(zp), _ptr(mu_hat),
                                  c_out, c_in, ld, bits, gran, group, _ptr(bias_in), _ptr(bias_out),
                                  _ptr(bias_out_f32), bias_dt, _ptr(st), _stream()))


def aweq_quant_act(X, rinv, bits, gran, tensor_lo_hi, Xq, step, zp, st=None):
    _check(_lib.aweq_quant_act(_ptr(X), dtype_tag(X), X.shape[0], X.shape[1], _ld(X), _ptr(rinv), bits, gran,
                               _ptr(tensor_lo_hi), _ptr(Xq), _ptr(step), _ptr(zp), _ptr(st), _stream()))


def aweq_plan_query(op: int, rows: int, cols: int):
    """Launch geometry for an operation on a rows x cols matrix as a tuple of 8 integers
    (see ``include/aweq.h``); host logic only."""
    plan = (_ll * 8)()
    _check(_lib.aweq_plan_query(op, rows, cols, ctypes.byref(plan)))
    return tuple(plan)


def aweq_relabel_signed(codes, out=None, zp=None, zp_out=None):
    """8-bit codes q -> q - 128 (an ``int8`` view of the result is the signed code) and zero-points
    Z -> Z - 128; in place when ``out`` / ``zp_out`` are None."""
    out = codes if out is None else out
    if zp is not None and zp_out is None:
        zp_out = zp
    _check(_lib.aweq_relabel_signed(_ptr(codes), codes.numel(), _ptr(out), _ptr(zp), 0 if zp is None else zp.numel(),
                                    _ptr(zp_out), _stream()))
    return out, zp_out


def aweq_fold_scale(P, rinv, out=None):
    """Scale row r of a 16-bit matrix (or element r of a vector) by ``rinv[r]``; in place when
    ``out`` is None."""
    out = P if out is None else out
    if P.dim() == 1:
        rows, cols, ld, ld_out = P.shape[0], 1, P.stride(0), out.stride(0)
    else:
        rows, cols, ld, ld_out = P.shape[0], P.shape[1], _ld(P), _ld(out)
    _check(_lib.aweq_fold_scale(_ptr(P), dtype_tag(P), rows, cols, ld, _ptr(rinv), _ptr(out), ld_out, _stream()))
    return out


def forward_check_workspace_bytes(N: int, C_in: int, C_out: int) -> int:
    return int(_lib.aweq_forward_check_workspace_bytes(N, C_in, C_out))


def aweq_forward_check(Xq, act_step, act_zp, Wq, w_step, w_zp, bias_q, X, W, bias, mean_err, sums, ws=None):
    """Mean output error per output channel and sums of squares of the quantised layer
    against the 16-bit layer (argument marshalling only; see ``include/aweq.h``)."""
    N, C_in = X.shape
    C_out = W.shape[0]
    if not (X.is_contiguous() and W.is_contiguous() and Xq.is_contiguous() and Wq.is_contiguous()):
        raise ValueError("aweq_forward_check takes contiguous matrices")
    if ws is None:
        ws = workspace(forward_check_workspace_bytes(N, C_in, C_out), X.device)
    _check(_lib.aweq_forward_check(_ptr(Xq), _ptr(act_step), _ptr(act_zp), _ptr(Wq), _ptr(w_step), _ptr(w_zp),
                                   _ptr(bias_q), _ptr(X), _ptr(W), dtype_tag(X), _ptr(bias), N, C_in, C_out,
                                   _ptr(mean_err), _ptr(sums), _ptr(ws), ws.numel(), _stream()))
    return ws


def forward_check_weights_workspace_bytes(N: int, C_in: int, C_out: int) -> int:
    return int(_lib.aweq_forward_check_weights_workspace_bytes(N, C_in, C_out))


def aweq_forward_check_weights(codes, step, zp, bits, gran, group, rinv, bias_q, X, W, bias, mean_err, sums, ws=None):
    """Forward check of a weight-only layer (argument marshalling only; see ``include/aweq.h``)."""
    N, C_in = X.shape
    C_out = W.shape[0]
    if not (X.is_contiguous() and W.is_contiguous() and codes.is_contiguous()):
        raise ValueError("aweq_forward_check_weights takes contiguous matrices")
    if ws is None:
        ws = workspace(forward_check_weights_workspace_bytes(N, C_in, C_out), X.device)
    _check(_lib.aweq_forward_check_weights(_ptr(codes), _ptr(step), _ptr(zp), bits, gran, group, _ptr(rinv), _ptr(bias_q),
                                           _ptr(X), _ptr(W), dtype_tag(X), _ptr(bias), N, C_in, C_out, _ptr(mean_err),
                                           _ptr(sums), _ptr(ws), ws.numel(), _stream()))
    return ws


def _parr(tensors: Optional[Sequence[Optional[torch.Tensor]]], n: int):
    if tensors is None:
        return None
    arr = (_vp * n)()
    for i, t in enumerate(tensors):
        arr[i] = _ptr(t)
    return arr


class LayerPass:
    """Marshals the arguments of ``aweq_layer_pass`` once so that the call can be
    repeated cheaply; keeps the tensors alive."""

    def __init__(self, X, Ws, bits, gran, group, codes, step, zp, epsmu, bias_in, bias_out, bias_out_f32,
                 xmin, xmax, xmean, wmin, wmax, s, rinv, mu_hat, pX=None, pW=None, scalars=None,
                 Xq=None, act_step=None, act_zp=None, act_bits=8, flags=0, stat_negmin_max=None, stat_sum_count=None):
        n = len(Ws)
        self._keep = (X, Ws, codes, step, zp, epsmu, bias_in, bias_out, bias_out_f32, xmin, xmax, xmean, wmin, wmax,
                      s, rinv, mu_hat, pX, pW, scalars, Xq, act_step, act_zp, stat_negmin_max, stat_sum_count)
        a = LayerArgs()
        a.X, a.dt, a.N, a.C_in, a.ldx = _ptr(X), dtype_tag(X), X.shape[0], X.shape[1], _ld(X)
        a.n_w = n
        self._arrs = dict(
            W=_parr(Ws, n), C_out=(_ll * n)(*[w.shape[0] for w in Ws]), ldw=(_ll * n)(*[_ld(w) for w in Ws]),
            bias_in=_parr(bias_in, n), bias_out=_parr(bias_out, n), bias_out_f32=_parr(bias_out_f32, n),
            codes=_parr(codes, n), step=_parr(step, n), zp=_parr(zp, n), epsmu=_parr(epsmu, n))
        for k, v in self._arrs.items():
            if v is not None:
                setattr(a, k, v)
        a.bits, a.gran, a.group = bits, gran, group
        for k, v in dict(xmin=xmin, xmax=xmax, xmean=xmean, wmin=wmin, wmax=wmax, s=s, rinv=rinv, mu_hat=mu_hat,
                         pX=pX, pW=pW, scalars=scalars, Xq=Xq, act_step=act_step, act_zp=act_zp,
                         stat_negmin_max=stat_negmin_max, stat_sum_count=stat_sum_count).items():
            setattr(a, k, _ptr(v))
        a.act_bits, a.flags = act_bits, flags
        self.args = a
        self.ws_bytes = int(_lib.aweq_layer_pass_workspace_bytes(ctypes.byref(a)))
        # steps 1 and 2 in one launch (the hooks around step 1 then cover the weight ranges too)
        self.fused_ranges = bool(_lib.aweq_layer_pass_fuses_ranges(ctypes.byref(a)))
        self.weight_bytes = sum(w.numel() * w.element_size() for w in Ws)

    def set_events(self, stats=None, act=None) -> None:
        """Profiling hooks: pairs of recorded-once ``torch.cuda.Event(enable_timing=True)``
        (or None) that the library records around step 1 and step 6."""
        def h(e):
            return None if e is None else e.cuda_event
        self._events = (stats, act)
        self.args.ev_stats_begin, self.args.ev_stats_end = (h(stats[0]), h(stats[1])) if stats else (None, None)
        self.args.ev_act_begin, self.args.ev_act_end = (h(act[0]), h(act[1])) if act else (None, None)

    def __call__(self, ws: torch.Tensor, st: Optional[torch.Tensor] = None, phases: int = 0) -> None:
        """``phases``: 0 = the whole pass, or a mask of ``FLAG_PHASE_*`` (see ``include/aweq.h``)."""
        base = self.args.flags & ~(FLAG_PHASE_REDUCE | FLAG_PHASE_QUANT | FLAG_PHASE_ACT)
        self.args.flags = base | phases
        try:
            _check(_lib.aweq_layer_pass(ctypes.byref(self.args), _ptr(ws), ws.numel(), _ptr(st), _stream()))
        finally:
            self.args.flags = base


def aweq_layer_pass(lp: LayerPass, ws: torch.Tensor, st: Optional[torch.Tensor] = None) -> None:
    lp(ws, st)
