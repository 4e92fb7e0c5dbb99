"""Buffer management around ``aweq_layer_pass`` for a whole workload.

A workload (``synth.Workload``) is a set of calibration inputs, each feeding
one or more linear layers.  ``LayerCalibrator`` allocates, once, every output
the C library writes for such a workload (statistics, factors, packed codes,
Step / zero-point arrays, corrected biases, quantised activations) plus one
scratch buffer, marshals the arguments of ``aweq_layer_pass`` once per input,
and ``run()`` then issues one library call per input on the current stream.
It performs no arithmetic of its own.
"""
from __future__ import annotations

from typing import Dict, List, Optional

import torch

from . import aweq, synth


def algorithmic_bytes(wl: synth.Workload, bits: int) -> int:
    """Bytes one layer pass must move: X once for the statistics; every W once
    for its column ranges and once more, plus the packed codes and the
    (Step, Z) pairs, for the fused rescale-quantise-pack; for W8A8 X a second
    time plus one byte per element and a (Step, Z) pair per token."""
    total = 0
    for inp in wl.inputs:
        total += 2 * inp.n_tokens * inp.c_in
        if wl.act_quant:
            total += 3 * inp.n_tokens * inp.c_in + 8 * inp.n_tokens
    for lin in wl.linears:
        n = lin.c_out * lin.c_in
        pairs = lin.c_out if wl.w_gran == "row" else lin.c_out * (lin.c_in // wl.group)
        total += 2 * n + 2 * n + n * bits // 8 + 8 * pairs
    return total


class LayerCalibrator:
    def __init__(self, wl: synth.Workload, bits: int, X: Dict[str, torch.Tensor], W: Dict[str, torch.Tensor],
                 bias: Optional[Dict[str, torch.Tensor]] = None, flags: int = 0, diagnostics: bool = True):
        self.wl, self.bits = wl, bits
        dev = next(iter(X.values())).device
        td = synth.torch_dtype(wl.dtype)
        gran = aweq.PER_ROW if wl.w_gran == "row" else aweq.PER_GROUP
        f32 = dict(dtype=torch.float32, device=dev)
        self.out: Dict[str, Dict[str, torch.Tensor]] = {}
        self.passes: List[aweq.LayerPass] = []
        ws_bytes = 256
        for inp in wl.inputs:
            lins = [l for l in wl.linears if l.input == inp.name]
            if not lins:
                continue
            x = X[inp.name]
            C = inp.c_in
            o = {k: torch.empty(C, **f32) for k in ("xmin", "xmax", "xmean", "wmin", "wmax", "s", "rinv", "mu_hat")}
            if diagnostics:
                o["pX"] = torch.empty(C, **f32)
                o["pW"] = torch.empty(C, **f32)
                o["scalars"] = torch.empty(8, dtype=torch.float64, device=dev)
            if wl.act_quant:
                o["Xq"] = torch.empty((x.shape[0], C), dtype=torch.uint8, device=dev)
                o["act_step"] = torch.empty(x.shape[0], **f32)
                o["act_zp"] = torch.empty(x.shape[0], dtype=torch.int32, device=dev)
            self.out[inp.name] = o
            codes, step, zp, epsmu, b_in, b_out, b_out32 = [], [], [], [], [], [], []
            for l in lins:
                pairs = l.c_out if gran == aweq.PER_ROW else l.c_out * (l.c_in // wl.group)
                lo = {
                    "codes": torch.empty((l.c_out, l.c_in * bits // 8), dtype=torch.uint8, device=dev),
                    "step": torch.empty(pairs, **f32),
                    "zp": torch.empty(pairs, dtype=torch.int32, device=dev),
                    "epsmu": torch.empty(l.c_out, **f32),
                    "bias": torch.empty(l.c_out, dtype=td, device=dev),
                    "bias_f32": torch.empty(l.c_out, **f32),
                }
                self.out[l.name] = lo
                codes.append(lo["codes"]); step.append(lo["step"]); zp.append(lo["zp"]); epsmu.append(lo["epsmu"])
                b_in.append(None if bias is None else bias.get(l.name))
                b_out.append(lo["bias"]); b_out32.append(lo["bias_f32"])
            lp = aweq.LayerPass(
                x, [W[l.name] for l in lins], bits, gran, wl.group, codes, step, zp, epsmu, b_in, b_out, b_out32,
                o["xmin"], o["xmax"], o["xmean"], o["wmin"], o["wmax"], o["s"], o["rinv"], o["mu_hat"],
                o.get("pX"), o.get("pW"), o.get("scalars"), o.get("Xq"), o.get("act_step"), o.get("act_zp"), 8,
                flags)
            ws_bytes = max(ws_bytes, lp.ws_bytes)
            self.passes.append(lp)
        self.ws = aweq.workspace(ws_bytes, dev)
        self.status = aweq.new_status(dev)

    def run(self) -> None:
        """One calibration pass of the whole layer: one library call per input."""
        for lp in self.passes:
            lp(self.ws, self.status)
