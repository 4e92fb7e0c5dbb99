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
import torch.distributed as dist

from . import aweq, synth


algorithmic_bytes = synth.algorithmic_bytes


def exchange_layout(wl: synth.Workload):
    """Where each fed input's statistics sit in the two flat exchange buffers of a token-sharded
    pass: ({input name: (offset into the float32 buffer, offset into the float64 buffer)},
    float32 elements, float64 elements).  An input with C_in channels takes 2 C_in floats
    ({-xmin, xmax}) and C_in + 1 doubles ({column sums, token count}) plus one pad double, so
    every slice starts on a 16-byte boundary.  Sizes only."""
    off, mm, sc = {}, 0, 0
    for inp in wl.inputs:
        if any(l.input == inp.name for l in wl.linears):
            off[inp.name] = (mm, sc)
            mm += 2 * inp.c_in
            sc += inp.c_in + 2
    return off, mm, sc


def schedule_order(wl: synth.Workload) -> List[str]:
    """Order in which the two-stream schedule takes the layer inputs (names).  The weight kernels
    of an input run beside the next input's statistics sweep and those of the last input have
    nothing to hide under, so the input that feeds the fewest weight bytes goes last and the
    one that feeds the most is followed by the longest sweep.  Sizes only; every output is the
    same in any order."""
    fed = [i for i in wl.inputs if any(l.input == i.name for l in wl.linears)]
    if len(fed) < 3:
        return [i.name for i in fed]
    wbytes = {i.name: sum(2 * l.c_out * l.c_in for l in wl.linears if l.input == i.name) for i in fed}
    xbytes = {i.name: 2 * i.n_tokens * i.c_in for i in fed}
    last = min(reversed(fed), key=lambda i: wbytes[i.name])
    rest = [i for i in fed if i is not last]
    heavy = max(rest, key=lambda i: wbytes[i.name])
    long_sweep = max(rest, key=lambda i: xbytes[i.name])
    if long_sweep is not heavy:
        rest.remove(long_sweep)
        rest.insert(rest.index(heavy) + 1, long_sweep)
    return [i.name for i in rest] + [last.name]


class LayerCalibrator:
    def __init__(self, wl: synth.Workload, bits: int, X: Dict[str, torch.Tensor], W: Dict[str, torch.Tensor],
                 bias: Optional[Dict[str, torch.Tensor]] = None, flags: int = 0, diagnostics: bool = True,
                 overlap: bool = False, exchange_buffers: bool = False, order: Optional[List[str]] = None):
        """``overlap``: split every pass into its parts (``FLAG_PHASE_*``) and issue the
        shared-memory-staged, HBM-bound kernels (the column reductions of steps 1-2 and step 6) on
        one CUDA stream and the short kernels of steps 3-5 (factors, weight quantiser) on others,
        each with its own scratch and ordered by events, so that the weight kernels of one input
        fill the tails of the following sweeps;
        ``run()`` forks from and joins back into the current stream.
        ``exchange_buffers``: give every pass the exchange form of its statistics (one flat
        ``float32`` buffer {-xmin, xmax} and one flat ``float64`` buffer {sums, count} over all
        inputs; see ``ShardedLayerCalibrator``).
        ``order``: names of the fed inputs in the order ``run()`` takes them (default: as the
        workload lists them, or ``schedule_order`` with two streams)."""
        self.wl, self.bits = wl, bits
        dev = next(iter(X.values())).device
        td = synth.torch_dtype(wl.dtype)
        gran = aweq.PER_ROW if wl.w_gran == "row" else aweq.PER_GROUP
        f32 = dict(dtype=torch.float32, device=dev)
        self.out: Dict[str, Dict[str, torch.Tensor]] = {}
        self.passes: List[aweq.LayerPass] = []
        ws_bytes = 256
        fed = [i for i in wl.inputs if any(l.input == i.name for l in wl.linears)]
        if order is None and overlap:
            order = schedule_order(wl)
        if order is not None:
            by_name = {i.name: i for i in fed}
            assert sorted(order) == sorted(by_name), "order must name every fed input once"
            fed = [by_name[n] for n in order]
        self.stat_negmin_max = self.stat_sum_count = None
        self._slices = []
        if exchange_buffers:
            layout, n_mm, n_sc = exchange_layout(wl)
            self.stat_negmin_max = torch.empty(n_mm, **f32)
            self.stat_sum_count = torch.zeros(n_sc, dtype=torch.float64, device=dev)
            flags |= aweq.FLAG_MERGED_STATS
        for inp in fed:
            lins = [l for l in wl.linears if l.input == inp.name]
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
            mm = sc = None
            if exchange_buffers:
                mm_off, sc_off = layout[inp.name]
                mm = self.stat_negmin_max[mm_off:mm_off + 2 * C]
                sc = self.stat_sum_count[sc_off:sc_off + C + 1]
                self._slices.append((mm, sc))
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
                flags, mm, sc)
            ws_bytes = max(ws_bytes, lp.ws_bytes)
            self.passes.append(lp)
        self.ws = aweq.workspace(ws_bytes, dev)
        self.status = aweq.new_status(dev)
        self.overlap = bool(overlap) and len(self.passes) > 1 and dev.type == "cuda"
        if self.overlap:
            # One stream for the sweeps; for the weight kernels one stream per input when there is no
            # step 6 (whatever is left when the last sweep ends -- the weight kernels only run in the tails
            # of the sweeps -- then runs side by side: LLaMA-7B pass 1.986 -> 1.969 ms), else a single one
            # (W8A8 passes gained nothing or lost 1 %).  Every stream has scratch of its own.
            nsmall = 1 if wl.act_quant else len(self.passes)
            self._streams = (torch.cuda.Stream(device=dev), [torch.cuda.Stream(device=dev) for _ in range(nsmall)])
            self._ws2 = (self.ws, [aweq.workspace(ws_bytes, dev) for _ in range(nsmall)])
            self._fork = torch.cuda.Event()
            self._ev_stats = [torch.cuda.Event() for _ in self.passes]
            self._ev_weights = [torch.cuda.Event() for _ in self.passes]
        self._fc_ws, self._fc_out = None, {}
        self.equalized = not (flags & aweq.FLAG_NO_EQUALIZE)

    def _exchange(self, i: int) -> None:
        """Between the REDUCE and the QUANT part of pass ``i``, on the stream that runs QUANT:
        nothing for a single device (see ``ShardedLayerCalibrator``)."""

    _split_parts = False            # a subclass with an exchange must run the parts separately

    def run(self) -> None:
        """One calibration pass of the whole layer: one library call per input (or one per part
        of every input, when the parts go to two streams)."""
        if not self.overlap:
            for i, lp in enumerate(self.passes):
                if self._split_parts:
                    lp(self.ws, self.status, aweq.FLAG_PHASE_REDUCE)
                    self._exchange(i)
                    lp(self.ws, self.status, aweq.FLAG_PHASE_QUANT | aweq.FLAG_PHASE_ACT)
                else:
                    lp(self.ws, self.status)
            return
        cur = torch.cuda.current_stream()
        big, smalls = self._streams
        ws_big, ws_smalls = self._ws2
        self._fork.record(cur)
        big.wait_event(self._fork)
        for small in smalls:
            small.wait_event(self._fork)
        n = len(self.passes)

        def stats(i):
            with torch.cuda.stream(big):
                self.passes[i](ws_big, self.status, aweq.FLAG_PHASE_REDUCE)
                self._ev_stats[i].record(big)

        stats(0)
        for i, lp in enumerate(self.passes):
            small, ws_small = smalls[i % len(smalls)], ws_smalls[i % len(smalls)]
            with torch.cuda.stream(small):
                small.wait_event(self._ev_stats[i])
                self._exchange(i)                  # sharded: beside the next input's sweep
                lp(ws_small, self.status, aweq.FLAG_PHASE_QUANT)
                self._ev_weights[i].record(small)
            if i + 1 < n:
                stats(i + 1)                       # the next sweep goes ahead of this input's step 6
            if self.wl.act_quant:
                with torch.cuda.stream(big):
                    big.wait_event(self._ev_weights[i])
                    lp(ws_big, self.status, aweq.FLAG_PHASE_ACT)
        cur.wait_stream(big)
        for small in smalls:
            cur.wait_stream(small)

    def capture(self, events=None) -> "torch.cuda.CUDAGraph":
        """Record one ``run()`` (both streams and their events when ``overlap`` is on) into a CUDA
        graph; ``graph.replay()`` then re-issues the whole pass with one launch.  The library's
        calls are capture-safe (no allocation, no synchronisation).  ``events``: one (stats pair,
        act pair or None) of timing events per pass for the profiling hooks; inside a graph they
        are recorded anew on every replay and hold the times of the latest one.  One ordinary
        ``run()`` happens first (it sets the kernels' shared-memory attributes outside the capture)."""
        for i, lp in enumerate(self.passes):
            if events is None:
                lp.set_events(None, None)
            else:
                lp.set_events(events[i][0], events[i][1])
        self.run()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.run()
        return graph

    def launch_trial(self, graph, steps: int = 3) -> dict:
        """Device time per pass of ``run()`` and of ``graph.replay()`` over ``steps`` passes each
        (CUDA events, a synchronise around each measurement): ``{"eager_ms": .., "graph_ms": ..}``.
        A graph removes the launch gaps, but it also orders the kernels of its branches in its own
        way, so which of the two is faster depends on the workload; a caller that repeats the pass
        (one call per decoder layer) times both once and keeps the faster."""
        def ms(step_fn):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            for _ in range(steps):
                step_fn()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / steps
        return {"eager_ms": ms(self.run), "graph_ms": ms(graph.replay)}

    def forward_check(self, X, W, bias=None, corrected: bool = True):
        """The forward check of every linear after ``run()``: {linear name: (mean_err[C_out],
        sums[4])} as binary64 device tensors.  W8A8 workloads with row-wise 8-bit weights go
        through ``aweq_forward_check`` (integer GEMM on the codes of steps 4 and 6), everything
        else through ``aweq_forward_check_weights`` (16-bit activations).  ``corrected`` gives the
        quantised layer the step-5 bias; otherwise it keeps the original one."""
        wl = self.wl
        w8a8 = wl.act_quant and self.bits == 8 and wl.w_gran == "row"
        gran = aweq.PER_ROW if wl.w_gran == "row" else aweq.PER_GROUP
        dev = self.ws.device
        size = aweq.forward_check_workspace_bytes if w8a8 else aweq.forward_check_weights_workspace_bytes
        need = max(size(X[l.input].shape[0], l.c_in, l.c_out) for l in wl.linears)
        if self._fc_ws is None or self._fc_ws.numel() < need:
            self._fc_ws = aweq.workspace(need, dev)
        res = {}
        for l in wl.linears:
            o, lo = self.out[l.input], self.out[l.name]
            if l.name not in self._fc_out:
                self._fc_out[l.name] = (torch.empty(l.c_out, dtype=torch.float64, device=dev),
                                        torch.empty(4, dtype=torch.float64, device=dev))
            mean_err, sums = self._fc_out[l.name]
            b = None if bias is None else bias.get(l.name)
            bq = lo["bias_f32"] if corrected else None
            if w8a8:
                aweq.aweq_forward_check(o["Xq"], o["act_step"], o["act_zp"], lo["codes"], lo["step"], lo["zp"], bq,
                                        X[l.input], W[l.name], b, mean_err, sums, ws=self._fc_ws)
            else:
                aweq.aweq_forward_check_weights(lo["codes"], lo["step"], lo["zp"], self.bits, gran, wl.group,
                                                o["rinv"] if self.equalized else None, bq, X[l.input], W[l.name], b,
                                                mean_err, sums, ws=self._fc_ws)
            res[l.name] = (mean_err, sums)
        return res


class DecoderWalk:
    """Calibration of one decoder layer in the order that folding diag(s)^-1 into the
    producers requires (Section 3.1: the division by s is fused into the previous block).

    An input produced by a linear layer (``o_in`` by ``v``, ``down_in`` by ``up``, ``fc2_in`` by
    ``fc1``) changes that layer's weights: its factors are computed first (steps 1-3 on the
    input and its consumers), rows of the producer's weight and bias are scaled by 1/s with
    ``aweq_fold_scale``, and only then is every input calibrated with ``aweq_layer_pass`` -- the
    producer is quantised with the fold already in it.  Inputs produced by a normalisation
    layer get the fold in the gain and shift.  ``W`` and ``bias`` are copied; ``artifacts()``
    returns everything a quantised layer needs.  Buffer management and call order only."""

    def __init__(self, wl: synth.Workload, bits: int, X, W, bias=None, norms=None, flags: int = 0):
        self.wl, self.bits, self.X = wl, bits, X
        self.W = {k: v.clone() for k, v in W.items()}
        self.bias = None if bias is None else {k: v.clone() for k, v in bias.items()}
        self.norms = {} if norms is None else {k: tuple(None if t is None else t.clone() for t in v)
                                               for k, v in norms.items()}
        self.producers = synth.producers(wl)
        self.cal = LayerCalibrator(wl, bits, X, self.W, self.bias, flags)
        self.folded = []

    def run(self) -> None:
        wl, cal = self.wl, self.cal
        # 1. inputs whose producer is a linear layer of this workload: factors, then fold
        for inp in wl.inputs:
            kind, prod = self.producers[inp.name]
            if kind != "linear":
                continue
            o = cal.out[inp.name]
            aweq.aweq_stats(self.X[inp.name], o["xmin"], o["xmax"], o["xmean"], ws=cal.ws, st=cal.status)
            for i, l in enumerate(l for l in wl.linears if l.input == inp.name):
                aweq.aweq_wrange(self.W[l.name], o["wmin"], o["wmax"], accumulate=i > 0, ws=cal.ws, st=cal.status)
            aweq.aweq_factors(o["xmin"], o["xmax"], o["xmean"], o["wmin"], o["wmax"], o["s"], o["rinv"], o["mu_hat"],
                              st=cal.status)
            aweq.aweq_fold_scale(self.W[prod], o["rinv"])
            if self.bias is not None and self.bias.get(prod) is not None:
                aweq.aweq_fold_scale(self.bias[prod], o["rinv"])
            self.folded.append((inp.name, "linear", prod))
        # 2. every input with the folded producers in place
        cal.run()
        # 3. normalisation layers take the fold in their gain and shift
        for inp in wl.inputs:
            kind, prod = self.producers[inp.name]
            if kind == "norm" and prod in self.norms:
                for t in self.norms[prod]:
                    if t is not None:
                        aweq.aweq_fold_scale(t, cal.out[inp.name]["rinv"])
                self.folded.append((inp.name, "norm", prod))

    def artifacts(self) -> dict:
        """{linear: codes, step, zp, bias}, {input: s, rinv, act_step, act_zp ...}, folded norms."""
        return {"linears": {l.name: self.cal.out[l.name] for l in self.wl.linears},
                "inputs": {i.name: self.cal.out[i.name] for i in self.wl.inputs if i.name in self.cal.out},
                "norms": self.norms, "folded": list(self.folded)}


def exchange_stats(negmin_max: torch.Tensor, sum_count: torch.Tensor, group=None) -> None:
    """The one exchange of a token-sharded calibration pass, in place, on any backend (NCCL on
    GPUs, gloo on CPU tensors): ``negmin_max`` = {-xmin_j, xmax_j} merges with an element-wise
    MAX, ``sum_count`` = {binary64 column sums, token count} with a SUM."""
    dist.all_reduce(negmin_max, op=dist.ReduceOp.MAX, group=group)
    dist.all_reduce(sum_count, op=dist.ReduceOp.SUM, group=group)


class ShardedLayerCalibrator(LayerCalibrator):
    """Token-sharded pass: every rank holds its own N tokens of each layer input and a replica
    of the weights.  It is the pass of ``LayerCalibrator`` -- same library calls, same two-stream
    schedule -- with one exchange per input between its REDUCE and its QUANT part: the REDUCE
    part leaves the shard's statistics in exchange form, ``exchange_stats`` merges them over the
    ranks (two all-reduces of 2 C_in floats and C_in + 1 doubles), and the QUANT part re-forms
    min / max / mean of the whole calibration set from the merged buffers
    (``FLAG_MERGED_STATS``).  With two streams the exchange sits on the stream of the weight
    kernels, so it runs beside the next input's sweep and only the last one is exposed.  Steps
    2-5 are replicated (W is a few per cent of the bytes); step 6 works on the local shard."""

    _split_parts = True

    def __init__(self, wl, bits, X, W, bias=None, flags=0, group=None, overlap=False):
        super().__init__(wl, bits, X, W, bias, flags, diagnostics=True, overlap=overlap, exchange_buffers=True)
        self.group = group

    def _exchange(self, i: int) -> None:
        mm, sc = self._slices[i]
        exchange_stats(mm, sc, self.group)
