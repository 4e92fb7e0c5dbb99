#!/usr/bin/env python
"""Benchmark of the AWEQ per-linear-layer calibration pass (arXiv 2311.01305).

    python bench.py --gpus N --steps K --warmup W [--workload NAME] [--bits B]
    python bench.py --impl reference ...       # the CPU oracle on a bounded sample

One step is one calibration pass over a whole decoder layer of the workload:
for every distinct layer input, statistics of X, column ranges of the weight
matrices it feeds, equalisation factors, the fused rescale + quantise + pack of
every matrix with its bias correction and, for W8A8 workloads, the per-token
8-bit quantisation of the equalised input.  Inputs are seeded synthetic tensors
with the shapes and value distributions of the named model layer; they are
resident in HBM before the timed region and are far larger than L2.

The metric is layer-pass HBM GB/s: algorithmic bytes of the pass divided by its
device time (CUDA events, max over ranks).  At one GPU the pass runs on two streams and the
steps that carry no profiling hooks replay it from a CUDA graph (--eager, --no-overlap).  With N > 1 every rank calibrates
its own token shard of the same layer (weak scaling); the one exchange of the method, the merge of the
per-channel statistics over the ranks, is an all-reduce inside the timed step.

After the headline region the default 1-GPU run also times, briefly, every other configuration (the same
layer at 3 bits, the two OPT-125M cases, the LLaMA-13B layer, the OPT-66B FFN pair) and the forward check
of two calibrated layers, and reports them under "workloads" / "forward_checks" of the same JSON line
(--no-extras skips that).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2311_01305_b200 import synth  # noqa: E402

DEFAULT_WORKLOAD = "llama7b_layer_w4w3_g128"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1400.0


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


generate = synth.generate


def oracle_pass(wl: synth.Workload, bits: int, Xb, Wb):
    """One layer pass through the CPU oracle on raw-bit arrays (the reference arm
    and the cpu_baseline leg)."""
    from oracle import aweq_oracle as orc
    dt = orc.F16 if wl.dtype == "f16" else orc.BF16
    gran = orc.PER_ROW if wl.w_gran == "row" else orc.PER_GROUP
    for inp in wl.inputs:
        lins = [l for l in wl.linears if l.input == inp.name]
        xs = orc.stats(Xb[inp.name], dt)
        wr = None
        for l in lins:
            wr = orc.wrange(Wb[l.name], dt, prev=wr)
        f = orc.factors(xs[0], xs[1], xs[2], wr[0], wr[1])
        for l in lins:
            codes, step, zp, delta = orc.equalize_quantize(Wb[l.name], dt, f["s"], f["mu_hat"], bits, gran, wl.group)
            orc.bias_correct(delta, None, dt)
        if wl.act_quant:
            orc.quant_act(Xb[inp.name], dt, f["rinv"], orc.PER_ROW)


def cpu_sample(wl_full: synth.Workload, sample_tokens: int):
    """The same layer with only the first ``sample_tokens`` tokens of every input."""
    import dataclasses
    inputs = tuple(dataclasses.replace(i, n_tokens=min(sample_tokens, i.n_tokens)) for i in wl_full.inputs)
    return dataclasses.replace(wl_full, inputs=inputs)


def workload_config(wl: synth.Workload, bits: int, world: int) -> dict:
    """The ``config`` object of the JSON line: what is calibrated, the same for both arms."""
    return {"workload": wl.name, "w_bits": bits, "w_gran": wl.w_gran, "group": wl.group,
            "act_quant": wl.act_quant, "storage": wl.dtype, "tokens_per_gpu": wl.inputs[0].n_tokens,
            "algorithmic_bytes_per_gpu": synth.algorithmic_bytes(wl, bits),
            "cache": "inputs (GBs) far larger than the 126 MB L2",
            "parallelism": "token shards, one per GPU" if world > 1 else "single GPU"}


def sample_text(wl: synth.Workload, sample_tokens: int) -> str:
    n = min(sample_tokens, wl.inputs[0].n_tokens)
    return "first %d of %d tokens of every layer input, all weight matrices at full size" % (n, wl.inputs[0].n_tokens)


def run_reference(args, wl, bits):
    """The oracle arm: the CPU oracle alone (this process never loads the CUDA library)."""
    from oracle import aweq_oracle as orc
    if int(os.environ.get("RANK", "0")) != 0:
        return
    swl = cpu_sample(wl, args.cpu_sample_tokens)
    X, W = generate(swl, "cpu", 0)
    Xb = {k: synth.raw_bits(v) for k, v in X.items()}
    Wb = {k: synth.raw_bits(v) for k, v in W.items()}
    nbytes = synth.algorithmic_bytes(swl, bits)
    for _ in range(args.warmup):
        oracle_pass(swl, bits, Xb, Wb)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_pass(swl, bits, Xb, Wb)
    dt = (time.perf_counter() - t0) / args.steps
    gbs = nbytes / dt / 1e9
    sample = sample_text(wl, args.cpu_sample_tokens)
    line = {
        "impl": "reference", "metric": "aweq_layer_pass_hbm_gbs", "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(wl, bits, max(1, args.gpus)),
        "tokens_per_s": swl.inputs[0].n_tokens / dt,
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": orc.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def gemm_peak():
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        try:
            return float(json.load(open(pk))["bf16_tflops_sustained"]), "measured (sustained)"
        except Exception:
            pass
    return FALLBACK_BF16_TFLOPS, "fallback"


def time_forward_check(wl, bits, X, W, steps, warmup):
    """Forward check of every linear of the calibrated layer: (summary dict, last results, calibrator)."""
    from paper_2311_01305_b200 import aweq, calibrate
    cal = calibrate.LayerCalibrator(wl, bits, X, W, None)
    cal.run()
    res = None
    for _ in range(max(1, warmup)):
        res = cal.forward_check(X, W)
    torch.cuda.synchronize()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    time.sleep(0.15)
    n0 = aweq.launch_count()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        res = cal.forward_check(X, W)
    b.record()
    torch.cuda.synchronize()
    launches = aweq.launch_count() - n0
    clocks = sampler.stop()
    ms = a.elapsed_time(b) / steps
    tokens = {i.name: i.n_tokens for i in wl.inputs}
    flops = sum(4.0 * tokens[l.input] * l.c_in * l.c_out for l in wl.linears)
    p16, kind = gemm_peak()
    w8a8 = wl.act_quant and bits == 8 and wl.w_gran == "row"
    peak = p16 * 2.0 / 1.5 if w8a8 else p16           # weight-only: both contractions are 16-bit
    tf = flops / ms / 1e9
    out = {"ms_per_step": ms, "tflops": tf, "w8a8": w8a8, "launches": int(launches), "clocks": clocks,
           "tokens": tokens, "steps": steps,
           "roofline": {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
                        "peak_kind": ("16-bit GEMM rate of %s x 4/3 for the 8-bit / 16-bit mix" if w8a8
                                      else "16-bit GEMM rate of %s") % kind, "traffic": None}}
    return out, res, cal


def run_forward_check(args, wl, bits):
    """Secondary benchmark: the forward check of every linear of a calibrated layer.
    A step is one check of the whole layer; the work is two dense contractions per linear
    (2 N C_in C_out flops each), so the bound is the tensor pipe.  For W8A8 layers the peak is
    the measured 16-bit GEMM rate scaled for the mix: the 8-bit half runs at twice the 16-bit
    rate (nominal ratio), so 2F flops take at best 1.5 F / P16."""
    from paper_2311_01305_b200 import aweq, calibrate
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    X, W = generate(wl, dev, 0)
    fc, res, cal = time_forward_check(wl, bits, X, W, args.steps, args.warmup)
    worst = {n: float((me.abs().max() / (s4[1] / s4[3]).sqrt()).item()) for n, (me, s4) in res.items()}
    sqnr = {n: float(10.0 * torch.log10(s4[1] / s4[0]).item()) for n, (me, s4) in res.items()}
    # ablation (outside the timed region): equalisation and bias correction switched on and off
    del cal
    ablation = {}
    for eq in (True, "absmax", False):
        for bc in (True, False):
            if eq == "absmax" and not bc:
                continue
            flags = (0 if eq else aweq.FLAG_NO_EQUALIZE) | (0 if bc else aweq.FLAG_NO_BIAS_CORRECT)
            flags |= aweq.FLAG_ABSMAX_CRITERION if eq == "absmax" else 0
            c = calibrate.LayerCalibrator(wl, bits, X, W, None, flags=flags)
            c.run()
            r = c.forward_check(X, W, corrected=bc)
            torch.cuda.synchronize()
            name = "abs-max criterion" if eq == "absmax" else ("AWE" if eq else "no AWE")
            ablation[name + (" + BC" if bc else "")] = {
                "output_sqnr_db": {n: round(float(10.0 * torch.log10(s4[1] / s4[0]).item()), 3)
                                   for n, (me, s4) in r.items()},
                "rms_mean_err_over_output_rms": {n: float(((s4[2] / me.numel()) / (s4[1] / s4[3])).sqrt().item())
                                                 for n, (me, s4) in r.items()}}
            del c, r
    print(json.dumps({
        "metric": "aweq_forward_check_tflops", "value": fc["tflops"], "unit": "TFLOP/s", "n_gpus": 1,
        "steps": args.steps, "warmup": max(1, args.warmup), "ms_per_step": fc["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": ("u8 x u8 -> s32 and %s -> f32" if fc["w8a8"] else "%s -> f32 (two contractions)") % wl.dtype,
        "data": "synthetic",
        "config": {"workload": wl.name, "tokens": fc["tokens"], "linears": [l.name for l in wl.linears],
                   "cache": "operands (GBs) far larger than the 126 MB L2"},
        "roofline": fc["roofline"], "clocks": fc["clocks"], "gpu_launches": fc["launches"],
        "max_abs_mean_err_over_output_rms": worst, "output_sqnr_db": sqnr, "ablation": ablation}))


# ncu DRAM counters of ONE whole layer pass at full size, as scheduled in the timed region (two
# streams, eager), taken as a single profiler range (dram__bytes_read.sum, dram__bytes_write.sum):
# {(workload, bits): (bytes read, bytes written)}.  Compared with the algorithmic bytes they say how
# much of the pass the L2 served.  The kernels have not changed since the counters were taken.
PASS_DRAM_BYTES = {("llama7b_layer_w4w3_g128", 4): (13027861248, 108804096),
                   ("llama7b_layer_w4w3_g128", 3): (13019588864, 86600960),
                   ("llama13b_layer_w8a8", 8): (31903268608, 7977698304),
                   ("opt66b_ffn_w8a8", 8): (26883141376, 6708150784),
                   ("opt125m_model_w8a8", 8): (5662176768, 1417811968)}
# Share of the second read of W (step 4, after step 2 has streamed the same matrices) that the L2 serves
# instead of HBM.  "scheduled": from the range capture above (algorithmic read bytes minus DRAM read bytes,
# over one read of W); a statistics sweep of the next input runs between the two reads and flushes the L2.
# "one_stream": per-kernel DRAM read bytes of the step-4 kernels with every kernel of a pass serialised
# (one stream, 1/32 of the tokens; weights are full size at any token count): what the L2 could serve.
W_SECOND_READ_FROM_L2 = {("llama7b_layer_w4w3_g128", 4): {"scheduled": 0.0, "one_stream": 0.605},
                         ("llama7b_layer_w4w3_g128", 3): {"scheduled": 0.009, "one_stream": 0.618}}
# DRAM traffic of the statistics sweep per launch, from a one-kernel capture at 1/8 of the tokens
# (268.44 MB of X and 100.66 MB of W in one launch: 369.21 MB read): reads grow with the rows; the few MB written during the launch are
# dirty lines of earlier kernels leaving the L2, not traffic of the sweep.
STATS_DRAM_READ_RATIO = 1.0003


def time_layer_pass(wl, bits, X, W, steps, warmup, *, rank=0, world=1, local=0, dist=None,
                    overlap=True, eager=False, graph_only=False):
    """Times ``steps`` layer passes of one workload (CUDA events on the launching stream, max over
    ranks) and, on every fourth of them, the dominant kernel through the library's event hooks.
    Returns (calibrator, result dict)."""
    from paper_2311_01305_b200 import aweq, calibrate
    dev = next(iter(X.values())).device
    cal = (calibrate.ShardedLayerCalibrator(wl, bits, X, W, None, overlap=overlap) if world > 1
           else calibrate.LayerCalibrator(wl, bits, X, W, None, overlap=overlap))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # profiling hooks around step 1 (and step 6) of every library call in the timed region
    def ev_pair():
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); b.record()              # create the handles
        return a, b
    # every fourth timed step carries the hooks (two event records per sweep cost 0.7 % of a pass, because
    # a record between two kernels undoes their programmatic overlap); the others run without them
    hooked = [k for k in range(steps) if k % 4 == 0]
    hooks = {k: [(ev_pair(), ev_pair() if wl.act_quant else None) for _ in cal.passes] for k in hooked}
    torch.cuda.synchronize()

    for _ in range(warmup):
        cal.run()
    graph = None
    if world == 1 and not eager:
        try:
            graph = cal.capture()           # without the event hooks: as graph nodes they cost 3 % of the pass
            for _ in range(warmup):
                graph.replay()
        except Exception as exc:            # a capture that fails leaves the eager pass as it was
            sys.stderr.write("CUDA graph capture failed (%s); timing eager launches\n" % exc)
            graph = None
            torch.cuda.synchronize()
    # Replaying the pass from a graph removes the launch gaps, but the graph also orders the kernels of the
    # two streams in its own way, which some workloads pay for (more weight kernels beside the per-token
    # quantiser): a short trial of both launch modes before the timed region picks the one that is timed.
    trial = None
    if graph is not None and not graph_only:
        trial = cal.launch_trial(graph, 3)
        if trial["eager_ms"] < 0.995 * trial["graph_ms"]:
            graph = None
    mixed = graph is not None and not graph_only
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.15)
    n0 = aweq.launch_count()
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_begin.record()
    for k in range(steps):
        if graph is not None and not (mixed and k in hooks):
            graph.replay()
        else:
            for i, lp in enumerate(cal.passes):
                es, ea = hooks[k][i] if k in hooks else (None, None)
                lp.set_events(es, ea)
            cal.run()                       # N > 1: the statistics are merged over the ranks inside the step
    t_end.record()
    barrier()
    launches = aweq.launch_count() - n0
    clocks = sampler.stop()
    if mixed:
        # replays go through no library call: a replay launches what an eager step launches
        launches = launches // len(hooks) * steps
    elif graph is not None:
        # replays go through no library call: a replay launches what one eager pass launches.  The
        # dominant kernel is timed in eager passes after the timed region (hooks inside the graph
        # would be recorded by every replay, but as graph nodes of their own they slow it down).
        torch.cuda.synchronize()
        n1 = aweq.launch_count()
        for k in range(steps):
            for i, lp in enumerate(cal.passes):
                es, ea = hooks[k][i] if k in hooks else (None, None)
                lp.set_events(es, ea)
            cal.run()
        torch.cuda.synchronize()
        launches = aweq.launch_count() - n1
    for lp in cal.passes:
        lp.set_events(None, None)
    ms = t_begin.elapsed_time(t_end) / steps
    if dist is not None:
        t = torch.tensor([ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    status = aweq.read_status(cal.status)
    if status["wait_timeout"]:
        raise SystemExit("a bounded wait inside a kernel gave up: results invalid")

    # dominant kernel: the statistics sweep (W8A8 workloads: the activation quantiser moves more bytes)
    stats_ms = [sum(es[0].elapsed_time(es[1]) for es, _ in hk) for hk in hooks.values()]
    # where steps 1 and 2 of an input share one launch, the hooks around step 1 time both: count the weights too
    fused_w = sum(lp.weight_bytes for lp in cal.passes if lp.fused_ranges)
    stats_bytes = sum(2 * i.n_tokens * i.c_in for i in wl.inputs) + fused_w
    dom = {"kernel": "colreduce_kernel (aweq_stats" + (" + aweq_wrange, one launch" if fused_w else "") + ")", "bytes": stats_bytes, "ms": statistics.mean(stats_ms),
           "launches_per_step": len(cal.passes)}
    if wl.act_quant:
        act_ms = [sum(ea[0].elapsed_time(ea[1]) for _, ea in hk) for hk in hooks.values()]
        act_bytes = sum(3 * i.n_tokens * i.c_in + 8 * i.n_tokens for i in wl.inputs)
        dom = {"kernel": "per-token quantiser: rowdirect_kernel (aweq_quant_act)", "bytes": act_bytes,
               "ms": statistics.mean(act_ms), "launches_per_step": len(cal.passes),
               "stats_gbs": stats_bytes / statistics.mean(stats_ms) / 1e6}
    peak, peak_kind = measured_peaks()
    achieved = dom["bytes"] / dom["ms"] / 1e6
    roofline = {"bound": "hbm", "kernel": dom["kernel"], "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": "of " + peak_kind, "traffic": None,
                "launch_ms": dom["ms"] / dom["launches_per_step"], "timed_steps": sorted(hooks.keys()),
                "bytes_per_launch": dom["bytes"] / dom["launches_per_step"]}
    if "stats_gbs" in dom:
        roofline["stats_gbs"] = dom["stats_gbs"]
    nbytes = synth.algorithmic_bytes(wl, bits)
    gbs = world * nbytes / ms / 1e6
    l2_both = W_SECOND_READ_FROM_L2.get((wl.name, bits))
    overlap_on = bool(getattr(cal, "overlap", False))
    l2 = None if l2_both is None else l2_both["scheduled" if overlap_on else "one_stream"]
    roofline["w_second_read_from_l2"] = l2
    roofline["w_second_read_from_l2_one_stream"] = None if l2_both is None else l2_both["one_stream"]
    if not wl.act_quant and world == 1:
        roofline["traffic"] = STATS_DRAM_READ_RATIO * roofline["bytes_per_launch"]
    dram = PASS_DRAM_BYTES.get((wl.name, bits)) if (overlap_on and world == 1 and wl.inputs[0].n_tokens == synth.workloads()[wl.name].inputs[0].n_tokens) else None
    res = {"ms": ms, "gbs": gbs, "nbytes": nbytes, "launches": int(launches), "clocks": clocks, "status": status,
           "roofline": roofline, "peak": peak,
           "pass_dram": None if dram is None else {"read_bytes": dram[0], "write_bytes": dram[1],
                                                   "over_algorithmic": (dram[0] + dram[1]) / nbytes},
           "gbs_hbm_basis": None if l2 is None else world * (nbytes - l2 * synth.weight_bytes(wl)) / ms / 1e6,
           "launch": ("CUDA graph replay; every fourth step eager, with the event hooks" if mixed
                      else "one CUDA graph replay per step" if graph is not None else "eager"),
           "launch_trial": trial,
           "schedule": ("column reductions and step 6 on one stream, factors and weight quantisers on others (one per input for weight-only workloads, one in all for W8A8)"
                        if getattr(cal, "overlap", False) else "one stream")}
    return cal, res


EXTRA_WORKLOADS = (("llama7b_layer_w4w3_g128", 3), ("opt125m_linear_w8a8", 8), ("opt125m_model_w8a8", 8),
                   ("llama13b_layer_w8a8", 8), ("opt66b_ffn_w8a8", 8))
EXTRA_FORWARD_CHECKS = (("llama7b_layer_w4w3_g128", 4), ("llama13b_layer_w8a8", 8))


def run_extras(args, dev, skip):
    """Every configuration other than the headline one, timed briefly on the same box with the same
    code as the headline region (one GPU), and the forward check of two calibrated layers."""
    table, checks = {}, {}
    wls = synth.workloads(args.tokens_scale)
    for name, bits in EXTRA_WORKLOADS:
        if (name, bits) == skip:
            continue
        wl = wls[name]
        X, W = generate(wl, dev, 0)
        cal, r = time_layer_pass(wl, bits, X, W, args.extra_steps, args.warmup, overlap=not args.no_overlap,
                                 eager=args.eager, graph_only=args.graph)
        rf = r["roofline"]
        table["%s@w%d" % (name, bits)] = {
            "bits": bits, "ms_per_step": r["ms"], "gbs": r["gbs"], "gbs_hbm_basis": r["gbs_hbm_basis"],
            "pass_dram": r["pass_dram"],
            "pct_of_8000_gbs": 100.0 * r["gbs"] / NOMINAL_HBM_GBS,
            "pct_of_measured_copy": 100.0 * r["gbs"] / r["peak"], "tokens_per_s": wl.inputs[0].n_tokens / (r["ms"] / 1e3),
            "algorithmic_bytes": r["nbytes"], "steps": args.extra_steps, "gpu_launches": r["launches"],
            "dominant_kernel": rf["kernel"], "frac": rf["frac"], "dominant_gbs": rf["achieved"],
            "stats_gbs": rf.get("stats_gbs", rf["achieved"]), "launch": r["launch"], "launch_trial": r["launch_trial"],
            "sm_mhz": r["clocks"].get("sm_mhz"), "reasons": r["clocks"].get("reasons")}
        del cal, X, W
        torch.cuda.empty_cache()
    if not args.no_forward_check:
        for name, bits in EXTRA_FORWARD_CHECKS:
            wl = wls[name]
            X, W = generate(wl, dev, 0)
            fc, res, cal = time_forward_check(wl, bits, X, W, 2, 1)
            checks["%s@w%d" % (name, bits)] = {
                "ms_per_step": fc["ms_per_step"], "tflops": fc["tflops"], "frac": fc["roofline"]["frac"],
                "peak": fc["roofline"]["peak"], "peak_kind": fc["roofline"]["peak_kind"], "steps": fc["steps"],
                "gpu_launches": fc["launches"], "sm_mhz": fc["clocks"].get("sm_mhz"),
                "reasons": fc["clocks"].get("reasons"),
                "output_sqnr_db": {n: round(float(10.0 * torch.log10(s4[1] / s4[0]).item()), 3)
                                   for n, (me, s4) in res.items()}}
            del cal, res, X, W
            torch.cuda.empty_cache()
    return table, checks


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--bits", type=int, default=0, help="weight bit-width (default: the workload's first)")
    ap.add_argument("--tokens-scale", type=float, default=1.0, help="shrink the token count (profiling captures)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-sample-tokens", type=int, default=262144)
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the short timed passes of the other configurations after the headline region")
    ap.add_argument("--extra-steps", type=int, default=8, help="timed steps of each of those passes")
    ap.add_argument("--no-forward-check", action="store_true", help="leave the forward checks out of the extras")
    ap.add_argument("--no-overlap", action="store_true",
                    help="issue every input's pass on one stream (default: two alternating streams)")
    ap.add_argument("--eager", action="store_true",
                    help="launch every timed step eagerly (default at 1 GPU: the steps that carry the event hooks "
                         "are eager, the others replay the pass from a CUDA graph)")
    ap.add_argument("--graph", action="store_true",
                    help="replay the pass as one CUDA graph in the timed region (1 GPU; the dominant kernel is then "
                         "timed in eager passes after it)")
    ap.add_argument("--profile-pass", action="store_true",
                    help="after the timed region, issue one more eager pass between cudaProfilerStart and "
                         "cudaProfilerStop (a range for a profiler started with profiling off; not timed)")
    ap.add_argument("--op", default="layer_pass", choices=["layer_pass", "forward_check"],
                    help="forward_check: time the forward check of the calibrated layer instead (1 GPU)")
    args = ap.parse_args()

    wl = synth.workloads(args.tokens_scale)[args.workload]
    bits = args.bits or wl.w_bits[0]
    if args.impl == "reference":
        return run_reference(args, wl, bits)

    from paper_2311_01305_b200 import build as _build
    _build.build()                      # no-op when libaweq.so is up to date
    from paper_2311_01305_b200 import aweq  # noqa: F401  (fails loudly when the library is missing)

    if args.op == "forward_check":
        return run_forward_check(args, wl, bits)
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the calibration pass has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    X, W = generate(wl, dev, rank)
    cal, r = time_layer_pass(wl, bits, X, W, args.steps, args.warmup, rank=rank, world=world, local=local, dist=dist,
                             overlap=not args.no_overlap, eager=args.eager, graph_only=args.graph)
    ms, gbs, nbytes, peak = r["ms"], r["gbs"], r["nbytes"], r["peak"]
    tokens = wl.inputs[0].n_tokens
    line = {
        "metric": "aweq_layer_pass_hbm_gbs", "value": gbs, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": workload_config(wl, bits, world),
        "launch_config": {"launch": r["launch"], "launch_trial": r["launch_trial"], "schedule": r["schedule"]},
        "tokens_per_s": world * tokens / (ms / 1e3),
        "pct_of_8000_gbs": 100.0 * gbs / world / NOMINAL_HBM_GBS,
        "pct_of_measured_copy": 100.0 * gbs / world / peak,
        "value_hbm_basis": r["gbs_hbm_basis"], "pass_dram": r["pass_dram"],
        "basis_note": ("value counts every algorithmic byte; value_hbm_basis leaves out the part of the second read "
                       "of W that the L2 serves (roofline.w_second_read_from_l2, from ncu DRAM counters of one whole "
                       "pass as scheduled: pass_dram). A percentage of the measured copy bandwidth above 100 is a "
                       "read-mostly stream against a read+write copy, not more than the HBM can deliver"),
        "roofline": r["roofline"], "clocks": r["clocks"], "gpu_launches": r["launches"], "device_status": r["status"],
    }

    if args.profile_pass and world == 1:
        torch.cuda.synchronize()
        torch.cuda.profiler.start()
        cal.run()
        torch.cuda.synchronize()
        torch.cuda.profiler.stop()

    # ---------------------------------------------------------------- end to end: host buffers in, results out
    if not args.no_e2e:
        hostX = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v) for k, v in X.items()}
        hostW = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v) for k, v in W.items()}
        res_names = {l.name: ("codes", "step", "zp", "bias") for l in wl.linears}
        res_names.update({i.name: ("s",) + (("Xq", "act_step", "act_zp") if wl.act_quant else ()) for i in wl.inputs})
        host_out = {n: {k: torch.empty(cal.out[n][k].shape, dtype=cal.out[n][k].dtype, pin_memory=True)
                        for k in ks} for n, ks in res_names.items() if n in cal.out}
        h2d = sum(v.numel() * v.element_size() for v in list(hostX.values()) + list(hostW.values()))
        d2h = sum(t.numel() * t.element_size() for d in host_out.values() for t in d.values())

        def e2e_step():
            for k, v in hostW.items():
                W[k].copy_(v, non_blocking=True)
            for k, v in hostX.items():
                X[k].copy_(v, non_blocking=True)
            cal.run()
            for n, d in host_out.items():
                for k, t in d.items():
                    t.copy_(cal.out[n][k], non_blocking=True)
        e2e_step()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.e2e_steps):
            e2e_step()
        b.record()
        barrier()
        ems = a.elapsed_time(b) / args.e2e_steps
        if dist is not None:
            t = torch.tensor([ems], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ems = float(t.item())
        line["e2e"] = {"value": world * nbytes / ems / 1e6, "unit": "GB/s", "ms_per_step": ems,
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps}
        del hostX, hostW, host_out

    # ---------------------------------------------------------------- the oracle beside it (rank 0, 1 GPU)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import aweq_oracle as orc
        swl = cpu_sample(wl, args.cpu_sample_tokens)
        Xb = {i.name: synth.raw_bits(X[i.name][:i.n_tokens]) for i in swl.inputs}
        Wb = {k: synth.raw_bits(v) for k, v in W.items()}
        t0 = time.perf_counter()
        oracle_pass(swl, bits, Xb, Wb)
        dt = time.perf_counter() - t0
        sbytes = synth.algorithmic_bytes(swl, bits)
        line["cpu_baseline"] = {"value": sbytes / dt / 1e9, "unit": "GB/s", "cores": orc.threads(), "kind": "oracle",
                                "seconds": dt, "tokens_per_s": swl.inputs[0].n_tokens / dt,
                                "sample": sample_text(wl, args.cpu_sample_tokens)}
        del Xb, Wb

    # ---------------------------------------------------------------- the other configurations, briefly
    if world == 1 and not args.no_extras:
        del cal, X, W
        torch.cuda.empty_cache()
        line["workloads"], line["forward_checks"] = run_extras(args, dev, (wl.name, bits))
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
