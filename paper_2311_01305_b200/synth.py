"""Seeded synthetic inputs for the AWEQ calibration pass.

Stand-ins for the OPT / LLaMA linear layers and calibration activations the
paper evaluates on (its Section 4): the real weights and calibration text are
not available, so shapes, dtypes and value distributions are reproduced and
the values are drawn from a seeded generator.  This module holds no part of
the method's arithmetic; it only draws numbers and casts them to 16 bits.
The resulting 16-bit values are the canonical inputs: a test generates them
once (on the CPU, or on the GPU for the full-size cases), and hands the same
bits to the CUDA library and to the CPU oracle.

Activations: i.i.d. per element from a base distribution (standard normal,
Student-t with nu degrees of freedom, or Laplace(0, 1)), then a seeded choice
of "outlier" columns is multiplied by a factor (fixed, or uniform in a range),
which is the structure Section 2 ("Quantization Difficulty") describes: a few
activation channels carry values tens of times larger than the rest.
Weights: i.i.d. normal with a small standard deviation.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence, Tuple, Union

import torch

F16_MAX = 65504.0


@dataclasses.dataclass(frozen=True)
class ActSpec:
    """One calibration input X[N, C_in]."""
    name: str
    n_tokens: int
    c_in: int
    dist: str                      # "normal" | "student_t" | "laplace"
    nu: int = 0                    # degrees of freedom for student_t
    n_outliers: int = 0            # number of outlier columns
    outlier_scale: Union[float, Tuple[float, float]] = 1.0   # fixed, or U[lo, hi] per column


@dataclasses.dataclass(frozen=True)
class LinearSpec:
    """One linear layer W[C_out, C_in] fed by the input called ``input``."""
    name: str
    c_out: int
    c_in: int
    input: str
    w_std: float


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    dtype: str                     # "f16" | "bf16"
    seed: int
    inputs: Tuple[ActSpec, ...]
    linears: Tuple[LinearSpec, ...]
    w_bits: Tuple[int, ...]        # weight bit-widths to run
    w_gran: str                    # "row" (per output channel) | "group"
    group: int                     # group size when w_gran == "group"
    act_quant: bool                # W8A8: also quantise activations per token
    layers: int = 1                # identical layers (distinct seeds) in the model


def _opt125m_layer(n_tokens: int, dist: str, nu: int, frac: float, scale) -> Tuple[Tuple[ActSpec, ...], Tuple[LinearSpec, ...]]:
    h, f = 768, 3072
    def k(c):
        return max(1, math.ceil(c * frac))
    inputs = (
        ActSpec("attn_in", n_tokens, h, dist, nu, k(h), scale),
        ActSpec("o_in", n_tokens, h, dist, nu, k(h), scale),
        ActSpec("fc1_in", n_tokens, h, dist, nu, k(h), scale),
        ActSpec("fc2_in", n_tokens, f, dist, nu, k(f), scale),
    )
    linears = (
        LinearSpec("q", h, h, "attn_in", 0.02), LinearSpec("k", h, h, "attn_in", 0.02),
        LinearSpec("v", h, h, "attn_in", 0.02), LinearSpec("o", h, h, "o_in", 0.02),
        LinearSpec("fc1", f, h, "fc1_in", 0.02), LinearSpec("fc2", h, f, "fc2_in", 0.02),
    )
    return inputs, linears


def _llama_layer(n_tokens: int, h: int, f: int, dist: str, nu: int, n_out, scale, w_std: float):
    inputs = (
        ActSpec("attn_in", n_tokens, h, dist, nu, n_out(h), scale),
        ActSpec("o_in", n_tokens, h, dist, nu, n_out(h), scale),
        ActSpec("mlp_in", n_tokens, h, dist, nu, n_out(h), scale),
        ActSpec("down_in", n_tokens, f, dist, nu, n_out(f), scale),
    )
    linears = (
        LinearSpec("q", h, h, "attn_in", w_std), LinearSpec("k", h, h, "attn_in", w_std),
        LinearSpec("v", h, h, "attn_in", w_std), LinearSpec("o", h, h, "o_in", w_std),
        LinearSpec("gate", f, h, "mlp_in", w_std), LinearSpec("up", f, h, "mlp_in", w_std),
        LinearSpec("down", h, f, "down_in", w_std),
    )
    return inputs, linears


def workloads(n_tokens_scale: float = 1.0) -> dict:
    """The five benchmark configurations.  ``n_tokens_scale`` shrinks the token
    counts (tests use it to get the same shapes at sizes a CPU finishes fast)."""
    def nt(n):
        return max(8, int(n * n_tokens_scale))
    w = {}
    w["opt125m_linear_w8a8"] = Workload(
        "opt125m_linear_w8a8", "f16", 0,
        (ActSpec("x", nt(2048), 768, "normal", 0, 6, 40.0),),
        (LinearSpec("linear", 768, 768, "x", 0.02),),
        (8,), "row", 0, True)
    i, l = _opt125m_layer(nt(128 * 2048), "student_t", 4, 0.01, (20.0, 60.0))
    w["opt125m_model_w8a8"] = Workload("opt125m_model_w8a8", "f16", 2, i, l, (8,), "row", 0, True, layers=12)
    i, l = _llama_layer(nt(128 * 2048), 4096, 11008, "student_t", 3, lambda c: math.ceil(c / 512), 50.0, 0.02)
    w["llama7b_layer_w4w3_g128"] = Workload("llama7b_layer_w4w3_g128", "bf16", 3, i, l, (4, 3), "group", 128, False)
    i, l = _llama_layer(nt(128 * 2048), 5120, 13824, "normal", 0, lambda c: math.ceil(c * 0.005), 80.0, 0.015)
    w["llama13b_layer_w8a8"] = Workload("llama13b_layer_w8a8", "f16", 4, i, l, (8,), "row", 0, True)
    w["opt66b_ffn_w8a8"] = Workload(
        "opt66b_ffn_w8a8", "f16", 5,
        (ActSpec("fc1_in", nt(64 * 2048), 9216, "laplace", 0, 8, 100.0),
         ActSpec("fc2_in", nt(64 * 2048), 36864, "laplace", 0, 8, 100.0)),
        (LinearSpec("fc1", 36864, 9216, "fc1_in", 0.01), LinearSpec("fc2", 9216, 36864, "fc2_in", 0.01)),
        (8,), "row", 0, True)
    return w


def algorithmic_bytes(wl: Workload, bits: int) -> int:
    """Bytes one layer pass must move: X once for the statistics; every W once
    for its column ranges and once more, plus the packed codes and the
    (Step, Z) pairs, for the fused rescale-quantise-pack; for W8A8 X a second
    time plus one byte per element and a (Step, Z) pair per token.  Bookkeeping
    for the benchmark: sizes only."""
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


def weight_bytes(wl: Workload) -> int:
    """Bytes of all 16-bit weight matrices of the workload (one read of W)."""
    return sum(2 * lin.c_out * lin.c_in for lin in wl.linears)


def generate(wl: Workload, device, rank: int = 0):
    """Every input and weight tensor of a workload: ({input name: X}, {linear name: W}).
    ``rank`` selects the token shard (its own seed); the weights are the same on every rank."""
    X, W = {}, {}
    for i, inp in enumerate(wl.inputs):
        X[inp.name] = make_activations(inp, wl.dtype, tensor_seed(wl.seed, rank, i), device)
    for i, lin in enumerate(wl.linears):
        W[lin.name] = make_weight(lin, wl.dtype, tensor_seed(wl.seed, 0, 100 + i), device)
    return X, W


def producers(wl: Workload) -> dict:
    """What produces each layer input of a decoder-shaped workload: {input name: (kind, name)}
    with kind "norm" (a normalisation layer's output: its gain and shift take 1/s) or
    "linear" (channel j of the input is a positive multiple of output channel j of that
    linear layer: the value projection seen through the attention weights, ``up`` through the
    gate, ``fc1`` through ReLU).  Structure only; the folding itself is the library's."""
    table = {"attn_in": ("norm", "ln_attn"), "o_in": ("linear", "v"), "mlp_in": ("norm", "ln_mlp"),
             "down_in": ("linear", "up"), "fc1_in": ("norm", "ln_mlp"), "fc2_in": ("linear", "fc1"),
             "x": ("norm", "ln")}
    names = {l.name for l in wl.linears}
    out = {}
    for i in wl.inputs:
        kind, name = table[i.name]
        if kind == "linear" and name not in names:
            kind, name = "none", ""            # the producer is not part of this workload
        out[i.name] = (kind, name)
    return out


def make_norm(c: int, dtype: str, seed: int, device="cpu", shift: bool = True):
    """Gain (around 1) and shift (around 0) of a normalisation layer, 16-bit."""
    g = _generator(seed, "cpu")
    gain = (1.0 + 0.1 * torch.randn(c, generator=g)).to(torch_dtype(dtype)).to(device)
    beta = (0.05 * torch.randn(c, generator=g)).to(torch_dtype(dtype)).to(device) if shift else None
    return gain, beta


def torch_dtype(name: str) -> torch.dtype:
    return {"f16": torch.float16, "bf16": torch.bfloat16}[name]


def _generator(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _base(shape, dist: str, nu: int, g: torch.Generator, device) -> torch.Tensor:
    if dist == "normal":
        return torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    if dist == "student_t":
        # z / sqrt(chi2_nu / nu), chi2 as a sum of nu squared normals
        z = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
        chi2 = torch.zeros(shape, device=device, dtype=torch.float32)
        for _ in range(nu):
            chi2 += torch.randn(shape, generator=g, device=device, dtype=torch.float32) ** 2
        return z / torch.sqrt(chi2 / nu)
    if dist == "laplace":
        # inverse CDF of Laplace(0, 1) on u in (-1/2, 1/2)
        u = torch.rand(shape, generator=g, device=device, dtype=torch.float32) - 0.5
        return -torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp(max=0.5 - 1e-7))
    raise ValueError(dist)


def outlier_columns(c_in: int, n_outliers: int, scale, seed: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """Seeded choice of outlier column indices and their factors (CPU tensors)."""
    g = _generator(seed * 7919 + 17, "cpu")
    idx = torch.randperm(c_in, generator=g)[:n_outliers].sort().values
    if isinstance(scale, tuple):
        lo, hi = scale
        fac = lo + (hi - lo) * torch.rand(n_outliers, generator=g)
    else:
        fac = torch.full((n_outliers,), float(scale))
    return idx, fac.to(torch.float32)


def make_activations(spec: ActSpec, dtype: str, seed: int, device="cpu", *,
                     channel_offset: Optional[torch.Tensor] = None,
                     chunk_elems: int = 1 << 25) -> torch.Tensor:
    """X[N, C_in] in the 16-bit ``dtype``; saturated to the largest finite value."""
    td = torch_dtype(dtype)
    g = _generator(seed, device)
    X = torch.empty((spec.n_tokens, spec.c_in), dtype=td, device=device)
    mult = torch.ones(spec.c_in, dtype=torch.float32)
    if spec.n_outliers:
        idx, fac = outlier_columns(spec.c_in, spec.n_outliers, spec.outlier_scale, seed)
        mult[idx] = fac
    mult = mult.to(device)
    off = None if channel_offset is None else channel_offset.to(device=device, dtype=torch.float32)
    rows = max(1, chunk_elems // spec.c_in)
    for r0 in range(0, spec.n_tokens, rows):
        r1 = min(spec.n_tokens, r0 + rows)
        v = _base((r1 - r0, spec.c_in), spec.dist, spec.nu, g, device) * mult
        if off is not None:
            v = v + off
        if td == torch.float16:
            v = v.clamp_(-F16_MAX, F16_MAX)
        X[r0:r1] = v.to(td)
    return X


def make_weight(spec: LinearSpec, dtype: str, seed: int, device="cpu", *, chunk_elems: int = 1 << 25) -> torch.Tensor:
    """W[C_out, C_in] ~ N(0, w_std^2) in the 16-bit ``dtype``."""
    td = torch_dtype(dtype)
    g = _generator(seed, device)
    W = torch.empty((spec.c_out, spec.c_in), dtype=td, device=device)
    rows = max(1, chunk_elems // spec.c_in)
    for r0 in range(0, spec.c_out, rows):
        r1 = min(spec.c_out, r0 + rows)
        W[r0:r1] = (torch.randn((r1 - r0, spec.c_in), generator=g, device=device, dtype=torch.float32)
                    * spec.w_std).to(td)
    return W


def tensor_seed(workload_seed: int, layer: int, tensor_index: int) -> int:
    """Distinct seed for every tensor of a workload."""
    return (workload_seed * 1000003 + layer * 1009 + tensor_index * 31 + 12345) & 0x7FFFFFFF


def raw_bits(t: torch.Tensor):
    """The 16-bit payload of a tensor as a NumPy uint16 array (host copy)."""
    import numpy as np
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)
