"""Seeded synthetic inputs for the Muon step: shapes, dtypes and value
distributions of the benchmark configurations.  This module holds no part of
the optimizer's arithmetic; the tests feed the same tensors to the CUDA path
and (widened to float64 on the host) to the CPU oracle.

Configurations (synthetic stand-ins, by shape and value distribution, for the
parameter sets of the paper's models; no dataset or trained weight is used):
  1  one fp32 128x256 weight, gradient ~ N(0,1), momentum zero
  2  dense transformer, 24 layers, d = 2048: per layer four 2048x2048
     attention matrices and SwiGLU matrices 2048x8192 (x2) and 8192x2048;
     bf16 weights ~ N(0, 0.02), bf16 gradients ~ N(0, 1e-3)
  3  one MoE layer's expert bucket: (64 routed + 2 shared) x (2048x1408,
     2048x1408, 1408x2048) = 198 matrices; gradients N(0, 1e-3) times a
     per-expert LogNormal(0, 1) scale (uneven routing)
  4  shape sweep: single matrices, squares 512..8192, 4096x16384, 16384x4096;
     gradients ~ N(0, 1)
  5  Moonlight-shaped full set (about 15.3 G parameters): 27 layers of
     attention projections 2048x1536, 1536x3072, 2048x576, 512x4096,
     2048x2048; layer 0 dense MLP 2048x11264 (x2) and 11264x2048; layers 1-26
     66 experts x (2048x1408 x2, 1408x2048)
  6  the five dense Llama-style models of the paper's scaling-law study
     (hidden 1536 / 1792 / 2048 / 2304 / 2560 with 12 / 14 / 16 / 18 / 20
     layers): per layer four H x H attention matrices and SwiGLU matrices
     H x F (x2) and F x H with F = 2.6 H rounded to a multiple of 128
"""

from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Tuple

import torch


@dataclass(frozen=True)
class GroupSpec:
    rows: int
    cols: int
    count: int
    w_dtype: torch.dtype = torch.bfloat16
    g_dtype: torch.dtype = torch.bfloat16
    w_std: float = 0.02
    g_std: float = 1e-3
    lognormal_scale: bool = False  # per-matrix gradient scale exp(N(0,1))
    name: str = ""


def config_groups(cfg: int, layers: Optional[int] = None) -> List[GroupSpec]:
    """Group list of a configuration.  ``layers`` shrinks configs 2 and 5 for
    tests (same shapes, fewer layers)."""
    bf = torch.bfloat16
    if cfg == 1:
        return [GroupSpec(128, 256, 1, torch.float32, torch.float32, 0.02, 1.0, name="w")]
    if cfg == 2:
        L = 24 if layers is None else layers
        return [
            GroupSpec(2048, 2048, 4 * L, bf, bf, name="attn"),
            GroupSpec(2048, 8192, 2 * L, bf, bf, name="mlp_up_gate"),
            GroupSpec(8192, 2048, 1 * L, bf, bf, name="mlp_down"),
        ]
    if cfg == 3:
        E = 66
        return [
            GroupSpec(2048, 1408, 2 * E, bf, bf, lognormal_scale=True, name="expert_up_gate"),
            GroupSpec(1408, 2048, 1 * E, bf, bf, lognormal_scale=True, name="expert_down"),
        ]
    if cfg == 4:
        out = [GroupSpec(n, n, 1, bf, bf, g_std=1.0, name="sq%d" % n) for n in (512, 1024, 2048, 4096, 8192)]
        out.append(GroupSpec(4096, 16384, 1, bf, bf, g_std=1.0, name="wide"))
        out.append(GroupSpec(16384, 4096, 1, bf, bf, g_std=1.0, name="tall"))
        return out
    if cfg == 5:
        L = 27 if layers is None else layers
        moe_layers = max(L - 1, 0)
        out = [
            GroupSpec(2048, 1536, L, bf, bf, name="q_a"),
            GroupSpec(1536, 3072, L, bf, bf, name="q_b"),
            GroupSpec(2048, 576, L, bf, bf, name="kv_a"),
            GroupSpec(512, 4096, L, bf, bf, name="kv_b"),
            GroupSpec(2048, 2048, L, bf, bf, name="o"),
            GroupSpec(2048, 11264, 2, bf, bf, name="dense_up_gate"),
            GroupSpec(11264, 2048, 1, bf, bf, name="dense_down"),
        ]
        if moe_layers:
            out.append(GroupSpec(2048, 1408, 2 * 66 * moe_layers, bf, bf, lognormal_scale=True, name="expert_up_gate"))
            out.append(GroupSpec(1408, 2048, 1 * 66 * moe_layers, bf, bf, lognormal_scale=True, name="expert_down"))
        return out
    if cfg == 6:
        out = []
        for hidden, n_layers in ((1536, 12), (1792, 14), (2048, 16), (2304, 18), (2560, 20)):
            L = n_layers if layers is None else layers
            ffn = int(round(2.6 * hidden / 128.0)) * 128
            out.append(GroupSpec(hidden, hidden, 4 * L, bf, bf, name="attn%d" % hidden))
            out.append(GroupSpec(hidden, ffn, 2 * L, bf, bf, name="mlp_up_gate%d" % hidden))
            out.append(GroupSpec(ffn, hidden, 1 * L, bf, bf, name="mlp_down%d" % hidden))
        return out
    raise ValueError("unknown config %r" % (cfg,))


def group_params(specs: List[GroupSpec]) -> int:
    return sum(s.rows * s.cols * s.count for s in specs)


def ns_flops(specs: List[GroupSpec], ns_steps: int = 5) -> Tuple[float, float]:
    """(algorithmic, dense-equivalent) Newton-Schulz FLOPs of one step:
    per iteration 3 m^2 n + m^3 with the symmetric products halved, and
    4 m^2 n + 2 m^3 without."""
    alg = dense = 0.0
    for s in specs:
        m, n = min(s.rows, s.cols), max(s.rows, s.cols)
        alg += s.count * ns_steps * (3.0 * m * m * n + float(m) ** 3)
        dense += s.count * ns_steps * (4.0 * m * m * n + 2.0 * float(m) ** 3)
    return alg, dense


def stream_bytes(specs: List[GroupSpec]) -> float:
    """Algorithmic HBM bytes of the momentum kernel: G read, M read + write,
    bf16 X write."""
    total = 0.0
    for s in specs:
        gb = 2 if s.g_dtype == torch.bfloat16 else 4
        total += s.rows * s.cols * s.count * (gb + 4 + 4 + 2)
    return total


def _randn(shape, std, gen, device, dtype, chunk_elems=1 << 26):
    """N(0, std) drawn in fp32 with the given generator, rounded to dtype.
    Large tensors are filled slab by slab to bound temporary memory."""
    out = torch.empty(shape, dtype=dtype, device=device)
    flat = out.view(-1)
    n = flat.numel()
    for s in range(0, n, chunk_elems):
        e = min(n, s + chunk_elems)
        flat[s:e] = (torch.randn(e - s, generator=gen, device=device, dtype=torch.float32) * std).to(dtype)
    return out


def make_group(spec: GroupSpec, seed: int, device="cpu", zero_momentum: bool = True):
    """Tensors of one group: stacked [count, rows, cols] W, G, M plus the
    per-matrix views the binding takes."""
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    shape = (spec.count, spec.rows, spec.cols)
    W = _randn(shape, spec.w_std, gen, device, spec.w_dtype)
    G = make_grads(spec, gen, device)
    if zero_momentum:
        M = torch.zeros(shape, dtype=torch.float32, device=device)
    else:
        M = _randn(shape, spec.g_std, gen, device, torch.float32)
    return W, G, M


def make_grads(spec: GroupSpec, gen, device="cpu"):
    """A fresh gradient batch [count, rows, cols] for one group."""
    shape = (spec.count, spec.rows, spec.cols)
    if not spec.lognormal_scale:
        return _randn(shape, spec.g_std, gen, device, spec.g_dtype)
    z = torch.randn(spec.count, generator=gen, device=device, dtype=torch.float32)
    G = torch.empty(shape, dtype=spec.g_dtype, device=device)
    for i in range(spec.count):
        G[i] = (torch.randn(spec.rows, spec.cols, generator=gen, device=device, dtype=torch.float32)
                * (spec.g_std * float(torch.exp(z[i])))).to(spec.g_dtype)
    return G


def views(stacked: torch.Tensor) -> List[torch.Tensor]:
    return [stacked[i] for i in range(stacked.shape[0])]


def make_config(cfg: int, device="cpu", layers: Optional[int] = None, seed_base: Optional[int] = None):
    """All groups of a configuration: list of (spec, W, G, M) with seeds
    1000*cfg + group index (config 1: seed 0)."""
    base = (0 if cfg == 1 else 1000 * cfg) if seed_base is None else seed_base
    out = []
    for gi, spec in enumerate(config_groups(cfg, layers)):
        W, G, M = make_group(spec, base + gi, device)
        out.append((spec, W, G, M))
    return out
