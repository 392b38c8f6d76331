"""Seeded synthetic inputs shaped like the workloads HiF4 is evaluated on.

This module only draws random tensors (shapes, value distributions, outlier structure, MoE routing);
it contains none of the format's arithmetic.  Both the CUDA path and the CPU oracle are fed from it,
so that they see the same bits: generate once (on any torch device), copy to the other side.

The model names only lend their linear-layer shapes; all weights and activations are random.
"""
from __future__ import annotations

import math
from typing import Dict, List, Tuple

import torch

# (K, N) of the Llama-3-8B-shaped linears: q/o, k/v, gate/up, down.
LLAMA3_8B_LINEARS: List[Tuple[str, int, int]] = [
    ("qo", 4096, 4096),
    ("kv", 4096, 1024),
    ("gate_up", 4096, 14336),
    ("down", 14336, 4096),
]
LLAMA3_8B_M = [1, 16, 4096]

# (K, N) of the Qwen2.5-32B / Mistral-like dense prefill linears, M = 8192 tokens.
DENSE_PREFILL_LINEARS: List[Tuple[str, int, int]] = [
    ("attn", 5120, 5120),
    ("gate_up", 5120, 27648),
    ("down", 27648, 5120),
]
DENSE_PREFILL_M = 8192

# DeepSeek-V3-shaped MoE layer.
MOE_HIDDEN, MOE_EXPERTS, MOE_INTER, MOE_TOPK, MOE_TOKENS = 7168, 256, 2048, 8, 4096


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def gaussian(rows: int, cols: int, std: float, seed: int, device="cpu", dtype=torch.bfloat16) -> torch.Tensor:
    """Weights ~ N(0, std^2)."""
    g = _gen(seed, device)
    return (torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32) * std).to(dtype)


def student_t(rows: int, cols: int, nu: int, g: torch.Generator, device) -> torch.Tensor:
    """Student-t(nu) = normal / sqrt(chi2_nu / nu), FP32."""
    z = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
    chi2 = torch.zeros(rows, cols, device=device, dtype=torch.float32)
    for _ in range(nu):
        chi2 += torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32) ** 2
    return z / torch.sqrt(chi2 / nu)


def single_layer(seed: int = 1001, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """Config 1: X 128x512 ~ N(0,1) with 4 outlier columns x40; W [N=512, K=512] ~ N(0, 0.02)."""
    g = _gen(seed, device)
    x = torch.randn(128, 512, generator=g, device=device, dtype=torch.float32)
    for c in (7, 130, 257, 500):
        x[:, c] *= 40.0
    w = torch.randn(512, 512, generator=g, device=device, dtype=torch.float32) * 0.02
    return x.to(torch.bfloat16), w.to(torch.bfloat16)


def llama_activations(M: int, K: int, seed: int = 1002, device="cpu", dtype=torch.bfloat16) -> torch.Tensor:
    """Config 2 activations: Student-t(nu=4), 0.5 % of the channels (columns) scaled x50."""
    g = _gen(seed, device)
    x = student_t(M, K, 4, g, device)
    n_out = math.ceil(0.005 * K)
    cols = torch.randperm(K, generator=g, device=device)[:n_out]
    x[:, cols] *= 50.0
    return x.to(dtype)


def quantize_sweep(n_elems: int, seed: int = 1003, device="cpu", dtype=torch.bfloat16) -> torch.Tensor:
    """Config 3: [n/4096, 4096]; rows cycle Gaussian / Student-t(3) / U[-1,1]; 1 % of the 64-element
    units hold one element scaled x1000 (which pushes the rest of the unit to the low scale levels)."""
    cols = 4096
    assert n_elems % cols == 0
    rows = n_elems // cols
    g = _gen(seed, device)
    out = torch.empty(rows, cols, device=device, dtype=dtype)
    chunk = 4096
    for r0 in range(0, rows, chunk):
        r1 = min(rows, r0 + chunk)
        n = r1 - r0
        kind = (torch.arange(r0, r1, device=device) % 3).view(n, 1)
        xg = torch.randn(n, cols, generator=g, device=device, dtype=torch.float32)
        xt = student_t(n, cols, 3, g, device)
        xu = torch.rand(n, cols, generator=g, device=device, dtype=torch.float32) * 2.0 - 1.0
        x = torch.where(kind == 0, xg, torch.where(kind == 1, xt, xu))
        units = x.view(n, cols // 64, 64)
        spike_unit = torch.rand(n, cols // 64, generator=g, device=device) < 0.01
        pos = torch.randint(0, 64, (n, cols // 64), generator=g, device=device)
        onehot = torch.nn.functional.one_hot(pos, 64).bool() & spike_unit.unsqueeze(-1)
        units = torch.where(onehot, units * 1000.0, units)
        out[r0:r1] = units.reshape(n, cols).to(dtype)
    return out


def prefill_activations(M: int, K: int, seed: int = 1004, device="cpu", dtype=torch.bfloat16) -> torch.Tensor:
    """Config 4 activations: row t ~ N(0,1) * r_t with log2 r_t uniform in [-4, 4]."""
    g = _gen(seed, device)
    r = torch.exp2(torch.rand(M, 1, generator=g, device=device, dtype=torch.float32) * 8.0 - 4.0)
    x = torch.randn(M, K, generator=g, device=device, dtype=torch.float32) * r
    return x.to(dtype)


def moe_routing(tokens: int = MOE_TOKENS, experts: int = MOE_EXPERTS, topk: int = MOE_TOPK,
                seed: int = 1005, device="cpu") -> Dict[str, torch.Tensor]:
    """Config 5 routing: expert popularity p_rank ~ rank^-1.1 (Zipf), expert ids a seeded permutation
    of the ranks, top-k per token by Gumbel-top-k on log p.  Returns the per-expert row counts, the
    int64 prefix sums (`offsets`, experts+1) and, per sorted row, its token id."""
    g = _gen(seed, device)
    ranks = torch.arange(1, experts + 1, device=device, dtype=torch.float64)
    logp_by_rank = -1.1 * torch.log(ranks)
    perm = torch.randperm(experts, generator=g, device=device)
    logp = torch.empty(experts, device=device, dtype=torch.float64)
    logp[perm] = logp_by_rank
    u = torch.rand(tokens, experts, generator=g, device=device, dtype=torch.float64).clamp_(1e-300, 1.0)
    gumbel = -torch.log((-torch.log(u)).clamp_min(1e-300))
    choice = torch.topk(logp.unsqueeze(0) + gumbel, topk, dim=1).indices      # [tokens, topk]
    flat_expert = choice.reshape(-1)
    flat_token = torch.arange(tokens, device=device).repeat_interleave(topk)
    order = torch.argsort(flat_expert, stable=True)
    counts = torch.bincount(flat_expert, minlength=experts)
    offsets = torch.zeros(experts + 1, device=device, dtype=torch.int64)
    offsets[1:] = torch.cumsum(counts, 0)
    return {"counts": counts, "offsets": offsets, "token_of_row": flat_token[order]}


def outlier_channel_activations(rows: int, K: int, seed: int, device="cpu", dtype=torch.bfloat16) -> torch.Tensor:
    """Config 5 activations: N(0,1) with 0.5 % outlier channels x50."""
    g = _gen(seed, device)
    x = torch.randn(rows, K, generator=g, device=device, dtype=torch.float32)
    n_out = math.ceil(0.005 * K)
    cols = torch.randperm(K, generator=g, device=device)[:n_out]
    x[:, cols] *= 50.0
    return x.to(dtype)


# ---- storage views (no arithmetic): torch <-> numpy bit patterns
def bf16_to_u16_numpy(t: torch.Tensor):
    """BF16 tensor -> numpy uint16 bit patterns (host)."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")


def u16_numpy_to_bf16(a, device="cpu") -> torch.Tensor:
    import numpy as np
    return torch.from_numpy(np.ascontiguousarray(a).view("int16")).view(torch.bfloat16).to(device)
