"""Seeded synthetic inputs for the Lynx hot path (shared by tests, oracle checks and bench).

This module only draws numbers: it holds none of the method's arithmetic (no
quantisation, no attention) and imports neither the oracle nor the CUDA binding.
Each recipe stands in for the KV statistics the paper describes: a few outlier
channels that stay fixed over tokens and dominate the range (Section 2.3, "The
Challenge of Activation Outliers"), channel-wise magnitude structure, and heavy
tails (Section 3, KV distribution figures).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

BASE_SEED = 20260701
D = 128


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration (shapes as the benchmark's `configs` state them)."""
    name: str
    layers: int
    batch: int
    num_kv_heads: int
    num_q_heads: int
    context: int            # tokens per sequence (max when ragged)
    recipe: str             # see kv_block_values
    k_list: tuple           # speculation depths exercised
    ragged: bool = False    # lengths drawn uniformly in [min_context, context]
    min_context: int = 0
    block_tokens: int = 16
    shuffled_blocks: bool = False
    anchor_steps: int = 0   # decode steps outside verify windows (config 2)
    extra: dict = field(default_factory=dict)


WORKLOADS = {
    1: Workload("c1_single_layer_4k", 1, 1, 8, 32, 4096, "normal_outlier4x8", (4,)),
    2: Workload("c2_llama8b_32k", 32, 1, 8, 32, 32768, "lognormal_channels", (4,), anchor_steps=64),
    3: Workload("c3_llama8b_128k", 32, 1, 8, 32, 131072, "lognormal_channels", (2, 4, 8)),
    4: Workload("c4_serving_mix", 32, 16, 8, 32, 65536, "student_t4", (4,), ragged=True,
                min_context=8192, shuffled_blocks=True),
    5: Workload("c5_70b_128k", 80, 2, 8, 64, 131072, "normal_outlier2pct_x10", (8,)),
}


def _gen(device, *key) -> torch.Generator:
    """A generator seeded from BASE_SEED and an integer/string key (stable across runs)."""
    h = BASE_SEED
    for part in key:
        if isinstance(part, str):
            part = sum((i + 1) * ord(c) for i, c in enumerate(part))
        h = (h * 1000003 + int(part) + 12345) % (2 ** 62)
    g = torch.Generator(device=device)
    g.manual_seed(h)
    return g


def channel_scale(recipe: str, num_kv_heads: int, device, *key) -> torch.Tensor:
    """Per-(head, channel) multiplier, float32 [Hkv][1][128], fixed over tokens."""
    g = _gen("cpu", "chan", recipe, *key)
    s = torch.ones(num_kv_heads, 1, D, dtype=torch.float32)
    if recipe == "normal_outlier4x8":
        for h in range(num_kv_heads):
            idx = torch.randperm(D, generator=g)[:4]
            s[h, 0, idx] = 8.0
    elif recipe == "normal_outlier2pct_x10":
        for h in range(num_kv_heads):
            idx = torch.randperm(D, generator=g)[:3]   # 3 of 128 channels = 2 %
            s[h, 0, idx] = 10.0
    elif recipe == "lognormal_channels":
        s = torch.exp(0.5 * torch.randn(num_kv_heads, 1, D, generator=g, dtype=torch.float32))
    elif recipe in ("student_t4", "normal"):
        pass
    else:
        raise ValueError(f"unknown recipe {recipe}")
    return s.to(device)


def kv_block_values(recipe: str, num_blocks: int, num_kv_heads: int, block_tokens: int, device,
                    *key, out: torch.Tensor | None = None) -> torch.Tensor:
    """BF16 [num_blocks][Hkv][block_tokens][128] drawn per the recipe.

    normal_outlier4x8       N(0,1), 4 fixed channels per head scaled x8
    normal_outlier2pct_x10  N(0,1), 3 of 128 channels per head scaled x10
    lognormal_channels      N(0, sigma_c^2), sigma_c ~ LogNormal(0, 0.5) per (head, channel)
    student_t4              Student-t with 4 degrees of freedom
    normal                  N(0,1)
    `out` (optional) is a preallocated BF16 tensor of that shape to fill.
    """
    dev = torch.device(device)
    g = _gen(dev, "kv", recipe, *key)
    cs = channel_scale(recipe, num_kv_heads, dev, *key)
    if out is None:
        out = torch.empty(num_blocks, num_kv_heads, block_tokens, D, dtype=torch.bfloat16, device=dev)
    assert tuple(out.shape) == (num_blocks, num_kv_heads, block_tokens, D) and out.dtype == torch.bfloat16
    step = max(1, (1 << 24) // (num_kv_heads * block_tokens * D))   # ~16 M elements at a time
    for b0 in range(0, num_blocks, step):
        nb = min(step, num_blocks - b0)
        z = torch.randn(nb, num_kv_heads, block_tokens, D, generator=g, device=dev,
                        dtype=torch.float32)
        if recipe == "student_t4":
            w = torch.randn(4, nb, num_kv_heads, block_tokens, D, generator=g, device=dev,
                            dtype=torch.float32)
            z = z / torch.sqrt((w * w).mean(dim=0))
            del w
        out[b0:b0 + nb] = (z * cs).to(torch.bfloat16)
    return out


def queries(batch: int, n_q: int, num_q_heads: int, device, *key) -> torch.Tensor:
    """BF16 N(0,1) queries [B][n_q][Hq][128]."""
    dev = torch.device(device)
    g = _gen(dev, "q", *key)
    return torch.randn(batch, n_q, num_q_heads, D, generator=g, device=dev,
                       dtype=torch.float32).to(torch.bfloat16)


def seq_lens(batch: int, lo: int, hi: int, *key) -> torch.Tensor:
    """int32 [B] lengths uniform in [lo, hi] (CPU tensor)."""
    g = _gen("cpu", "lens", *key)
    if lo >= hi:
        return torch.full((batch,), hi, dtype=torch.int32)
    return torch.randint(lo, hi + 1, (batch,), generator=g, dtype=torch.int64).to(torch.int32)


def block_table(lens: torch.Tensor, block_tokens: int, shuffled: bool, *key):
    """Block table for the given lengths.

    Returns (table int32 [B][max_blocks] on CPU, num_blocks).  Each sequence owns
    ceil(len / block_tokens) distinct blocks of a pool of exactly that many blocks in
    total; `shuffled` assigns them by a seeded random permutation of the pool, otherwise
    in order.  Unused table entries are 0 (a valid block id, never read for a valid token).
    """
    need = [(int(l) + block_tokens - 1) // block_tokens for l in lens.tolist()]
    total = max(1, sum(need))
    max_blocks = max(1, max(need) if need else 1)
    if shuffled:
        perm = torch.randperm(total, generator=_gen("cpu", "blocks", *key))
    else:
        perm = torch.arange(total)
    table = torch.zeros(len(need), max_blocks, dtype=torch.int32)
    pos = 0
    for b, n in enumerate(need):
        table[b, :n] = perm[pos:pos + n].to(torch.int32)
        pos += n
    return table, total
