"""Seeded synthetic inputs for the Orthrus generation-step hot path.

This module only draws random tensors and lays them out; it holds none of the
method's arithmetic (no attention, no argmax, no consensus).  Both the CUDA
path and the CPU oracle are fed the very same bytes produced here.

Shapes follow the paper's decoding setting (Section 4.1: Qwen3-class GQA models,
block width K in {8,16,32}; Section 4.4: context up to tens of thousands of
tokens).  The public evaluation suites of Section 4.1 are not reproduced: random
tensors with a controlled draft/AR agreement rate stand in for them.

Layouts (row-major, innermost last):
  q_diff, q_ar            [B][K][Hq][d]
  k_diff_blk, v_diff_blk  [B][K][Hkv][d]   transient diffusion-view block KV
  k_ar_blk,  v_ar_blk     [B][K][Hkv][d]   AR-view block KV (committed on accept)
  k_cache, v_cache        [B][Hkv][capacity][d]   shared prefix cache
  cache_len               [B] int32
  logits                  [B][K][V]
  draft                   [B][K] int32
"""
from __future__ import annotations

import dataclasses
import hashlib
import math
from typing import Dict, Optional

import torch

BASE_SEED = 12825


@dataclasses.dataclass(frozen=True)
class Workload:
    """Static description of one synthetic workload (one layer's shapes)."""

    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    block: int
    vocab: int
    prefix_min: int
    prefix_max: int          # == prefix_min for fixed-length workloads
    layers: int = 1
    value_std: float = 1.0   # std of Q/K/V entries
    logit_std: float = 1.0
    match_min: float = 0.5   # per-sequence draft agreement rate drawn U[min,max]
    match_max: float = 0.5
    dtype: str = "bf16"      # "bf16" or "fp32"

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def capacity(self) -> int:
        # room for one full block beyond the longest prefix, rounded to 64 rows
        need = self.prefix_max + self.block
        return (need + 63) // 64 * 64

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five synthetic configurations, smallest first (the second is the one the headline metric is quoted on).
CONFIGS: Dict[str, Workload] = {
    "cfg1_tiny": Workload("cfg1_tiny", 1, 8, 2, 64, 8, 1000, 512, 512,
                          layers=1, value_std=1.0 / 8, logit_std=1.0,
                          match_min=0.7, match_max=0.7),
    "cfg2_8b_b1": Workload("cfg2_8b_b1", 1, 32, 8, 128, 16, 151936, 4096, 4096,
                           layers=36, value_std=1.0 / math.sqrt(128), logit_std=2.0,
                           match_min=0.6, match_max=0.6),
    "cfg3_ragged": Workload("cfg3_ragged", 32, 32, 8, 128, 32, 128256, 1024, 8192,
                            layers=1, value_std=1.0 / math.sqrt(128), logit_std=1.0,
                            match_min=0.3, match_max=0.9),
    "cfg4_long": Workload("cfg4_long", 4, 64, 8, 128, 16, 151936, 32768, 32768,
                          layers=1, value_std=1.0 / math.sqrt(128), logit_std=1.0,
                          match_min=0.5, match_max=0.5),
    # attention/consensus shapes of the end-to-end decoder configuration
    "cfg5_loop": Workload("cfg5_loop", 8, 16, 4, 128, 16, 32000, 2048, 2048,
                          layers=12, value_std=1.0 / math.sqrt(128), logit_std=1.0,
                          match_min=0.65, match_max=0.65),
}


def sub_seed(seed: int, workload: str, layer: int, tensor: str) -> int:
    """Independent 63-bit seed for one tensor of one layer of one workload."""
    h = hashlib.sha256(f"{seed}/{workload}/{layer}/{tensor}".encode()).digest()
    return int.from_bytes(h[:8], "little") & ((1 << 63) - 1)


def _gen(seed: int, wl: Workload, layer: int, tensor: str) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(sub_seed(seed, wl.name, layer, tensor))
    return g


def torch_dtype(wl: Workload) -> torch.dtype:
    return torch.bfloat16 if wl.dtype == "bf16" else torch.float32


def _normal(shape, std, gen, dtype, chunk_rows: int = 0) -> torch.Tensor:
    """N(0, std) in fp32, rounded once to `dtype`."""
    out = torch.empty(shape, dtype=dtype)
    flat = out.view(-1)
    n = flat.numel()
    step = 1 << 24
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        flat[lo:hi] = (torch.randn(hi - lo, generator=gen, dtype=torch.float32) * std).to(dtype)
    return out


def prefix_lengths(wl: Workload, seed: int = BASE_SEED) -> torch.Tensor:
    """Per-sequence prefix lengths P_b, int32 [B] (uniform integers, inclusive)."""
    if wl.prefix_min == wl.prefix_max:
        return torch.full((wl.batch,), wl.prefix_min, dtype=torch.int32)
    g = _gen(seed, wl, 0, "prefix_len")
    return torch.randint(wl.prefix_min, wl.prefix_max + 1, (wl.batch,), generator=g,
                         dtype=torch.int64).to(torch.int32)


def attention_inputs(wl: Workload, layer: int = 0, seed: int = BASE_SEED,
                     q_gain: float = 1.0, fill_tail: Optional[float] = None
                     ) -> Dict[str, torch.Tensor]:
    """All attention-side tensors of one layer.

    `q_gain` scales the queries (a "peaked" variant that makes the softmax
    concentrate).  Cache rows at positions >= P_b are filled with `fill_tail`
    (default: random values, so that a kernel reading past the prefix is caught).
    """
    dt = torch_dtype(wl)
    B, K, Hq, Hkv, d, cap = (wl.batch, wl.block, wl.n_q_heads, wl.n_kv_heads,
                             wl.head_dim, wl.capacity)
    s = wl.value_std
    t = {}
    t["cache_len"] = prefix_lengths(wl, seed)
    t["k_cache"] = _normal((B, Hkv, cap, d), s, _gen(seed, wl, layer, "k_cache"), dt)
    t["v_cache"] = _normal((B, Hkv, cap, d), s, _gen(seed, wl, layer, "v_cache"), dt)
    if fill_tail is not None:
        for b in range(B):
            p = int(t["cache_len"][b])
            t["k_cache"][b, :, p:, :] = fill_tail
            t["v_cache"][b, :, p:, :] = fill_tail
    t["q_diff"] = _normal((B, K, Hq, d), s * q_gain, _gen(seed, wl, layer, "q_diff"), dt)
    t["q_ar"] = _normal((B, K, Hq, d), s * q_gain, _gen(seed, wl, layer, "q_ar"), dt)
    for name in ("k_diff_blk", "v_diff_blk", "k_ar_blk", "v_ar_blk"):
        t[name] = _normal((B, K, Hkv, d), s, _gen(seed, wl, layer, name), dt)
    return t


def logits(wl: Workload, seed: int = BASE_SEED) -> torch.Tensor:
    """AR-view logits [B][K][V], N(0, logit_std), rounded once to the dtype."""
    return _normal((wl.batch, wl.block, wl.vocab), wl.logit_std,
                   _gen(seed, wl, 0, "logits"), torch_dtype(wl))


def match_rates(wl: Workload, seed: int = BASE_SEED) -> torch.Tensor:
    """Per-sequence draft agreement rate p_b, float64 [B]."""
    if wl.match_min == wl.match_max:
        return torch.full((wl.batch,), wl.match_min, dtype=torch.float64)
    g = _gen(seed, wl, 0, "match_rate")
    u = torch.rand(wl.batch, generator=g, dtype=torch.float64)
    return wl.match_min + (wl.match_max - wl.match_min) * u


def drafts(wl: Workload, greedy_ids: torch.Tensor, seed: int = BASE_SEED) -> torch.Tensor:
    """Draft tokens [B][K] int32.

    `greedy_ids` [B][K] are token ids supplied by the caller (the per-position
    greedy token of the logits, computed outside this module).  Each draft copies
    the supplied id with the sequence's agreement rate and is otherwise uniform
    over the vocabulary (it may coincide with the supplied id by chance).
    """
    B, K, V = wl.batch, wl.block, wl.vocab
    g = _gen(seed, wl, 0, "draft")
    rates = match_rates(wl, seed).view(B, 1)
    coin = torch.rand((B, K), generator=g, dtype=torch.float64)
    rand_tok = torch.randint(0, V, (B, K), generator=g, dtype=torch.int64)
    out = torch.where(coin < rates, greedy_ids.to(torch.int64), rand_tok)
    return out.to(torch.int32).contiguous()
