"""The five workload shapes (Llama-3-8B / Mistral-7B shaped KV caches and a tiny fp32 case).

Shapes follow the model families the paper evaluates (32 layers, 32 query / 8 KV heads,
head dim 128) and its hyper-parameters (max-pool kernel 7, budgets of 128..2048 entries per
head, contexts up to 128K).  They stand in for the paper's LongBench / needle / 128K inputs,
which need datasets and weights.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass, field
from typing import List, Optional

POOL_NONE, POOL_MAX, POOL_AVG = 0, 1, 2


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str                      # "f32" or "bf16"
    seq_lens: tuple                 # one entry per sequence in the batch
    window: int
    pool_kind: int
    pool_kernel: int
    budget_per_head: int            # average retained rows per KV head per layer (window incl.)
    seed: int
    # value structure
    sink_positions: tuple = ()      # keys scaled x4 at these positions
    heavy_frac: float = 0.0         # Bernoulli fraction of key rows scaled x3
    drift: bool = False             # per-head random walk along position added to K
    v_lognormal_sigma: float = 0.0  # V row scale exp(sigma * z)
    needle: bool = False            # one planted key per sequence aligned with the window queries
    n_spans: int = 0                # heavy-hitter spans of span_len tokens scaled x3
    span_len: int = 16
    dynamic_layers: bool = True
    d_model: int = 0                # for W_O (unused by the hot path; only C-hat)
    ragged_range: Optional[tuple] = None

    @property
    def batch(self) -> int:
        return len(self.seq_lens)

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seq_lens))

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def total_budget(self, seq: int = 0) -> int:
        """Model-wide budget of one sequence, in KV-head rows (window rows included)."""
        return int(self.budget_per_head) * self.n_kv_heads * self.n_layers

    def scaled(self, **kw) -> "WorkloadConfig":
        """A copy with some fields replaced (smaller n / fewer layers for oracle-sized tests)."""
        return dataclasses.replace(self, **kw)


def _ragged_lengths(seed: int, batch: int, lo: int, hi: int) -> tuple:
    # small LCG so the lengths do not depend on any library's generator
    state = (seed * 6364136223846793005 + 1442695040888963407) & ((1 << 64) - 1)
    out = []
    for _ in range(batch):
        state = (state * 6364136223846793005 + 1442695040888963407) & ((1 << 64) - 1)
        out.append(lo + (state >> 33) % (hi - lo + 1))
    return tuple(int(x) for x in out)


CONFIGS = {
    # 1: tiny single layer, fp32, planted sinks
    "tiny": WorkloadConfig(
        name="tiny", n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=64, dtype="f32",
        seq_lens=(512,), window=16, pool_kind=POOL_MAX, pool_kernel=5, budget_per_head=64,
        seed=0, sink_positions=(0, 1, 2, 3), d_model=256),
    # 2: Llama-3-8B shaped, 8K context
    "llama8b_8k": WorkloadConfig(
        name="llama8b_8k", n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128, dtype="bf16",
        seq_lens=(8192,), window=32, pool_kind=POOL_MAX, pool_kernel=7, budget_per_head=512,
        seed=2, heavy_frac=0.01, drift=True, v_lognormal_sigma=0.5, d_model=4096),
    # 3: Llama-3-8B shaped, 32K context, dynamic head and layer budgets
    "llama8b_32k": WorkloadConfig(
        name="llama8b_32k", n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128, dtype="bf16",
        seq_lens=(32768,), window=32, pool_kind=POOL_MAX, pool_kernel=7, budget_per_head=2048,
        seed=3, heavy_frac=0.01, drift=True, v_lognormal_sigma=0.5, d_model=4096),
    # 4: Mistral-7B shaped, batch of 8 ragged sequences, avg-pool, needle
    "mistral7b_ragged": WorkloadConfig(
        name="mistral7b_ragged", n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128,
        dtype="bf16", seq_lens=_ragged_lengths(4, 8, 4096, 16384), window=64,
        pool_kind=POOL_AVG, pool_kernel=5, budget_per_head=128, seed=4, heavy_frac=0.01,
        drift=True, v_lognormal_sigma=0.5, needle=True, d_model=4096,
        ragged_range=(4096, 16384)),
    # 5: long-context stress, GQA 7
    "gqa7_128k": WorkloadConfig(
        name="gqa7_128k", n_layers=28, n_q_heads=28, n_kv_heads=4, head_dim=128, dtype="bf16",
        seq_lens=(131072,), window=32, pool_kind=POOL_MAX, pool_kernel=7, budget_per_head=1024,
        seed=5, heavy_frac=0.01, drift=True, v_lognormal_sigma=0.5, n_spans=64, span_len=16,
        d_model=3584),
}


def get_config(name: str) -> WorkloadConfig:
    return CONFIGS[name]
