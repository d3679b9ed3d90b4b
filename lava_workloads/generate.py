"""Seeded tensor generation for the workload configs (torch generators, CPU or CUDA).

Layout of one layer (``generate_layer``):
  q_win : [batch, H_q, w, d]        last-w queries of every sequence
  k, v  : [H_kv, total_tokens, d]   sequences concatenated along the token axis
  cu_seqlens : int32 [batch + 1]    token offsets of the sequences
The same (config, layer, device type) always yields the same bits.  Tensors are drawn in fp32
and rounded once to the config's dtype; every consumer reads those rounded bits.
"""
from __future__ import annotations

import math

import numpy as np
import torch

from .configs import WorkloadConfig


def _gen(cfg: WorkloadConfig, layer: int, stream: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((cfg.seed * 1_000_003 + layer * 10_007 + stream * 101 + 17) & 0x7FFFFFFF)
    return g


def _torch_dtype(cfg: WorkloadConfig):
    return torch.float32 if cfg.dtype == "f32" else torch.bfloat16


def needle_position(cfg: WorkloadConfig, seq: int) -> int:
    """Prefix position of the planted key of sequence ``seq`` (same in every layer)."""
    n = cfg.seq_lens[seq]
    prefix = n - cfg.window
    return int((cfg.seed * 7919 + seq * 104729 + 12345) % max(1, prefix - 64)) + 32


def span_starts(cfg: WorkloadConfig, seq: int):
    """Start positions of the non-overlapping heavy-hitter spans of sequence ``seq``."""
    n = cfg.seq_lens[seq]
    prefix = n - cfg.window
    if cfg.n_spans <= 0:
        return []
    cell = prefix // cfg.n_spans
    if cell < cfg.span_len:
        return []
    rng = np.random.RandomState(cfg.seed * 31 + seq)
    return [int(c * cell + rng.randint(0, cell - cfg.span_len + 1)) for c in range(cfg.n_spans)]


def generate_layer(cfg: WorkloadConfig, layer: int, device="cpu"):
    """Draw one layer's Q window, K and V.  Returns a dict of torch tensors on ``device``."""
    device = torch.device(device)
    d, w = cfg.head_dim, cfg.window
    total = cfg.total_tokens
    cu = [0]
    for n in cfg.seq_lens:
        cu.append(cu[-1] + int(n))
    gq, gk, gv, gx = (_gen(cfg, layer, s, device) for s in range(4))

    q = torch.randn((cfg.batch, cfg.n_q_heads, w, d), generator=gq, device=device,
                    dtype=torch.float32)
    k = torch.randn((cfg.n_kv_heads, total, d), generator=gk, device=device, dtype=torch.float32)
    v = torch.randn((cfg.n_kv_heads, total, d), generator=gv, device=device, dtype=torch.float32)

    for b, n in enumerate(cfg.seq_lens):
        lo, hi = cu[b], cu[b + 1]
        if cfg.drift:
            # per-head random walk along position, unit variance per dim at the end
            steps = torch.randn((cfg.n_kv_heads, n, d), generator=gx, device=device,
                                dtype=torch.float32) * (1.0 / math.sqrt(n))
            steps[:, 0, :] = 0.0
            k[:, lo:hi, :] += torch.cumsum(steps, dim=1)
            del steps
        if cfg.heavy_frac > 0.0:
            heavy = torch.rand((cfg.n_kv_heads, n), generator=gx, device=device) < cfg.heavy_frac
            k[:, lo:hi, :] *= torch.where(heavy, 3.0, 1.0).unsqueeze(-1)
        for p in cfg.sink_positions:
            if p < n:
                k[:, lo + p, :] *= 4.0
        for s0 in span_starts(cfg, b):
            k[:, lo + s0: lo + s0 + cfg.span_len, :] *= 3.0
        if cfg.needle:
            p = needle_position(cfg, b)
            c = torch.randn((cfg.n_kv_heads, d), generator=gx, device=device, dtype=torch.float32)
            c = c / c.norm(dim=1, keepdim=True)
            r = torch.randn((cfg.n_kv_heads, d), generator=gx, device=device, dtype=torch.float32)
            r = r - (r * c).sum(dim=1, keepdim=True) * c
            r = r / r.norm(dim=1, keepdim=True)
            k[:, lo + p, :] = math.sqrt(d) * (0.9 * c + math.sqrt(0.19) * r)
            grp = cfg.group
            q[b] += math.sqrt(d) * c.repeat_interleave(grp, dim=0).unsqueeze(1)
    if cfg.v_lognormal_sigma > 0.0:
        z = torch.randn((cfg.n_kv_heads, total, 1), generator=gx, device=device,
                        dtype=torch.float32)
        v *= torch.exp(cfg.v_lognormal_sigma * z)

    dt = _torch_dtype(cfg)
    out = {
        "q_win": q.to(dt).contiguous(),
        "k": k.to(dt).contiguous(),
        "v": v.to(dt).contiguous(),
        "cu_seqlens": torch.tensor(cu, dtype=torch.int32, device=device),
    }
    return out


def generate_wo(cfg: WorkloadConfig, layer: int, device="cpu"):
    """W_O ~ N(0, 1/sqrt(d_model)) of shape [d_model, d_model] (enters only through C-hat)."""
    g = _gen(cfg, layer, 9, torch.device(device))
    dm = cfg.d_model
    return torch.randn((dm, dm), generator=g, device=device, dtype=torch.float32) / math.sqrt(
        math.sqrt(dm))


def generate_model(cfg: WorkloadConfig, device="cpu", layers=None):
    """All layers (or the listed ones) as a list of ``generate_layer`` dicts."""
    layers = range(cfg.n_layers) if layers is None else layers
    return [generate_layer(cfg, l, device) for l in layers]


def to_numpy64(t: torch.Tensor) -> np.ndarray:
    """Exact fp64 copy of a tensor's values on the host (bf16 and fp32 widen exactly)."""
    return t.detach().to("cpu").to(torch.float64).numpy()
