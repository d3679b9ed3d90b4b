"""Layer-wide selection with the KV heads of a layer split over the ranks of a process group.

The local steps run in the library's kernels (lava_select_shard_*); this module only places the
two collectives between them: an all-reduce of the digit histograms after each of the three radix
passes, and an all-gather of the ranks' tie counts before the emit.  Both move a few KB per
(layer, sequence); no rank reads another rank's memory.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding as _lib


class _LibrarySteps:
    """The CUDA library's steps on device tensors."""

    def state(self, desc, n_layers, device):
        state = torch.zeros(_lib.lava_select_shard_bytes(desc, n_layers), dtype=torch.uint8, device=device)
        h0, hb, t0, tb = _lib.lava_select_shard_layout(desc, n_layers)
        return state, state[h0:h0 + hb].view(torch.int32), state[t0:t0 + tb].view(torch.int64)

    begin = staticmethod(_lib.lava_select_shard_begin)
    hist = staticmethod(_lib.lava_select_shard_hist)
    step = staticmethod(_lib.lava_select_shard_step)
    count = staticmethod(_lib.lava_select_shard_count)
    emit = staticmethod(_lib.lava_select_shard_emit)


def ties_before_this_rank(gathered, rank: int) -> torch.Tensor:
    """Exclusive prefix over ranks of the per-rank tie counts ([problems] each)."""
    out = torch.zeros_like(gathered[0])
    for r in range(rank):
        out += gathered[r]
    return out


def sharded_select(desc, n_layers, total_kv_heads, scores, layer_budget, keep_idx, head_offsets,
                   layer_row_offset=None, group=None, _steps=None):
    """Selection of this rank's heads of every (layer, sequence); see lava.h, lava_select_shard_*.

    desc describes the LOCAL heads; scores, keep_idx, head_offsets, layer_row_offset are local;
    layer_budget is the whole layer's.  `_steps` is a test hook (the choreography of the
    collectives can be driven on CPU ranks with stand-in steps); the default is the CUDA library.
    """
    steps = _steps or _LibrarySteps()
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    state, hist, ties = steps.state(desc, n_layers, scores.device)
    steps.begin(desc, n_layers, total_kv_heads, layer_budget, state)
    for p in range(3):
        steps.hist(desc, n_layers, scores, p, state)
        if world > 1:
            dist.all_reduce(hist, op=dist.ReduceOp.SUM, group=group)
        steps.step(desc, n_layers, p, state)
    steps.count(desc, n_layers, scores, state)
    if world > 1:
        gathered = [torch.empty_like(ties) for _ in range(world)]
        dist.all_gather(gathered, ties, group=group)
        before = ties_before_this_rank(gathered, rank)
    else:
        before = torch.zeros_like(ties)
    steps.emit(desc, n_layers, scores, before, keep_idx, head_offsets, layer_row_offset, state)
    return state
