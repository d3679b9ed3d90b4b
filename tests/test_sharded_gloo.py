"""Choreography of the sharded selection on two CPU ranks (gloo): stand-in steps written from the
radix-select definition take the place of the CUDA kernels, so what is tested is the order of
the collectives, the rank offsets of the ties and that both ranks agree on the threshold."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SHIFT, WIDTH = (21, 10, 0), (11, 11, 10)


class NumpySteps:
    """One (layer, sequence) problem per call site; scores [problems, heads_local, P] float32."""

    def __init__(self, w):
        self.w = w

    def state(self, desc, n_layers, device):
        st = {"hist": torch.zeros((desc["problems"], 2048), dtype=torch.int32),
              "ties": torch.zeros(desc["problems"], dtype=torch.int64)}
        return st, st["hist"], st["ties"]

    def begin(self, desc, n_layers, total_heads, budget, st):
        p = desc["prefix"]
        st["k"] = [max(0, min(int(b) - total_heads * self.w, total_heads * p)) for b in budget]
        st["k_rem"] = list(st["k"])
        st["val"] = [0] * len(budget)
        st["mask"] = [0] * len(budget)

    def hist(self, desc, n_layers, scores, p, st):
        keys = scores.numpy().view(np.uint32)
        st["hist"].zero_()
        for i in range(keys.shape[0]):
            if st["k"][i] == 0:
                continue
            kk = keys[i].reshape(-1)
            sel = kk[(kk & np.uint32(st["mask"][i])) == np.uint32(st["val"][i])]
            d = (sel >> np.uint32(SHIFT[p])) & np.uint32((1 << WIDTH[p]) - 1)
            st["hist"][i] += torch.from_numpy(np.bincount(d, minlength=2048).astype(np.int32))

    def step(self, desc, n_layers, p, st):
        for i in range(st["hist"].shape[0]):
            if st["k"][i] == 0:
                continue
            h = st["hist"][i].numpy()
            before = 0
            for d in range(2047, -1, -1):
                if before < st["k_rem"][i] <= before + h[d]:
                    st["val"][i] |= d << SHIFT[p]
                    st["mask"][i] |= ((1 << WIDTH[p]) - 1) << SHIFT[p]
                    st["k_rem"][i] -= before
                    break
                before += int(h[d])

    def count(self, desc, n_layers, scores, st):
        keys = scores.numpy().view(np.uint32)
        for i in range(keys.shape[0]):
            tau = st["val"][i] if st["k"][i] > 0 else 0xFFFFFFFF
            st["ties"][i] = int((keys[i] == np.uint32(tau)).sum())

    def emit(self, desc, n_layers, scores, before, keep, hoff, roff, st):
        keys = scores.numpy().view(np.uint32)
        for i in range(keys.shape[0]):
            tau = st["val"][i] if st["k"][i] > 0 else 0xFFFFFFFF
            wanted = st["k_rem"][i] if st["k"][i] > 0 else 0
            seen = int(before[i])
            out = []
            for g in range(keys.shape[1]):
                kept = []
                for pos, key in enumerate(keys[i, g]):
                    if key > tau or (key == tau and seen < wanted):
                        kept.append(pos)
                    seen += int(key == tau)
                out.append(kept)
            keep[i] = out


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    from paper_2509_09754_b200.sharded import sharded_select
    rng = np.random.RandomState(3)
    heads, hl, P, w, problems = 4, 2, 300, 8, 3
    full = np.round(rng.rand(problems, heads, P), 1).astype(np.float32)          # many ties
    budget = [heads * w + 137, heads * w, heads * (w + P)]
    local = torch.from_numpy(full[:, rank * hl:(rank + 1) * hl].copy())
    keep = [None] * problems
    sharded_select({"problems": problems, "prefix": P}, 1, heads, local, budget, keep, None,
                   _steps=NumpySteps(w))
    q.put((rank, keep, full, budget))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_with_the_unsplit_selection():
    sys.path.insert(0, ROOT)
    from oracle import lava_oracle as O
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict()
    for _ in range(2):
        rank, keep, full, budget = q.get(timeout=120)
        got[rank] = keep
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for i in range(full.shape[0]):
        want, _ = O.select_topk(full[i].astype(np.float64), budget[i], 8)
        for r in range(2):
            for gl in range(2):
                assert list(want[r * 2 + gl]) == got[r][i][gl], (i, r, gl)
