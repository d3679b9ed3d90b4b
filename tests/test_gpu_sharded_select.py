"""KV-head-sharded layer-wide selection: the local steps of every rank run one after the other
on one GPU (no kernel waits for another), the histogram all-reduce and the tie all-gather are
plain tensor sums, and the union of the ranks' outputs must equal the oracle's select_topk on the
unsplit layer, ties included."""
import numpy as np
import pytest
import torch

import paper_2509_09754_b200 as lava
from oracle import lava_oracle as O

pytestmark = pytest.mark.gpu


def _desc(hkv, lens, w, cu):
    total = sum(lens)
    return lava.LayerDesc(n_q_heads=hkv, n_kv_heads=hkv, head_dim=128, window=w, batch=len(lens),
                          max_seqlen=max(lens), cu_seqlens=cu, total_tokens=total,
                          k_stride_head=total * 128, k_stride_tok=128, v_stride_head=total * 128,
                          v_stride_tok=128)


@pytest.mark.parametrize("ranks,hkv,lens,w,L", [
    (2, 8, (3000,), 32, 2),
    (4, 8, (2100, 700, 40), 32, 2),          # ragged batch, one sequence barely above the window
    (2, 4, (9000, 32), 32, 1),               # a sequence of exactly the window: nothing to select
])
def test_sharded_select_equals_the_unsplit_selection(ranks, hkv, lens, w, L):
    rng = np.random.RandomState(ranks * 100 + hkv)
    hl = hkv // ranks
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
    d_loc = _desc(hl, lens, w, cu)
    prefixes = [max(n - w, 0) for n in lens]
    # full scores per (layer, sequence): [hkv, P], heavily tied
    full = [[np.round(rng.rand(hkv, p), 2).astype(np.float32) for p in prefixes] for _ in range(L)]
    budgets = np.array([[hkv * min(w, n) + int(rng.randint(0, hkv * p + 1)) for n, p in zip(lens, prefixes)]
                        for _ in range(L)], dtype=np.int64)
    lb = torch.from_numpy(budgets).cuda()
    probs = L * len(lens)
    # local score arrays in the library's layout for hl heads
    loc_scores, states, hists, ties, keeps, hoffs, roffs = [], [], [], [], [], [], []
    h0, hb, t0, tb = lava.lava_select_shard_layout(d_loc, L)
    for r in range(ranks):
        rows = [np.concatenate([full[l][b][r * hl:(r + 1) * hl].reshape(-1) for b in range(len(lens))])
                for l in range(L)]
        loc_scores.append(torch.from_numpy(np.stack(rows)).cuda())
        st = torch.zeros(lava.lava_select_shard_bytes(d_loc, L), dtype=torch.uint8, device="cuda")
        states.append(st)
        hists.append(st[h0:h0 + hb].view(torch.int32))
        ties.append(st[t0:t0 + tb].view(torch.int64))
        keeps.append(torch.full((L, d_loc.total_scores), -1, dtype=torch.int32, device="cuda"))
        hoffs.append(torch.zeros((L, len(lens), hl + 1), dtype=torch.int32, device="cuda"))
        roffs.append(torch.zeros(probs + 1, dtype=torch.int64, device="cuda"))
        lava.lava_select_shard_begin(d_loc, L, hkv, lb, st)
    for p in range(3):
        for r in range(ranks):
            lava.lava_select_shard_hist(d_loc, L, loc_scores[r], p, states[r])
        total = sum(hists)                         # stands in for the all-reduce
        for r in range(ranks):
            hists[r].copy_(total)
            lava.lava_select_shard_step(d_loc, L, p, states[r])
    for r in range(ranks):
        lava.lava_select_shard_count(d_loc, L, loc_scores[r], states[r])
    gathered = [t.clone() for t in ties]           # stands in for the all-gather
    from paper_2509_09754_b200.sharded import ties_before_this_rank
    for r in range(ranks):
        lava.lava_select_shard_emit(d_loc, L, loc_scores[r], ties_before_this_rank(gathered, r), keeps[r],
                                    hoffs[r], roffs[r], states[r])
    torch.cuda.synchronize()
    for l in range(L):
        tok0 = 0
        for b, n in enumerate(lens):
            win = min(w, n)
            want_keep, want_off = O.select_topk(full[l][b].astype(np.float64), int(budgets[l, b]), win)
            so_loc = hl * (tok0 - b * w) if n >= w else hl * (tok0 - b * w)
            for r in range(ranks):
                off = hoffs[r][l, b].cpu().numpy()
                seg = keeps[r][l].cpu().numpy()
                rows_r = 0
                for gl in range(hl):
                    g = r * hl + gl
                    a, e = int(off[gl]) - gl * win, int(off[gl + 1]) - (gl + 1) * win
                    base = hl * (tok0 - b * w)
                    np.testing.assert_array_equal(seg[base + a: base + e], want_keep[g],
                                                  err_msg="layer %d seq %d rank %d head %d" % (l, b, r, gl))
                    rows_r += len(want_keep[g]) + win
                ro = roffs[r].cpu().numpy()
                assert int(ro[l * len(lens) + b + 1] - ro[l * len(lens) + b]) == rows_r == int(off[hl])
            tok0 += n
