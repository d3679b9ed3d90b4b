"""Parity at the full size of every workload shape, in the launch configuration the benchmark
times: one score launch over all layers, one budget launch, one selection launch, one compaction
launch.

The fp64 oracle cannot score millions of entries per layer for every layer in seconds, so
  * a few whole (layer, sequence) problems and a few more (layer, sequence, KV head) triples are
    scored by the oracle and compared entry by entry (scores, value norms, and for the whole
    problems entropy, selection on the device's own scores, head offsets and the gathered rows);
  * every (layer, sequence) is checked through properties that hold at any size: the budgets are
    the oracle's rule applied to the device's entropies, the kept set is a valid top-k of the
    device's scores with ties resolved to the lower flat index, kept positions ascend inside
    each head, and the packed cache is a bit-exact gather.
Inputs are drawn on the device by the seeded generator (the oracle reads the same bits back).
"""
import numpy as np
import pytest
import torch

import paper_2509_09754_b200 as lava
from lava_workloads import generate_layer, get_config, to_numpy64
from lava_workloads.generate import needle_position
from oracle import lava_oracle as O
from tests.parity_harness import SCORE_ATOL, SCORE_RTOL, ENTROPY_RTOL

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32)


def _bits_u32(scores_f32):
    # non-negative floats order like their bit patterns; int64 keeps the comparison unsigned
    return scores_f32.contiguous().view(torch.int32).long()


def run_full_size(name, whole, sampled, expect_path=None, check_needle=False):
    """whole: (layer, sequence) pairs compared in full; sampled: (layer, sequence, KV head)."""
    cfg = get_config(name)
    dev = torch.device("cuda", 0)
    L, hkv, hq, d, w = cfg.n_layers, cfg.n_kv_heads, cfg.n_q_heads, cfg.head_dim, cfg.window
    G, B, T = hq // hkv, cfg.batch, cfg.total_tokens
    q = torch.empty((L, B, hq, w, d), dtype=torch.bfloat16, device=dev)
    k = torch.empty((L, hkv, T, d), dtype=torch.bfloat16, device=dev)
    v = torch.empty((L, hkv, T, d), dtype=torch.bfloat16, device=dev)
    cu = None
    for l in range(L):
        t = generate_layer(cfg, l, dev)
        q[l], k[l], v[l] = t["q_win"], t["k"], t["v"]
        cu = t["cu_seqlens"]
        del t
    desc = lava.LayerDesc.for_tensors(q[0], k[0], v[0], w, cfg.pool_kind, cfg.pool_kernel,
                                      cu_seqlens=cu if B > 1 else None,
                                      max_seqlen=max(cfg.seq_lens))
    if expect_path is not None:
        assert lava.lava_score_path(desc) == expect_path
    budgets = [cfg.total_budget(b) for b in range(B)]
    plan = lava.EvictionPlan.create(desc, L, budgets, cfg.seq_lens, device=dev)
    plan.keep_idx.fill_(-12345)
    plan.k_out.fill_(7.0)
    plan.v_out.fill_(7.0)
    mode = lava.LAVA_BUDGET_DYNAMIC if cfg.dynamic_layers else lava.LAVA_BUDGET_UNIFORM
    lava.evict_model(plan, q, k, v, mode)
    torch.cuda.synchronize()
    assert lava.lava_poll_status(plan.workspace) == 0

    tok0 = [0]
    for n in cfg.seq_lens:
        tok0.append(tok0[-1] + n)
    soff = [hkv * (tok0[b] - b * w) for b in range(B)]
    g_ent = plan.entropy.cpu().numpy()
    g_budget = plan.layer_budget.cpu().numpy()
    g_rowoff = plan.layer_row_offset.cpu().numpy()
    g_hoff = plan.head_offsets.cpu().numpy()
    g_vbar = plan.vbar.cpu().numpy()

    def dev_scores(l, b):
        n = cfg.seq_lens[b]
        return plan.scores[l, soff[b]: soff[b] + hkv * (n - w)].view(hkv, n - w)

    # ---- oracle on sampled heads and whole problems ---------------------------------------
    def oracle_heads(l, b, heads):
        lo, hi = tok0[b], tok0[b + 1]
        out = []
        for g in heads:
            s = O.lava_scores(to_numpy64(q[l, b, g * G:(g + 1) * G]),
                              to_numpy64(k[l, g:g + 1, lo:hi]), to_numpy64(v[l, g:g + 1, lo:hi]),
                              w, cfg.pool_kind, cfg.pool_kernel)
            gs = dev_scores(l, b)[g].cpu().numpy().astype(np.float64)
            err = np.abs(gs - s[0])
            tol = SCORE_RTOL * np.abs(s[0]) + SCORE_ATOL
            assert np.all(err <= tol), "layer %d seq %d head %d: score error %g at %d" % (
                l, b, g, err.max(), int(np.argmax(err - tol)))
            vb = O.value_norm(to_numpy64(v[l, g:g + 1, lo:hi]))
            np.testing.assert_allclose(g_vbar[l, b, g], vb[0], rtol=1e-5)
            out.append(s[0])
        return np.stack(out)

    def compare_whole(l, b):
        """Every output of one (layer, sequence) against the oracle; returns the oracle's scores."""
        n = cfg.seq_lens[b]
        prefix = n - w
        o_scores = oracle_heads(l, b, range(hkv))
        o_ent = O.layer_entropy(o_scores, n)
        assert abs(g_ent[l, b] - o_ent) <= ENTROPY_RTOL * abs(o_ent) + 1e-15
        # selection of the device's own scores: exact
        gs32 = dev_scores(l, b).cpu().numpy()
        keep_exact, off_exact = O.select_topk(gs32.astype(np.float64), int(g_budget[l, b]), w)
        assert [int(x) for x in g_hoff[l, b]] == [int(x) for x in off_exact]
        seg = plan.keep_idx[l, soff[b]: soff[b] + hkv * prefix].cpu().numpy()
        got = []
        for g in range(hkv):
            a, e = int(g_hoff[l, b, g]) - g * w, int(g_hoff[l, b, g + 1]) - (g + 1) * w
            np.testing.assert_array_equal(seg[a:e], keep_exact[g])
            got.append(seg[a:e])
        n_sel = int(g_hoff[l, b, -1]) - hkv * w
        assert np.all(seg[n_sel:] == -12345)
        lo, hi = tok0[b], tok0[b + 1]
        ko, vo = O.compact_kv(_bits(k[l, :, lo:hi]).cpu().numpy(), _bits(v[l, :, lo:hi]).cpu().numpy(),
                              got, w)
        r0, rows = int(g_rowoff[l * B + b]), int(g_hoff[l, b, -1])
        np.testing.assert_array_equal(_bits(plan.k_out[r0:r0 + rows]).cpu().numpy(), ko)
        np.testing.assert_array_equal(_bits(plan.v_out[r0:r0 + rows]).cpu().numpy(), vo)
        return o_scores

    for l, b, g in sampled:
        oracle_heads(l, b, [g])
    for l, b in whole:
        compare_whole(l, b)

    # ---- budgets: the oracle's rule on the device's entropies, bit-exact ---------------------
    for b in range(B):
        n = cfg.seq_lens[b]
        want = O.layer_budgets(list(g_ent[:, b]), budgets[b], hkv * w, hkv * n, mode)
        assert [int(x) for x in g_budget[:, b]] == want
        assert int(g_budget[:, b].sum()) == budgets[b]
    assert sum(budgets) == plan.k_out.shape[0]
    np.testing.assert_array_equal(g_rowoff, np.concatenate([[0], np.cumsum(g_budget.reshape(-1))]))

    # ---- every (layer, sequence): valid top-k, ordered, exact gather --------------------------
    needle_kept = {}
    for l in range(L):
        for b in range(B):
            n = cfg.seq_lens[b]
            prefix = n - w
            hoff = g_hoff[l, b]
            assert int(hoff[0]) == 0 and int(hoff[-1]) == int(g_budget[l, b])
            n_sel = int(g_budget[l, b]) - hkv * w
            flat = _bits_u32(dev_scores(l, b).reshape(-1))
            kept = torch.zeros(hkv * prefix, dtype=torch.bool, device=dev)
            r0 = int(g_rowoff[l * B + b])
            win_pos = torch.arange(prefix, n, device=dev)
            keep_l = plan.keep_idx[l, soff[b]: soff[b] + hkv * prefix]
            needle = needle_position(cfg, b) if check_needle else None
            for g in range(hkv):
                a, e = int(hoff[g]) - g * w, int(hoff[g + 1]) - (g + 1) * w
                assert 0 <= a <= e <= n_sel
                pos = keep_l[a:e].long()
                if e > a:
                    assert int(pos.min()) >= 0 and int(pos.max()) < prefix
                    assert bool((pos[1:] > pos[:-1]).all()), "kept positions must ascend"
                if needle is not None:
                    needle_kept[(l, b, g)] = bool((pos == needle).any())
                kept[g * prefix + pos] = True
                rows_all = torch.cat([pos, win_pos]) + tok0[b]
                o0 = r0 + int(hoff[g])
                assert torch.equal(_bits(plan.k_out[o0:o0 + rows_all.numel()]), _bits(k[l, g, rows_all]))
                assert torch.equal(_bits(plan.v_out[o0:o0 + rows_all.numel()]), _bits(v[l, g, rows_all]))
            assert int(kept.sum()) == n_sel
            if 0 < n_sel < hkv * prefix:
                tau = int(flat[kept].min())
                assert int(flat[~kept].max()) <= tau, "an entry above the threshold was dropped"
                ties = (flat == tau).nonzero().flatten()
                tk = kept[ties]
                n_tk = int(tk.sum())
                assert bool(tk[:n_tk].all()), "ties must resolve to the lower flat index"
    if check_needle:
        # At full length the planted key (logit about 0.9 sqrt(d) = 10) competes with the 1 % of
        # key rows that are scaled x3 (logits of standard deviation about 4, a hundred and more of
        # them per head), so a 128-row budget does not always retain it.  Where it is retained
        # the device and the oracle must agree, and where it is not, too: the decision is checked
        # against the oracle's own scores and selection on problems of both kinds.
        lost = list(dict.fromkeys((l, b) for (l, b, g), was_kept in needle_kept.items() if not was_kept))
        held = list(dict.fromkeys((l, b) for (l, b, g), was_kept in needle_kept.items() if was_kept))
        for l, b in [x for x in lost if x not in whole][:2] + [x for x in held if x not in whole][:1]:
            o_scores = compare_whole(l, b)
            keep_o, _ = O.select_topk(o_scores, int(g_budget[l, b]), w)
            p = needle_position(cfg, b)
            for g in range(hkv):
                assert bool(p in keep_o[g]) == needle_kept[(l, b, g)], (
                    "device and oracle disagree on the planted key (layer %d seq %d head %d)" % (l, b, g))
    del plan, q, k, v
    torch.cuda.empty_cache()


def test_llama8b_8k_all_layers_in_one_launch():
    # selection: 65 280 candidates per layer (16 keys per thread, clusters of 8)
    run_full_size("llama8b_8k", whole=[(3, 0), (30, 0)],
                  sampled=[(0, 0, 0), (11, 0, 5), (17, 0, 2), (31, 0, 7)], expect_path=1)


def test_llama8b_32k_all_layers_in_one_launch():
    run_full_size("llama8b_32k", whole=[(5, 0), (31, 0)],
                  sampled=[(0, 0, 0), (12, 0, 3), (16, 0, 7), (23, 0, 4)], expect_path=1)


def test_mistral7b_ragged_all_layers_in_one_launch():
    # w 64 x G 4 = 256 window-query rows per KV head (two units), avg-pool, eight ragged
    # sequences, a planted key per sequence
    cfg = get_config("mistral7b_ragged")
    order = sorted(range(cfg.batch), key=lambda b: cfg.seq_lens[b])
    shortest, longest, middle = order[0], order[-1], order[len(order) // 2]
    run_full_size("mistral7b_ragged", whole=[(2, shortest), (29, middle)],
                  sampled=[(0, longest, 0), (15, longest, 6), (31, order[1], 3), (20, order[-2], 7)],
                  expect_path=2, check_needle=True)


def test_gqa7_128k_all_layers_in_one_launch():
    # G 7 x w 32 = 224 window-query rows (units of 4 and 3 heads); 524 160 selection candidates
    # per layer (64 keys per thread, clusters of 16)
    run_full_size("gqa7_128k", whole=[(9, 0)], sampled=[(0, 0, 0), (27, 0, 3), (14, 0, 2)],
                  expect_path=2)
