"""Parity at the full 32K-token, 32-layer size, in the launch configuration the benchmark times:
one score launch over all layers, one budget launch, one selection launch, one compaction launch.

The fp64 oracle cannot score 8.4 million entries per layer for 32 layers in seconds, so
  * two whole layers and four more (layer, KV head) pairs are scored by the oracle and compared
    entry by entry (scores, value norms, and for the whole layers entropy, selection on the
    device's own scores, head offsets and the gathered rows);
  * every layer is checked through properties that hold at any size: the budgets are the
    oracle's rule applied to the device's entropies, the kept set is a valid top-k of the
    device's scores with ties resolved to the lower flat index, kept positions ascend inside
    each head, and the packed cache is a bit-exact gather.
"""
import numpy as np
import pytest
import torch

import paper_2509_09754_b200 as lava
from lava_workloads import generate_layer, get_config, to_numpy64
from oracle import lava_oracle as O
from tests.parity_harness import SCORE_ATOL, SCORE_RTOL, ENTROPY_RTOL

pytestmark = pytest.mark.gpu

WHOLE_LAYERS = (5, 31)
SAMPLED_HEADS = ((0, 0), (12, 3), (16, 7), (23, 4))


def _bits(t):
    return t.view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32)


def test_llama8b_32k_all_layers_in_one_launch():
    cfg = get_config("llama8b_32k")
    dev = torch.device("cuda", 0)
    L, hkv, hq, d, w, n = (cfg.n_layers, cfg.n_kv_heads, cfg.n_q_heads, cfg.head_dim, cfg.window,
                           cfg.seq_lens[0])
    G, prefix = hq // hkv, n - w
    q = torch.empty((L, 1, hq, w, d), dtype=torch.bfloat16, device=dev)
    k = torch.empty((L, hkv, n, d), dtype=torch.bfloat16, device=dev)
    v = torch.empty((L, hkv, n, d), dtype=torch.bfloat16, device=dev)
    for l in range(L):
        t = generate_layer(cfg, l, dev)
        q[l], k[l], v[l] = t["q_win"], t["k"], t["v"]
        del t
    desc = lava.LayerDesc.for_tensors(q[0], k[0], v[0], w, cfg.pool_kind, cfg.pool_kernel,
                                      max_seqlen=n)
    total_budget = cfg.total_budget(0)
    plan = lava.EvictionPlan.create(desc, L, [total_budget], cfg.seq_lens, device=dev)
    plan.keep_idx.fill_(-12345)
    plan.k_out.fill_(7.0)
    plan.v_out.fill_(7.0)
    lava.evict_model(plan, q, k, v, lava.LAVA_BUDGET_DYNAMIC)
    torch.cuda.synchronize()
    assert lava.lava_poll_status(plan.workspace) == 0

    g_scores = plan.scores.view(L, hkv, prefix)
    g_ent = plan.entropy.cpu().numpy()[:, 0]
    g_budget = plan.layer_budget.cpu().numpy()[:, 0]
    g_rowoff = plan.layer_row_offset.cpu().numpy()
    g_hoff = plan.head_offsets.cpu().numpy()[:, 0]
    g_vbar = plan.vbar.cpu().numpy()[:, 0]

    # ---- oracle on sampled heads and whole layers -----------------------------------------
    def oracle_heads(l, heads):
        out = []
        for g in heads:
            s = O.lava_scores(to_numpy64(q[l, 0, g * G:(g + 1) * G]), to_numpy64(k[l, g:g + 1]),
                              to_numpy64(v[l, g:g + 1]), w, cfg.pool_kind, cfg.pool_kernel)
            gs = g_scores[l, g].cpu().numpy().astype(np.float64)
            err = np.abs(gs - s[0])
            tol = SCORE_RTOL * np.abs(s[0]) + SCORE_ATOL
            assert np.all(err <= tol), "layer %d head %d: score error %g at %d" % (
                l, g, err.max(), int(np.argmax(err - tol)))
            vb = O.value_norm(to_numpy64(v[l, g:g + 1]))
            np.testing.assert_allclose(g_vbar[l, g], vb[0], rtol=1e-5)
            out.append(s[0])
        return np.stack(out)

    for l, g in SAMPLED_HEADS:
        oracle_heads(l, [g])
    for l in WHOLE_LAYERS:
        o_scores = oracle_heads(l, range(hkv))
        o_ent = O.layer_entropy(o_scores, n)
        assert abs(g_ent[l] - o_ent) <= ENTROPY_RTOL * abs(o_ent) + 1e-15
        # selection of the device's own scores: exact
        gs32 = g_scores[l].cpu().numpy()
        keep_exact, off_exact = O.select_topk(gs32.astype(np.float64), int(g_budget[l]), w)
        assert [int(x) for x in g_hoff[l]] == [int(x) for x in off_exact]
        seg = plan.keep_idx[l].cpu().numpy()
        got = []
        for g in range(hkv):
            a, e = int(g_hoff[l, g]) - g * w, int(g_hoff[l, g + 1]) - (g + 1) * w
            np.testing.assert_array_equal(seg[a:e], keep_exact[g])
            got.append(seg[a:e])
        n_sel = int(g_hoff[l, -1]) - hkv * w
        assert np.all(seg[n_sel:] == -12345)
        ko, vo = O.compact_kv(_bits(k[l]).cpu().numpy(), _bits(v[l]).cpu().numpy(), got, w)
        r0, rows = int(g_rowoff[l]), int(g_hoff[l, -1])
        np.testing.assert_array_equal(_bits(plan.k_out[r0:r0 + rows]).cpu().numpy(), ko)
        np.testing.assert_array_equal(_bits(plan.v_out[r0:r0 + rows]).cpu().numpy(), vo)

    # ---- budgets: the oracle's rule on the device's entropies, bit-exact ---------------------
    want = O.layer_budgets(list(g_ent), total_budget, hkv * w, hkv * n, O.BUDGET_DYNAMIC)
    assert [int(x) for x in g_budget] == want
    assert int(g_budget.sum()) == total_budget == plan.k_out.shape[0]
    np.testing.assert_array_equal(g_rowoff, np.concatenate([[0], np.cumsum(g_budget)]))

    # ---- every layer: valid top-k, ordered, exact gather ---------------------------------------
    win_pos = torch.arange(prefix, n, device=dev)
    for l in range(L):
        hoff = g_hoff[l]
        assert int(hoff[0]) == 0 and int(hoff[-1]) == int(g_budget[l])
        n_sel = int(g_budget[l]) - hkv * w
        flat = _bits_u32(g_scores[l].reshape(-1))
        kept = torch.zeros(hkv * prefix, dtype=torch.bool, device=dev)
        r0 = int(g_rowoff[l])
        for g in range(hkv):
            a, e = int(hoff[g]) - g * w, int(hoff[g + 1]) - (g + 1) * w
            assert 0 <= a <= e <= n_sel
            pos = plan.keep_idx[l, a:e].long()
            if e > a:
                assert int(pos.min()) >= 0 and int(pos.max()) < prefix
                assert bool((pos[1:] > pos[:-1]).all()), "kept positions must ascend"
            kept[g * prefix + pos] = True
            rows_all = torch.cat([pos, win_pos])
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


def _bits_u32(scores_f32):
    # non-negative floats order like their bit patterns; int64 keeps the comparison unsigned
    return scores_f32.contiguous().view(torch.int32).long()
