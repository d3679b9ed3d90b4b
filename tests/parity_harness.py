"""GPU-vs-oracle comparison of one full eviction (all four steps) on a workload config.

Used by the GPU parity tests and by the smoke check.  Inputs are drawn on the CPU by the
seeded generator, uploaded, pushed through the C ABI, and every output is compared with the
fp64 oracle run on the same bits.
"""
from __future__ import annotations

import numpy as np
import torch

import paper_2509_09754_b200 as lava
from lava_workloads import WorkloadConfig, generate_layer, to_numpy64
from oracle import lava_oracle as O

SCORE_RTOL, SCORE_ATOL = 1e-3, 1e-6      # the stated floating-point tolerance for scores
ENTROPY_RTOL = 1e-5


def upload_model(cfg: WorkloadConfig, device="cuda", gen_device="cpu"):
    """Stack all layers: q [L,B,Hq,w,d], k/v [L,Hkv,T,d]; returns device tensors + cu_seqlens."""
    layers = [generate_layer(cfg, l, gen_device) for l in range(cfg.n_layers)]
    q = torch.stack([x["q_win"] for x in layers]).to(device)
    k = torch.stack([x["k"] for x in layers]).to(device)
    v = torch.stack([x["v"] for x in layers]).to(device)
    cu = layers[0]["cu_seqlens"].to(device)
    return q, k, v, cu


def make_plan(cfg: WorkloadConfig, q, k, v, cu, budgets=None, c_hat=0.0):
    desc = lava.LayerDesc.for_tensors(
        q[0], k[0], v[0], cfg.window, cfg.pool_kind, cfg.pool_kernel,
        cu_seqlens=cu if cfg.batch > 1 else None, max_seqlen=max(cfg.seq_lens), c_hat=c_hat)
    if budgets is None:
        budgets = [cfg.total_budget(b) for b in range(cfg.batch)]
    plan = lava.EvictionPlan.create(desc, cfg.n_layers, budgets, cfg.seq_lens, device=q.device,
                                    kv_dtype=k.dtype)
    return plan


def oracle_sequence(cfg: WorkloadConfig, q, k, v, b: int, c_hat=1.0):
    """Oracle scores and entropies of sequence b for every layer (fp64, from the same bits)."""
    lo = sum(cfg.seq_lens[:b])
    hi = lo + cfg.seq_lens[b]
    scores, ent = [], []
    for l in range(cfg.n_layers):
        s = O.lava_scores(to_numpy64(q[l, b]), to_numpy64(k[l, :, lo:hi]),
                          to_numpy64(v[l, :, lo:hi]), cfg.window, cfg.pool_kind, cfg.pool_kernel,
                          c_hat=c_hat)
        scores.append(s)
        ent.append(O.layer_entropy(s, cfg.seq_lens[b]))
    return scores, ent


def compare_eviction(cfg: WorkloadConfig, mode=lava.LAVA_BUDGET_DYNAMIC, budgets=None,
                     device="cuda", c_hat=0.0):
    """Runs the CUDA path and the oracle; raises AssertionError on any mismatch.

    Returns a small report dict (max score error, band sizes, budget deltas).
    """
    q, k, v, cu = upload_model(cfg, device)
    plan = make_plan(cfg, q, k, v, cu, budgets, c_hat)
    canary_k = plan.k_out.clone().fill_(7.0)
    plan.k_out.copy_(canary_k)
    plan.v_out.fill_(7.0)
    plan.keep_idx.fill_(-12345)
    lava.evict_model(plan, q, k, v, mode)
    status = lava.lava_poll_status(plan.workspace)
    assert status == 0, "device status word = %d" % status

    hkv, w, d = cfg.n_kv_heads, cfg.window, cfg.head_dim
    g_scores = plan.scores.cpu().numpy()
    g_ent = plan.entropy.cpu().numpy()
    g_budget = plan.layer_budget.cpu().numpy()
    g_rowoff = plan.layer_row_offset.cpu().numpy()
    g_keep = plan.keep_idx.cpu().numpy()
    g_hoff = plan.head_offsets.cpu().numpy()
    g_vbar = plan.vbar.cpu().numpy()
    k_out = plan.k_out.cpu()
    v_out = plan.v_out.cpu()
    k_host, v_host = k.cpu(), v.cpu()
    report = {"max_rel_err": 0.0, "band_entries": 0, "budget_delta": 0}
    total_budget = budgets if budgets is not None else [cfg.total_budget(b) for b in range(cfg.batch)]
    tok0 = 0
    for b, n in enumerate(cfg.seq_lens):
        prefix = n - w
        soff = hkv * (tok0 - b * w)
        o_scores, o_ent = oracle_sequence(cfg, q, k, v, b, c_hat if c_hat > 0 else 1.0)
        # --- scores, value norms and entropies -------------------------------------------
        for l in range(cfg.n_layers):
            gs = g_scores[l, soff: soff + hkv * prefix].reshape(hkv, prefix).astype(np.float64)
            err = np.abs(gs - o_scores[l])
            tol = SCORE_RTOL * np.abs(o_scores[l]) + SCORE_ATOL
            assert np.all(err <= tol), "layer %d seq %d: score error %g exceeds tolerance at %s" % (
                l, b, err.max(), np.unravel_index(np.argmax(err - tol), err.shape))
            report["max_rel_err"] = max(report["max_rel_err"],
                                        float((err / np.maximum(np.abs(o_scores[l]), 1e-30)).max())
                                        if prefix else 0.0)
            o_vbar = O.value_norm(to_numpy64(v[l, :, tok0: tok0 + n]))
            np.testing.assert_allclose(g_vbar[l, b], o_vbar, rtol=1e-5)
            assert abs(g_ent[l, b] - o_ent[l]) <= ENTROPY_RTOL * abs(o_ent[l]) + 1e-15
        # --- budgets: bit-exact given the GPU's entropies; close to the oracle's own -------
        lo_b, hi_b = hkv * w, hkv * n
        want = O.layer_budgets(list(g_ent[:, b]), total_budget[b], lo_b, hi_b, mode)
        assert [int(x) for x in g_budget[:, b]] == want, "budgets differ from the oracle's rule"
        pure = O.layer_budgets(o_ent, total_budget[b], lo_b, hi_b, mode)
        delta = max(abs(int(x) - y) for x, y in zip(g_budget[:, b], pure))
        assert delta <= 1, "budgets differ by %d from the oracle run on its own entropies" % delta
        report["budget_delta"] = max(report["budget_delta"], delta)
        # --- selection and compaction -----------------------------------------------------
        for l in range(cfg.n_layers):
            bl = int(g_budget[l, b])
            gs32 = g_scores[l, soff: soff + hkv * prefix].reshape(hkv, prefix)
            keep_exact, off_exact = O.select_topk(gs32.astype(np.float64), bl, w)
            hoff = g_hoff[l, b]
            assert [int(x) for x in hoff] == [int(x) for x in off_exact], "head offsets differ"
            assert hoff[-1] == min(bl, hkv * n)
            seg = g_keep[l, soff: soff + hkv * prefix]
            n_sel = int(hoff[-1]) - hkv * w
            got = []
            for g in range(hkv):
                a = int(hoff[g]) - g * w
                e = int(hoff[g + 1]) - (g + 1) * w
                got.append(seg[a:e])
                np.testing.assert_array_equal(seg[a:e], keep_exact[g])   # bit-exact on its scores
            assert np.all(seg[n_sel:] == -12345), "keep_idx written beyond the selected count"
            # against the oracle's own scores: only entries near the k-th score may differ
            keep_o, _ = O.select_topk(o_scores[l], bl, w)
            flat_o = o_scores[l].reshape(-1)
            set_g = set(int(g * prefix + i) for g in range(hkv) for i in got[g])
            set_o = set(int(g * prefix + i) for g in range(hkv) for i in keep_o[g])
            diff = set_g ^ set_o
            if diff:
                kth = np.sort(flat_o)[::-1][n_sel - 1]
                band = SCORE_RTOL * abs(kth) + SCORE_ATOL
                for f in diff:
                    assert abs(flat_o[f] - kth) <= band, "selection differs outside the tie band"
                report["band_entries"] += len(diff)
            # compaction: bit-exact gather in (kept ascending, then window) order
            ko, vo = O.compact_kv(k_host[l, :, tok0: tok0 + n].view(torch.int16 if k.dtype == torch.bfloat16 else torch.int32).numpy(),
                                  v_host[l, :, tok0: tok0 + n].view(torch.int16 if k.dtype == torch.bfloat16 else torch.int32).numpy(),
                                  got, w)
            r0 = int(g_rowoff[l * cfg.batch + b])
            rows = int(hoff[-1])
            bits = torch.int16 if k.dtype == torch.bfloat16 else torch.int32
            np.testing.assert_array_equal(k_out[r0: r0 + rows].view(bits).numpy(), ko)
            np.testing.assert_array_equal(v_out[r0: r0 + rows].view(bits).numpy(), vo)
        tok0 += n
    # prefix sums and the packed size
    flat_b = g_budget.reshape(-1)
    np.testing.assert_array_equal(g_rowoff[:-1], np.concatenate([[0], np.cumsum(flat_b)[:-1]]))
    assert g_rowoff[-1] == sum(total_budget) == plan.k_out.shape[0]
    return report
