"""Algorithm 2 on the GPU, one layer per call: after every step the state is compared with the
oracle's cascade (same stored scores, same entropies), and the final cache with the one-shot
result whenever every layer's budget only ever shrank."""
import numpy as np
import pytest
import torch

import paper_2509_09754_b200 as lava
from lava_workloads import get_config
from oracle import lava_oracle as O
from tests.parity_harness import make_plan, upload_model

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.cpu().view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32).numpy()


def _check_state(cfg, view, k, v, keep_by_seq, budgets_by_seq, layers):
    """Device state after `layers` steps == the oracle's cascade after the same steps."""
    hkv, w, batch = cfg.n_kv_heads, cfg.window, cfg.batch
    hoff = view["head_offsets"].cpu().numpy()
    roff = view["layer_row_offset"].cpu().numpy()
    bud = view["layer_budget"].cpu().numpy()
    pos = view["kept_pos"].cpu().numpy()
    tok0 = 0
    for b, n in enumerate(cfg.seq_lens):
        for l in range(layers):
            assert int(bud[l, b]) == budgets_by_seq[b][l]
            r0 = int(roff[l * batch + b])
            assert int(roff[l * batch + b + 1]) - r0 == budgets_by_seq[b][l]
            keep = keep_by_seq[b][l]
            for g in range(hkv):
                a, e = int(hoff[l, b, g]) - g * w, int(hoff[l, b, g + 1]) - (g + 1) * w
                np.testing.assert_array_equal(pos[r0 + a: r0 + e], keep[g])
            rows = int(hoff[l, b, hkv])
            ko, vo = O.compact_kv(_bits(k[l, :, tok0:tok0 + n]), _bits(v[l, :, tok0:tok0 + n]), keep, w)
            np.testing.assert_array_equal(_bits(view["k_out"][r0:r0 + rows]), ko)
            np.testing.assert_array_equal(_bits(view["v_out"][r0:r0 + rows]), vo)
        tok0 += n


@pytest.mark.parametrize("name,kw,mode", [
    ("llama8b_8k", dict(seq_lens=(3000,), n_layers=6, budget_per_head=256), lava.LAVA_BUDGET_DYNAMIC),
    ("llama8b_8k", dict(seq_lens=(1500,), n_layers=4, budget_per_head=1200), lava.LAVA_BUDGET_DYNAMIC),
    ("mistral7b_ragged", dict(seq_lens=(640, 901, 333), n_layers=5, budget_per_head=96),
     lava.LAVA_BUDGET_DYNAMIC),
    ("mistral7b_ragged", dict(seq_lens=(520, 777), n_layers=4, budget_per_head=128),
     lava.LAVA_BUDGET_UNIFORM),
    ("tiny", dict(seq_lens=(300,), n_layers=4, budget_per_head=40), lava.LAVA_BUDGET_DYNAMIC),
])
def test_cascade_matches_the_oracle_and_the_one_shot_result(name, kw, mode):
    cfg = get_config(name).scaled(**kw)
    q, k, v, cu = upload_model(cfg)
    L, hkv, w, batch = cfg.n_layers, cfg.n_kv_heads, cfg.window, cfg.batch
    # one-shot path: scores and entropies (the cascade runs the same score kernels), final cache
    plan = make_plan(cfg, q, k, v, cu)
    lava.evict_model(plan, q, k, v, mode)
    assert lava.lava_poll_status(plan.workspace) == 0
    g_scores = plan.scores.cpu().numpy()
    g_ent = plan.entropy.cpu().numpy()
    budgets = [cfg.total_budget(b) for b in range(batch)]

    cas = lava.Cascade(plan.desc, L, sum(budgets), mode, kv_dtype=k.dtype)
    cas.begin(plan.total_budget)
    o_mode = O.BUDGET_DYNAMIC if mode == lava.LAVA_BUDGET_DYNAMIC else O.BUDGET_UNIFORM
    per_seq_scores = []
    tok0 = 0
    for b, n in enumerate(cfg.seq_lens):
        so = hkv * (tok0 - b * w)
        per_seq_scores.append([g_scores[l, so: so + hkv * (n - w)].reshape(hkv, n - w).astype(np.float64)
                               for l in range(L)])
        tok0 += n
    all_monotone = True
    for l in range(L):
        cas.step(q[l], k[l], v[l])
        assert lava.lava_poll_status(cas.workspace) == 0
        view = cas.view()
        assert view["layers_done"] == l + 1
        np.testing.assert_array_equal(view["entropy"].cpu().numpy(), g_ent[:l + 1])
        keep_by_seq, bud_by_seq = [], []
        for b, n in enumerate(cfg.seq_lens):
            keep, bud, mono = O.cascade_evict(per_seq_scores[b][:l + 1], n, w, budgets[b], o_mode,
                                              entropy=g_ent[:l + 1, b])
            keep_by_seq.append(keep)
            bud_by_seq.append(bud)
            all_monotone = all_monotone and mono
        _check_state(cfg, view, k, v, keep_by_seq, bud_by_seq, l + 1)
    # the one-shot result, bit for bit, when no budget ever grew
    assert all_monotone, "these cases were chosen with budgets that only shrink"
    view = cas.view()
    np.testing.assert_array_equal(view["layer_budget"].cpu().numpy(), plan.layer_budget.cpu().numpy())
    np.testing.assert_array_equal(view["layer_row_offset"].cpu().numpy(), plan.layer_row_offset.cpu().numpy())
    np.testing.assert_array_equal(view["head_offsets"].cpu().numpy(), plan.head_offsets.cpu().numpy())
    rows = sum(budgets)
    np.testing.assert_array_equal(_bits(view["k_out"][:rows]), _bits(plan.k_out[:rows]))
    np.testing.assert_array_equal(_bits(view["v_out"][:rows]), _bits(plan.v_out[:rows]))
    one_keep = plan.keep_idx.cpu().numpy()
    hoff = plan.head_offsets.cpu().numpy()
    roff = plan.layer_row_offset.cpu().numpy()
    pos = view["kept_pos"].cpu().numpy()
    tok0 = 0
    for b, n in enumerate(cfg.seq_lens):
        so = hkv * (tok0 - b * w)
        for l in range(L):
            kept = int(hoff[l, b, hkv]) - hkv * w
            r0 = int(roff[l * batch + b])
            np.testing.assert_array_equal(pos[r0:r0 + kept], one_keep[l, so: so + kept])
        tok0 += n
    cas.close()


def test_cascade_while_the_live_layers_cannot_hold_the_total():
    """A total above two layers' caps: the first layers keep everything (budget = cap, nothing to
    drop) until enough layers share the total; the state follows the oracle at every step."""
    cfg = get_config("tiny").scaled(seq_lens=(200,), n_layers=3, budget_per_head=150)
    q, k, v, cu = upload_model(cfg)
    L, hkv, w = cfg.n_layers, cfg.n_kv_heads, cfg.window
    plan = make_plan(cfg, q, k, v, cu)
    lava.evict_model(plan, q, k, v)          # the device's scores and entropies
    g_scores = plan.scores.cpu().numpy()
    g_ent = plan.entropy.cpu().numpy()
    n = cfg.seq_lens[0]
    scores = [g_scores[l, : hkv * (n - w)].reshape(hkv, n - w).astype(np.float64) for l in range(L)]
    total = cfg.total_budget(0)
    assert total > 2 * hkv * n
    cas = lava.Cascade(plan.desc, L, total, kv_dtype=k.dtype)
    cas.begin(plan.total_budget)
    for l in range(L):
        cas.step(q[l], k[l], v[l])
        keep, bud, _ = O.cascade_evict(scores[:l + 1], n, w, total, entropy=g_ent[:l + 1, 0])
        if l < 2:
            assert bud == [hkv * n] * (l + 1)
        _check_state(cfg, cas.view(), k, v, [keep], [bud], l + 1)
    assert lava.lava_poll_status(cas.workspace) == 0
    cas.close()


def test_cascade_rejects_what_it_does_not_cover_and_steps_out_of_order():
    cfg = get_config("tiny").scaled(seq_lens=(100,), n_layers=2)
    q, k, v, cu = upload_model(cfg)
    plan = make_plan(cfg, q, k, v, cu)
    with pytest.raises(lava.LavaError):
        lava.Cascade(plan.desc, 2, cfg.total_budget(0), lava.LAVA_BUDGET_PYRAMID, kv_dtype=k.dtype)
    with pytest.raises(lava.LavaError):
        lava.Cascade(plan.desc, 2, 3, kv_dtype=k.dtype)                  # arena below the window rows
    cas = lava.Cascade(plan.desc, 2, cfg.total_budget(0), kv_dtype=k.dtype)
    with pytest.raises(lava.LavaError):
        cas.step(q[0], k[0], v[0])                                       # begin has not run
    cas.begin(plan.total_budget)
    cas.step(q[0], k[0], v[0])
    cas.step(q[1], k[1], v[1])
    with pytest.raises(lava.LavaError):
        cas.step(q[1], k[1], v[1])                                       # all layers taken
    torch.cuda.synchronize()
    cas.close()


def test_a_sequence_shorter_than_the_window_stops_the_batch():
    """The score layout has no room for a sequence shorter than the window, and only the device
    knows the lengths: every kernel that addresses scores leaves such a batch alone, the status
    word says why, and nothing is written (the outputs keep their fill)."""
    cfg = get_config("mistral7b_ragged").scaled(seq_lens=(900, 40), n_layers=2, budget_per_head=128)
    q, k, v, cu = upload_model(cfg)
    plan = make_plan(cfg, q, k, v, cu)
    plan.scores.fill_(-7.0)
    plan.keep_idx.fill_(-7)
    plan.k_out.fill_(3.0)
    lava.evict_model(plan, q, k, v)
    assert lava.lava_poll_status(plan.workspace) & 1            # LAVA_DEV_SHORT_SEQUENCE
    # (query groups scored as two halves start from a cleared score array: zeros, not the fill)
    assert bool(((plan.scores == -7.0) | (plan.scores == 0.0)).all()) and bool((plan.keep_idx == -7).all())
    assert bool((plan.k_out == 3.0).all())
    cas = lava.Cascade(plan.desc, cfg.n_layers, sum(cfg.total_budget(b) for b in range(cfg.batch)),
                       kv_dtype=k.dtype)
    cas.begin(plan.total_budget)
    for l in range(cfg.n_layers):
        cas.step(q[l], k[l], v[l])
    assert lava.lava_poll_status(cas.workspace) & 1
    cas.close()
    # the CUDA-core path (fp32) behaves the same
    cfg = get_config("tiny").scaled(seq_lens=(300, 9), n_layers=1)
    q, k, v, cu = upload_model(cfg)
    plan = make_plan(cfg, q, k, v, cu)
    plan.scores.fill_(-7.0)
    lava.evict_model(plan, q, k, v)
    assert lava.lava_poll_status(plan.workspace) & 1
    assert bool((plan.scores == -7.0).all())
