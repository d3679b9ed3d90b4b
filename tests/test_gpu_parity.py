"""GPU parity: the CUDA path through the C ABI against the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

import paper_2509_09754_b200 as lava
from lava_workloads import get_config
from oracle import lava_oracle as O
from tests.parity_harness import compare_eviction, make_plan, upload_model

pytestmark = pytest.mark.gpu


def test_tiny_config_full():
    rep = compare_eviction(get_config("tiny"))
    assert rep["max_rel_err"] < 1e-3


def test_llama_shape_several_tiles_and_ragged_tail():
    cfg = get_config("llama8b_8k").scaled(seq_lens=(1733,), n_layers=3, budget_per_head=160)
    compare_eviction(cfg)
    compare_eviction(cfg, mode=lava.LAVA_BUDGET_UNIFORM)


def test_ragged_batch_avgpool_needle():
    cfg = get_config("mistral7b_ragged").scaled(seq_lens=(777, 1290, 515), n_layers=2,
                                                budget_per_head=128)
    compare_eviction(cfg)
    # the planted key survives in every layer of every sequence
    from lava_workloads.generate import needle_position
    q, k, v, cu = upload_model(cfg)
    plan = make_plan(cfg, q, k, v, cu)
    lava.evict_model(plan, q, k, v)
    hoff = plan.head_offsets.cpu().numpy()
    keep = plan.keep_idx.cpu().numpy()
    tok0 = 0
    for b, n in enumerate(cfg.seq_lens):
        soff = cfg.n_kv_heads * (tok0 - b * cfg.window)
        p = needle_position(cfg, b)
        for l in range(cfg.n_layers):
            for g in range(cfg.n_kv_heads):
                a = hoff[l, b, g] - g * cfg.window
                e = hoff[l, b, g + 1] - (g + 1) * cfg.window
                assert p in keep[l, soff + a: soff + e]
        tok0 += n


def test_gqa7_shape():
    cfg = get_config("gqa7_128k").scaled(seq_lens=(2100,), n_layers=2, budget_per_head=200)
    compare_eviction(cfg)


@pytest.mark.parametrize("kw", [
    dict(seq_lens=(16,), budget_per_head=16),                                   # n == w: nothing to score
    dict(seq_lens=(17,), budget_per_head=17),                                   # one candidate per head
    dict(seq_lens=(300,), budget_per_head=300),             # budget == n: keep all
    dict(seq_lens=(300,), budget_per_head=16),              # window only
    dict(seq_lens=(513,), pool_kind=lava.LAVA_POOL_NONE, pool_kernel=1),
    dict(seq_lens=(600,), n_q_heads=2, n_kv_heads=2),       # MHA (G = 1)
    dict(seq_lens=(531,), pool_kind=lava.LAVA_POOL_AVG, pool_kernel=9, n_layers=4),
    dict(seq_lens=(1024,), head_dim=128),
])
def test_edge_cases(kw):
    cfg = get_config("tiny").scaled(**kw)
    compare_eviction(cfg)


def test_bf16_head_dim_64_and_c_hat():
    cfg = get_config("tiny").scaled(dtype="bf16", seq_lens=(900,), n_layers=2)
    compare_eviction(cfg, c_hat=3.25)


def test_budget_over_capacity_is_flagged_and_keeps_everything():
    cfg = get_config("tiny").scaled(seq_lens=(200,))
    q, k, v, cu = upload_model(cfg)
    plan = make_plan(cfg, q, k, v, cu, budgets=[2 * 200 + 50])
    lava.evict_model(plan, q, k, v)
    assert lava.lava_poll_status(plan.workspace) & 2
    assert int(plan.layer_budget[0, 0]) == 400
    bits = plan.k_out[:400].view(torch.int32)
    assert torch.equal(bits, k[0].reshape(400, 64).view(torch.int32))


def test_select_is_exact_on_heavily_tied_scores():
    rng = np.random.RandomState(3)
    hkv, n, w = 4, 5000, 32
    prefix = n - w
    cases = [np.round(rng.rand(hkv, prefix), 2).astype(np.float32),        # ~100 distinct values
             np.full((hkv, prefix), 0.25, dtype=np.float32),               # pure tie-break
             (rng.rand(hkv, prefix) ** 8).astype(np.float32),
             np.zeros((hkv, prefix), dtype=np.float32)]
    desc = lava.LayerDesc(n_q_heads=hkv, n_kv_heads=hkv, head_dim=128, window=w, total_tokens=n,
                          k_stride_head=n * 128, k_stride_tok=128, v_stride_head=n * 128,
                          v_stride_tok=128)
    for s in cases:
        for budget in (hkv * w, hkv * w + 1, hkv * w + 777, hkv * n - 1, hkv * n, 5 * hkv * n):
            scores = torch.from_numpy(s).cuda().reshape(-1)
            keep = torch.full((hkv * prefix,), -1, dtype=torch.int32, device="cuda")
            hoff = torch.zeros(hkv + 1, dtype=torch.int32, device="cuda")
            lb = torch.tensor([budget], dtype=torch.int64, device="cuda")
            lava.lava_select_topk(desc, scores, lb, keep, hoff)
            want_keep, want_off = O.select_topk(s.astype(np.float64), budget, w)
            got_off = hoff.cpu().numpy()
            np.testing.assert_array_equal(got_off, want_off)
            got = keep.cpu().numpy()
            for g in range(hkv):
                a, e = got_off[g] - g * w, got_off[g + 1] - (g + 1) * w
                np.testing.assert_array_equal(got[a:e], want_keep[g])
            assert np.all(got[got_off[-1] - hkv * w:] == -1)


def test_budgets_are_bit_exact_against_the_oracle_rule():
    rng = np.random.RandomState(4)
    for trial in range(40):
        nl = int(rng.randint(1, 40))
        batch = int(rng.randint(1, 5))
        e = rng.rand(nl, batch) ** (1 + trial % 5)
        if trial % 7 == 0:
            e[:, 0] = 0.0
        lo = rng.randint(0, 50, size=batch)
        hi = lo + rng.randint(1, 400, size=batch)
        total = np.array([rng.randint(nl * lo[b], nl * hi[b] + 1) for b in range(batch)])
        for mode in (0, 1):
            ent = torch.from_numpy(e).cuda()
            out = torch.empty((nl, batch), dtype=torch.int64, device="cuda")
            off = torch.empty(nl * batch + 1, dtype=torch.int64, device="cuda")
            lava.lava_layer_budgets(nl, batch, ent, torch.from_numpy(total).cuda(),
                                    torch.from_numpy(lo).cuda(), torch.from_numpy(hi).cuda(), mode,
                                    out, off)
            got = out.cpu().numpy()
            for b in range(batch):
                want = O.layer_budgets(list(e[:, b]), int(total[b]), int(lo[b]), int(hi[b]), mode)
                assert [int(x) for x in got[:, b]] == want
            flat = got.reshape(-1)
            np.testing.assert_array_equal(off.cpu().numpy(),
                                          np.concatenate([[0], np.cumsum(flat)]))


def test_results_are_bitwise_reproducible():
    cfg = get_config("llama8b_8k").scaled(seq_lens=(2222,), n_layers=2, budget_per_head=100)
    q, k, v, cu = upload_model(cfg)
    plan = make_plan(cfg, q, k, v, cu)
    lava.evict_model(plan, q, k, v)
    ref = [plan.scores.clone(), plan.entropy.clone(), plan.keep_idx.clone(), plan.k_out.clone()]
    for _ in range(5):
        lava.evict_model(plan, q, k, v)
        assert torch.equal(plan.scores, ref[0]) and torch.equal(plan.entropy, ref[1])
        assert torch.equal(plan.keep_idx, ref[2])
        assert torch.equal(plan.k_out.view(torch.int16), ref[3].view(torch.int16))


def test_per_layer_calls_equal_the_batched_calls():
    cfg = get_config("llama8b_8k").scaled(seq_lens=(1100,), n_layers=2, budget_per_head=90)
    q, k, v, cu = upload_model(cfg)
    plan = make_plan(cfg, q, k, v, cu)
    lava.evict_model(plan, q, k, v)
    d = plan.desc
    ws = torch.zeros(lava.lava_workspace_bytes(d, 1), dtype=torch.uint8, device="cuda")
    for l in range(cfg.n_layers):
        sc = torch.empty_like(plan.scores[l])
        ent = torch.empty(1, dtype=torch.float64, device="cuda")
        vb = torch.empty(1, d.n_kv_heads, device="cuda")
        lava.lava_score_layer(d, q[l], k[l], v[l], None, sc, vb, ent, ws)
        assert torch.equal(sc, plan.scores[l]) and torch.equal(ent, plan.entropy[l])
        keep = torch.empty_like(plan.keep_idx[l])
        hoff = torch.empty_like(plan.head_offsets[l])
        lava.lava_select_topk(d, sc, plan.layer_budget[l], keep, hoff)
        nsel = int(hoff[0, -1]) - d.n_kv_heads * d.window
        assert torch.equal(keep[:nsel], plan.keep_idx[l][:nsel]) and torch.equal(hoff, plan.head_offsets[l])
        ko, vo = torch.zeros_like(plan.k_out), torch.zeros_like(plan.v_out)
        lava.lava_compact_kv(d, k[l], v[l], keep, hoff, plan.layer_row_offset[l: l + 1], ko, vo)
        r0, r1 = int(plan.layer_row_offset[l]), int(plan.layer_row_offset[l + 1])
        assert torch.equal(ko[r0:r1].view(torch.int16), plan.k_out[r0:r1].view(torch.int16))
        assert torch.equal(vo[r0:r1].view(torch.int16), plan.v_out[r0:r1].view(torch.int16))
        # a caller-supplied value norm replaces the pass over V
        sc2 = torch.empty_like(sc)
        lava.lava_score_layer(d, q[l], k[l], None, vb, sc2, None, ent, ws)
        assert torch.equal(sc2, sc)


def test_wo_norm():
    from lava_workloads.generate import generate_wo
    w_o = generate_wo(get_config("tiny"), 0).cuda()
    out = torch.zeros(1, device="cuda")
    lava.lava_wo_norm(w_o, out)
    assert abs(float(out) - O.wo_norm(w_o.cpu().numpy())) < 1e-4 * float(out)


def test_host_buffer_path_equals_device_path():
    cfg = get_config("mistral7b_ragged").scaled(seq_lens=(640, 901), n_layers=3, budget_per_head=96)
    q, k, v, cu = upload_model(cfg)
    plan = make_plan(cfg, q, k, v, cu)
    lava.evict_model(plan, q, k, v)
    rows = plan.k_out.shape[0]
    L, hkv = cfg.n_layers, cfg.n_kv_heads
    pin = lambda x: x.cpu().pin_memory()
    out_budget = torch.empty((L, cfg.batch), dtype=torch.int64).pin_memory()
    out_hoff = torch.empty((L, cfg.batch, hkv + 1), dtype=torch.int32).pin_memory()
    out_k = torch.empty((rows, cfg.head_dim), dtype=k.dtype).pin_memory()
    out_v = torch.empty((rows, cfg.head_dim), dtype=k.dtype).pin_memory()
    budgets = [cfg.total_budget(b) for b in range(cfg.batch)]
    arena = torch.empty(lava.lava_host_arena_bytes(plan.desc, L, rows), dtype=torch.uint8, device="cuda")
    for _ in range(2):
        lava.lava_evict_model_host(plan.desc, L, pin(q), pin(k), pin(v),
                                   torch.tensor(cfg.seq_lens, dtype=torch.int32),
                                   torch.tensor(budgets, dtype=torch.int64), 0, out_budget, out_hoff,
                                   out_k, out_v, arena)
        torch.cuda.synchronize()
        assert torch.equal(out_budget, plan.layer_budget.cpu())
        assert torch.equal(out_hoff, plan.head_offsets.cpu())
        assert torch.equal(out_k.view(torch.int16), plan.k_out.cpu().view(torch.int16))
        assert torch.equal(out_v.view(torch.int16), plan.v_out.cpu().view(torch.int16))

@pytest.mark.parametrize("kw", [
    # query groups of more than 128 window-query rows: two halves per KV head on the tensor-core path
    dict(n_q_heads=8, n_kv_heads=2, window=64, seq_lens=(1500,)),                    # G 4 x w 64, max-pool
    dict(n_q_heads=14, n_kv_heads=2, window=32, seq_lens=(1100, 700)),               # G 7: halves of 4 and 3
    dict(n_q_heads=4, n_kv_heads=2, window=128, seq_lens=(1300,)),                   # G 2 x w 128: one head each
    dict(n_q_heads=32, n_kv_heads=2, window=16, seq_lens=(900,)),                    # G 16 x w 16: 8 heads each
    dict(n_q_heads=6, n_kv_heads=2, window=64, seq_lens=(1000,), pool_kind=lava.LAVA_POOL_AVG,
         pool_kernel=5),                                                             # G 3: halves of 2 and 1, avg
    dict(n_q_heads=8, n_kv_heads=2, window=64, seq_lens=(64,)),                      # n == w
    dict(n_q_heads=8, n_kv_heads=2, window=64, seq_lens=(65, 200)),                  # one candidate
])
def test_split_query_groups(kw):
    budget = min(max(kw["window"], 96), min(kw["seq_lens"]))   # between the window and the shortest n
    cfg = get_config("llama8b_8k").scaled(n_layers=2, budget_per_head=budget, **kw)
    n, d = cfg.total_tokens, cfg.head_dim
    desc = lava.LayerDesc(n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads, head_dim=d,
                          window=cfg.window, pool_kind=cfg.pool_kind, pool_kernel=cfg.pool_kernel,
                          batch=cfg.batch, max_seqlen=max(cfg.seq_lens),
                          cu_seqlens=torch.zeros(cfg.batch + 1, dtype=torch.int32) if cfg.batch > 1 else None,
                          total_tokens=n, k_stride_head=n * d, k_stride_tok=d, v_stride_head=n * d,
                          v_stride_tok=d)
    assert lava.lava_score_path(desc) == 2, "this geometry must run as two units per KV head"
    compare_eviction(cfg)



@pytest.mark.parametrize("kw", [
    dict(seq_lens=(1733,), n_layers=3, budget_per_head=160),                              # G 4 x w 32
    dict(seq_lens=(777, 1290, 515), n_layers=2, budget_per_head=128, window=64,
         pool_kind=lava.LAVA_POOL_AVG, pool_kernel=5),                                    # two units, avg-pool, ragged
    dict(seq_lens=(2100,), n_layers=2, budget_per_head=200, n_q_heads=14, n_kv_heads=2),  # G 7: units of 4 and 3
    dict(seq_lens=(900,), n_layers=2, budget_per_head=64, n_q_heads=32, n_kv_heads=2, window=16),  # 8 heads per unit
    dict(seq_lens=(1300,), n_layers=1, budget_per_head=140, n_q_heads=4, n_kv_heads=2, window=128),
    dict(seq_lens=(33, 64), n_layers=2, budget_per_head=33),                              # one candidate / n == 2w
])
def test_single_pass_score_kernel(kw):
    """The opt-in single-pass kernel (exponentials kept in tensor memory as fp16) against the
    oracle on the geometries it covers, whole eviction."""
    cfg = get_config("llama8b_8k").scaled(**kw)
    lava.lava_set_option("score_kernel", 2)
    try:
        rep = compare_eviction(cfg)
        assert rep["max_rel_err"] < 1e-3
    finally:
        lava.lava_set_option("score_kernel", 0)
