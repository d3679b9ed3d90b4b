"""Decode-time attention over the packed, per-head ragged cache against the oracle, on the cache
the eviction itself produced (one-shot path and the layer-by-layer cascade)."""
import numpy as np
import pytest
import torch

import paper_2509_09754_b200 as lava
from lava_workloads import get_config, to_numpy64
from oracle import lava_oracle as O
from tests.parity_harness import make_plan, upload_model

pytestmark = pytest.mark.gpu

# bf16 tensor path: probabilities are rounded to bf16 (unit roundoff 2^-9) before they multiply
# V, everything else is fp32: |err| <= 2^-8 * sum_i p_i |V[i][c]| with room for the fp32 sums
P_ROUND = 2.0 ** -8


def _check(cfg, q_new, k_out, v_out, hoff, roff, out, L):
    hq, hkv, w = cfg.n_q_heads, cfg.n_kv_heads, cfg.window
    hoff, roff = hoff.cpu().numpy(), roff.cpu().numpy()
    got = out.cpu().numpy().astype(np.float64)
    kh, vh = to_numpy64(k_out), to_numpy64(v_out)
    for l in range(L):
        for b in range(cfg.batch):
            r0 = int(roff[l * cfg.batch + b])
            kr = [kh[r0 + int(hoff[l, b, g]): r0 + int(hoff[l, b, g + 1])] for g in range(hkv)]
            vr = [vh[r0 + int(hoff[l, b, g]): r0 + int(hoff[l, b, g + 1])] for g in range(hkv)]
            want = O.decode_attention(to_numpy64(q_new[l, b]), kr, vr)
            mag = O.decode_attention(to_numpy64(q_new[l, b]), kr, [np.abs(x) for x in vr])
            tol = (P_ROUND if k_out.dtype == torch.bfloat16 else 1e-5) * mag + 1e-6
            assert np.all(np.abs(got[l, b] - want) <= tol), (l, b, np.abs(got[l, b] - want).max())


@pytest.mark.parametrize("name,kw", [
    ("llama8b_8k", dict(seq_lens=(4000,), n_layers=3, budget_per_head=700)),      # several warps per head
    ("mistral7b_ragged", dict(seq_lens=(640, 901, 333), n_layers=2, budget_per_head=96)),
    ("gqa7_128k", dict(seq_lens=(2500,), n_layers=2, budget_per_head=300)),       # 7 queries per KV head
    ("tiny", dict(seq_lens=(300,), n_layers=2, budget_per_head=40)),              # fp32, d = 64: plain kernel
])
def test_decode_attention_matches_the_oracle_on_the_evicted_cache(name, kw):
    cfg = get_config(name).scaled(**kw)
    q, k, v, cu = upload_model(cfg)
    L = cfg.n_layers
    plan = make_plan(cfg, q, k, v, cu)
    lava.evict_model(plan, q, k, v)
    assert lava.lava_poll_status(plan.workspace) == 0
    gen = torch.Generator().manual_seed(21)
    q_new = torch.randn(L, cfg.batch, cfg.n_q_heads, cfg.head_dim, generator=gen).to(k.dtype).cuda()
    out = torch.full((L, cfg.batch, cfg.n_q_heads, cfg.head_dim), float("nan"), device="cuda")
    ws = torch.empty(max(256, lava.lava_decode_workspace_bytes(plan.desc, L)), dtype=torch.uint8, device="cuda")
    lava.lava_decode_attention_layers(plan.desc, L, q_new, plan.k_out, plan.v_out, plan.head_offsets,
                                      plan.layer_row_offset, out, ws)
    torch.cuda.synchronize()
    _check(cfg, q_new, plan.k_out, plan.v_out, plan.head_offsets, plan.layer_row_offset, out, L)
    # the one-layer form on the last layer
    one = torch.full((cfg.batch, cfg.n_q_heads, cfg.head_dim), float("nan"), device="cuda")
    lava.lava_decode_attention(plan.desc, q_new[L - 1], plan.k_out, plan.v_out, plan.head_offsets[L - 1],
                               plan.layer_row_offset[(L - 1) * cfg.batch:], one, ws)
    torch.cuda.synchronize()
    assert torch.equal(one, out[L - 1])


def test_decode_attention_reads_a_cascade_state():
    cfg = get_config("llama8b_8k").scaled(seq_lens=(1800,), n_layers=3, budget_per_head=200)
    q, k, v, cu = upload_model(cfg)
    plan = make_plan(cfg, q, k, v, cu)
    cas = lava.Cascade(plan.desc, cfg.n_layers, cfg.total_budget(0), kv_dtype=k.dtype)
    cas.begin(plan.total_budget)
    for l in range(cfg.n_layers):
        cas.step(q[l], k[l], v[l])
    view = cas.view()
    L = cfg.n_layers
    gen = torch.Generator().manual_seed(22)
    q_new = torch.randn(L, 1, cfg.n_q_heads, cfg.head_dim, generator=gen).to(k.dtype).cuda()
    out = torch.empty((L, 1, cfg.n_q_heads, cfg.head_dim), device="cuda")
    ws = torch.empty(lava.lava_decode_workspace_bytes(plan.desc, L), dtype=torch.uint8, device="cuda")
    lava.lava_decode_attention_layers(plan.desc, L, q_new, view["k_out"], view["v_out"],
                                      view["head_offsets"], view["layer_row_offset"], out, ws)
    torch.cuda.synchronize()
    _check(cfg, q_new, view["k_out"], view["v_out"], view["head_offsets"], view["layer_row_offset"], out, L)
    cas.close()


def test_decode_attention_with_eight_queries_per_kv_head():
    """G = 8 fills the eight real rows of the padded query operand; w = 16 keeps the score path
    on one unit."""
    cfg = get_config("llama8b_8k").scaled(seq_lens=(1500,), n_layers=2, n_q_heads=32, n_kv_heads=4,
                                          window=16, budget_per_head=300)
    q, k, v, cu = upload_model(cfg)
    L = cfg.n_layers
    plan = make_plan(cfg, q, k, v, cu)
    lava.evict_model(plan, q, k, v)
    assert lava.lava_poll_status(plan.workspace) == 0
    gen = torch.Generator().manual_seed(23)
    q_new = torch.randn(L, 1, cfg.n_q_heads, cfg.head_dim, generator=gen).to(k.dtype).cuda()
    out = torch.empty((L, 1, cfg.n_q_heads, cfg.head_dim), device="cuda")
    ws = torch.empty(lava.lava_decode_workspace_bytes(plan.desc, L), dtype=torch.uint8, device="cuda")
    lava.lava_decode_attention_layers(plan.desc, L, q_new, plan.k_out, plan.v_out, plan.head_offsets,
                                      plan.layer_row_offset, out, ws)
    torch.cuda.synchronize()
    _check(cfg, q_new, plan.k_out, plan.v_out, plan.head_offsets, plan.layer_row_offset, out, L)
