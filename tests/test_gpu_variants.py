"""The ablation axes of the paper as modes of the CUDA path, each against its oracle function:
per-head top-k ("- head dynamic", Sec. 5.4), PyramidKV layer budgets (LAVa-Pyramid of the
layer-allocation comparison), the SnapKV / AdaKV score (value term 1) and the VATP score
(per-token value norms) of the paper's table of methods."""
import numpy as np
import pytest
import torch

import paper_2509_09754_b200 as lava
from lava_workloads import get_config, to_numpy64
from oracle import lava_oracle as O
from tests.parity_harness import ENTROPY_RTOL, SCORE_ATOL, SCORE_RTOL, upload_model

pytestmark = pytest.mark.gpu


def _desc(cfg, q, k, v, cu, flags):
    return lava.LayerDesc.for_tensors(q[0], k[0], v[0], cfg.window, cfg.pool_kind, cfg.pool_kernel,
                                      cu_seqlens=cu if cfg.batch > 1 else None,
                                      max_seqlen=max(cfg.seq_lens), flags=flags)


@pytest.mark.parametrize("name,kw", [
    ("llama8b_8k", dict(seq_lens=(1733,), n_layers=2)),                              # tensor-core path
    ("mistral7b_ragged", dict(seq_lens=(700, 1301), n_layers=2)),                    # two units, avg-pool, ragged
    ("tiny", dict(n_layers=2)),                                                      # CUDA-core path, fp32
])
@pytest.mark.parametrize("term", [O.VALUE_NORM_UNIT, O.VALUE_NORM_TOKEN])
def test_value_term_variants_match_the_oracle(name, kw, term):
    cfg = get_config(name).scaled(**kw)
    q, k, v, cu = upload_model(cfg)
    flags = lava.LAVA_FLAG_UNIT_VALUE_NORM if term == O.VALUE_NORM_UNIT else lava.LAVA_FLAG_TOKEN_VALUE_NORM
    desc = _desc(cfg, q, k, v, cu, flags)
    L, hkv, w = cfg.n_layers, cfg.n_kv_heads, cfg.window
    ws = torch.zeros(lava.lava_workspace_bytes(desc, L), dtype=torch.uint8, device="cuda")
    scores = torch.zeros((L, desc.total_scores), dtype=torch.float32, device="cuda")
    vbar = torch.zeros((L, cfg.batch, hkv), dtype=torch.float32, device="cuda")
    ent = torch.zeros((L, cfg.batch), dtype=torch.float64, device="cuda")
    v_arg = None if term == O.VALUE_NORM_UNIT else v          # the unit term never reads V
    lava.lava_score_layers(desc, L, q, k, v_arg, q.stride(0), k.stride(0), v.stride(0), None, scores,
                           vbar, ent, ws)
    assert lava.lava_poll_status(ws) == 0
    g_scores, g_ent = scores.cpu().numpy(), ent.cpu().numpy()
    tok0 = 0
    for b, n in enumerate(cfg.seq_lens):
        so = hkv * (tok0 - b * w)
        for l in range(L):
            want = O.variant_scores(to_numpy64(q[l, b]), to_numpy64(k[l, :, tok0:tok0 + n]),
                                    to_numpy64(v[l, :, tok0:tok0 + n]), w, cfg.pool_kind,
                                    cfg.pool_kernel, value_term=term)
            got = g_scores[l, so: so + hkv * (n - w)].reshape(hkv, n - w).astype(np.float64)
            assert np.all(np.abs(got - want) <= SCORE_RTOL * np.abs(want) + SCORE_ATOL)
            o_ent = O.layer_entropy(want, n)
            assert abs(g_ent[l, b] - o_ent) <= ENTROPY_RTOL * abs(o_ent) + 1e-15
        tok0 += n


@pytest.mark.parametrize("name,kw", [
    ("llama8b_8k", dict(seq_lens=(2222,), n_layers=2, budget_per_head=100)),
    ("mistral7b_ragged", dict(seq_lens=(640, 901, 333), n_layers=2, budget_per_head=96)),
    ("tiny", dict(seq_lens=(300,), budget_per_head=30)),
    ("tiny", dict(seq_lens=(40,), budget_per_head=38)),            # shares larger than the heads
])
def test_per_head_topk_matches_the_oracle(name, kw):
    """Whole eviction with LAVA_FLAG_PER_HEAD_TOPK: selection and compaction bit-exact against
    select_topk_per_head on the device's own scores."""
    cfg = get_config(name).scaled(**kw)
    q, k, v, cu = upload_model(cfg)
    desc = _desc(cfg, q, k, v, cu, lava.LAVA_FLAG_PER_HEAD_TOPK)
    L, hkv, w = cfg.n_layers, cfg.n_kv_heads, cfg.window
    budgets = [cfg.total_budget(b) for b in range(cfg.batch)]
    plan = lava.EvictionPlan.create(desc, L, budgets, cfg.seq_lens, kv_dtype=k.dtype)
    plan.keep_idx.fill_(-12345)
    lava.evict_model(plan, q, k, v)
    assert lava.lava_poll_status(plan.workspace) == 0
    g_scores = plan.scores.cpu().numpy()
    g_budget = plan.layer_budget.cpu().numpy()
    g_hoff = plan.head_offsets.cpu().numpy()
    g_keep = plan.keep_idx.cpu().numpy()
    g_rowoff = plan.layer_row_offset.cpu().numpy()
    bits = torch.int16 if k.dtype == torch.bfloat16 else torch.int32
    tok0 = 0
    for b, n in enumerate(cfg.seq_lens):
        prefix, so = n - w, hkv * (tok0 - b * w)
        for l in range(L):
            s = g_scores[l, so: so + hkv * prefix].reshape(hkv, prefix).astype(np.float64)
            keep, off = O.select_topk_per_head(s, int(g_budget[l, b]), w)
            np.testing.assert_array_equal(g_hoff[l, b], off)
            seg = g_keep[l, so: so + hkv * prefix]
            got = []
            for g in range(hkv):
                a, e = int(off[g]) - g * w, int(off[g + 1]) - (g + 1) * w
                np.testing.assert_array_equal(seg[a:e], keep[g])
                got.append(seg[a:e])
            assert np.all(seg[int(off[-1]) - hkv * w:] == -12345)
            ko, vo = O.compact_kv(k[l, :, tok0:tok0 + n].cpu().view(bits).numpy(),
                                  v[l, :, tok0:tok0 + n].cpu().view(bits).numpy(), got, w)
            r0 = int(g_rowoff[l * cfg.batch + b])
            rows = int(off[-1])
            np.testing.assert_array_equal(plan.k_out[r0:r0 + rows].cpu().view(bits).numpy(), ko)
            np.testing.assert_array_equal(plan.v_out[r0:r0 + rows].cpu().view(bits).numpy(), vo)
        tok0 += n


def test_pyramid_budgets_are_bit_exact_against_the_oracle_rule():
    rng = np.random.RandomState(7)
    for trial in range(30):
        nl = int(rng.randint(1, 40))
        batch = int(rng.randint(1, 4))
        beta = int(rng.choice([0, 2, 5, 20, 33]))
        lo = rng.randint(0, 50, size=batch)
        hi = lo + rng.randint(1, 400, size=batch)
        total = np.array([rng.randint(nl * lo[b], nl * hi[b] + 1) for b in range(batch)])
        ent = torch.from_numpy(rng.rand(nl, batch)).cuda()              # ignored by the mode
        out = torch.empty((nl, batch), dtype=torch.int64, device="cuda")
        off = torch.empty(nl * batch + 1, dtype=torch.int64, device="cuda")
        lava.lava_layer_budgets(nl, batch, ent, torch.from_numpy(total).cuda(),
                                torch.from_numpy(lo).cuda(), torch.from_numpy(hi).cuda(),
                                lava.LAVA_BUDGET_PYRAMID | (beta << 8), out, off)
        got = out.cpu().numpy()
        for b in range(batch):
            want = O.layer_budgets([0.0] * nl, int(total[b]), int(lo[b]), int(hi[b]),
                                   O.BUDGET_PYRAMID, beta=float(beta) if beta else 20.0)
            assert [int(x) for x in got[:, b]] == want
