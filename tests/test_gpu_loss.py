"""Layer attention output loss (Lemma 1, p = 1, last token) and the bound of Theorem 1 on the
GPU against the oracle's evaluators, for the selection the eviction itself made."""
import numpy as np
import pytest
import torch

import paper_2509_09754_b200 as lava
from lava_workloads import get_config, to_numpy64
from oracle import lava_oracle as O
from tests.parity_harness import make_plan, upload_model

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,kw,w_dtype", [
    ("tiny", dict(seq_lens=(300,), n_layers=2, budget_per_head=40), torch.float32),
    ("llama8b_8k", dict(seq_lens=(1100,), n_layers=2, budget_per_head=128), torch.bfloat16),
    ("mistral7b_ragged", dict(seq_lens=(400, 650), n_layers=2, budget_per_head=100), torch.float32),
])
def test_loss_and_bound_match_the_oracle(name, kw, w_dtype):
    cfg = get_config(name).scaled(**kw)
    q, k, v, cu = upload_model(cfg)
    L, hq, hkv, w, d = cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.window, cfg.head_dim
    plan = make_plan(cfg, q, k, v, cu)
    lava.evict_model(plan, q, k, v)
    assert lava.lava_poll_status(plan.workspace) == 0
    d_model = 192
    gen = torch.Generator().manual_seed(5)
    w_o = (torch.randn(hq * d, d_model, generator=gen) / 8).to(w_dtype).cuda()
    loss = torch.zeros(cfg.batch, dtype=torch.float64, device="cuda")
    bound = torch.zeros(cfg.batch, dtype=torch.float64, device="cuda")
    hoff = plan.head_offsets.cpu().numpy()
    keep_idx = plan.keep_idx.cpu().numpy()
    group = hq // hkv
    for l in range(L):
        lava.lava_layer_output_loss(plan.desc, q[l], k[l], v[l], plan.keep_idx[l], plan.head_offsets[l],
                                    plan.vbar[l], w_o, loss, bound)
        g_loss, g_bound = loss.cpu().numpy(), bound.cpu().numpy()
        tok0 = 0
        for b, n in enumerate(cfg.seq_lens):
            so = hkv * (tok0 - b * w)
            kk, vv = to_numpy64(k[l, :, tok0:tok0 + n]), to_numpy64(v[l, :, tok0:tok0 + n])
            att = O.window_attention(to_numpy64(q[l, b]), kk)[:, w - 1, :]          # [H_q, n]
            masks = np.zeros((hkv, n))
            masks[:, n - w:] = 1.0
            for g in range(hkv):
                a, e = int(hoff[l, b, g]) - g * w, int(hoff[l, b, g + 1]) - (g + 1) * w
                masks[g, keep_idx[l, so + a: so + e]] = 1.0
            heads = [h // group for h in range(hq)]
            o_loss = O.layer_output_loss(att, vv[heads], to_numpy64(w_o), masks[heads])
            o_bound = O.loss_upper_bound(att, vv[heads], to_numpy64(w_o), masks[heads])
            assert abs(g_loss[b] - o_loss) <= 1e-6 * abs(o_loss) + 1e-12
            assert abs(g_bound[b] - o_bound) <= 1e-5 * abs(o_bound) + 1e-12
            assert g_loss[b] <= g_bound[b] * (1 + 1e-9)                              # Theorem 1
            tok0 += n
