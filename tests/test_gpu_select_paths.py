"""Every code path of the layer-wide selection (Algorithm 1, Evict) against the oracle's
``select_topk`` on synthetic score arrays: the register-resident kernel at 8, 16, 32 and 64 keys
per thread with clusters of 8 and 16 CTAs, and the streaming kernel for layers beyond 524 288
candidates.  Scores are heavily tied, constant, zero or skewed, and the budgets sit on every edge
(window only, one more, mid, all but one, all, more than all)."""
import numpy as np
import pytest
import torch

import paper_2509_09754_b200 as lava
from oracle import lava_oracle as O

pytestmark = pytest.mark.gpu


def _score_cases(rng, hkv, prefix):
    yield "rounded", np.round(rng.rand(hkv, prefix), 2).astype(np.float32)     # ~100 distinct values
    yield "constant", np.full((hkv, prefix), 0.25, dtype=np.float32)          # pure tie-break
    yield "skewed", (rng.rand(hkv, prefix) ** 8).astype(np.float32)
    yield "zeros", np.zeros((hkv, prefix), dtype=np.float32)
    runs = np.repeat(rng.rand(hkv, prefix // 7 + 1).astype(np.float32), 7, axis=1)[:, :prefix]
    yield "runs_of_7", np.ascontiguousarray(runs)                             # what max-pool 7 leaves


def _check(hkv, n, w, cluster, seed):
    prefix = n - w
    rng = np.random.RandomState(seed)
    desc = lava.LayerDesc(n_q_heads=hkv, n_kv_heads=hkv, head_dim=128, window=w, total_tokens=n,
                          k_stride_head=n * 128, k_stride_tok=128, v_stride_head=n * 128,
                          v_stride_tok=128)
    lava.lava_set_option("select_cluster", cluster)
    try:
        for name, s in _score_cases(rng, hkv, prefix):
            scores = torch.from_numpy(s).cuda().reshape(-1)
            flat64 = s.astype(np.float64)
            for budget in (hkv * w, hkv * w + 1, hkv * w + 777, hkv * (w + prefix // 3),
                           hkv * n - 1, hkv * n, 5 * hkv * n):
                keep = torch.full((hkv * prefix,), -1, dtype=torch.int32, device="cuda")
                hoff = torch.zeros(hkv + 1, dtype=torch.int32, device="cuda")
                lb = torch.tensor([budget], dtype=torch.int64, device="cuda")
                lava.lava_select_topk(desc, scores, lb, keep, hoff)
                want_keep, want_off = O.select_topk(flat64, budget, w)
                got_off = hoff.cpu().numpy()
                np.testing.assert_array_equal(got_off, want_off, err_msg="%s budget %d" % (name, budget))
                got = keep.cpu().numpy()
                for g in range(hkv):
                    a, e = got_off[g] - g * w, got_off[g + 1] - (g + 1) * w
                    np.testing.assert_array_equal(got[a:e], want_keep[g],
                                                  err_msg="%s budget %d head %d" % (name, budget, g))
                assert np.all(got[got_off[-1] - hkv * w:] == -1), "written beyond the selected count"
    finally:
        lava.lava_set_option("select_cluster", 0)


@pytest.mark.parametrize("hkv,n,w,cluster,what", [
    (8, 8192, 32, 0, "16 keys per thread, clusters of 8 (the 8K workload)"),
    (8, 8192, 32, 16, "8 keys per thread, clusters of 16"),
    (8, 32768, 32, 0, "32 keys per thread, clusters of 16 (the 32K workload)"),
    (8, 32768, 32, 8, "64 keys per thread, clusters of 8"),
    (4, 131072, 32, 0, "64 keys per thread, clusters of 16 (the 128K workload)"),
    (8, 70000, 32, 0, "streaming kernel: 559 744 candidates"),
    (3, 40001, 16, 0, "odd sizes, heads not aligned with threads"),
])
def test_select_paths_are_exact(hkv, n, w, cluster, what):
    _check(hkv, n, w, cluster, seed=hkv * 1000 + n % 997)


def test_select_many_problems_in_one_launch():
    """Several (layer, sequence) problems of different sizes in one launch, ragged batch."""
    hkv, w, L = 4, 32, 3
    lens = (5000, 20000, 777, 33)
    total = sum(lens)
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
    desc = lava.LayerDesc(n_q_heads=hkv, n_kv_heads=hkv, head_dim=128, window=w, batch=len(lens),
                          max_seqlen=max(lens), cu_seqlens=cu, total_tokens=total,
                          k_stride_head=total * 128, k_stride_tok=128, v_stride_head=total * 128,
                          v_stride_tok=128)
    ts = desc.total_scores
    rng = np.random.RandomState(11)
    s = np.round(rng.rand(L, ts), 3).astype(np.float32)
    budgets = rng.randint(hkv * w, hkv * 600, size=(L, len(lens))).astype(np.int64)
    budgets[:, 3] = hkv * 33                                 # the shortest keeps everything
    scores = torch.from_numpy(s).cuda()
    keep = torch.full((L, ts), -1, dtype=torch.int32, device="cuda")
    hoff = torch.zeros((L, len(lens), hkv + 1), dtype=torch.int32, device="cuda")
    lava.lava_select_topk_layers(desc, L, scores, torch.from_numpy(budgets).cuda(), keep, hoff)
    got, got_off = keep.cpu().numpy(), hoff.cpu().numpy()
    tok0 = 0
    for b, n in enumerate(lens):
        prefix, so = n - w, hkv * (tok0 - b * w)
        for l in range(L):
            seg = s[l, so: so + hkv * prefix].reshape(hkv, prefix).astype(np.float64)
            want_keep, want_off = O.select_topk(seg, int(budgets[l, b]), w)
            np.testing.assert_array_equal(got_off[l, b], want_off)
            for g in range(hkv):
                a, e = want_off[g] - g * w, want_off[g + 1] - (g + 1) * w
                np.testing.assert_array_equal(got[l, so + a: so + e], want_keep[g])
        tok0 += n
