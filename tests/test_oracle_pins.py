"""Pins for the CPU oracle: closed forms, library routines, invariants and brute force.

None of these tests re-types the oracle's own formula: each compares it with something the
paper or the mathematics fixes independently.
"""
import itertools
import math

import numpy as np
import pytest
import scipy.stats
import torch

from oracle import lava_oracle as O


def _rand_layer(seed, hq, hkv, n, w, d, vscale=None):
    rng = np.random.RandomState(seed)
    q = rng.randn(hq, w, d)
    k = rng.randn(hkv, n, d)
    v = rng.randn(hkv, n, d)
    if vscale is not None:
        v *= np.asarray(vscale, dtype=np.float64)[:, None, None]
    return q, k, v


# ---------------------------------------------------------------- attention rows (Sec. 2)
def test_attention_rows_match_library_softmax():
    """Causal softmax built with torch ops on the full [n, n] problem, last w rows taken."""
    hq, hkv, n, w, d = 4, 2, 37, 5, 8
    q, k, v = _rand_layer(1, hq, hkv, n, w, d)
    att = O.window_attention(q, k)
    g = hq // hkv
    for h in range(hq):
        # embed the window queries as the last w rows of a full query matrix
        qfull = torch.zeros(n, d, dtype=torch.float64)
        qfull[n - w:] = torch.from_numpy(q[h])
        logits = qfull @ torch.from_numpy(k[h // g]).T / math.sqrt(d)
        causal = torch.tril(torch.ones(n, n, dtype=torch.bool))
        logits = logits.masked_fill(~causal, float("-inf"))
        ref = torch.softmax(logits, dim=-1)[n - w:].numpy()
        np.testing.assert_allclose(att[h], ref, rtol=1e-12, atol=1e-15)


def test_attention_rows_sum_to_one_and_are_causal():
    q, k, v = _rand_layer(2, 2, 2, 50, 7, 16)
    att = O.window_attention(q, k)
    np.testing.assert_allclose(att.sum(axis=2), 1.0, rtol=1e-12)
    prefix = 50 - 7
    for t in range(7):
        assert np.all(att[:, t, prefix + t + 1:] == 0.0)
        assert np.all(att[:, t, : prefix + t + 1] > 0.0)
    a = O.window_mean_prefix(att, 7)
    assert np.all(a.sum(axis=1) < 1.0)          # the window itself holds some of the mass


def test_transposed_or_unscaled_logits_would_be_caught():
    """sm_scale really scales the logits: doubling q with half the scale changes nothing."""
    q, k, v = _rand_layer(3, 2, 1, 40, 4, 8)
    a1 = O.window_attention(q, k, sm_scale=0.25)
    a2 = O.window_attention(2.0 * q, k, sm_scale=0.125)
    np.testing.assert_allclose(a1, a2, rtol=1e-12)
    a3 = O.window_attention(q, k)               # default = 1/sqrt(d)
    a4 = O.window_attention(q, k, sm_scale=1.0 / math.sqrt(8))
    np.testing.assert_array_equal(a3, a4)


# ---------------------------------------------------------------- closed form: Q = 0
@pytest.mark.parametrize("pool_kind,kernel", [(O.POOL_MAX, 7), (O.POOL_AVG, 5), (O.POOL_NONE, 1)])
def test_zero_queries_give_harmonic_closed_form(pool_kind, kernel):
    """Uniform attention A^j[i] = 1/(j+1) => s = Vbar * (H_n - H_P) / w for every prefix i."""
    hq, hkv, n, w, d = 4, 2, 64, 8, 16
    q, k, v = _rand_layer(4, hq, hkv, n, w, d, vscale=[1.0, 3.0])
    q[:] = 0.0
    s = O.lava_scores(q, k, v, w, pool_kind, kernel)
    prefix = n - w
    harm = sum(1.0 / (j + 1) for j in range(prefix, n))      # positions P..n-1 see j+1 keys
    vbar = np.array([np.linalg.norm(v[g].T, 1) for g in range(hkv)])
    base = vbar[:, None] * harm / w * np.ones((hkv, prefix))
    if pool_kind == O.POOL_AVG:
        r = kernel // 2
        taps = np.array([min(prefix, i + r + 1) - max(0, i - r) for i in range(prefix)])
        base = base * taps[None, :] / kernel
    np.testing.assert_allclose(s, base, rtol=1e-12)


# ---------------------------------------------------------------- pooling vs library
@pytest.mark.parametrize("kernel", [1, 3, 5, 7])
def test_pooling_matches_torch(kernel):
    rng = np.random.RandomState(5)
    a = rng.rand(3, 29)
    t = torch.from_numpy(a).unsqueeze(0)
    mx = torch.nn.functional.max_pool1d(t, kernel, stride=1, padding=kernel // 2)[0].numpy()
    av = torch.nn.functional.avg_pool1d(t, kernel, stride=1, padding=kernel // 2,
                                        count_include_pad=True)[0].numpy()
    np.testing.assert_array_equal(O.pool1d(a, O.POOL_MAX, kernel), mx)
    np.testing.assert_allclose(O.pool1d(a, O.POOL_AVG, kernel), av, rtol=1e-14)
    np.testing.assert_array_equal(O.pool1d(a, O.POOL_NONE, kernel), a)


def test_pool_kernel_wider_than_prefix():
    a = np.array([[0.1, 0.7, 0.2]])
    np.testing.assert_array_equal(O.pool1d(a, O.POOL_MAX, 7), [[0.7, 0.7, 0.7]])
    np.testing.assert_allclose(O.pool1d(a, O.POOL_AVG, 7), [[1.0 / 7] * 3])


# ---------------------------------------------------------------- value norm (Theorem 1)
def test_value_norm_is_matrix_one_norm_of_v_transposed():
    rng = np.random.RandomState(6)
    v = rng.randn(3, 17, 9)
    ref = [np.linalg.norm(v[g].T, 1) for g in range(3)]        # max column abs-sum of V^T
    np.testing.assert_allclose(O.value_norm(v), ref, rtol=1e-14)
    v[1, 16] = 100.0                                           # a window row counts too
    assert O.value_norm(v)[1] == pytest.approx(900.0)


# ---------------------------------------------------------------- GQA group maximum (Sec. 4.3)
def test_gqa_score_is_max_of_single_head_scores():
    hq, hkv, n, w, d = 6, 2, 45, 6, 8
    q, k, v = _rand_layer(7, hq, hkv, n, w, d, vscale=[2.0, 0.5])
    s = O.lava_scores(q, k, v, w, O.POOL_AVG, 5)
    g = hq // hkv
    for kv in range(hkv):
        singles = [O.lava_scores(q[h:h + 1], k[kv:kv + 1], v[kv:kv + 1], w, O.POOL_AVG, 5)[0]
                   for h in range(kv * g, (kv + 1) * g)]
        np.testing.assert_allclose(s[kv], np.max(np.stack(singles), axis=0), rtol=1e-13)


def test_maxpool_commutes_with_group_max():
    hq, hkv, n, w, d = 4, 1, 60, 4, 8
    q, k, v = _rand_layer(8, hq, hkv, n, w, d)
    att = O.window_attention(q, k)
    a = O.window_mean_prefix(att, w)
    pool_then_max = O.pool1d(a, O.POOL_MAX, 7).max(axis=0)
    max_then_pool = O.pool1d(a.max(axis=0, keepdims=True), O.POOL_MAX, 7)[0]
    np.testing.assert_array_equal(pool_then_max, max_then_pool)
    s = O.lava_scores(q, k, v, w, O.POOL_MAX, 7)
    np.testing.assert_allclose(s[0], O.value_norm(v)[0] * max_then_pool, rtol=1e-14)


def test_equal_value_norms_reduce_to_window_attention_ranking():
    """Table 1: with one common Vbar, LAVa ranks exactly like pooled window-mean attention."""
    hq, hkv, n, w, d = 4, 4, 80, 8, 16
    q, k, v = _rand_layer(9, hq, hkv, n, w, d)
    for g in range(hkv):                       # give every head the same largest row L1 norm
        v[g] *= 10.0 / np.abs(v[g]).sum(axis=1).max()
    s = O.lava_scores(q, k, v, w, O.POOL_MAX, 7)
    snap = O.pool1d(O.window_mean_prefix(O.window_attention(q, k), w), O.POOL_MAX, 7)
    np.testing.assert_allclose(s, 10.0 * snap, rtol=1e-12)
    keep_l, _ = O.select_topk(s, 4 * w + 40, w)
    keep_s, _ = O.select_topk(snap, 4 * w + 40, w)
    for a, b in zip(keep_l, keep_s):
        np.testing.assert_array_equal(a, b)


def test_c_hat_scales_scores_but_changes_no_decision():
    q, k, v = _rand_layer(10, 4, 2, 70, 6, 8)
    s1 = O.lava_scores(q, k, v, 6, O.POOL_MAX, 5, c_hat=1.0)
    s2 = O.lava_scores(q, k, v, 6, O.POOL_MAX, 5, c_hat=3.5)
    np.testing.assert_allclose(s2, 3.5 * s1, rtol=1e-14)
    assert O.layer_entropy(s1, 70) == pytest.approx(O.layer_entropy(s2, 70), rel=1e-12)


# ---------------------------------------------------------------- entropy (Sec. 4.2)
def test_entropy_matches_library_and_closed_forms():
    rng = np.random.RandomState(11)
    s = rng.rand(3, 41)
    n = 50
    ref = scipy.stats.entropy(s.reshape(-1)) / (3 * n)        # natural log, normalises itself
    assert O.layer_entropy(s, n) == pytest.approx(ref, rel=1e-12)
    flat = np.full((3, 41), 0.37)
    assert O.layer_entropy(flat, n) == pytest.approx(math.log(3 * 41) / (3 * n), rel=1e-12)
    onehot = np.zeros((3, 41))
    onehot[1, 7] = 2.0
    assert O.layer_entropy(onehot, n) == 0.0
    assert O.layer_entropy(np.zeros((3, 41)), n) == 0.0


# ---------------------------------------------------------------- budgets (Algorithm 2)
def test_budgets_sum_and_proportionality():
    e = [0.3, 0.1, 0.25, 0.35]
    b = O.layer_budgets(e, 1000, 10, 10_000)
    assert sum(b) == 1000
    for bl, el in zip(b, e):
        assert abs(bl - 1000 * el / sum(e)) < 1.0
    # equal uncertainty -> equal budgets (+-1), and uniform mode ignores e
    b = O.layer_budgets([0.2] * 7, 1000, 1, 1000)
    assert sum(b) == 1000 and max(b) - min(b) <= 1
    assert b == sorted(b, reverse=True)                       # remainders go to lower layers
    b = O.layer_budgets(e, 1001, 10, 10_000, mode=O.BUDGET_UNIFORM)
    assert b == [251, 250, 250, 250]
    # scale of e (log base, constant divisors) is irrelevant
    assert O.layer_budgets(e, 777, 10, 10_000) == O.layer_budgets([7 * x for x in e], 777, 10, 10_000)
    # all-zero uncertainty -> uniform
    assert O.layer_budgets([0.0] * 4, 40, 1, 100) == [10, 10, 10, 10]


def test_budgets_clamping_keeps_sum_and_bounds():
    b = O.layer_budgets([0.9, 0.01, 0.01, 0.08], 450, 100, 200)
    assert sum(b) == 450 and min(b) >= 100 and max(b) <= 200
    assert b == [150, 100, 100, 100]
    b = O.layer_budgets([0.9, 0.05, 0.05], 500, 10, 200)
    assert sum(b) == 500 and b == [200, 150, 150]
    rng = np.random.RandomState(12)
    for _ in range(200):
        nl = rng.randint(1, 9)
        lo = rng.randint(0, 20)
        hi = lo + rng.randint(0, 50)
        total = rng.randint(nl * lo, nl * hi + 1)
        e = rng.rand(nl) ** 4
        b = O.layer_budgets(e, total, lo, hi)
        assert sum(b) == total and min(b) >= lo and max(b) <= hi
    with pytest.raises(ValueError):
        O.layer_budgets([0.5, 0.5], 10, 6, 20)


# ---------------------------------------------------------------- selection (Algorithm 1)
def test_selection_counts_and_window_always_kept():
    hq, hkv, n, w, d = 4, 2, 90, 10, 8
    q, k, v = _rand_layer(13, hq, hkv, n, w, d, vscale=[1.0, 4.0])
    s = O.lava_scores(q, k, v, w, O.POOL_MAX, 7)
    for budget in (hkv * w, hkv * w + 1, 57, hkv * n - 1, hkv * n, hkv * n + 50):
        keep, off = O.select_topk(s, budget, w)
        want = min(budget, hkv * n)
        assert off[-1] == want
        assert sum(len(x) for x in keep) == want - hkv * w
        ko, vo = O.compact_kv(k, v, keep, w)
        assert ko.shape[0] == want
        for g in range(hkv):                                   # window rows close every head
            np.testing.assert_array_equal(ko[off[g + 1] - w: off[g + 1]], k[g, n - w:])
            assert np.all(np.diff(keep[g]) > 0)
    keep, off = O.select_topk(s, hkv * n, w)                    # keep-all preserves the input
    ko, vo = O.compact_kv(k, v, keep, w)
    np.testing.assert_array_equal(ko, k.reshape(-1, d))
    np.testing.assert_array_equal(vo, v.reshape(-1, d))


def test_selection_matches_library_topk_and_tie_rule():
    rng = np.random.RandomState(14)
    s = rng.rand(3, 50)
    keep, _ = O.select_topk(s, 3 * 4 + 20, 4)
    top = torch.topk(torch.from_numpy(s.reshape(-1)), 20).indices.numpy()
    got = np.concatenate([keep[g] + g * 50 for g in range(3)])
    np.testing.assert_array_equal(np.sort(top), got)
    # ties: the lower flat index (lower head, then lower position) wins
    s = np.zeros((2, 6))
    s[0, 2] = s[0, 4] = s[1, 1] = s[1, 3] = 0.5
    s[1, 5] = 0.9
    keep, off = O.select_topk(s, 2 * 1 + 3, 1)
    np.testing.assert_array_equal(keep[0], [2, 4])
    np.testing.assert_array_equal(keep[1], [5])
    np.testing.assert_array_equal(off, [0, 3, 5])


def test_selection_nesting():
    rng = np.random.RandomState(15)
    s = np.round(rng.rand(2, 40), 1)                           # many ties
    prev = set()
    for ksel in range(0, 81, 7):
        keep, _ = O.select_topk(s, 2 * 3 + ksel, 3)
        cur = {(g, int(i)) for g in range(2) for i in keep[g]}
        assert prev <= cur and len(cur) == min(ksel, 80)
        prev = cur


def test_head_permutation_permutes_selection():
    hq, hkv, n, w, d = 6, 3, 70, 6, 8
    q, k, v = _rand_layer(16, hq, hkv, n, w, d, vscale=[1.0, 2.0, 0.7])
    perm = [2, 0, 1]
    g = hq // hkv
    qp = np.concatenate([q[p * g:(p + 1) * g] for p in perm])
    s = O.lava_scores(q, k, v, w, O.POOL_AVG, 3)
    sp = O.lava_scores(qp, k[perm], v[perm], w, O.POOL_AVG, 3)
    np.testing.assert_array_equal(sp, s[perm])
    keep, _ = O.select_topk(s, hkv * w + 50, w)
    keep_p, _ = O.select_topk(sp, hkv * w + 50, w)
    for new, old in enumerate(perm):
        np.testing.assert_array_equal(keep_p[new], keep[old])


def test_scaling_one_heads_values_never_shrinks_its_budget():
    hq, hkv, n, w, d = 4, 2, 100, 8, 8
    q, k, v = _rand_layer(17, hq, hkv, n, w, d)
    last = -1
    for c in (0.25, 0.5, 1.0, 2.0, 8.0):
        vv = v.copy()
        vv[1] *= c
        s = O.lava_scores(q, k, vv, w, O.POOL_MAX, 7)
        keep, _ = O.select_topk(s, hkv * w + 60, w)
        assert len(keep[1]) >= last
        last = len(keep[1])
    assert last > 30


def test_planted_key_captures_the_mass():
    hq, hkv, n, w, d = 2, 1, 200, 8, 16
    q, k, v = _rand_layer(18, hq, hkv, n, w, d)
    c = np.ones(d) / math.sqrt(d)
    q += 4.0 * math.sqrt(d) * c
    k[0, 77] = 4.0 * math.sqrt(d) * c
    s = O.lava_scores(q, k, v, w, O.POOL_NONE, 1)
    assert int(np.argmax(s[0])) == 77
    keep, _ = O.select_topk(s, w + 1, w)
    np.testing.assert_array_equal(keep[0], [77])


# ---------------------------------------------------------------- Lemma 1 / Theorem 1, brute force
def test_masked_attention_distance_identity():
    """Proof of Theorem 1: ||A - A_hat||_1 = 2 * (evicted attention mass)."""
    rng = np.random.RandomState(19)
    a = rng.rand(11)
    a /= a.sum()
    for bits in itertools.product([0, 1], repeat=11):
        if sum(bits) == 0:
            continue
        m = np.array(bits, dtype=np.float64)
        lhs = np.abs(a - O.masked_attention(a, m)).sum()
        assert lhs == pytest.approx(2.0 * (a * (1 - m)).sum(), abs=1e-13)


def test_layer_output_loss_closed_form_with_identity_values_and_projection():
    """Lemma 1 with V_h = I (d_h = n) and W_O = I: the concatenated rows are A_h - A_hat_h, so
    the loss is sum_h ||A_h - A_hat_h||_1 = 2 * (evicted attention mass over all heads), by the
    identity in the proof of Theorem 1.  A version that drops a head or a term fails."""
    rng = np.random.RandomState(31)
    n_heads, n = 3, 7
    att = rng.rand(n_heads, n)
    att /= att.sum(axis=1, keepdims=True)
    v = np.stack([np.eye(n)] * n_heads)
    w_o = np.eye(n_heads * n)
    for trial in range(20):
        masks = (rng.rand(n_heads, n) < 0.6).astype(np.float64)
        masks[:, -1] = 1.0                                   # something is always kept
        want = 2.0 * float((att * (1.0 - masks)).sum())
        assert O.layer_output_loss(att, v, w_o, masks) == pytest.approx(want, abs=1e-13)
    # per-head contributions add up: with one head's mask full, that head contributes nothing
    masks = np.ones((n_heads, n))
    masks[1, :3] = 0.0
    assert O.layer_output_loss(att, v, w_o, masks) == pytest.approx(2.0 * att[1, :3].sum(), abs=1e-13)


def test_layer_output_loss_hand_worked_two_heads_with_projection():
    """Lemma 1 by hand: 2 heads, n = 3, d_h = 2, a W_O that mixes and flips signs.

    head 0: A = (.5, .3, .2), mask (1, 0, 1) -> A_hat = (5/7, 0, 2/7), A - A_hat = (-3/14, 3/10, -3/35)
            V = [[1, 0], [0, 2], [1, 1]]     -> (A - A_hat) V = (-3/10, 18/35)
    head 1: A = (.2, .2, .6), mask (0, 1, 1) -> A_hat = (0, 1/4, 3/4), A - A_hat = (1/5, -1/20, -3/20)
            V = [[2, 1], [0, 1], [1, 0]]     -> (A - A_hat) V = (1/4, 3/20)
    Cat = (-3/10, 18/35, 1/4, 3/20);  W_O = [[1, -1], [2, 0], [0, 3], [-1, 1]]
    Cat W_O = (-3/10 + 36/35 - 3/20,  3/10 + 3/4 + 3/20) = (81/140, 6/5);  L1 norm = 249/140.
    """
    att = np.array([[0.5, 0.3, 0.2], [0.2, 0.2, 0.6]])
    masks = np.array([[1.0, 0.0, 1.0], [0.0, 1.0, 1.0]])
    v = np.array([[[1.0, 0.0], [0.0, 2.0], [1.0, 1.0]], [[2.0, 1.0], [0.0, 1.0], [1.0, 0.0]]])
    w_o = np.array([[1.0, -1.0], [2.0, 0.0], [0.0, 3.0], [-1.0, 1.0]])
    assert O.layer_output_loss(att, v, w_o, masks) == pytest.approx(249.0 / 140.0, abs=1e-14)
    # the bound of Theorem 1 for the same case: C_hat = max row sum of |W_O| = 3,
    # Vbar = (2, 3), evicted mass (.3, .2): 2 * 3 * (2 * .3 + 3 * .2) = 7.2
    assert O.wo_norm(w_o) == 3.0
    assert O.loss_upper_bound(att, v, w_o, masks) == pytest.approx(7.2, abs=1e-14)


def test_bound_holds_and_topk_minimises_it_by_enumeration():
    """w = 1, MHA, no pooling: every subset obeys Theorem 1; top-k minimises the bound."""
    hq = hkv = 2
    n, w, d, dm = 9, 1, 4, 8
    q, k, v = _rand_layer(20, hq, hkv, n, w, d, vscale=[1.0, 2.5])
    rng = np.random.RandomState(21)
    w_o = rng.randn(hq * d, dm)
    att = O.window_attention(q, k)[:, 0, :]                    # [H, n] last query
    s = O.lava_scores(q, k, v, w, O.POOL_NONE, 1)               # [H, P]
    prefix = n - w
    k_sel = 5
    best_bound, best_set = None, None
    for subset in itertools.combinations(range(hq * prefix), k_sel):
        masks = np.zeros((hq, n))
        masks[:, prefix:] = 1.0                                 # window always kept
        for f in subset:
            masks[f // prefix, f % prefix] = 1.0
        loss = O.layer_output_loss(att, v, w_o, masks)
        bound = O.loss_upper_bound(att, v, w_o, masks)
        assert loss <= bound * (1 + 1e-12)
        # the bound is 2*C_hat * (sum of evicted scores): Definition 1 with w = 1
        evicted = s.sum() - s.reshape(-1)[list(subset)].sum()
        assert bound == pytest.approx(2.0 * O.wo_norm(w_o) * evicted, rel=1e-11)
        if best_bound is None or bound < best_bound - 1e-15:
            best_bound, best_set = bound, subset
    keep, _ = O.select_topk(s, hq * w + k_sel, w)
    got = tuple(sorted(int(g * prefix + i) for g in range(hq) for i in keep[g]))
    assert got == tuple(best_set)


def test_topk_minimises_window_averaged_bound_by_enumeration():
    """n <= 12, G = 1, w > 1: the selected set maximises retained score mass over all subsets."""
    hq = hkv = 2
    n, w, d = 11, 3, 4
    q, k, v = _rand_layer(22, hq, hkv, n, w, d, vscale=[1.0, 0.4])
    s = O.lava_scores(q, k, v, w, O.POOL_NONE, 1)
    prefix = n - w
    for k_sel in (1, 4, 7):
        best, mass = O.best_subset_by_enumeration(s, k_sel)
        brute = max(itertools.combinations(range(hq * prefix), k_sel),
                    key=lambda c: sum(s.reshape(-1)[i] for i in c))
        assert tuple(best) == tuple(brute)
        keep, _ = O.select_topk(s, hq * w + k_sel, w)
        got = tuple(sorted(int(g * prefix + i) for g in range(hq) for i in keep[g]))
        assert got == tuple(best)
    # wo_norm is the induced norm that makes ||x W||_1 <= ||x||_1 * C_hat tight on a unit row
    rng = np.random.RandomState(23)
    w_o = rng.randn(6, 5)
    c_hat = O.wo_norm(w_o)
    worst = max(np.abs(np.eye(6)[i] @ w_o).sum() for i in range(6))
    assert c_hat == pytest.approx(worst)


# ---------------------------------------------------------------- Algorithm 2 cascade
def test_cascade_equals_one_shot_when_budgets_shrink():
    rng = np.random.RandomState(24)
    n_layers, hq, hkv, n, w, d = 5, 4, 2, 60, 4, 8
    qs, ks, vs = [], [], []
    for l in range(n_layers):
        q, k, v = _rand_layer(100 + l, hq, hkv, n, w, d, vscale=rng.rand(hkv) + 0.5)
        qs.append(q), ks.append(k), vs.append(v)
    total = 40 * hkv * n_layers // 2
    one = O.evict_model(qs, ks, vs, w, total, O.POOL_MAX, 5)
    assert sum(one["budgets"]) == total
    for l in range(n_layers):
        assert one["head_offsets"][l][-1] == one["budgets"][l]
    keep_c, budgets_c, monotone = O.cascade_evict(one["scores"], n, w, total)
    assert budgets_c == one["budgets"]
    assert monotone
    for l in range(n_layers):
        for g in range(hkv):
            np.testing.assert_array_equal(keep_c[l][g], one["keep"][l][g])


def test_model_level_invariants():
    n_layers, hq, hkv, n, w, d = 3, 4, 2, 48, 4, 8
    qs, ks, vs = [], [], []
    for l in range(n_layers):
        q, k, v = _rand_layer(200 + l, hq, hkv, n, w, d)
        qs.append(q), ks.append(k), vs.append(v)
    total = 3 * 31
    out = O.evict_model(qs, ks, vs, w, total, O.POOL_MAX, 7)
    assert sum(out["budgets"]) == total
    for l in range(n_layers):
        heads = np.diff(out["head_offsets"][l])
        assert heads.sum() == out["budgets"][l] and np.all(heads >= w)
        assert out["k_out"][l].shape == (out["budgets"][l], d)
        for g in range(hkv):
            rows = out["k_out"][l][out["head_offsets"][l][g]: out["head_offsets"][l][g + 1]]
            pos = np.concatenate([out["keep"][l][g], np.arange(n - w, n)])
            np.testing.assert_array_equal(rows, ks[l][g][pos])
    uni = O.evict_model(qs, ks, vs, w, total, O.POOL_MAX, 7, mode=O.BUDGET_UNIFORM)
    assert uni["budgets"] == [31, 31, 31]


# ---------------------------------------------------------------- ablation modes (Sec. 5.4; table of methods)
def test_per_head_selection_is_the_layer_rule_on_each_head_alone():
    """"- head dynamic": every head keeps its own share; with one head the two rules coincide,
    and a head's choice never depends on the other heads' scores."""
    rng = np.random.RandomState(41)
    hkv, prefix, w = 3, 40, 4
    s = rng.rand(hkv, prefix)
    one, off1 = O.select_topk_per_head(s[:1], w + 13, w)
    ref, off2 = O.select_topk(s[:1], w + 13, w)
    np.testing.assert_array_equal(one[0], ref[0])
    np.testing.assert_array_equal(off1, off2)
    budget = hkv * w + 20                                    # 20 = 3 * 6 + 2: shares 7, 7, 6
    keep, off = O.select_topk_per_head(s, budget, w)
    assert [len(x) for x in keep] == [7, 7, 6]
    np.testing.assert_array_equal(off, [0, 11, 22, 32])
    for g in range(hkv):
        np.testing.assert_array_equal(np.sort(keep[g]), keep[g])
        want = np.sort(np.argsort(-s[g], kind="stable")[:len(keep[g])])
        np.testing.assert_array_equal(keep[g], want)
    s2 = s.copy()
    s2[1] *= 1000.0                                          # another head's scale changes nothing
    keep2, _ = O.select_topk_per_head(s2, budget, w)
    for g in range(hkv):
        np.testing.assert_array_equal(keep2[g], keep[g])
    # a head with fewer candidates than its share keeps all of them; the rest is not handed on
    keep3, off3 = O.select_topk_per_head(s[:, :5], hkv * w + 20, w)
    assert [len(x) for x in keep3] == [5, 5, 5] and off3[-1] == hkv * (5 + w)
    # layer-wide selection of the same budget differs once one head dominates
    wide, _ = O.select_topk(s2, budget, w)
    assert len(wide[1]) == 20 and len(wide[0]) == 0


def test_pyramid_weights_follow_the_quoted_rule():
    """PyramidKV paragraph: B_{L-1} = B/(beta L), B_0 = 2B/L - B_{L-1}, a straight line between."""
    for n_layers, beta in ((32, 20.0), (5, 2.0), (2, 4.0)):
        wts = O.pyramid_weights(n_layers, beta)
        assert sum(wts) == pytest.approx(1.0, abs=1e-12)
        assert wts[-1] == pytest.approx(1.0 / (beta * n_layers), abs=1e-15)
        assert wts[0] == pytest.approx(2.0 / n_layers - 1.0 / (beta * n_layers), abs=1e-15)
        steps = np.diff(wts)
        assert np.all(steps < 0) and np.allclose(steps, steps[0], atol=1e-15)
    assert O.pyramid_weights(1) == [1.0]
    # hand-worked: L = 4, beta = 2, B = 800 -> B_3 = 100, B_0 = 300, line 300, 233.33, 166.67, 100
    want = O.layer_budgets([0.0] * 4, 800, 0, 10_000, O.BUDGET_PYRAMID, beta=2.0)
    assert want == [300, 233, 167, 100]
    # the entropies play no part, the floor still binds (the last layer is lifted to it)
    assert O.layer_budgets([9.0, 1.0, 5.0, 2.0], 800, 0, 10_000, O.BUDGET_PYRAMID, beta=2.0) == want
    clamped = O.layer_budgets([0.0] * 4, 800, 150, 10_000, O.BUDGET_PYRAMID, beta=2.0)
    assert clamped[-1] == 150 and sum(clamped) == 800 and clamped[0] > clamped[1] > clamped[2] >= 150


def test_value_term_variants():
    """VALUE_NORM_MAX is Definition 1; UNIT is the pooled window mean alone (the SnapKV / AdaKV
    score of the paper's table); TOKEN weights position i by ||V[i]||_1 (VATP)."""
    hq, hkv, n, w, d = 4, 2, 30, 4, 8
    q, k, v = _rand_layer(51, hq, hkv, n, w, d, vscale=[1.0, 3.0])
    base = O.lava_scores(q, k, v, w, O.POOL_MAX, 5)
    np.testing.assert_array_equal(O.variant_scores(q, k, v, w, O.POOL_MAX, 5), base)
    unit = O.variant_scores(q, k, v, w, O.POOL_MAX, 5, value_term=O.VALUE_NORM_UNIT)
    vbar = O.value_norm(v)
    np.testing.assert_allclose(unit * vbar[:, None], base, rtol=1e-13)
    # unit scores are pooled window means: with max-pool 1 each head's row sums to at most 1
    plain = O.variant_scores(q, k, v, w, O.POOL_NONE, 1, value_term=O.VALUE_NORM_UNIT)
    att = O.window_attention(q, k)
    a = O.window_mean_prefix(att, w)
    np.testing.assert_allclose(plain, np.maximum(a[0::2], a[1::2]), rtol=1e-13)
    # per-token weights: with rows of V of equal norm c the score is c times the unit score;
    # scaling ONE row of V scales only that position's score (no pooling), unlike Vbar
    v_eq = np.sign(v) * 0.5
    tok = O.variant_scores(q, k, v_eq, w, O.POOL_NONE, 1, value_term=O.VALUE_NORM_TOKEN)
    np.testing.assert_allclose(tok, 0.5 * d * plain, rtol=1e-13)
    v_one = v_eq.copy()
    v_one[1, 7] *= 10.0
    tok2 = O.variant_scores(q, k, v_one, w, O.POOL_NONE, 1, value_term=O.VALUE_NORM_TOKEN)
    np.testing.assert_allclose(tok2[1, 7], 10.0 * tok[1, 7], rtol=1e-13)
    tok2[1, 7] = tok[1, 7]
    np.testing.assert_array_equal(tok2, tok)
    np.testing.assert_allclose(O.token_value_norms(v_one)[1, 7], 5.0 * d, rtol=1e-13)


# ------------------------------------------------------------------ the consumer: decode attention
def test_decode_attention_special_cases_and_library_softmax():
    rng = np.random.RandomState(11)
    d, hq, hkv = 8, 4, 2
    q = rng.randn(hq, d)
    # one retained row: the output is that row of V, whatever the logit
    k1 = [rng.randn(1, d) for _ in range(hkv)]
    v1 = [rng.randn(1, d) for _ in range(hkv)]
    out = O.decode_attention(q, k1, v1)
    for h in range(hq):
        np.testing.assert_allclose(out[h], v1[h // 2][0], rtol=1e-13)
    # identical keys: uniform weights, the plain mean of the value rows
    kk = [np.tile(rng.randn(1, d), (5, 1)), np.tile(rng.randn(1, d), (3, 1))]
    vv = [rng.randn(5, d), rng.randn(3, d)]
    out = O.decode_attention(q, kk, vv)
    for h in range(hq):
        np.testing.assert_allclose(out[h], vv[h // 2].mean(axis=0), rtol=1e-12)
    # a head with no rows gives zeros; lengths differ per head
    out = O.decode_attention(q, [np.zeros((0, d)), kk[1]], [np.zeros((0, d)), vv[1]])
    assert np.all(out[:2] == 0.0) and np.any(out[2:] != 0.0)
    # against the library softmax, with an explicit scale (a transposed product, a missing scale
    # or the wrong head grouping would show)
    kr = [rng.randn(7, d), rng.randn(4, d)]
    vr = [rng.randn(7, d), rng.randn(4, d)]
    out = O.decode_attention(q, kr, vr, sm_scale=0.37)
    for h in range(hq):
        g = h // 2
        p = torch.softmax(torch.tensor(0.37 * kr[g] @ q[h]), dim=0).numpy()
        np.testing.assert_allclose(out[h], p @ vr[g], rtol=1e-12)
    # row order does not matter
    perm = rng.permutation(7)
    out2 = O.decode_attention(q, [kr[0][perm], kr[1]], [vr[0][perm], vr[1]], sm_scale=0.37)
    np.testing.assert_allclose(out2, out, rtol=1e-12)


def test_decode_attention_over_a_full_cache_is_the_last_attention_row_times_v():
    """Nothing evicted: the new token's output equals the (already pinned) attention row of a
    query at the last position applied to V."""
    rng = np.random.RandomState(12)
    hq, hkv, n, d, w = 4, 2, 19, 8, 3
    q_win = rng.randn(hq, w, d)
    k, v = rng.randn(hkv, n, d), rng.randn(hkv, n, d)
    att = O.window_attention(q_win, k)[:, w - 1, :]                      # sees all n keys
    out = O.decode_attention(q_win[:, w - 1, :], list(k), list(v))
    for h in range(hq):
        np.testing.assert_allclose(out[h], att[h] @ v[h // 2], rtol=1e-12)
