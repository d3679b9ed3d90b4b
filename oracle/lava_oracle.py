"""CPU oracle for LAVa prefill-time KV-cache eviction.

TEST INFRASTRUCTURE ONLY.  This module is a plain, slow, fp64 restatement of what the paper
defines.  It shares no code with the CUDA path and must never be imported by the product
package; only the tests, the smoke check and the benchmark's CPU-baseline leg may call it.

Every function cites the passage it follows.  Nothing here is blocked, fused or reordered:
the steps appear in the order the paper states them, so a reader can check each against the
text by eye.  numpy's matmul, sort and exp serve as library steps.

Readings adopted where the paper is silent or ambiguous (each one is pinned by a test):

* window = the last ``w`` positions; there are exactly ``w`` window queries and
  ``P = n - w`` prefix candidates (Definition 1 writes a ``w+1``-term sum divided by ``w``).
* softmax of window query ``j`` runs over every key ``i <= j`` (Sec. 2, definition of
  ``A^N``): the prefix and the causal part of the window; only prefix columns are scored.
* pooling: stride 1, centred, same length, over the prefix only.  max-pool ignores taps that
  fall outside ``[0, P)``; avg-pool counts them as zero and divides by the kernel size.
* order inside a KV group: pool each query head's window mean, scale by the group's value
  norm, then take the maximum over the group's query heads (Sec. 4.3).
* the value norm of a KV head is the largest row L1 norm over all ``n`` rows (Theorem 1).
* a layer budget counts the always-kept window rows: ``B_l - H_kv*w`` prefix entries are
  selected, so a layer retains exactly ``B_l`` rows (constraints of Eq. 1).
* equal scores: the lower flat index ``g*P + i`` wins.
* integer budgets: largest-remainder apportionment, ties to the lower layer, clamped to
  ``[lo, hi]`` per layer with one-sided re-apportionment rounds (see ``layer_budgets``).

Parity status: the absolute score values on realistic inputs are pinned by closed forms
(uniform attention / harmonic numbers), by a library softmax + library pooling cross-check
and by brute force on tiny inputs, not by numbers printed in the paper (it prints none).
"""
from __future__ import annotations

import itertools
import math

import numpy as np

POOL_NONE, POOL_MAX, POOL_AVG = 0, 1, 2
BUDGET_DYNAMIC, BUDGET_UNIFORM, BUDGET_PYRAMID = 0, 1, 2
VALUE_NORM_MAX, VALUE_NORM_UNIT, VALUE_NORM_TOKEN = 0, 1, 2


# --------------------------------------------------------------------------------------------
# Step 1: attention of the window queries (Sec. 2: A^j = Softmax(Q^j K^T / sqrt(d_h)), i <= j)
# --------------------------------------------------------------------------------------------
def window_attention(q_win, k, sm_scale=None):
    """Attention rows of the last ``w`` queries of every query head.

    q_win : [H_q, w, d]   queries at absolute positions P..n-1 (P = n - w)
    k     : [H_kv, n, d]  keys; query head h reads KV head h // (H_q // H_kv)
    returns A : [H_q, w, n] fp64, row t is the softmax over keys 0..P+t and zero beyond.
    """
    q_win = np.asarray(q_win, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    n_q_heads, w, d = q_win.shape
    n_kv_heads, n, _ = k.shape
    group = n_q_heads // n_kv_heads
    prefix = n - w
    scale = (1.0 / math.sqrt(d)) if sm_scale in (None, 0, 0.0) else float(sm_scale)
    att = np.zeros((n_q_heads, w, n), dtype=np.float64)
    for h in range(n_q_heads):
        g = h // group
        logits = scale * (q_win[h] @ k[g].T)              # [w, n]
        for t in range(w):
            j = prefix + t                                 # absolute position of this query
            z = logits[t, : j + 1]
            z = z - z.max()
            ez = np.exp(z)
            att[h, t, : j + 1] = ez / ez.sum()
    return att


# --------------------------------------------------------------------------------------------
# Step 2: window mean over the prefix (Definition 1, the (1/w) * sum over the window)
# --------------------------------------------------------------------------------------------
def window_mean_prefix(att, w):
    """a_h[i] = (1/w) * sum_t A_{h,t}[i] for prefix positions i < P.  att: [H_q, w, n]."""
    n = att.shape[2]
    prefix = n - w
    return att[:, :, :prefix].sum(axis=1) / float(w)


# --------------------------------------------------------------------------------------------
# Step 3: pooling along the token axis (Sec. 5.1 "Pooling operators": maxpool, kernel 7)
# --------------------------------------------------------------------------------------------
def pool1d(a, kind, kernel):
    """Stride-1 centred pooling of every row of ``a`` ([rows, P]) with an odd kernel."""
    a = np.asarray(a, dtype=np.float64)
    if kind == POOL_NONE or kernel <= 1:
        return a.copy()
    if kernel % 2 == 0:
        raise ValueError("pool kernel must be odd")
    r = kernel // 2
    rows, p = a.shape
    out = np.empty_like(a)
    for i in range(p):
        lo, hi = max(0, i - r), min(p, i + r + 1)
        if kind == POOL_MAX:
            out[:, i] = a[:, lo:hi].max(axis=1)
        elif kind == POOL_AVG:
            out[:, i] = a[:, lo:hi].sum(axis=1) / float(kernel)
        else:
            raise ValueError("unknown pooling kind")
    return out


# --------------------------------------------------------------------------------------------
# Step 4: value norm (Theorem 1: V-bar_{l,h} = max_k ||V_{l,h}[k]||_1)
# --------------------------------------------------------------------------------------------
def value_norm(v):
    """v: [H_kv, n, d] -> [H_kv], the largest row L1 norm of each KV head."""
    v = np.asarray(v, dtype=np.float64)
    return np.abs(v).sum(axis=2).max(axis=1)


# --------------------------------------------------------------------------------------------
# Step 5: LAVa score with GQA group maximum (Definition 1; Sec. 4.3)
# --------------------------------------------------------------------------------------------
def token_value_norms(v):
    """Row L1 norms ||V_g[i]||_1 of every cached position: [H_kv, n] (the VATP weight)."""
    return np.abs(np.asarray(v, dtype=np.float64)).sum(axis=2)


def variant_scores(q_win, k, v, w, pool_kind=POOL_MAX, pool_kernel=7, sm_scale=None,
                   c_hat=1.0, value_term=VALUE_NORM_MAX):
    """The score with the value term of the methods the paper compares against (its table of
    score functions and the related-work paragraph on VATP):

    VALUE_NORM_MAX    LAVa, Definition 1: the head's largest row L1 norm (same as lava_scores)
    VALUE_NORM_UNIT   SnapKV / AdaKV: the pooled window-mean attention alone (value term 1)
    VALUE_NORM_TOKEN  VATP: every position weighted by its own ||V_g[i]||_1
    In all three the pooled window mean of each query head is weighted first and the group
    maximum (Sec. 4.3) is taken last.  Returns [H_kv, P].
    """
    q_win = np.asarray(q_win, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    n_q_heads = q_win.shape[0]
    n_kv_heads, n, _ = k.shape
    group = n_q_heads // n_kv_heads
    prefix = n - w
    att = window_attention(q_win, k, sm_scale)
    pooled = pool1d(window_mean_prefix(att, w), pool_kind, pool_kernel)      # [H_q, P]
    if value_term == VALUE_NORM_MAX:
        weight = np.repeat(value_norm(v)[:, None], prefix, axis=1)
    elif value_term == VALUE_NORM_UNIT:
        weight = np.ones((n_kv_heads, prefix))
    elif value_term == VALUE_NORM_TOKEN:
        weight = token_value_norms(v)[:, :prefix]
    else:
        raise ValueError("unknown value-norm variant")
    scores = np.empty((n_kv_heads, prefix), dtype=np.float64)
    for g in range(n_kv_heads):
        scaled = float(c_hat) * weight[g][None, :] * pooled[g * group:(g + 1) * group]
        scores[g] = scaled.max(axis=0)
    return scores


def lava_scores(q_win, k, v, w, pool_kind=POOL_MAX, pool_kernel=7, sm_scale=None,
                c_hat=1.0, vbar=None):
    """s_g[i] = c_hat * Vbar_g * max_{h in group g} pool(a_h)[i], i < P.  Returns [H_kv, P]."""
    q_win = np.asarray(q_win, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    n_q_heads = q_win.shape[0]
    n_kv_heads, n, _ = k.shape
    group = n_q_heads // n_kv_heads
    prefix = n - w
    att = window_attention(q_win, k, sm_scale)
    a = window_mean_prefix(att, w)                          # [H_q, P]
    pooled = pool1d(a, pool_kind, pool_kernel)              # [H_q, P]
    if vbar is None:
        vbar = value_norm(v)
    vbar = np.asarray(vbar, dtype=np.float64)
    scores = np.empty((n_kv_heads, prefix), dtype=np.float64)
    for g in range(n_kv_heads):
        scaled = float(c_hat) * vbar[g] * pooled[g * group:(g + 1) * group]   # [G, P]
        scores[g] = scaled.max(axis=0)
    return scores


# --------------------------------------------------------------------------------------------
# Step 6: layer uncertainty (Sec. 4.2: normalised scores and normalised entropy)
# --------------------------------------------------------------------------------------------
def layer_entropy(scores, n):
    """e_l = -sum(s_hat * ln s_hat) / (H_kv * n), s_hat = s / sum(s), 0*ln 0 = 0."""
    s = np.asarray(scores, dtype=np.float64)
    n_kv_heads = s.shape[0]
    total = s.sum()
    if not (total > 0.0):
        return 0.0
    s_hat = s.reshape(-1) / total
    nz = s_hat[s_hat > 0.0]
    ent = -(nz * np.log(nz)).sum()
    return float(ent / (n_kv_heads * n))


# --------------------------------------------------------------------------------------------
# Step 7: layer budgets (Algorithm 2: B_l = e_l / sum_l e_l * B) made integral
# --------------------------------------------------------------------------------------------
def _largest_remainder(shares, total):
    """Integers that sum to ``total``: floors, then +1 to the largest fractions (ties: lower)."""
    base = [int(math.floor(x)) for x in shares]
    rest = total - sum(base)
    frac = [shares[i] - base[i] for i in range(len(shares))]
    order = sorted(range(len(shares)), key=lambda i: (-frac[i], i))
    # rest is in [0, len) for exact shares; rounding noise can push it slightly outside
    idx = 0
    while rest > 0:
        base[order[idx % len(order)]] += 1
        rest -= 1
        idx += 1
    idx = len(order) - 1
    while rest < 0:
        base[order[idx % len(order)]] -= 1
        rest += 1
        idx -= 1
    return base


def pyramid_weights(n_layers, beta=20.0):
    """Relative layer budgets of the PyramidKV rule the paper quotes (its paragraph on
    PyramidKV): B_{L-1} = B / (beta L), B_0 = 2 B / L - B_{L-1}, and a straight line between
    them, descending with depth (the printed interpolation has its sign garbled; the line from
    B_0 at layer 0 to B_{L-1} at the last layer is what "like a pyramid" describes).  Returned
    for B = 1; the weights are positive and sum to 1."""
    n_layers = int(n_layers)
    if n_layers == 1:
        return [1.0]
    last = 1.0 / (float(beta) * n_layers)
    first = 2.0 / n_layers - last
    return [first + (last - first) * l / (n_layers - 1) for l in range(n_layers)]


def layer_budgets(entropy, total_budget, lo, hi, mode=BUDGET_DYNAMIC, beta=20.0):
    """Integer layer budgets with sum == total_budget and lo <= B_l <= hi.

    entropy      : [L] layer uncertainties e_l
    total_budget : the model-wide budget (KV-head entries, window rows included)
    lo, hi       : per-layer floor (H_kv*w: the window is always kept) and cap (H_kv*n)
    mode         : BUDGET_DYNAMIC -> shares e_l / sum e ; BUDGET_UNIFORM -> equal shares ;
                   BUDGET_PYRAMID -> shares pyramid_weights(L, beta) (the entropies are ignored)

    Rule.  Layers start "active".  Each round the remaining budget R (total minus what clamped
    layers hold) is shared among active layers in proportion to e_l (equally if their e sum to
    zero or mode is uniform) and made integral by largest remainder.  If any active layer is
    below lo or above hi, the total shortfall D = sum(lo - B_l) and total excess
    X = sum(B_l - hi) are compared; the side with the larger total (shortfall on a tie) is
    clamped and leaves the active set, and the round repeats.  One-sided clamping keeps the
    remaining problem feasible whenever L*lo <= total <= L*hi.
    """
    e = [float(x) for x in entropy]
    n_layers = len(e)
    if mode == BUDGET_PYRAMID:
        e = pyramid_weights(n_layers, beta)
    total_budget, lo, hi = int(total_budget), int(lo), int(hi)
    if not (n_layers * lo <= total_budget <= n_layers * hi):
        raise ValueError("infeasible budget: need L*lo <= total <= L*hi")
    budget = [0] * n_layers
    active = list(range(n_layers))
    remaining = total_budget
    while active:
        esum = 0.0
        for l in active:
            esum += e[l]
        if mode == BUDGET_UNIFORM or not (esum > 0.0) or not math.isfinite(esum):
            shares = [remaining / len(active) for _ in active]
        else:
            shares = [remaining * e[l] / esum for l in active]
        ints = _largest_remainder(shares, remaining)
        short = sum(lo - b for b in ints if b < lo)
        excess = sum(b - hi for b in ints if b > hi)
        if short == 0 and excess == 0:
            for l, b in zip(active, ints):
                budget[l] = b
            break
        still = []
        if short >= excess:
            for l, b in zip(active, ints):
                if b < lo:
                    budget[l] = lo
                    remaining -= lo
                else:
                    still.append(l)
        else:
            for l, b in zip(active, ints):
                if b > hi:
                    budget[l] = hi
                    remaining -= hi
                else:
                    still.append(l)
        active = still
    return budget


# --------------------------------------------------------------------------------------------
# Step 8: layer-wide selection (Algorithm 1, Evict: the B_l largest entries of the flat s_l)
# --------------------------------------------------------------------------------------------
def select_topk(scores, layer_budget, w):
    """Keep the ``layer_budget - H_kv*w`` best prefix entries of the flat score array.

    scores : [H_kv, P].  Order: score descending, flat index g*P + i ascending.
    returns (keep, head_offsets): keep[g] = ascending kept prefix positions of head g;
    head_offsets[g] = exclusive scan of (len(keep[g]) + w), length H_kv + 1.
    """
    s = np.asarray(scores, dtype=np.float64)
    n_kv_heads, prefix = s.shape
    k_sel = int(layer_budget) - n_kv_heads * int(w)
    k_sel = max(0, min(k_sel, n_kv_heads * prefix))
    flat = s.reshape(-1)
    # stable sort on the negated score: equal scores stay in ascending flat-index order
    order = np.argsort(-flat, kind="stable")
    chosen = np.sort(order[:k_sel])
    keep = []
    for g in range(n_kv_heads):
        sel = chosen[(chosen >= g * prefix) & (chosen < (g + 1) * prefix)] - g * prefix
        keep.append(sel.astype(np.int64))
    head_offsets = np.zeros(n_kv_heads + 1, dtype=np.int64)
    for g in range(n_kv_heads):
        head_offsets[g + 1] = head_offsets[g] + len(keep[g]) + int(w)
    return keep, head_offsets


# --------------------------------------------------------------------------------------------
# Step 9: compaction (Algorithm 1: K-hat = K (.) I, V-hat = V (.) I, physically a gather)
# --------------------------------------------------------------------------------------------
def select_topk_per_head(scores, layer_budget, w):
    """The paper's "- head dynamic" ablation (Sec. 5.4): the layer budget is split evenly over
    the heads and every head keeps its own best entries, with no comparison across heads.

    The ``layer_budget - H_kv*w`` selectable entries are shared as evenly as integers allow (the
    first ``remainder`` heads get one more); a head with fewer candidates than its share keeps
    all of them (the surplus is not handed on: budgets are fixed).  Same return as select_topk.
    """
    s = np.asarray(scores, dtype=np.float64)
    n_kv_heads, prefix = s.shape
    k_sel = max(0, int(layer_budget) - n_kv_heads * int(w))
    base, extra = divmod(k_sel, n_kv_heads)
    keep = []
    for g in range(n_kv_heads):
        k_g = min(prefix, base + (1 if g < extra else 0))
        one, _ = select_topk(s[g:g + 1], k_g + int(w), w)        # the layer-wide rule on one head
        keep.append(one[0])
    head_offsets = np.zeros(n_kv_heads + 1, dtype=np.int64)
    for g in range(n_kv_heads):
        head_offsets[g + 1] = head_offsets[g] + len(keep[g]) + int(w)
    return keep, head_offsets


def compact_kv(k, v, keep, w):
    """Rows of every head in temporal order: kept prefix rows, then the w window rows.

    k, v : [H_kv, n, d] arrays of any dtype (copied bit for bit).
    returns (k_out, v_out), each [sum_g (len(keep[g]) + w), d], heads in order.
    """
    n_kv_heads, n, _ = k.shape
    prefix = n - int(w)
    rows_k, rows_v = [], []
    for g in range(n_kv_heads):
        pos = np.concatenate([np.asarray(keep[g], dtype=np.int64),
                              np.arange(prefix, n, dtype=np.int64)])
        rows_k.append(k[g][pos])
        rows_v.append(v[g][pos])
    return np.concatenate(rows_k, axis=0), np.concatenate(rows_v, axis=0)


# --------------------------------------------------------------------------------------------
# Whole model, one shot: scores -> entropies -> budgets -> selection -> compaction
# --------------------------------------------------------------------------------------------
def evict_model(q_win, k, v, w, total_budget, pool_kind=POOL_MAX, pool_kernel=7,
                sm_scale=None, mode=BUDGET_DYNAMIC, c_hat=1.0):
    """q_win/k/v are lists over layers ([H_q,w,d], [H_kv,n,d], [H_kv,n,d]).  Returns a dict."""
    n_layers = len(k)
    n_kv_heads, n, _ = k[0].shape
    scores = [lava_scores(q_win[l], k[l], v[l], w, pool_kind, pool_kernel, sm_scale, c_hat)
              for l in range(n_layers)]
    ent = [layer_entropy(scores[l], n) for l in range(n_layers)]
    budgets = layer_budgets(ent, total_budget, n_kv_heads * w, n_kv_heads * n, mode)
    keep, offsets, k_out, v_out = [], [], [], []
    for l in range(n_layers):
        kp, ho = select_topk(scores[l], budgets[l], w)
        ko, vo = compact_kv(k[l], v[l], kp, w)
        keep.append(kp)
        offsets.append(ho)
        k_out.append(ko)
        v_out.append(vo)
    return {"scores": scores, "entropy": ent, "budgets": budgets, "keep": keep,
            "head_offsets": offsets, "k_out": k_out, "v_out": v_out}


# --------------------------------------------------------------------------------------------
# Algorithm 2, streaming form: after each new layer, re-budget layers 0..l and re-evict them
# --------------------------------------------------------------------------------------------
def cascade_evict(scores, n, w, total_budget, mode=BUDGET_DYNAMIC, entropy=None):
    """Follow Algorithm 2 on stored scores.  scores: list of [H_kv, P] arrays.  ``entropy``
    (optional, [L]) supplies the e_l instead of layer_entropy(s_l): Algorithm 2 takes them as
    given once computed, and a caller that compares integer budgets fixes them this way.

    After layer l arrives the budgets of layers 0..l are recomputed from e_0..e_l (the sum in
    the denominator runs over the layers prefilled so far) and every one of them is evicted
    again with its own stored scores.  A repeated eviction can only drop entries: it keeps the
    best ``B - H_kv*w`` of what the layer still holds.  Returns (keep per layer, budgets,
    monotone) where ``monotone`` tells whether every layer's budget sequence was non-increasing.
    """
    n_kv_heads, prefix = scores[0].shape
    lo, hi = n_kv_heads * w, n_kv_heads * n
    held = []            # per layer: sorted flat indices currently retained
    ent = []
    last_budget = []
    monotone = True
    budgets = []
    for l, s in enumerate(scores):
        ent.append(layer_entropy(s, n) if entropy is None else float(entropy[l]))
        held.append(np.arange(n_kv_heads * prefix, dtype=np.int64))
        last_budget.append(hi)
        live = l + 1
        total_now = min(int(total_budget), live * hi)
        total_now = max(total_now, live * lo)
        budgets = layer_budgets(ent, total_now, lo, hi, mode)
        for lt in range(live):
            if budgets[lt] > last_budget[lt]:
                monotone = False
            last_budget[lt] = budgets[lt]
            k_sel = max(0, min(budgets[lt] - lo, len(held[lt])))
            flat = np.asarray(scores[lt], dtype=np.float64).reshape(-1)[held[lt]]
            order = np.argsort(-flat, kind="stable")       # held[] is ascending, so ties keep
            held[lt] = np.sort(held[lt][order[:k_sel]])    # the lower flat index first
    keep = []
    for lt in range(len(scores)):
        per_head = []
        for g in range(n_kv_heads):
            sel = held[lt][(held[lt] >= g * prefix) & (held[lt] < (g + 1) * prefix)] - g * prefix
            per_head.append(sel)
        keep.append(per_head)
    return keep, budgets, monotone


# --------------------------------------------------------------------------------------------
# The consumer of the compressed cache: one decoding step's attention (Sec. 2 attention over
# the retained entries K-hat, V-hat of Algorithm 1; each KV head keeps its own number of rows)
# --------------------------------------------------------------------------------------------
def decode_attention(q, k_rows, v_rows, sm_scale=None):
    """out[h] = softmax_i(sm_scale * q[h] . K-hat_g[i]) V-hat_g, g = h // (H_q // H_kv).

    q      : [H_q, d] the new token's query heads
    k_rows : list over KV heads of [len_g, d] retained key rows (any order: a softmax-weighted
             sum does not depend on it); v_rows likewise
    returns [H_q, d] fp64; a head with no rows gives zeros.
    """
    q = np.asarray(q, dtype=np.float64)
    n_q_heads, d = q.shape
    group = n_q_heads // len(k_rows)
    scale = (1.0 / math.sqrt(d)) if sm_scale in (None, 0, 0.0) else float(sm_scale)
    out = np.zeros((n_q_heads, d), dtype=np.float64)
    for h in range(n_q_heads):
        kk = np.asarray(k_rows[h // group], dtype=np.float64)
        vv = np.asarray(v_rows[h // group], dtype=np.float64)
        if kk.shape[0] == 0:
            continue
        z = scale * (kk @ q[h])
        z = z - z.max()
        e = np.exp(z)
        out[h] = (e / e.sum()) @ vv
    return out


# --------------------------------------------------------------------------------------------
# Lemma 1 and Theorem 1 evaluators (used only to pin the scoring rule on tiny inputs)
# --------------------------------------------------------------------------------------------
def masked_attention(att_row, mask):
    """Lemma 1: attention after eviction = (A (.) I) / ||A (.) I||_1."""
    kept = np.asarray(att_row, dtype=np.float64) * np.asarray(mask, dtype=np.float64)
    return kept / kept.sum()


def wo_norm(w_o):
    """C-hat = ||W_O^T||_1, the largest absolute row sum of W_O (Theorem 1 and its proof)."""
    return float(np.abs(np.asarray(w_o, dtype=np.float64)).sum(axis=1).max())


def layer_output_loss(att_last, v, w_o, masks):
    """Lemma 1 with p = 1 for the last query: || Cat_h[(A_h - A-hat_h) V_h] W_O ||_1.

    att_last : [H, n] attention of the last query per head (MHA: one V head per query head)
    v        : [H, n, d_h];  w_o : [H*d_h, d_model];  masks : [H, n] in {0, 1}
    """
    n_heads = att_last.shape[0]
    parts = []
    for h in range(n_heads):
        diff = np.asarray(att_last[h], dtype=np.float64) - masked_attention(att_last[h], masks[h])
        parts.append(diff @ np.asarray(v[h], dtype=np.float64))
    cat = np.concatenate(parts)
    return float(np.abs(cat @ np.asarray(w_o, dtype=np.float64)).sum())


def loss_upper_bound(att_last, v, w_o, masks):
    """Theorem 1: 2 * C-hat * sum_h sum_i A_h[i] * Vbar_h * (1 - I_h[i])."""
    vbar = value_norm(v)
    total = 0.0
    for h in range(att_last.shape[0]):
        total += vbar[h] * float((np.asarray(att_last[h]) * (1.0 - np.asarray(masks[h]))).sum())
    return 2.0 * wo_norm(w_o) * total


def best_subset_by_enumeration(scores, k_sel):
    """Exhaustive minimiser of sum of evicted scores over all subsets of size k_sel (tiny only).

    Returns the set (as a sorted tuple of flat indices) whose retained score mass is largest;
    among equal masses the lexicographically smallest tuple.
    """
    flat = np.asarray(scores, dtype=np.float64).reshape(-1)
    best, best_mass = None, -1.0
    for subset in itertools.combinations(range(flat.size), k_sel):
        mass = float(flat[list(subset)].sum())
        if mass > best_mass:
            best, best_mass = subset, mass
    return best, best_mass
