"""Dense brute force for tiny inputs: a second, differently written statement of the same
definitions, used only to cross-check the C oracle.  Test infrastructure only.

* ``plan_tokens`` / ``plan_pages``: Algorithm 1's budgeted selection written with Python sets
  (the C oracle uses a flag array and an insertion sort; this uses ``sorted`` with a key).
* ``dense_attention``: gathers the whole context of a sequence into dense [L, d] matrices through
  the block table, builds an explicit 0/1 visibility vector per query row, sets the logits of
  invisible tokens to -inf and applies a plain softmax (Section 3.2: the proposal path sees the
  plan's pages, the verifier sees everything up to the row's own position).
"""
from __future__ import annotations

import numpy as np


def _bf16_to_f64(bits):
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def plan_tokens(L, spans, budget, n_sink, n_recent):
    """spans: list of (start, length, score).  Returns (set of selected tokens, over_budget)."""
    chosen = set(range(0, min(n_sink, L))) | set(range(max(0, L - n_recent), L)) | {L - 1}
    if len(chosen) > budget:
        return chosen, True
    clipped = []
    for idx, (start, length, score) in enumerate(spans):
        lo, hi = max(0, int(start)), min(L, int(start) + int(length))
        if hi > lo:
            clipped.append((-float(np.float32(score)), lo, idx, hi))
    for _, lo, _, hi in sorted(clipped):
        fresh = set(range(lo, hi)) - chosen
        if len(chosen) + len(fresh) <= budget:
            chosen |= fresh
    return chosen, False


def plan_pages(L, spans, budget, n_sink, n_recent, page_size=16, force_full=False):
    """Returns (ascending logical page list, number of selected tokens, over_budget)."""
    if force_full:
        return list(range((L + page_size - 1) // page_size)), L, False
    tokens, over = plan_tokens(L, spans, budget, n_sink, n_recent)
    return sorted({t // page_size for t in tokens}), len(tokens), over


def dense_attention(q_bits, pool_bits, bt_pages, L, visible_pages, n_q, scale=None,
                    visible_tokens=None):
    """One sequence.  q_bits [n_q, Hq, d]; pool_bits [pages, 2, Hkv, P, d]; bt_pages: the
    sequence's block table (logical -> physical); visible_pages: iterable of logical pages the
    rows may see (all pages for verification); visible_tokens, when given, replaces it by an
    explicit set of token positions.  Row j sits at position L - n_q + j.
    Returns (out [n_q, Hq, d], lse [n_q, Hq], weights [n_q, Hq, L])."""
    q = _bf16_to_f64(q_bits)
    pool = _bf16_to_f64(pool_bits)
    _, _, Hkv, P, d = pool.shape
    Hq = q.shape[1]
    G = Hq // Hkv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    n_pages = (L + P - 1) // P
    phys = np.asarray(bt_pages[:n_pages], dtype=np.int64)
    # dense [L, Hkv, d]
    K = pool[phys, 0].transpose(0, 2, 1, 3).reshape(n_pages * P, Hkv, d)[:L]
    V = pool[phys, 1].transpose(0, 2, 1, 3).reshape(n_pages * P, Hkv, d)[:L]
    page_vis = np.zeros(n_pages, dtype=bool)
    page_vis[list(visible_pages)] = True
    tok_vis = np.repeat(page_vis, P)[:L]
    if visible_tokens is not None:
        tok_vis = np.zeros(L, dtype=bool)
        tok_vis[sorted(visible_tokens)] = True
    out = np.zeros((n_q, Hq, d))
    lse = np.zeros((n_q, Hq))
    weights = np.zeros((n_q, Hq, L))
    for j in range(n_q):
        pos = L - n_q + j
        vis = tok_vis & (np.arange(L) <= pos)
        for h in range(Hq):
            z = scale * (K[:, h // G, :] @ q[j, h])
            z = np.where(vis, z, -np.inf)
            m = z.max()
            e = np.exp(z - m)
            weights[j, h] = e / e.sum()
            out[j, h] = weights[j, h] @ V[:, h // G, :]
            lse[j, h] = m + np.log(e.sum())
    return out, lse, weights


def append_kv(pool_bits, bt_pages, L, k_new_bits, v_new_bits, page_size=16):
    """Slot mapping written out (Section 3.1, "Selected-KV view materialization": newly scheduled
    tokens go to their physical KV slots): token j of the n_new new tokens is stored at logical
    position L + j, i.e. page bt_pages[(L + j) // P], slot (L + j) % P, for K and V and every KV
    head.  pool_bits [pages, 2, Hkv, P, d] uint16 is modified in place; returns the new length."""
    n_new = k_new_bits.shape[0]
    for j in range(n_new):
        pos = L + j
        page = int(bt_pages[pos // page_size])
        pool_bits[page, 0, :, pos % page_size, :] = k_new_bits[j]
        pool_bits[page, 1, :, pos % page_size, :] = v_new_bits[j]
    return L + n_new


def top3_accept(logits, row_indptr, proposed):
    """Tolerant acceptance (Section 3.2, Eq. 2 with the Top-3 rule): per row the three best
    candidates (value descending, lower index first on ties, NaN below every number, -inf included); m = number of
    proposed tokens accepted consecutively from the start of each sequence's window; next carry =
    the best candidate of row m.  A window without any row (row_indptr[b+1] == row_indptr[b]) has
    nothing to accept and no row to take a carry from: accepted = 0, next = -1.
    logits float32 [rows, V].  Returns (top3, accepted, next)."""
    x = np.asarray(logits, dtype=np.float32)
    rows, V = x.shape
    nan = np.isnan(x)
    val = np.where(nan, 0.0, x).astype(np.float64)
    top3 = np.zeros((rows, 3), dtype=np.int32)
    for r in range(rows):
        # rank: numbers before NaN, then value descending, then index ascending
        order = np.lexsort((np.arange(V), -val[r], nan[r]))
        top3[r] = order[:3]
    B = len(row_indptr) - 1
    accepted = np.zeros(B, dtype=np.int32)
    nxt = np.zeros(B, dtype=np.int32)
    for b in range(B):
        r0, n = int(row_indptr[b]), int(row_indptr[b + 1] - row_indptr[b])
        if n <= 0:
            accepted[b], nxt[b] = 0, -1
            continue
        m = 0
        while m < n - 1 and int(proposed[r0 + m]) in top3[r0 + m].tolist():
            m += 1
        accepted[b] = m
        nxt[b] = top3[r0 + m, 0]
    return top3, accepted, nxt


def phase_model(k, h, s, w_main, w_prop, kv):
    """Section 4.1-4.2 written out: Eq. 3 Cost_full, Eq. 6 Cost_base, Eq. 7 Cost_plan, their ratio,
    Eq. 13 phase slack, the break-even KV scale of Eq. 12 (general form), the Eq. 8 verdict and
    the Eq. 11 margin.  Plain Python floats (fp64)."""
    cost_full = w_main + kv
    cost_base = (1 + k * h) * (w_main + kv)
    cost_plan = k * (w_prop + s * kv) + (w_main + kv)
    slack = h * (w_main + kv) - (w_prop + s * kv)
    rhs = w_prop - h * w_main
    if h > s:
        kv_crit = rhs / (h - s) if rhs > 0 else 0.0
    else:
        kv_crit = 0.0 if rhs < 0 else float("inf")
    return dict(cost_full=cost_full, cost_base=cost_base, cost_plan=cost_plan,
                speedup=cost_base / cost_plan if cost_plan > 0 else float("inf"), slack=slack,
                kv_crit=kv_crit, beneficial=1.0 if cost_plan < cost_base else 0.0, h_minus_s=h - s)


def materialize_view(pool_bits, plan_phys_pages):
    """The selected-KV view as a copy (Section 3.1, "Selected-KV view materialization"): compact
    page i holds the plan's i-th page; returns (compact pool, compact page ids)."""
    phys = np.asarray(plan_phys_pages, dtype=np.int64)
    return pool_bits[phys].copy(), np.arange(len(phys), dtype=np.int32)


# reasons for falling back to full-context access (Section 3.2, "Runtime stability and fallback")
FB_CAPACITY, FB_METADATA, FB_CONFIDENCE, FB_S_HIGH, FB_H_LOW, FB_NO_MARGIN, FB_SLACK = 1, 2, 4, 8, 16, 32, 64
RT_OVER_CAPACITY, RT_UNSTABLE_METADATA = 1, 2     # runtime_flags given by the caller
_PLAN_S_HIGH = 4                                  # the compiler's "retained ratio above s_max" flag


def fallback_decide(accepted_sum, proposed_sum, min_proposed, h_prior, s, kv, w_main, w_prop,
                    h_min, s_max, plan_flags=None, runtime_flags=None, confidence=None,
                    confidence_min=0.0):
    """The fallback rule of Section 3.2 ("Runtime stability and fallback") with the quantities of
    Section 4, one sequence at a time.  A sequence takes full-context access when
      * its plan exceeds the compact workspace, or breaks the metadata-stability assumptions
        (both reported by the caller in runtime_flags),
      * its prior confidence is below confidence_min,
      * it retains too much KV: s > s_max, or the compiler already flagged that,
      * its observed acceptance is low: h < h_min, where h = accepted / proposed (Eq. 5) once at
        least min_proposed proposals were verified and h_prior before that,
      * h <= s: no KV-side margin (Eq. 11), whatever the context length,
      * the phase slack of Eq. 13, h (W_main + KV) - (W_prop + s KV), is not positive.
    Besides the decision the function returns the slack and the factor by which s could be
    multiplied before the slack reaches zero (room to widen the budget when > 1, the cut needed when
    < 1): scale = (h (W_main + KV) - W_prop) / (s KV).
    Returns a list of dicts: force_full, reasons, h, slack, budget_scale."""
    res = []
    for b in range(len(s)):
        n_prop, n_acc = int(proposed_sum[b]), int(accepted_sum[b])
        h = n_acc / n_prop if n_prop >= max(int(min_proposed), 1) else float(h_prior)
        kv_b, s_b = float(kv[b]), float(s[b])
        slack = h * (w_main + kv_b) - (w_prop + s_b * kv_b)
        room = h * (w_main + kv_b) - w_prop
        if s_b * kv_b > 0:
            scale = max(room, 0.0) / (s_b * kv_b)
        else:
            scale = float("inf") if room > 0 else 0.0
        why = 0
        rt = 0 if runtime_flags is None else int(runtime_flags[b])
        if rt & RT_OVER_CAPACITY:
            why |= FB_CAPACITY
        if rt & RT_UNSTABLE_METADATA:
            why |= FB_METADATA
        if confidence is not None and float(confidence[b]) < confidence_min:
            why |= FB_CONFIDENCE
        if s_b > s_max or (plan_flags is not None and int(plan_flags[b]) & _PLAN_S_HIGH):
            why |= FB_S_HIGH
        if h < h_min:
            why |= FB_H_LOW
        if h <= s_b:
            why |= FB_NO_MARGIN
        if not slack > 0:
            why |= FB_SLACK
        res.append(dict(force_full=1 if why else 0, reasons=why, h=h, slack=slack, budget_scale=scale))
    return res
