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
