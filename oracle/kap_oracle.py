"""ctypes binding of the C oracle (oracle/kap_oracle.c).  Test infrastructure only.

Every function takes and returns numpy arrays; bf16 tensors travel as uint16 bit patterns and are
widened exactly to double inside the C code.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build

OK, INVALID, CAPACITY = 0, 1, 2
PLAN_FULL, PLAN_OVER_BUDGET, PLAN_S_HIGH = 1, 2, 4

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
    return _lib


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(C.POINTER(ct))


def _arr(a, dt):
    return None if a is None else np.ascontiguousarray(a, dtype=dt)


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle status {code}")
        self.code = code


def compile_plan(ctx_len, span_indptr, span_start, span_len, span_score, budget_tokens, n_sink,
                 n_recent, force_full=None, s_max=1.0, bt_indptr=None, bt_pages=None,
                 page_size=16, capacity=None):
    """Algorithm 1 (budgeted span selection -> page list).  Returns a dict with plan_indptr,
    plan_logical_pages, plan_phys_pages (None without a block table), plan_flags,
    selected_tokens, plan_token_masks (uint16 per listed page: bit t set when token
    page*page_size + t is in the selected union U; page_size <= 16 only, else None)."""
    ctx_len = _arr(ctx_len, np.int32)
    B = ctx_len.shape[0]
    span_indptr = _arr(span_indptr, np.int32)
    span_start = _arr(span_start, np.int32)
    span_len = _arr(span_len, np.int32)
    span_score = _arr(span_score, np.float32)
    budget_tokens = _arr(budget_tokens, np.int32)
    n_sink = _arr(n_sink, np.int32)
    n_recent = _arr(n_recent, np.int32)
    force_full = _arr(force_full, np.uint8)
    bt_indptr = _arr(bt_indptr, np.int32)
    bt_pages = _arr(bt_pages, np.int32)
    if capacity is None:
        capacity = int(sum((int(L) + page_size - 1) // page_size for L in ctx_len if L > 0))
    indptr = np.full(B + 1, -1, dtype=np.int32)
    logical = np.full(max(1, capacity), -1, dtype=np.int32)
    phys = np.full(max(1, capacity), -1, dtype=np.int32) if bt_indptr is not None else None
    flags = np.full(B, -1, dtype=np.int32)
    sel = np.full(B, -1, dtype=np.int32)
    masks = np.zeros(max(1, capacity), dtype=np.uint16) if page_size <= 16 else None
    rc = lib().kap_oracle_compile_plan(
        C.c_int32(B), C.c_int32(page_size), _p(ctx_len, C.c_int32), _p(span_indptr, C.c_int32),
        _p(span_start, C.c_int32), _p(span_len, C.c_int32), _p(span_score, C.c_float),
        _p(budget_tokens, C.c_int32), _p(n_sink, C.c_int32), _p(n_recent, C.c_int32),
        _p(force_full, C.c_uint8), C.c_float(s_max), _p(bt_indptr, C.c_int32),
        _p(bt_pages, C.c_int32), C.c_int64(capacity), _p(indptr, C.c_int32),
        _p(logical, C.c_int32), _p(phys, C.c_int32), _p(flags, C.c_int32), _p(sel, C.c_int32),
        _p(masks, C.c_uint16))
    if rc != OK:
        raise OracleError(rc)
    n = int(indptr[-1])
    return dict(plan_indptr=indptr, plan_logical_pages=logical[:n].copy(),
                plan_phys_pages=None if phys is None else phys[:n].copy(), plan_flags=flags,
                selected_tokens=sel,
                plan_token_masks=None if masks is None else masks[:n].copy())


def compile_workload(w, capacity=None):
    return compile_plan(w.ctx_len, w.span_indptr, w.span_start, w.span_len, w.span_score,
                        w.budget_tokens, w.n_sink, w.n_recent, w.force_full, w.s_max,
                        w.bt_indptr, w.bt_pages, w.page_size, capacity)


def _attn_out(rows, Hq, d):
    return (np.zeros((rows, Hq, d), dtype=np.float64), np.zeros((rows, Hq), dtype=np.float64),
            np.zeros((rows, Hq), dtype=np.float64), np.zeros((rows, Hq), dtype=np.int64))


def selected_decode_attn(q_bits, pool_bits, plan_indptr, plan_phys_pages, plan_logical_pages,
                         ctx_len, scale=None, plan_token_masks=None):
    """q_bits [B, Hq, d] uint16, pool_bits [pages, 2, Hkv, P, d] uint16.  plan_token_masks
    (uint16 per listed page) narrows visibility from whole pages to the tokens whose bit is set.
    Returns (out f64 [B,Hq,d], lse f64 [B,Hq], weight_sum [B,Hq], n_visible [B,Hq])."""
    q_bits = _arr(q_bits, np.uint16)
    pool_bits = _arr(pool_bits, np.uint16)
    B, Hq, d = q_bits.shape
    n_pages, two, Hkv, P, d2 = pool_bits.shape
    assert two == 2 and d2 == d
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    out, lse, ws, nv = _attn_out(B, Hq, d)
    pi, pp = _arr(plan_indptr, np.int32), _arr(plan_phys_pages, np.int32)
    pl, cl = _arr(plan_logical_pages, np.int32), _arr(ctx_len, np.int32)
    pm = _arr(plan_token_masks, np.uint16)
    rc = lib().kap_oracle_selected_decode_attn(
        _p(q_bits, C.c_uint16), _p(pool_bits, C.c_uint16), C.c_int64(n_pages),
        _p(pi, C.c_int32), _p(pp, C.c_int32), _p(pl, C.c_int32), _p(pm, C.c_uint16),
        _p(cl, C.c_int32),
        C.c_int32(B), C.c_int32(Hq), C.c_int32(Hkv), C.c_int32(d), C.c_int32(P),
        C.c_double(scale), _p(out, C.c_double), _p(lse, C.c_double), _p(ws, C.c_double),
        _p(nv, C.c_int64))
    if rc != OK:
        raise OracleError(rc)
    return out, lse, ws, nv


def verify_attn(q_bits, q_indptr, pool_bits, bt_indptr, bt_pages, ctx_len, scale=None):
    """q_bits [sum n_q, Hq, d] uint16; rows of sequence b are q_indptr[b]..q_indptr[b+1]-1 and
    row j sits at logical position ctx_len[b] - n_q + j.  Returns as selected_decode_attn."""
    q_bits = _arr(q_bits, np.uint16)
    pool_bits = _arr(pool_bits, np.uint16)
    rows, Hq, d = q_bits.shape
    n_pages, two, Hkv, P, d2 = pool_bits.shape
    assert two == 2 and d2 == d
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    out, lse, ws, nv = _attn_out(rows, Hq, d)
    qi, bi = _arr(q_indptr, np.int32), _arr(bt_indptr, np.int32)
    bp, cl = _arr(bt_pages, np.int32), _arr(ctx_len, np.int32)
    rc = lib().kap_oracle_verify_attn(
        _p(q_bits, C.c_uint16), _p(qi, C.c_int32), _p(pool_bits, C.c_uint16), C.c_int64(n_pages),
        _p(bi, C.c_int32), _p(bp, C.c_int32), _p(cl, C.c_int32), C.c_int32(cl.shape[0]),
        C.c_int32(Hq), C.c_int32(Hkv), C.c_int32(d), C.c_int32(P), C.c_double(scale),
        _p(out, C.c_double), _p(lse, C.c_double), _p(ws, C.c_double), _p(nv, C.c_int64))
    if rc != OK:
        raise OracleError(rc)
    return out, lse, ws, nv


def num_threads() -> int:
    return int(lib().kap_oracle_num_threads())
