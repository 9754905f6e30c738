"""Thin Python binding of the C ABI in include/kap.h - argument marshalling only.

Host-side calls take numpy arrays; the attention calls take torch CUDA tensors (PyTorch is used
for device memory and streams only) and pass raw device pointers and the current CUDA stream.
The shared library must have been built (``python -m paper_2607_24260_b200.build`` or
``__graft_entry__.build()``); there is no fallback path: a missing library raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

OK, ERR_INVALID_ARG, ERR_CAPACITY, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT, ERR_DEVICE_INDEX = range(7)
PLAN_FULL, PLAN_OVER_BUDGET, PLAN_S_HIGH, PLAN_MOVES_WITH_LENGTH = 1, 2, 4, 8
KV_HND, KV_NHD = 0, 1

_i32p, _f32p, _u8p, _vp = C.POINTER(C.c_int32), C.POINTER(C.c_float), C.POINTER(C.c_uint8), C.c_void_p

# every symbol include/kap.h declares, with its signature
SIGNATURES = {
    "kap_compile_plan": (C.c_int, [C.c_int32, C.c_int32, _i32p, _i32p, _i32p, _i32p, _f32p, _i32p,
                                   _i32p, _i32p, _u8p, C.c_float, _i32p, _i32p, C.c_int64, _i32p,
                                   _i32p, _i32p, _i32p, _i32p, C.POINTER(C.c_uint16)]),
    "kap_compile_growing_plan": (C.c_int, [C.c_int32, C.c_int32, _i32p, _i32p, _i32p, _i32p, _f32p,
                                           _i32p, _i32p, _i32p, _u8p, C.c_float, _i32p, _i32p,
                                           C.c_int32, C.c_int64, _i32p, _i32p, _i32p,
                                           C.POINTER(C.c_uint16), _i32p, _i32p, _i32p]),
    "kap_refresh_recent": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int32,
                                     C.c_int64, _vp, _vp, _vp]),
    "kap_workspace_create": (C.c_int, [C.POINTER(_vp), C.c_int32, C.c_int32, C.c_int32, C.c_int32]),
    "kap_workspace_destroy": (None, [_vp]),
    "kap_schedule": (C.c_int, [_vp, C.c_int32, _i32p, _i32p, C.c_int32, C.c_int32, C.c_int32, _vp]),
    "kap_schedule_host": (C.c_int, [C.c_int32, _i32p, _i32p, C.c_int32, C.c_int32, C.c_int32,
                                    C.c_int32, C.c_int32, C.c_int32, _i32p, _i32p, _i32p, _i32p,
                                    _i32p]),
    "kap_schedule_info": (C.c_int, [_vp, _i32p, _i32p, _i32p, _i32p, _i32p]),
    "kap_selected_decode_attn": (C.c_int, [_vp, _vp, C.c_int64, _vp, _vp, _vp, _vp, _vp, C.c_int32,
                                           C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_float,
                                           _vp, _vp, _vp, _vp]),
    "kap_verify_attn": (C.c_int, [_vp, _vp, _vp, C.c_int64, _vp, _vp, _vp, C.c_int32, C.c_int32,
                                  C.c_int32, C.c_int32, C.c_int32, C.c_float, _vp, _vp, _vp, _vp]),
    "kap_selected_decode_attn_static": (C.c_int, [_vp, _vp, C.c_int64, _vp, _vp, _vp, _vp, C.c_int32,
                                                  C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                                  C.c_float, C.c_int32, _vp, _vp, _vp, _vp]),
    "kap_append_kv": (C.c_int, [_vp, _vp, _vp, _vp, C.c_int64, _vp, _vp, _vp, C.c_int32, C.c_int32,
                                C.c_int32, C.c_int32, C.c_int32, C.c_int32, _vp, _vp]),
    "kap_workspace_set_kv_layout": (C.c_int, [_vp, C.c_int32]),
    "kap_top3_accept": (C.c_int, [_vp, C.c_int64, _vp, _vp, C.c_int32, C.c_int32, C.c_int32, _vp, _vp,
                                  _vp, _vp, _vp]),
    "kap_phase_model": (C.c_int, [C.c_double] * 6 + [C.POINTER(C.c_double)]),
    "kap_fallback_decide": (C.c_int, [C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.c_int64,
                                      C.c_double, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                      C.c_double, C.c_double, C.c_double, C.c_double, _i32p, _i32p,
                                      C.POINTER(C.c_double), C.c_double, _u8p, _i32p,
                                      C.POINTER(C.c_double), C.POINTER(C.c_double),
                                      C.POINTER(C.c_double)]),
    "kap_materialize_view": (C.c_int, [_vp, C.c_int64, _vp, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                       _vp, C.c_int64, _vp, _vp, _vp]),
    "kap_device_sm_rates": (C.c_int, [C.c_int32, C.c_int32, _f32p, _i32p]),
    "kap_workspace_check": (C.c_int, [_vp, _vp]),
    "kap_set_launch_options": (C.c_int, [C.c_int32] * 5),
    "kap_set_verify_kernel": (C.c_int, [C.c_int32]),
    "kap_launch_count": (C.c_int64, []),
    "kap_last_error": (C.c_char_p, []),
    "kap_version": (C.c_char_p, []),
}

_lib = None


class KapError(RuntimeError):
    def __init__(self, code, message):
        super().__init__(f"kap status {code}: {message}")
        self.code = code


def lib():
    """Load libkap_b200.so (built in-tree).  Raises if it is missing: there is no fallback."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: build it with `python -m paper_2607_24260_b200.build`")
        handle = C.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _check(code):
    if code != OK:
        raise KapError(code, lib().kap_last_error().decode())


def _np(a, dt):
    return None if a is None else np.ascontiguousarray(a, dtype=dt)


def _ptr(a, ct):
    return None if a is None else a.ctypes.data_as(C.POINTER(ct))


def version() -> str:
    return lib().kap_version().decode()


def launch_count() -> int:
    return int(lib().kap_launch_count())


def set_launch_options(use_pdl: int = -1, early_kv: int = -1, ctas_per_sm: int = -1,
                       max_cluster: int = -1, ring_slots: int = -1):
    _check(lib().kap_set_launch_options(int(use_pdl), int(early_kv), int(ctas_per_sm),
                                        int(max_cluster), int(ring_slots)))


def set_verify_kernel(kernel: int):
    """kap_set_verify_kernel: 0 = the mma.sync split kernel, 1 = the tcgen05 kernel (schedules made
    afterwards; at most 64 query rows per KV head, else the split kernel is used)."""
    _check(lib().kap_set_verify_kernel(int(kernel)))


# ------------------------------------------------------------------------------- kap_compile_plan
def compile_plan(ctx_len, span_indptr, span_start, span_len, span_score, budget_tokens, n_sink,
                 n_recent, force_full=None, s_max=1.0, bt_indptr=None, bt_pages=None, page_size=16,
                 capacity=None):
    """kap_compile_plan on host arrays.  Returns a dict: plan_indptr, plan_logical_pages,
    plan_phys_pages (None without a block table), plan_flags, selected_tokens, plan_token_masks
    (uint16 per listed page, bit t = token t of the page is in the selected union; None when
    page_size > 16)."""
    ctx_len = _np(ctx_len, np.int32)
    B = int(ctx_len.shape[0])
    span_indptr, span_start = _np(span_indptr, np.int32), _np(span_start, np.int32)
    span_len, span_score = _np(span_len, np.int32), _np(span_score, np.float32)
    budget_tokens, n_sink = _np(budget_tokens, np.int32), _np(n_sink, np.int32)
    n_recent, force_full = _np(n_recent, np.int32), _np(force_full, np.uint8)
    bt_indptr, bt_pages = _np(bt_indptr, np.int32), _np(bt_pages, np.int32)
    if capacity is None:
        capacity = int(sum((max(int(L), 0) + page_size - 1) // max(page_size, 1) for L in ctx_len))
    indptr = np.full(B + 1, -1, dtype=np.int32)
    logical = np.full(max(1, capacity), -1, dtype=np.int32)
    phys = np.full(max(1, capacity), -1, dtype=np.int32) if bt_indptr is not None else None
    flags = np.full(B, -1, dtype=np.int32)
    sel = np.full(B, -1, dtype=np.int32)
    masks = np.zeros(max(1, capacity), dtype=np.uint16) if 0 < page_size <= 16 else None
    _check(lib().kap_compile_plan(
        B, page_size, _ptr(ctx_len, C.c_int32), _ptr(span_indptr, C.c_int32),
        _ptr(span_start, C.c_int32), _ptr(span_len, C.c_int32), _ptr(span_score, C.c_float),
        _ptr(budget_tokens, C.c_int32), _ptr(n_sink, C.c_int32), _ptr(n_recent, C.c_int32),
        _ptr(force_full, C.c_uint8), float(s_max), _ptr(bt_indptr, C.c_int32),
        _ptr(bt_pages, C.c_int32), int(capacity), _ptr(indptr, C.c_int32), _ptr(logical, C.c_int32),
        _ptr(phys, C.c_int32), _ptr(flags, C.c_int32), _ptr(sel, C.c_int32),
        _ptr(masks, C.c_uint16)))
    n = int(indptr[-1])
    return dict(plan_indptr=indptr, plan_logical_pages=logical[:n].copy(),
                plan_phys_pages=None if phys is None else phys[:n].copy(), plan_flags=flags,
                selected_tokens=sel,
                plan_token_masks=None if masks is None else masks[:n].copy())


def compile_growing_plan(ctx_len, span_indptr, span_start, span_len, span_score, budget_tokens,
                         n_sink, n_recent, bt_indptr, bt_pages, force_full=None, s_max=1.0,
                         page_size=16, max_growth=0, capacity=None):
    """kap_compile_growing_plan on host arrays.  Returns the dict of compile_plan (lists = fixed
    part + reserved entries) plus tail_desc int32 [B, 3]."""
    ctx_len = _np(ctx_len, np.int32)
    B = int(ctx_len.shape[0])
    span_indptr, span_start = _np(span_indptr, np.int32), _np(span_start, np.int32)
    span_len, span_score = _np(span_len, np.int32), _np(span_score, np.float32)
    budget_tokens, n_sink = _np(budget_tokens, np.int32), _np(n_sink, np.int32)
    n_recent, force_full = _np(n_recent, np.int32), _np(force_full, np.uint8)
    bt_indptr, bt_pages = _np(bt_indptr, np.int32), _np(bt_pages, np.int32)
    if capacity is None:
        ps = max(page_size, 1)
        capacity = int(sum((max(int(L), 0) + ps - 1) // ps + (max(int(r), 1) + ps - 2) // ps + 1
                           + (max_growth + ps - 1) // ps + 1 for L, r in zip(ctx_len, n_recent)))
    indptr = np.full(B + 1, -1, dtype=np.int32)
    logical = np.full(max(1, capacity), -1, dtype=np.int32)
    phys = np.full(max(1, capacity), -1, dtype=np.int32)
    masks = np.zeros(max(1, capacity), dtype=np.uint16)
    flags = np.full(B, -1, dtype=np.int32)
    sel = np.full(B, -1, dtype=np.int32)
    tail = np.full((B, 3), -1, dtype=np.int32)
    _check(lib().kap_compile_growing_plan(
        B, page_size, _ptr(ctx_len, C.c_int32), _ptr(span_indptr, C.c_int32),
        _ptr(span_start, C.c_int32), _ptr(span_len, C.c_int32), _ptr(span_score, C.c_float),
        _ptr(budget_tokens, C.c_int32), _ptr(n_sink, C.c_int32), _ptr(n_recent, C.c_int32),
        _ptr(force_full, C.c_uint8), float(s_max), _ptr(bt_indptr, C.c_int32),
        _ptr(bt_pages, C.c_int32), int(max_growth), int(capacity), _ptr(indptr, C.c_int32),
        _ptr(logical, C.c_int32), _ptr(phys, C.c_int32), _ptr(masks, C.c_uint16),
        _ptr(flags, C.c_int32), _ptr(sel, C.c_int32), _ptr(tail, C.c_int32)))
    n = int(indptr[-1])
    return dict(plan_indptr=indptr, plan_logical_pages=logical[:n].copy(),
                plan_phys_pages=phys[:n].copy(), plan_flags=flags, selected_tokens=sel,
                plan_token_masks=masks[:n].copy(), tail_desc=tail)


def refresh_recent(plan_indptr, plan_logical_pages, plan_phys_pages, plan_token_masks, tail_desc,
                   bt_indptr, bt_pages, ctx_len, num_pool_pages, ws: "Workspace | None" = None,
                   device_status=None, page_size=16, stream=None):
    """kap_refresh_recent on torch CUDA tensors (int32; masks as 16-bit words): rewrites the
    reserved entries of a growing plan from the current device ctx_len."""
    _check(lib().kap_refresh_recent(
        _dptr(plan_indptr), _dptr(plan_logical_pages), _dptr(plan_phys_pages),
        _dptr(plan_token_masks), _dptr(tail_desc), _dptr(bt_indptr), _dptr(bt_pages),
        _dptr(ctx_len), int(ctx_len.shape[0]), int(page_size), int(num_pool_pages),
        _dptr(device_status), None if ws is None else ws._h, _stream_ptr(stream)))


def compile_workload(w, capacity=None):
    """kap_compile_plan on a synth.Workload."""
    return compile_plan(w.ctx_len, w.span_indptr, w.span_start, w.span_len, w.span_score,
                        w.budget_tokens, w.n_sink, w.n_recent, w.force_full, w.s_max, w.bt_indptr,
                        w.bt_pages, w.page_size, capacity)


def schedule_host(list_len, n_q, num_q_heads, num_kv_heads, cta_slots, max_chunk_pages=0,
                  max_items=8192, max_cluster=1):
    """kap_schedule_host: the split-K work list as an [n_items, 8] int32 array (seq, kv_head,
    page_begin, page_end, group, slot, n_splits, n_q) plus (n_merge_groups, max_chunk) and, when
    max_cluster > 1, the chosen cluster size as a fourth value."""
    list_len = _np(list_len, np.int32)
    n_q = _np(n_q, np.int32)
    items = np.zeros((max_items, 8), dtype=np.int32)
    n_items, n_merge, max_chunk, cluster = C.c_int32(0), C.c_int32(0), C.c_int32(0), C.c_int32(1)
    _check(lib().kap_schedule_host(int(list_len.shape[0]), _ptr(list_len, C.c_int32),
                                   _ptr(n_q, C.c_int32), num_q_heads, num_kv_heads, cta_slots,
                                   max_cluster, max_chunk_pages, max_items, _ptr(items, C.c_int32),
                                   C.byref(n_items), C.byref(n_merge), C.byref(max_chunk),
                                   C.byref(cluster)))
    out = (items[:n_items.value].copy(), n_merge.value, max_chunk.value)
    return out if max_cluster <= 1 else out + (cluster.value,)


# ------------------------------------------------------------------------- workspace + attention
def _stream_ptr(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _dptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _pool_shape(kv_pool, ws):
    """(pages, Hkv, P) of a pool tensor in the layout the workspace is set to"""
    pages, _, a, b, _ = kv_pool.shape
    return (pages, b, a) if getattr(ws, "kv_layout", KV_HND) == KV_NHD else (pages, a, b)


class Workspace:
    """kap_workspace: split-K schedule + partial-result buffers for one launch shape."""

    def __init__(self, device=0, max_items=8192, max_rows_per_item=16, max_batch=256):
        self._h = C.c_void_p()
        self.device = int(device)
        self._destroy = lib().kap_workspace_destroy
        _check(lib().kap_workspace_create(C.byref(self._h), self.device, max_items,
                                          max_rows_per_item, max_batch))

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            self._destroy(self._h)           # bound at construction: module globals may be gone at exit
            self._h = None

    __del__ = close

    def schedule(self, list_len, n_q=None, num_q_heads=32, num_kv_heads=8, max_chunk_pages=0,
                 stream=None):
        list_len = _np(list_len, np.int32)
        n_q = _np(n_q, np.int32)
        _check(lib().kap_schedule(self._h, int(list_len.shape[0]), _ptr(list_len, C.c_int32),
                                  _ptr(n_q, C.c_int32), num_q_heads, num_kv_heads, max_chunk_pages,
                                  _stream_ptr(stream)))
        return self.info()

    def set_kv_layout(self, kv_layout):
        """KV_HND (default): pools are [pages, 2, Hkv, P, d]; KV_NHD: [pages, 2, P, Hkv, d]."""
        _check(lib().kap_workspace_set_kv_layout(self._h, int(kv_layout)))
        self.kv_layout = int(kv_layout)

    def info(self):
        v = [C.c_int32(0) for _ in range(5)]
        _check(lib().kap_schedule_info(self._h, *[C.byref(x) for x in v]))
        return dict(n_items=v[0].value, n_merge_groups=v[1].value, max_chunk_pages=v[2].value,
                    ctas_per_wave=v[3].value, cluster_size=v[4].value)

    def check(self, stream=None):
        _check(lib().kap_workspace_check(self._h, _stream_ptr(stream)))


def selected_decode_attn(q, kv_pool, plan_indptr, plan_phys_pages, plan_logical_pages, ctx_len, out,
                         ws: Workspace, lse=None, sm_scale=None, stream=None, plan_token_masks=None):
    """kap_selected_decode_attn on torch CUDA tensors: q/out bf16 [B, Hq, d]; kv_pool bf16
    [pages, 2, Hkv, P, d]; plan arrays and ctx_len int32 device tensors; plan_token_masks an
    optional uint16 device tensor (one word per listed page) for token-granular visibility."""
    B, Hq, d = q.shape
    pages, Hkv, P = _pool_shape(kv_pool, ws)
    sm_scale = float(d) ** -0.5 if sm_scale is None else float(sm_scale)
    _check(lib().kap_selected_decode_attn(
        _dptr(q), _dptr(kv_pool), int(pages), _dptr(plan_indptr), _dptr(plan_phys_pages),
        _dptr(plan_logical_pages), _dptr(plan_token_masks), _dptr(ctx_len), B, Hq, Hkv, d, P,
        sm_scale, _dptr(out), _dptr(lse), ws._h, _stream_ptr(stream)))
    return out


def verify_attn(q, q_indptr, kv_pool, bt_indptr, bt_pages, ctx_len, out, ws: Workspace, lse=None,
                sm_scale=None, stream=None):
    """kap_verify_attn on torch CUDA tensors: q/out bf16 [sum n_q, Hq, d]."""
    _, Hq, d = q.shape
    pages, Hkv, P = _pool_shape(kv_pool, ws)
    sm_scale = float(d) ** -0.5 if sm_scale is None else float(sm_scale)
    _check(lib().kap_verify_attn(
        _dptr(q), _dptr(q_indptr), _dptr(kv_pool), int(pages), _dptr(bt_indptr), _dptr(bt_pages),
        _dptr(ctx_len), int(ctx_len.shape[0]), Hq, Hkv, d, P, sm_scale, _dptr(out), _dptr(lse),
        ws._h, _stream_ptr(stream)))
    return out


def selected_decode_attn_static(q, kv_pool, plan_indptr, plan_phys_pages, plan_logical_pages, ctx_len,
                                out, num_splits, lse=None, device_status=None, sm_scale=None,
                                stream=None):
    """kap_selected_decode_attn_static: the proposal-path attention without a workspace, for
    callers that may not allocate device memory (scratch is a fixed array inside the library).
    `device_status`: optional int32 CUDA tensor of one element that receives the status bits."""
    B, Hq, d = q.shape
    pages, _, Hkv, P, _ = kv_pool.shape
    sm_scale = float(d) ** -0.5 if sm_scale is None else float(sm_scale)
    _check(lib().kap_selected_decode_attn_static(
        _dptr(q), _dptr(kv_pool), int(pages), _dptr(plan_indptr), _dptr(plan_phys_pages),
        _dptr(plan_logical_pages), _dptr(ctx_len), B, Hq, Hkv, d, P, sm_scale, int(num_splits),
        _dptr(out), _dptr(lse), _dptr(device_status), _stream_ptr(stream)))
    return out


def append_kv(k_new, v_new, kv_pool, bt_indptr, bt_pages, ctx_len, new_indptr=None, advance=True,
              device_status=None, stream=None, kv_layout=KV_HND):
    """kap_append_kv: write the new tokens' K/V rows (bf16 [sum n_new, Hkv, d]) into the paged pool
    at positions ctx_len[b] .. and, with advance, bump ctx_len on the device.  kv_pool has shape
    [pages, 2, Hkv, P, d] (KV_HND) or [pages, 2, P, Hkv, d] (KV_NHD)."""
    if kv_layout == KV_NHD:
        pages, _, P, Hkv, d = kv_pool.shape
    else:
        pages, _, Hkv, P, d = kv_pool.shape
    _check(lib().kap_append_kv(_dptr(k_new), _dptr(v_new), _dptr(new_indptr), _dptr(kv_pool), int(pages),
                               _dptr(bt_indptr), _dptr(bt_pages), _dptr(ctx_len), int(bool(advance)),
                               int(ctx_len.shape[0]), Hkv, d, P, int(kv_layout), _dptr(device_status),
                               _stream_ptr(stream)))


def top3_accept(logits, row_indptr, proposed, top3, accepted, next_token, stream=None, ctx_len=None):
    """kap_top3_accept on torch CUDA tensors: logits fp32 [rows, vocab] (row stride taken from the
    tensor), int32 row_indptr [B+1], proposed [rows]; outputs int32 top3 [rows, 3], accepted [B],
    next_token [B].  ctx_len (int32 [B], optional) is reduced by the number of rejected proposals."""
    rows, vocab = logits.shape
    _check(lib().kap_top3_accept(_dptr(logits), int(logits.stride(0)), _dptr(row_indptr), _dptr(proposed),
                                 int(row_indptr.shape[0]) - 1, int(rows), int(vocab), _dptr(top3),
                                 _dptr(accepted), _dptr(next_token), _dptr(ctx_len), _stream_ptr(stream)))


PHASE_FIELDS = ("cost_full", "cost_base", "cost_plan", "speedup", "slack", "kv_crit", "beneficial",
                "h_minus_s")


def phase_model(k, h, s, w_main, w_prop, kv):
    """kap_phase_model: dict of the cost model's quantities (Eqs. 3-15)."""
    out = (C.c_double * 8)()
    _check(lib().kap_phase_model(float(k), float(h), float(s), float(w_main), float(w_prop), float(kv), out))
    return dict(zip(PHASE_FIELDS, [float(x) for x in out]))


FALLBACK_CAPACITY, FALLBACK_METADATA, FALLBACK_CONFIDENCE, FALLBACK_S_HIGH, FALLBACK_H_LOW, \
    FALLBACK_NO_MARGIN, FALLBACK_SLACK = 1, 2, 4, 8, 16, 32, 64
RUNTIME_OVER_CAPACITY, RUNTIME_UNSTABLE_METADATA = 1, 2


def fallback_decide(accepted_sum, proposed_sum, s, kv, w_main=0.0, w_prop=0.0, min_proposed=1,
                    h_prior=1.0, h_min=0.0, s_max=1.0, plan_flags=None, runtime_flags=None,
                    confidence=None, confidence_min=0.0):
    """kap_fallback_decide on host arrays; returns a dict of numpy arrays: force_full (uint8, ready
    for compile_plan's force_full), reasons, h, slack, budget_scale."""
    acc, prop = _np(accepted_sum, np.int64), _np(proposed_sum, np.int64)
    s, kv = _np(s, np.float64), _np(kv, np.float64)
    B = int(s.shape[0])
    flags, rt, conf = _np(plan_flags, np.int32), _np(runtime_flags, np.int32), _np(confidence, np.float64)
    out = dict(force_full=np.zeros(B, dtype=np.uint8), reasons=np.zeros(B, dtype=np.int32),
               h=np.zeros(B), slack=np.zeros(B), budget_scale=np.zeros(B))
    _check(lib().kap_fallback_decide(
        B, _ptr(acc, C.c_int64), _ptr(prop, C.c_int64), int(min_proposed), float(h_prior),
        _ptr(s, C.c_double), _ptr(kv, C.c_double), float(w_main), float(w_prop), float(h_min),
        float(s_max), _ptr(flags, C.c_int32), _ptr(rt, C.c_int32), _ptr(conf, C.c_double),
        float(confidence_min), _ptr(out["force_full"], C.c_uint8), _ptr(out["reasons"], C.c_int32),
        _ptr(out["h"], C.c_double), _ptr(out["slack"], C.c_double), _ptr(out["budget_scale"], C.c_double)))
    return out


def device_sm_rates(device=0):
    """kap_device_sm_rates: numpy array of the relative streaming rate of every SM (mean 1)."""
    n = C.c_int32(0)
    _check(lib().kap_device_sm_rates(int(device), 0, None, C.byref(n)))
    out = np.zeros(n.value, dtype=np.float32)
    _check(lib().kap_device_sm_rates(int(device), n.value, _ptr(out, C.c_float), C.byref(n)))
    return out


def materialize_view(kv_pool, plan_phys_pages, compact_pool, compact_pages=None, device_status=None,
                     stream=None):
    """kap_materialize_view: copy the plan's pages into compact_pool in plan order."""
    pages, _, Hkv, P, d = kv_pool.shape
    _check(lib().kap_materialize_view(_dptr(kv_pool), int(pages), _dptr(plan_phys_pages),
                                      int(plan_phys_pages.shape[0]), Hkv, d, P, _dptr(compact_pool),
                                      int(compact_pool.shape[0]), _dptr(compact_pages),
                                      _dptr(device_status), _stream_ptr(stream)))
