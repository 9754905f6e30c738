"""Helpers for the GPU parity tests: move a workload to the device, run the library through its
C ABI binding, run the oracle on the same bits.  No method arithmetic here."""
from __future__ import annotations

import numpy as np
import torch

from oracle import kap_oracle as orc
from paper_2607_24260_b200 import kap, synth

DEV = "cuda:0"


def bits_to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch bf16 tensor on the GPU (bit-exact)."""
    return torch.from_numpy(np.array(bits, copy=True).view(np.int16)).to(DEV).view(torch.bfloat16)


def dev_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def dev_bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return synth.bf16_bits_to_f64(dev_to_bits(t))


def i32(a) -> torch.Tensor:
    return torch.from_numpy(np.array(a, dtype=np.int32, copy=True)).to(DEV)


def u16(a) -> torch.Tensor:
    """uint16 words -> device tensor of the same bits (carried as int16)."""
    return torch.from_numpy(np.array(a, dtype=np.uint16, copy=True).view(np.int16)).to(DEV)


def to_nhd(pool_bits: np.ndarray) -> np.ndarray:
    """[pages, 2, Hkv, P, d] (head-major) -> [pages, 2, P, Hkv, d] (token-major), same values"""
    return np.ascontiguousarray(pool_bits.transpose(0, 1, 3, 2, 4))


def run_decode(q_bits, pool_dev, plan, ctx_len, Hq=32, Hkv=8, max_chunk_pages=0, ws=None,
               logical=True, sm_scale=None, masks=None, kv_layout=kap.KV_HND):
    """Library proposal-path attention.  q_bits [B, Hq, d] uint16; pool_dev torch bf16
    [pages, 2, Hkv, P, d]; plan = dict from a plan compiler; masks = optional uint16 word per
    listed page (token-granular visibility).  Returns (out f64, lse f64)."""
    B = q_bits.shape[0]
    n = np.diff(plan["plan_indptr"])
    own = ws is None
    if own:
        ws = kap.Workspace(max_rows_per_item=Hq // Hkv, max_batch=max(B, 1))
        ws.set_kv_layout(kv_layout)
    ws.schedule(n, None, Hq, Hkv, max_chunk_pages)
    q = bits_to_dev(q_bits)
    out = torch.full_like(q, float("nan"))
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
    kap.selected_decode_attn(q, pool_dev, i32(plan["plan_indptr"]), i32(plan["plan_phys_pages"]),
                             i32(plan["plan_logical_pages"]) if logical else None, i32(ctx_len),
                             out, ws, lse=lse, sm_scale=sm_scale,
                             plan_token_masks=None if masks is None else u16(masks))
    ws.check()
    res = dev_bf16_to_f64(out), lse.double().cpu().numpy()
    if own:
        ws.close()
    return res


def run_verify(q_bits, n_q, pool_dev, bt_indptr, bt_pages, ctx_len, Hq=32, Hkv=8,
               max_chunk_pages=0, ws=None, page=16, sm_scale=None, kv_layout=kap.KV_HND):
    """Library verification attention.  q_bits [sum n_q, Hq, d] uint16."""
    n_q = np.asarray(n_q, dtype=np.int32)
    B = n_q.shape[0]
    q_indptr = np.zeros(B + 1, dtype=np.int32)
    np.cumsum(n_q, out=q_indptr[1:])
    own = ws is None
    if own:
        ws = kap.Workspace(max_rows_per_item=int(n_q.max()) * (Hq // Hkv), max_batch=max(B, 1))
        ws.set_kv_layout(kv_layout)
    n_pages = (np.asarray(ctx_len, dtype=np.int64) + page - 1) // page
    ws.schedule(n_pages, n_q, Hq, Hkv, max_chunk_pages)
    q = bits_to_dev(q_bits)
    out = torch.full_like(q, float("nan"))
    lse = torch.full((q.shape[0], Hq), float("nan"), dtype=torch.float32, device=DEV)
    kap.verify_attn(q, i32(q_indptr), pool_dev, i32(bt_indptr), i32(bt_pages), i32(ctx_len), out,
                    ws, lse=lse, sm_scale=sm_scale)
    ws.check()
    res = dev_bf16_to_f64(out), lse.double().cpu().numpy()
    if own:
        ws.close()
    return res


def oracle_decode(q_bits, pool_bits, plan, ctx_len, scale=None, masks=None):
    out, lse, _, _ = orc.selected_decode_attn(q_bits, pool_bits, plan["plan_indptr"],
                                              plan["plan_phys_pages"], plan["plan_logical_pages"],
                                              ctx_len, scale=scale, plan_token_masks=masks)
    return out, lse


def oracle_verify(q_bits, n_q, pool_bits, bt_indptr, bt_pages, ctx_len, scale=None):
    n_q = np.asarray(n_q, dtype=np.int32)
    q_indptr = np.zeros(n_q.shape[0] + 1, dtype=np.int32)
    np.cumsum(n_q, out=q_indptr[1:])
    out, lse, _, _ = orc.verify_attn(q_bits, q_indptr, pool_bits, bt_indptr, bt_pages, ctx_len,
                                     scale=scale)
    return out, lse


def normalised_error(got, ref):
    """max |got - ref| / max |ref| : the tolerance the benchmark spec states is loose for long contexts
    (outputs shrink like 1/sqrt(n_visible)), so the tests also bound this."""
    return float(np.max(np.abs(got - ref)) / max(np.max(np.abs(ref)), 1e-30))
