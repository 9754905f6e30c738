"""kap_selected_decode_attn_static: the allocation-free entry point (its scratch is a fixed array
inside the library).  Every result is compared with the fp64 oracle AND with the workspace entry
point.  Collected last on purpose, so that a run that stops at the first failure has already run
everything else.  The checks call through the C ABI binding, twice in a row with different
queries: the second call finds the first call's leftovers in the shared array and must not be
affected by them."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from helpers import assert_close
from paper_2607_24260_b200 import kap, synth

pytestmark = pytest.mark.gpu


def _case(seed):
    w = synth.config2(0, batch=3, L=6000, layers=1)
    q_bits, pool_bits = synth.host_qkv(w, seed)
    return w, q_bits[w.q_indptr[1:] - 1], pool_bits


def _identity_plan(ctx_len, bt_indptr, bt_pages, page=16):
    """the full-context plan: every page of every sequence, logical index = position in the list"""
    n = (np.asarray(ctx_len, dtype=np.int64) + page - 1) // page
    indptr = np.concatenate([[0], np.cumsum(n)]).astype(np.int32)
    phys = np.concatenate([bt_pages[bt_indptr[b]:bt_indptr[b] + n[b]] for b in range(len(n))]).astype(np.int32)
    logical = np.concatenate([np.arange(k, dtype=np.int32) for k in n])
    return {"plan_indptr": indptr, "plan_phys_pages": phys, "plan_logical_pages": logical}


def _check_against_both(got, got_lse, ref_oracle, ref_ws, what):
    assert not np.isnan(got).any(), what
    out_o, lse_o = ref_oracle
    assert_close(got, out_o, what=f"{what} out vs oracle")                   # 1e-2 + 1e-2 |ref|
    assert gu.normalised_error(got, out_o) <= 2e-2, what
    if got_lse is not None:
        assert_close(got_lse, lse_o, atol=1e-2, rtol=1e-3, what=f"{what} lse vs oracle")
    if ref_ws is not None:
        assert_close(got, ref_ws[0], what=f"{what} out vs workspace entry point")
        if got_lse is not None:
            assert_close(got_lse, ref_ws[1], atol=1e-2, rtol=1e-3, what=f"{what} lse vs workspace entry point")


def test_static_entry_matches_oracle_and_workspace_entry_twice_in_a_row():
    w, _, pool_bits = _case(0)
    pool = gu.bits_to_dev(pool_bits)
    plan = kap.compile_workload(w)
    d_indptr, d_phys = gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"])
    d_logical, d_ctx = gu.i32(plan["plan_logical_pages"]), gu.i32(w.ctx_len)
    status = torch.full((1,), -1, dtype=torch.int32, device=gu.DEV)
    for call, (seed, splits) in enumerate([(1, 5), (2, 3)]):
        _, qd_bits, _ = _case(seed)
        ref_ws = gu.run_decode(qd_bits, pool, plan, w.ctx_len)               # existing entry point
        ref_oracle = gu.oracle_decode(qd_bits, pool_bits, plan, w.ctx_len)
        q = gu.bits_to_dev(qd_bits)
        out = torch.full_like(q, float("nan"))
        lse = torch.full((w.batch, 32), float("nan"), dtype=torch.float32, device=gu.DEV)
        kap.selected_decode_attn_static(q, pool, d_indptr, d_phys, d_logical, d_ctx, out, splits,
                                        lse=lse, device_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        _check_against_both(gu.dev_bf16_to_f64(out), lse.double().cpu().numpy(), ref_oracle, ref_ws,
                            f"static call {call}")


def test_static_entry_single_split_and_capacity_limit():
    w, qd_bits, pool_bits = _case(3)
    pool = gu.bits_to_dev(pool_bits)
    plan = kap.compile_workload(w)
    args = (gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"]), gu.i32(plan["plan_logical_pages"]),
            gu.i32(w.ctx_len))
    q = gu.bits_to_dev(qd_bits)
    out = torch.zeros_like(q)
    ref_ws = gu.run_decode(qd_bits, pool, plan, w.ctx_len)
    ref_oracle = gu.oracle_decode(qd_bits, pool_bits, plan, w.ctx_len)
    kap.selected_decode_attn_static(q, pool, *args, out, 1)                  # no merge pass, lse = NULL
    torch.cuda.synchronize()
    _check_against_both(gu.dev_bf16_to_f64(out), None, ref_oracle, ref_ws, "static single split")
    before = kap.launch_count()
    with pytest.raises(kap.KapError) as e:                                   # 3*8*200 items > 4 MiB
        kap.selected_decode_attn_static(q, pool, *args, out, 200)
    assert e.value.code == kap.ERR_CAPACITY and "scratch" in str(e.value)
    assert kap.launch_count() == before


@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (16, 2)])
def test_static_entry_other_group_sizes_and_more_splits_than_pages(Hq, Hkv):
    """G = 1 and G = 8; one sequence of two pages cut into five slices (three of them empty);
    identity plan given without logical indices (the kernel's physical-ids-only mode)."""
    rng = synth.rng_for(Hq, "static-g")
    ctx = np.array([700, 20, 333], dtype=np.int32)
    n_pages = (ctx + 15) // 16
    bt_indptr = np.concatenate([[0], np.cumsum(n_pages)]).astype(np.int32)
    bt_pages = rng.permutation(int(n_pages.sum()) + 9)[:int(n_pages.sum())].astype(np.int32)
    pool_bits = synth.normal_bf16((int(n_pages.sum()) + 9, 2, Hkv, 16, 128), 0.5, rng)
    q_bits = synth.normal_bf16((3, Hq, 128), 1.0, rng)
    plan = _identity_plan(ctx, bt_indptr, bt_pages)
    ref_oracle = gu.oracle_decode(q_bits, pool_bits, plan, ctx)
    pool, q = gu.bits_to_dev(pool_bits), gu.bits_to_dev(q_bits)
    status = torch.full((1,), -1, dtype=torch.int32, device=gu.DEV)
    for logical in (gu.i32(plan["plan_logical_pages"]), None):
        out = torch.full_like(q, float("nan"))
        lse = torch.full((3, Hq), float("nan"), dtype=torch.float32, device=gu.DEV)
        kap.selected_decode_attn_static(q, pool, gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"]),
                                        logical, gu.i32(ctx), out, 5, lse=lse, device_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        _check_against_both(gu.dev_bf16_to_f64(out), lse.double().cpu().numpy(), ref_oracle, None,
                            f"static {Hq}/{Hkv} logical={'given' if logical is not None else 'NULL'}")


def test_static_entry_reports_a_slice_longer_than_a_cta_can_hold():
    """641 pages in one slice with logical indices (the CTA holds 640): the device cuts the slice,
    sets 1 << KAP_ERR_CAPACITY and nothing faults.  The same list without logical indices fits
    (1600) and matches the oracle; so does the first call with one more split."""
    rng = synth.rng_for(641, "static-long")
    Hq, Hkv, n = 8, 2, 641
    ctx = np.array([n * 16 - 5], dtype=np.int32)
    bt_pages = rng.permutation(n + 3)[:n].astype(np.int32)
    pool_bits = synth.normal_bf16((n + 3, 2, Hkv, 16, 128), 0.5, rng)
    q_bits = synth.normal_bf16((1, Hq, 128), 1.0, rng)
    plan = _identity_plan(ctx, np.array([0, n], dtype=np.int32), bt_pages)
    ref_oracle = gu.oracle_decode(q_bits, pool_bits, plan, ctx)
    pool, q = gu.bits_to_dev(pool_bits), gu.bits_to_dev(q_bits)
    d = (gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"]))
    d_logical, d_ctx = gu.i32(plan["plan_logical_pages"]), gu.i32(ctx)
    status = torch.full((1,), -1, dtype=torch.int32, device=gu.DEV)
    out = torch.zeros_like(q)
    kap.selected_decode_attn_static(q, pool, *d, d_logical, d_ctx, out, 1, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1 << kap.ERR_CAPACITY
    for logical, splits in ((None, 1), (d_logical, 2)):
        out = torch.full_like(q, float("nan"))
        kap.selected_decode_attn_static(q, pool, *d, logical, d_ctx, out, splits, device_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0                       # the status word starts from zero again
        _check_against_both(gu.dev_bf16_to_f64(out), None, ref_oracle, None, f"641 pages, {splits} split(s)")
