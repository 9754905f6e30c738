"""kap_selected_decode_attn_static: the allocation-free entry point (its scratch is a fixed array
inside the library) must give the same attention output as the workspace entry point.  Collected
last on purpose, so that a run that stops at the first failure has already run everything else.
The checks call through the C ABI binding, twice in a row with different queries: the second call
finds the first call's leftovers in the shared array and must not be affected by them."""
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


def test_static_entry_matches_workspace_entry_twice_in_a_row():
    w, _, pool_bits = _case(0)
    pool = gu.bits_to_dev(pool_bits)
    plan = kap.compile_workload(w)
    d_indptr, d_phys = gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"])
    d_logical, d_ctx = gu.i32(plan["plan_logical_pages"]), gu.i32(w.ctx_len)
    status = torch.full((1,), -1, dtype=torch.int32, device=gu.DEV)
    for call, (seed, splits) in enumerate([(1, 5), (2, 3)]):
        _, qd_bits, _ = _case(seed)
        ref_out, ref_lse = gu.run_decode(qd_bits, pool, plan, w.ctx_len)      # existing entry point
        q = gu.bits_to_dev(qd_bits)
        out = torch.full_like(q, float("nan"))
        lse = torch.full((w.batch, 32), float("nan"), dtype=torch.float32, device=gu.DEV)
        kap.selected_decode_attn_static(q, pool, d_indptr, d_phys, d_logical, d_ctx, out, splits,
                                        lse=lse, device_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got = gu.dev_bf16_to_f64(out)
        assert not np.isnan(got).any()
        assert_close(got, ref_out, what=f"static call {call} out")          # 1e-2 + 1e-2 |ref|
        assert gu.normalised_error(got, ref_out) <= 2e-2
        assert_close(lse.double().cpu().numpy(), ref_lse, atol=1e-2, rtol=1e-3, what=f"static call {call} lse")


def test_static_entry_single_split_and_capacity_limit():
    w, qd_bits, pool_bits = _case(3)
    pool = gu.bits_to_dev(pool_bits)
    plan = kap.compile_workload(w)
    args = (gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"]), gu.i32(plan["plan_logical_pages"]),
            gu.i32(w.ctx_len))
    q = gu.bits_to_dev(qd_bits)
    out = torch.zeros_like(q)
    ref_out, _ = gu.run_decode(qd_bits, pool, plan, w.ctx_len)
    kap.selected_decode_attn_static(q, pool, *args, out, 1)                  # no merge pass at all
    torch.cuda.synchronize()
    assert_close(gu.dev_bf16_to_f64(out), ref_out, what="static single split")
    before = kap.launch_count()
    with pytest.raises(kap.KapError) as e:                                   # 3*8*200 items > 4 MiB
        kap.selected_decode_attn_static(q, pool, *args, out, 200)
    assert e.value.code == kap.ERR_CAPACITY and "scratch" in str(e.value)
    assert kap.launch_count() == before
