"""kap_materialize_view: the copy is bit-exact against the oracle's indexing, and decode attention
over the compact view equals the in-place gather bit for bit (same pages, same order, same math)."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from oracle import brute
from paper_2607_24260_b200 import kap, synth

pytestmark = pytest.mark.gpu


def test_view_copy_and_attention_equivalence():
    w = synth.config3(0, batch=3, L=8192, layers=1, bt_mode="shuffled")
    q_bits, pool_bits = synth.host_qkv(w, 1)
    qd = q_bits[w.q_indptr[1:] - 1]
    plan = kap.compile_workload(w)
    n = int(plan["plan_indptr"][-1])
    pool = gu.bits_to_dev(pool_bits)
    compact = torch.zeros((n + 2,) + tuple(pool.shape[1:]), dtype=torch.bfloat16, device=gu.DEV)
    cpages = torch.full((n,), -1, dtype=torch.int32, device=gu.DEV)
    status = torch.zeros(1, dtype=torch.int32, device=gu.DEV)
    kap.materialize_view(pool, gu.i32(plan["plan_phys_pages"]), compact, cpages, status)
    torch.cuda.synchronize()
    ref_pool, ref_pages = brute.materialize_view(pool_bits, plan["plan_phys_pages"])
    assert int(status.item()) == 0
    np.testing.assert_array_equal(gu.dev_to_bits(compact[:n]), ref_pool)
    np.testing.assert_array_equal(cpages.cpu().numpy(), ref_pages)
    assert not gu.dev_to_bits(compact[n:]).any()                   # nothing written past the view
    in_place = gu.run_decode(qd, pool, plan, w.ctx_len)
    view_plan = dict(plan, plan_phys_pages=ref_pages)
    on_view = gu.run_decode(qd, compact, view_plan, w.ctx_len)
    np.testing.assert_array_equal(in_place[0], on_view[0])
    np.testing.assert_array_equal(in_place[1], on_view[1])


def test_view_capacity_and_bad_page():
    w = synth.config2(0, batch=1, L=1024, layers=1)
    _, pool_bits = synth.host_qkv(w, 2)
    pool = gu.bits_to_dev(pool_bits)
    plan = kap.compile_workload(w)
    n = int(plan["plan_indptr"][-1])
    small = torch.zeros((n - 1,) + tuple(pool.shape[1:]), dtype=torch.bfloat16, device=gu.DEV)
    before = kap.launch_count()
    with pytest.raises(kap.KapError) as e:
        kap.materialize_view(pool, gu.i32(plan["plan_phys_pages"]), small)
    assert e.value.code == kap.ERR_CAPACITY and kap.launch_count() == before
    bad = plan["plan_phys_pages"].copy()
    bad[1] = w.num_pool_pages + 5
    big = torch.zeros((n,) + tuple(pool.shape[1:]), dtype=torch.bfloat16, device=gu.DEV)
    status = torch.zeros(1, dtype=torch.int32, device=gu.DEV)
    kap.materialize_view(pool, gu.i32(bad), big, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1 << kap.ERR_DEVICE_INDEX
    assert not gu.dev_to_bits(big[1]).any()                        # the bad entry was skipped
    np.testing.assert_array_equal(gu.dev_to_bits(big[0]), pool_bits[plan["plan_phys_pages"][0]])
