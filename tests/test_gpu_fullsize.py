"""GPU parity at the full batch and context sizes of configurations 2-5, one layer each, in the
launch configuration bench.py times (default launch options, the library's own schedule):

* sampled outputs: for a few (sequence, KV head) pairs the pages of that sequence and head are
  copied to the host and the oracle computes those query heads' outputs one by one (proposal path
  over the plan's pages, verification over the whole context);
* a property that holds at any size, checked for EVERY (sequence, head): with q = 0 the
  log-sum-exp is ln(number of visible tokens), which counts the pages each kernel visited.

KV and Q are drawn on the device from a seeded generator; the oracle gets the same bits back."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from helpers import assert_close
from oracle import kap_oracle as orc
from paper_2607_24260_b200 import kap, synth

pytestmark = pytest.mark.gpu


def _device_case(name, seed=0):
    w = synth.CONFIGS[name](seed, layers=1)
    pool = torch.empty((w.num_pool_pages, 2, w.num_kv_heads, w.page_size, w.head_dim),
                       dtype=torch.bfloat16, device=gu.DEV)
    synth.device_fill_normal_(pool, 0.5, seed + 11)
    g = torch.Generator(device=gu.DEV)
    g.manual_seed(seed + 12)
    q = torch.randn((int(w.n_q.sum()), w.num_q_heads, w.head_dim), device=gu.DEV, generator=g).to(torch.bfloat16)
    if name == "c3":        # planted keys with a +2 sigma affinity to the decode queries, inside the plan's pages
        plan = kap.compile_workload(w)
        per_seq = [plan["plan_phys_pages"][plan["plan_indptr"][b]:plan["plan_indptr"][b + 1]] for b in range(w.batch)]
        qd = q[torch.from_numpy(w.q_indptr[1:] - 1).long().to(gu.DEV)].contiguous()
        assert synth.plant_affinity_keys_(pool, qd, w, per_seq, seed=seed, layer=0) > 0
    return w, pool, q


def _run_library(w, pool, q, plan):
    B, Hq, Hkv = w.batch, w.num_q_heads, w.num_kv_heads
    qd = q[torch.from_numpy(w.q_indptr[1:] - 1).long().to(gu.DEV)].contiguous()
    ws_d = kap.Workspace(max_rows_per_item=Hq // Hkv, max_batch=B)
    ws_v = kap.Workspace(max_rows_per_item=int(w.n_q.max()) * (Hq // Hkv), max_batch=B)
    info_d = ws_d.schedule(np.diff(plan["plan_indptr"]), None, Hq, Hkv)
    n_pages = (w.ctx_len.astype(np.int64) + 15) // 16
    info_v = ws_v.schedule(n_pages, w.n_q, Hq, Hkv)
    out_d, out_v = torch.zeros_like(qd), torch.zeros_like(q)
    lse_d = torch.zeros((B, Hq), dtype=torch.float32, device=gu.DEV)
    lse_v = torch.zeros((q.shape[0], Hq), dtype=torch.float32, device=gu.DEV)
    d = dict(indptr=gu.i32(plan["plan_indptr"]), phys=gu.i32(plan["plan_phys_pages"]),
             logical=gu.i32(plan["plan_logical_pages"]), ctx=gu.i32(w.ctx_len), q_indptr=gu.i32(w.q_indptr),
             bt_indptr=gu.i32(w.bt_indptr), bt_pages=gu.i32(w.bt_pages))
    kap.selected_decode_attn(qd, pool, d["indptr"], d["phys"], d["logical"], d["ctx"], out_d, ws_d, lse=lse_d)
    kap.verify_attn(q, d["q_indptr"], pool, d["bt_indptr"], d["bt_pages"], d["ctx"], out_v, ws_v, lse=lse_v)
    ws_d.check()
    ws_v.check()
    # the q = 0 property run, same schedules
    z_d, z_v = torch.zeros_like(qd), torch.zeros_like(q)
    zl_d, zl_v = torch.zeros_like(lse_d), torch.zeros_like(lse_v)
    kap.selected_decode_attn(z_d, pool, d["indptr"], d["phys"], d["logical"], d["ctx"], torch.zeros_like(qd), ws_d, lse=zl_d)
    kap.verify_attn(z_v, d["q_indptr"], pool, d["bt_indptr"], d["bt_pages"], d["ctx"], torch.zeros_like(q), ws_v, lse=zl_v)
    ws_d.check()
    ws_v.check()
    # the same property under the plan's token masks: only the selected union is visible
    zl_m = torch.zeros_like(lse_d)
    kap.selected_decode_attn(z_d, pool, d["indptr"], d["phys"], d["logical"], d["ctx"], torch.zeros_like(qd), ws_d,
                             lse=zl_m, plan_token_masks=gu.u16(plan["plan_token_masks"]))
    ws_d.check()
    res = dict(zl_m=zl_m.double().cpu().numpy(), qd=qd, out_d=out_d, out_v=out_v, lse_d=lse_d.double().cpu().numpy(),
               lse_v=lse_v.double().cpu().numpy(), zl_d=zl_d.double().cpu().numpy(),
               zl_v=zl_v.double().cpu().numpy(), info_d=info_d, info_v=info_v)
    ws_d.close()
    ws_v.close()
    return res


def _head_pool(pool, phys_pages, g):
    """host copy [n, 2, 1, P, d] of the given pages for KV head g"""
    idx = torch.from_numpy(np.asarray(phys_pages, dtype=np.int64)).to(gu.DEV)
    return gu.dev_to_bits(pool[idx][:, :, g:g + 1].contiguous())


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_full_size_configuration(name):
    w, pool, q = _device_case(name)
    plan = kap.compile_workload(w)
    ref_plan = orc.compile_workload(w)
    for k in ("plan_indptr", "plan_logical_pages", "plan_phys_pages", "plan_flags", "selected_tokens",
              "plan_token_masks"):
        np.testing.assert_array_equal(plan[k], ref_plan[k])
    r = _run_library(w, pool, q, plan)
    G = w.num_q_heads // w.num_kv_heads
    out_d, out_v = gu.dev_bf16_to_f64(r["out_d"]), gu.dev_bf16_to_f64(r["out_v"])
    assert not np.isnan(out_d).any() and not np.isnan(out_v).any()

    # ---- property at full size, every (sequence, head): lse(q = 0) = ln(visible tokens)
    n_sel = np.diff(plan["plan_indptr"])
    for b in range(w.batch):
        L = int(w.ctx_len[b])
        lp = plan["plan_logical_pages"][plan["plan_indptr"][b]:plan["plan_indptr"][b + 1]]
        vis = int(np.minimum(16, L - lp.astype(np.int64) * 16).sum())
        np.testing.assert_allclose(r["zl_d"][b], np.log(vis), atol=3e-5, err_msg=f"{name} decode seq {b}")
        # token-granular: exactly the tokens of the selected union (the oracle's count)
        np.testing.assert_allclose(r["zl_m"][b], np.log(int(ref_plan["selected_tokens"][b])), atol=3e-5,
                                   err_msg=f"{name} masked decode seq {b}")
        for j in range(int(w.n_q[b])):
            row = int(w.q_indptr[b]) + j
            np.testing.assert_allclose(r["zl_v"][row], np.log(L - int(w.n_q[b]) + j + 1), atol=3e-5,
                                       err_msg=f"{name} verify seq {b} row {j}")

    # ---- sampled (sequence, KV head) pairs against the oracle
    rng = synth.rng_for(0, name, "fullsize-sample")
    seqs = rng.choice(w.batch, size=min(3, w.batch), replace=False)
    if name == "c5":                                   # make sure a fallback sequence is sampled
        seqs[0] = int(np.nonzero(w.force_full)[0][0])
    qd_bits, q_bits = gu.dev_to_bits(r["qd"]), gu.dev_to_bits(q)
    for b in seqs:
        b = int(b)
        L = int(w.ctx_len[b])
        for g in rng.choice(w.num_kv_heads, size=2, replace=False):
            g = int(g)
            heads = slice(g * G, (g + 1) * G)
            # proposal path: only the plan's pages of this sequence and head
            lo, hi = plan["plan_indptr"][b], plan["plan_indptr"][b + 1]
            small = _head_pool(pool, plan["plan_phys_pages"][lo:hi], g)
            o, l, _, _ = orc.selected_decode_attn(qd_bits[b:b + 1, heads], small, [0, hi - lo],
                                                  np.arange(hi - lo), plan["plan_logical_pages"][lo:hi], [L])
            assert_close(out_d[b, heads], o[0], what=f"{name} decode seq {b} kv head {g}")
            assert gu.normalised_error(out_d[b, heads], o[0]) <= 2e-2
            assert_close(r["lse_d"][b, heads], l[0], atol=1e-2, rtol=1e-3, what=f"{name} decode lse")
            # verification: the whole context of this sequence and head
            n_pages = (L + 15) // 16
            small = _head_pool(pool, w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b] + n_pages], g)
            rows = slice(int(w.q_indptr[b]), int(w.q_indptr[b + 1]))
            o, l, _, _ = orc.verify_attn(q_bits[rows, heads], [0, int(w.n_q[b])], small, [0, n_pages],
                                         np.arange(n_pages), [L])
            assert_close(out_v[rows, heads], o, what=f"{name} verify seq {b} kv head {g}")
            assert gu.normalised_error(out_v[rows, heads], o) <= 2e-2
            assert_close(r["lse_v"][rows, heads], l, atol=1e-2, rtol=1e-3, what=f"{name} verify lse")
