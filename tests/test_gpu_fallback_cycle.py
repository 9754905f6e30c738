"""The fallback controller inside whole propose-k / verify cycles on the GPU (Section 3.2 "Runtime
stability and fallback", Section 4.2): after every cycle the accepted counts of kap_top3_accept
feed kap_fallback_decide, whose force_full goes into the next cycle's kap_compile_plan.  Synthetic
logits (there is no model here) let one sequence's acceptance collapse mid-run; from the next cycle
on it must run the identity plan.  Two independent chains are compared at every step:
    library: kap_top3_accept -> kap_fallback_decide -> kap_compile_plan -> kap_selected_decode_attn
    oracle : brute.top3_accept -> brute.fallback_decide -> oracle compile -> oracle attention
Integer results bit-exact, attention within the benchmark spec's tolerance."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from helpers import assert_close
from oracle import brute
from oracle import kap_oracle as orc
from paper_2607_24260_b200 import kap, synth
from test_gpu_append_loop import _cycle_case

pytestmark = pytest.mark.gpu
P = 16


@pytest.mark.parametrize("seed,k,cycles", [(2, 4, 5), (5, 3, 6)])
def test_acceptance_collapse_sends_a_sequence_to_full_context(seed, k, cycles):
    lens = (3000, 2500, 1777)
    w, _ = _cycle_case(seed, k * cycles, lens)
    B, Hq, Hkv, d, V = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, 211
    G = Hq // Hkv
    rng = synth.rng_for(seed, "fallback-cycle")
    q_bits, pool_bits = synth.host_qkv(w, seed, q_rows=cycles * 2 * k * B, q_std=4.0)
    q_dec = q_bits[:cycles * k * B].reshape(cycles, k, B, Hq, d)
    q_ver = q_bits[cycles * k * B:].reshape(cycles, B * k, Hq, d)
    k_new = synth.normal_bf16((cycles, k, B, Hkv, d), 0.5, rng)
    v_new = synth.normal_bf16((cycles, k, B, Hkv, d), 0.5, rng)
    logits = rng.standard_normal((cycles, B * (k + 1), V)).astype(np.float32)
    row_indptr = np.arange(0, B * (k + 1) + 1, k + 1, dtype=np.int32)
    best = logits.argmax(axis=2)
    worst = logits.argmin(axis=2)
    proposed = best.astype(np.int32).copy()                  # everything acceptable ...
    collapse_from, victim = 1, 1
    for c in range(collapse_from, cycles):                   # ... except the victim's, from cycle 1 on
        rows = slice(victim * (k + 1), victim * (k + 1) + k)
        proposed[c, rows] = worst[c, rows]
    h_min, min_proposed = 0.55, k

    pool = gu.bits_to_dev(pool_bits)
    host_pool = pool_bits.copy()
    d_bt_indptr, d_bt_pages = gu.i32(w.bt_indptr), gu.i32(w.bt_pages)
    d_ctx = gu.i32(w.ctx_len)
    status = torch.zeros(1, dtype=torch.int32, device=gu.DEV)
    ws_d = kap.Workspace(max_rows_per_item=G, max_batch=B)
    ws_v = kap.Workspace(max_rows_per_item=k * G, max_batch=B)
    q_indptr = gu.i32(np.arange(0, B * k + 1, k))
    n_q = np.full(B, k, dtype=np.int32)

    L = w.ctx_len.copy()
    force = {"lib": np.zeros(B, dtype=np.uint8), "ref": np.zeros(B, dtype=np.uint8)}
    acc_sum = {"lib": np.zeros(B, dtype=np.int64), "ref": np.zeros(B, dtype=np.int64)}
    prop_sum = np.zeros(B, dtype=np.int64)
    history = []
    for c in range(cycles):
        end = (L + k).astype(np.int32)
        comp = lambda fn, ff: fn(end, w.span_indptr, w.span_start, w.span_len, w.span_score,
                                 w.budget_tokens + k, w.n_sink, w.n_recent + k, ff, 1.0, w.bt_indptr, w.bt_pages)
        plan, ref_plan = comp(kap.compile_plan, force["lib"]), comp(orc.compile_plan, force["ref"])
        for key in ("plan_indptr", "plan_logical_pages", "plan_phys_pages", "plan_flags"):
            np.testing.assert_array_equal(plan[key], ref_plan[key], err_msg=f"cycle {c} {key}")
        for b in range(B):                                   # a fallen-back sequence lists every page
            if force["lib"][b]:
                assert plan["plan_flags"][b] & kap.PLAN_FULL
                assert plan["plan_indptr"][b + 1] - plan["plan_indptr"][b] == (end[b] + P - 1) // P
        ws_d.schedule(np.diff(plan["plan_indptr"]), None, Hq, Hkv)
        ws_v.schedule((end.astype(np.int64) + P - 1) // P, n_q, Hq, Hkv)
        args = (gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"]), gu.i32(plan["plan_logical_pages"]))
        for t in range(k):
            kap.append_kv(gu.bits_to_dev(k_new[c, t]), gu.bits_to_dev(v_new[c, t]), pool, d_bt_indptr, d_bt_pages,
                          d_ctx, advance=True, device_status=status)
            dq = gu.bits_to_dev(q_dec[c, t])
            out = torch.full_like(dq, float("nan"))
            kap.selected_decode_attn(dq, pool, *args, d_ctx, out, ws_d)
            for b in range(B):
                bt = w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b + 1]]
                L[b] = brute.append_kv(host_pool, bt, int(L[b]), k_new[c, t, b:b + 1], v_new[c, t, b:b + 1])
            # the plan was compiled for the end-of-cycle length: the oracle gets it trimmed to the
            # pages that exist at this step (the library masks them on the device)
            indptr, phys, logical = [0], [], []
            for b in range(B):
                lo, hi = ref_plan["plan_indptr"][b], ref_plan["plan_indptr"][b + 1]
                keep = ref_plan["plan_logical_pages"][lo:hi].astype(np.int64) * P < L[b]
                phys.append(ref_plan["plan_phys_pages"][lo:hi][keep])
                logical.append(ref_plan["plan_logical_pages"][lo:hi][keep])
                indptr.append(indptr[-1] + int(keep.sum()))
            ref, _, _, n_vis = orc.selected_decode_attn(q_dec[c, t], host_pool, indptr, np.concatenate(phys),
                                                        np.concatenate(logical), L)
            got = gu.dev_bf16_to_f64(out)
            assert_close(got, ref, what=f"cycle {c} step {t} decode")
            assert gu.normalised_error(got, ref) <= 2e-2
            for b in range(B):                               # full-context access really sees every token
                if force["ref"][b]:
                    assert np.all(n_vis[b] == L[b])
        dq = gu.bits_to_dev(q_ver[c])
        out_v = torch.full_like(dq, float("nan"))
        kap.verify_attn(dq, q_indptr, pool, d_bt_indptr, d_bt_pages, d_ctx, out_v, ws_v)
        n_pages = (L.astype(np.int64) + P - 1) // P
        v_indptr = np.concatenate([[0], np.cumsum(n_pages)]).astype(np.int32)
        v_pages = np.concatenate([w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b] + n_pages[b]] for b in range(B)])
        ref_v, _, _, _ = orc.verify_attn(q_ver[c], np.arange(0, B * k + 1, k), host_pool, v_indptr, v_pages, L)
        assert_close(gu.dev_bf16_to_f64(out_v), ref_v, what=f"cycle {c} verify")
        top3 = torch.zeros((B * (k + 1), 3), dtype=torch.int32, device=gu.DEV)
        acc = torch.zeros(B, dtype=torch.int32, device=gu.DEV)
        nxt = torch.zeros(B, dtype=torch.int32, device=gu.DEV)
        kap.top3_accept(torch.from_numpy(logits[c]).to(gu.DEV), gu.i32(row_indptr), gu.i32(proposed[c]), top3, acc,
                        nxt, ctx_len=d_ctx)
        torch.cuda.synchronize()
        ws_d.check(); ws_v.check()
        assert int(status.item()) == 0
        _, r_m, _ = brute.top3_accept(logits[c], row_indptr, proposed[c])
        m = acc.cpu().numpy()
        np.testing.assert_array_equal(m, r_m)
        L = (L - (k - r_m)).astype(np.int32)
        np.testing.assert_array_equal(d_ctx.cpu().numpy(), L)
        # the controller: costs in pages (attention only, no weight term), observed acceptance
        acc_sum["lib"] += m
        acc_sum["ref"] += r_m
        prop_sum += k
        pages = ((L + P - 1) // P).astype(np.float64)
        s = np.diff(plan["plan_indptr"]) / ((end + P - 1) // P)
        dec = kap.fallback_decide(acc_sum["lib"], prop_sum, s, pages, min_proposed=min_proposed, h_prior=1.0,
                                  h_min=h_min, s_max=0.9, plan_flags=plan["plan_flags"])
        ref_dec = brute.fallback_decide(acc_sum["ref"], prop_sum, min_proposed, 1.0, s, pages, 0.0, 0.0, h_min, 0.9,
                                        plan_flags=ref_plan["plan_flags"])
        np.testing.assert_array_equal(dec["force_full"], [r["force_full"] for r in ref_dec])
        np.testing.assert_array_equal(dec["reasons"], [r["reasons"] for r in ref_dec])
        # once fallen back a sequence stays there (s = 1 >= any h is itself a reason)
        force["lib"] = np.maximum(force["lib"], dec["force_full"])
        force["ref"] = np.maximum(force["ref"], np.array([r["force_full"] for r in ref_dec], dtype=np.uint8))
        history.append(force["lib"].copy())
    history = np.array(history)
    assert history[0].sum() == 0                             # nobody falls back after the good cycle
    assert history[-1, victim] == 1 and history[-1].sum() == 1
    first = int(np.argmax(history[:, victim]))
    assert collapse_from <= first < cycles - 1               # ... and at least one later cycle ran the identity plan
    ws_d.close(); ws_v.close()
