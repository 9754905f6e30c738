"""Multi-step proposal loop on the GPU: k steps of "append the new token's K/V -> selected-KV decode
attention", captured into ONE CUDA graph, on a plan compiled once for the end-of-cycle length.
Every step's output is compared with the oracle run on a host pool that received the same appends
(slot mapping stated in oracle/brute.py) with that step's context length."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from helpers import assert_close
from oracle import brute
from oracle import kap_oracle as orc
from paper_2607_24260_b200 import kap, synth

pytestmark = pytest.mark.gpu


def _cycle_case(seed, k_steps, lens):
    """a batch whose block tables already hold pages for k_steps more tokens"""
    B = len(lens)
    w = synth.config2(seed, batch=B, L=max(lens), layers=1)
    w.ctx_len = np.asarray(lens, dtype=np.int32)
    end = w.ctx_len + k_steps
    w.bt_indptr, w.bt_pages, w.num_pool_pages = synth.block_tables(end, "shuffled", seed, "append", spare_pages=3)
    # spans were drawn for max(lens); clip happens in the compiler
    return w, end


@pytest.mark.parametrize("k_steps,lens", [(4, (1000, 2047, 2048, 333)), (8, (4090, 15, 16)), (6, (777,))])
def test_append_and_decode_loop_in_one_graph(k_steps, lens):
    w, end = _cycle_case(3, k_steps, lens)
    B, Hq, Hkv, d = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim
    rng = synth.rng_for(3, "append-loop", k_steps)
    q_bits, pool_bits = synth.host_qkv(w, 3, q_rows=k_steps * B)
    q_bits = q_bits.reshape(k_steps, B, Hq, d)
    k_new = synth.normal_bf16((k_steps, B, Hkv, d), 0.5, rng)
    v_new = synth.normal_bf16((k_steps, B, Hkv, d), 0.5, rng)
    # plan for the end-of-cycle length: recent window widened by k_steps, budget too
    plan = kap.compile_plan(end, w.span_indptr, w.span_start, w.span_len, w.span_score,
                            w.budget_tokens + k_steps, w.n_sink, w.n_recent + k_steps, None, 1.0,
                            w.bt_indptr, w.bt_pages)
    pool = gu.bits_to_dev(pool_bits)
    d_q, d_k, d_v = gu.bits_to_dev(q_bits), gu.bits_to_dev(k_new), gu.bits_to_dev(v_new)
    d_ctx = gu.i32(w.ctx_len)
    d_out = torch.zeros_like(d_q)
    status = torch.zeros(1, dtype=torch.int32, device=gu.DEV)
    args = (gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"]), gu.i32(plan["plan_logical_pages"]))
    d_bt_indptr, d_bt_pages = gu.i32(w.bt_indptr), gu.i32(w.bt_pages)
    ws = kap.Workspace(max_rows_per_item=Hq // Hkv, max_batch=B)
    ws.schedule(np.diff(plan["plan_indptr"]), None, Hq, Hkv)

    def cycle():
        for t in range(k_steps):
            kap.append_kv(d_k[t], d_v[t], pool, d_bt_indptr, d_bt_pages, d_ctx, advance=True, device_status=status)
            kap.selected_decode_attn(d_q[t], pool, *args, d_ctx, d_out[t], ws)

    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        cycle()                                   # eager warm-up (also proves the non-graph path)
    stream.synchronize()
    eager = gu.dev_bf16_to_f64(d_out)
    # reset state, capture, replay
    pool.copy_(gu.bits_to_dev(pool_bits))
    d_ctx.copy_(gu.i32(w.ctx_len))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        pass
    with torch.cuda.graph(graph, stream=stream):
        cycle()
    pool.copy_(gu.bits_to_dev(pool_bits))
    d_ctx.copy_(gu.i32(w.ctx_len))
    d_out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    ws.check()
    assert int(status.item()) == 0
    np.testing.assert_array_equal(d_ctx.cpu().numpy(), end)
    got = gu.dev_bf16_to_f64(d_out)
    np.testing.assert_array_equal(got, eager)    # graph replay == eager, bit for bit

    # oracle: same appends on the host, plan trimmed to the pages that exist at each step
    host_pool = pool_bits.copy()
    L = w.ctx_len.copy()
    for t in range(k_steps):
        for b in range(B):
            bt = w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b + 1]]
            L[b] = brute.append_kv(host_pool, bt, int(L[b]), k_new[t, b:b + 1], v_new[t, b:b + 1])
        indptr, phys, logical = [0], [], []
        for b in range(B):
            lo, hi = plan["plan_indptr"][b], plan["plan_indptr"][b + 1]
            keep = plan["plan_logical_pages"][lo:hi].astype(np.int64) * 16 < L[b]
            phys.append(plan["plan_phys_pages"][lo:hi][keep])
            logical.append(plan["plan_logical_pages"][lo:hi][keep])
            indptr.append(indptr[-1] + int(keep.sum()))
        ref, _, _, _ = orc.selected_decode_attn(q_bits[t], host_pool, indptr, np.concatenate(phys),
                                                np.concatenate(logical), L)
        assert_close(got[t], ref, what=f"step {t}")
        assert gu.normalised_error(got[t], ref) <= 2e-2
    # the device pool equals the host pool wherever tokens were appended
    np.testing.assert_array_equal(gu.dev_to_bits(pool), host_pool)
    ws.close()


def test_append_reports_missing_page():
    w, end = _cycle_case(4, 2, (31,))
    q_bits, pool_bits = synth.host_qkv(w, 4, q_rows=1)
    pool = gu.bits_to_dev(pool_bits)
    knew = gu.bits_to_dev(synth.normal_bf16((1, 8, 128), 0.5, synth.rng_for(4, "x")))
    status = torch.zeros(1, dtype=torch.int32, device=gu.DEV)
    short_bt = gu.i32(w.bt_pages[:2])                       # 2 pages = 32 tokens
    ctx = gu.i32([32])                                      # position 32 needs a third page
    kap.append_kv(knew, knew, pool, gu.i32([0, 2]), short_bt, ctx, advance=False, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1 << kap.ERR_DEVICE_INDEX
    np.testing.assert_array_equal(gu.dev_to_bits(pool), pool_bits)     # nothing was written


def test_bulk_append_then_decode_sees_every_new_token():
    """Several tokens per sequence appended by one call, the proposal-path attention enqueued right
    behind it on the same stream (programmatic dependent launch on): the attention must see all
    of them - its early page loads may not run ahead of the append."""
    w, end = _cycle_case(5, 7, (1000, 2040, 333))
    B, Hq, Hkv, d = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim
    rng = synth.rng_for(5, "bulk-append")
    n_new = np.array([7, 3, 5], dtype=np.int32)
    indptr = np.concatenate([[0], np.cumsum(n_new)]).astype(np.int32)
    q_bits, pool_bits = synth.host_qkv(w, 5, q_rows=B, q_std=4.0)
    k_new = synth.normal_bf16((int(n_new.sum()), Hkv, d), 0.5, rng)
    v_new = synth.normal_bf16((int(n_new.sum()), Hkv, d), 0.5, rng)
    final = (w.ctx_len + n_new).astype(np.int32)
    plan = kap.compile_plan(final, w.span_indptr, w.span_start, w.span_len, w.span_score,
                            w.budget_tokens + 7, w.n_sink, w.n_recent + 7, None, 1.0, w.bt_indptr, w.bt_pages)
    pool = gu.bits_to_dev(pool_bits)
    d_ctx = gu.i32(w.ctx_len)
    d_q = gu.bits_to_dev(q_bits)
    d_out = torch.zeros_like(d_q)
    ws = kap.Workspace(max_rows_per_item=Hq // Hkv, max_batch=B)
    ws.schedule(np.diff(plan["plan_indptr"]), None, Hq, Hkv)
    args = (gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"]), gu.i32(plan["plan_logical_pages"]))
    d_k, d_v, d_ind = gu.bits_to_dev(k_new), gu.bits_to_dev(v_new), gu.i32(indptr)
    d_bt_indptr, d_bt_pages = gu.i32(w.bt_indptr), gu.i32(w.bt_pages)
    for _ in range(3):                                      # repeat: a race would be intermittent
        pool.copy_(gu.bits_to_dev(pool_bits))
        d_ctx.copy_(gu.i32(w.ctx_len))
        kap.selected_decode_attn(d_q, pool, *args, d_ctx, d_out, ws)          # keeps the GPU busy in front
        kap.append_kv(d_k, d_v, pool, d_bt_indptr, d_bt_pages, d_ctx, new_indptr=d_ind, advance=True)
        kap.selected_decode_attn(d_q, pool, *args, d_ctx, d_out, ws)
        torch.cuda.synchronize()
        ws.check()
        host_pool = pool_bits.copy()
        for b in range(B):
            bt = w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b + 1]]
            brute.append_kv(host_pool, bt, int(w.ctx_len[b]), k_new[indptr[b]:indptr[b + 1]], v_new[indptr[b]:indptr[b + 1]])
        ref, _, _, _ = orc.selected_decode_attn(q_bits, host_pool, plan["plan_indptr"], plan["plan_phys_pages"],
                                                plan["plan_logical_pages"], final)
        assert_close(gu.dev_bf16_to_f64(d_out), ref, what="decode after a bulk append")
        np.testing.assert_array_equal(d_ctx.cpu().numpy(), final)
    ws.close()


def test_bulk_append_mark_belongs_to_its_stream():
    """Two streams in one process.  Stream A: a busy attention kernel, a several-token append, then
    the attention call that must see every new token.  Between A's append and A's attention the
    host issues an attention call on stream B (another workspace, another batch).  B's launch must
    not use up the "loads wait for the append" mark that belongs to A: A's output still matches
    the oracle, every repetition."""
    w, end = _cycle_case(6, 7, (1500, 2040, 900))
    B, Hq, Hkv, d = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim
    rng = synth.rng_for(6, "two-streams")
    n_new = np.array([6, 7, 4], dtype=np.int32)
    indptr = np.concatenate([[0], np.cumsum(n_new)]).astype(np.int32)
    q_bits, pool_bits = synth.host_qkv(w, 6, q_rows=B, q_std=4.0)
    k_new = synth.normal_bf16((int(n_new.sum()), Hkv, d), 0.5, rng)
    v_new = synth.normal_bf16((int(n_new.sum()), Hkv, d), 0.5, rng)
    final = (w.ctx_len + n_new).astype(np.int32)
    plan = kap.compile_plan(final, w.span_indptr, w.span_start, w.span_len, w.span_score,
                            w.budget_tokens + 7, w.n_sink, w.n_recent + 7, None, 1.0, w.bt_indptr, w.bt_pages)
    pool = gu.bits_to_dev(pool_bits)
    d_ctx, d_q = gu.i32(w.ctx_len), gu.bits_to_dev(q_bits)
    d_out = torch.zeros_like(d_q)
    ws_a = kap.Workspace(max_rows_per_item=Hq // Hkv, max_batch=B)
    ws_a.schedule(np.diff(plan["plan_indptr"]), None, Hq, Hkv)
    args = (gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"]), gu.i32(plan["plan_logical_pages"]))
    d_k, d_v, d_ind = gu.bits_to_dev(k_new), gu.bits_to_dev(v_new), gu.i32(indptr)
    d_bt_indptr, d_bt_pages = gu.i32(w.bt_indptr), gu.i32(w.bt_pages)
    # stream B's own, unrelated work
    wb = synth.config2(7, batch=2, L=3000, layers=1)
    qb_bits, poolb_bits = synth.host_qkv(wb, 7, q_rows=2)
    planb = kap.compile_workload(wb)
    poolb, d_qb = gu.bits_to_dev(poolb_bits), gu.bits_to_dev(qb_bits)
    d_outb = torch.zeros_like(d_qb)
    ws_b = kap.Workspace(max_rows_per_item=Hq // Hkv, max_batch=2)
    ws_b.schedule(np.diff(planb["plan_indptr"]), None, Hq, Hkv)
    argsb = (gu.i32(planb["plan_indptr"]), gu.i32(planb["plan_phys_pages"]), gu.i32(planb["plan_logical_pages"]),
             gu.i32(wb.ctx_len))
    ref_b, _ = gu.oracle_decode(qb_bits, poolb_bits, planb, wb.ctx_len)
    host_pool = pool_bits.copy()
    for b in range(B):
        bt = w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b + 1]]
        brute.append_kv(host_pool, bt, int(w.ctx_len[b]), k_new[indptr[b]:indptr[b + 1]], v_new[indptr[b]:indptr[b + 1]])
    ref_a, _, _, _ = orc.selected_decode_attn(q_bits, host_pool, plan["plan_indptr"], plan["plan_phys_pages"],
                                              plan["plan_logical_pages"], final)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(4):                                      # repeat: a race would be intermittent
        pool.copy_(gu.bits_to_dev(pool_bits))
        d_ctx.copy_(gu.i32(w.ctx_len))
        torch.cuda.synchronize()
        kap.selected_decode_attn(d_q, pool, *args, d_ctx, d_out, ws_a, stream=sa)      # keeps A busy in front
        kap.append_kv(d_k, d_v, pool, d_bt_indptr, d_bt_pages, d_ctx, new_indptr=d_ind, advance=True, stream=sa)
        kap.selected_decode_attn(d_qb, poolb, *argsb, d_outb, ws_b, stream=sb)         # the intruder
        kap.selected_decode_attn(d_q, pool, *args, d_ctx, d_out, ws_a, stream=sa)
        torch.cuda.synchronize()
        ws_a.check()
        ws_b.check()
        assert_close(gu.dev_bf16_to_f64(d_out), ref_a, what="stream A decode after its bulk append")
        assert_close(gu.dev_bf16_to_f64(d_outb), ref_b, what="stream B decode")
        np.testing.assert_array_equal(d_ctx.cpu().numpy(), final)
    ws_a.close()
    ws_b.close()
