"""Several propose-k / verify cycles on the GPU with everything driven from the device-side
ctx_len, captured into ONE CUDA graph: k x (append the draft's K/V -> refresh the plan's recent
entries -> selected-KV decode), verification of the k rows over the full context, Top-3 acceptance
with its commit step (rejected drafts leave the context; their slots are overwritten in the next
cycle).  A host mirror (oracle attention, brute-force append and acceptance) replays the same
cycles; every attention output and the final lengths must agree.  The logits are synthetic and
unrelated to the attention outputs - there is no model here; they only decide how many drafts
survive each cycle."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from helpers import assert_close
from oracle import brute
from oracle import kap_oracle as orc
from paper_2607_24260_b200 import kap, synth
from test_gpu_growing_plan import _Device, _lists_from_tokens
from test_host_growing_plan import _grow, _tokens, _window

pytestmark = pytest.mark.gpu
P = 16


@pytest.mark.parametrize("seed,k,cycles", [(1, 4, 3), (3, 3, 4)])
def test_cycles_with_rollback_in_one_graph(seed, k, cycles):
    growth = k * cycles
    w = synth.growing_random(seed, batch=5, max_doc=700, growth=growth)
    B, Hq, Hkv, d, V = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, 97
    g = _grow(w, growth)
    fixed = []
    for b in range(B):
        lo, hi = g["plan_indptr"][b], g["plan_indptr"][b + 1] - g["tail_desc"][b, 0]
        fixed.append(_tokens(g["plan_logical_pages"][lo:hi], g["plan_token_masks"][lo:hi]))
    rng = synth.rng_for(seed, "generation-loop")
    q_bits, pool_bits = synth.host_qkv(w, seed, q_rows=cycles * 2 * k * B, q_std=4.0)
    q_dec = q_bits[:cycles * k * B].reshape(cycles, k, B, Hq, d)
    q_ver = q_bits[cycles * k * B:].reshape(cycles, B * k, Hq, d)        # a sequence's k rows contiguous
    k_new = synth.normal_bf16((cycles, k, B, Hkv, d), 0.5, rng)
    v_new = synth.normal_bf16((cycles, k, B, Hkv, d), 0.5, rng)
    logits = rng.standard_normal((cycles, B * (k + 1), V)).astype(np.float32)
    row_indptr = np.arange(0, B * (k + 1) + 1, k + 1, dtype=np.int32)
    # proposals: the row's best token most of the time, so that prefixes of every length occur
    best = logits.argmax(axis=2)
    proposed = np.where(rng.random(best.shape) < 0.7, best, (best + 1) % V).astype(np.int32)

    dev = _Device(w, g, pool_bits)
    d_qd, d_qv = gu.bits_to_dev(q_dec), gu.bits_to_dev(q_ver)
    d_k, d_v = gu.bits_to_dev(k_new), gu.bits_to_dev(v_new)
    d_logits = torch.from_numpy(logits).to(gu.DEV)
    d_prop, d_rows = gu.i32(proposed), gu.i32(row_indptr)
    out_d, out_v = torch.zeros_like(d_qd), torch.zeros_like(d_qv)
    top3 = torch.zeros((cycles, B * (k + 1), 3), dtype=torch.int32, device=gu.DEV)
    acc = torch.zeros((cycles, B), dtype=torch.int32, device=gu.DEV)
    nxt = torch.zeros((cycles, B), dtype=torch.int32, device=gu.DEV)
    status = torch.zeros(1, dtype=torch.int32, device=gu.DEV)
    # verification schedule: sized for the longest context that can occur, k rows per sequence
    n_q = np.full(B, k, dtype=np.int32)
    q_indptr = gu.i32(np.arange(0, B * k + 1, k))
    ws_v = kap.Workspace(max_rows_per_item=k * (Hq // Hkv), max_batch=B)
    ws_v.schedule((w.ctx_len.astype(np.int64) + growth + P - 1) // P, n_q, Hq, Hkv)

    def run():
        for c in range(cycles):
            for t in range(k):
                kap.append_kv(d_k[c, t], d_v[c, t], dev.pool, dev.bt_indptr, dev.bt_pages, dev.ctx,
                              advance=True, device_status=status)
                dev.refresh()
                dev.decode(d_qd[c, t], out_d[c, t])
            kap.verify_attn(d_qv[c], q_indptr, dev.pool, dev.bt_indptr, dev.bt_pages, dev.ctx, out_v[c], ws_v)
            kap.top3_accept(d_logits[c], d_rows, d_prop[c], top3[c], acc[c], nxt[c], ctx_len=dev.ctx)

    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        run()                                               # eager pass: warm-up and comparison
    stream.synchronize()
    eager = (gu.dev_bf16_to_f64(out_d), gu.dev_bf16_to_f64(out_v), dev.ctx.cpu().numpy().copy())
    dev.pool.copy_(gu.bits_to_dev(pool_bits))
    dev.ctx.copy_(gu.i32(w.ctx_len))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        run()
    dev.pool.copy_(gu.bits_to_dev(pool_bits))
    dev.ctx.copy_(gu.i32(w.ctx_len))
    out_d.zero_(); out_v.zero_()
    graph.replay()
    torch.cuda.synchronize()
    dev.ws.check(); ws_v.check()
    assert int(status.item()) == 0
    got_d, got_v = gu.dev_bf16_to_f64(out_d), gu.dev_bf16_to_f64(out_v)
    np.testing.assert_array_equal(got_d, eager[0])
    np.testing.assert_array_equal(got_v, eager[1])

    # ---- host mirror
    host_pool = pool_bits.copy()
    L = w.ctx_len.copy()
    n_rejected = 0
    for c in range(cycles):
        for t in range(k):
            for b in range(B):
                bt = w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b + 1]]
                L[b] = brute.append_kv(host_pool, bt, int(L[b]), k_new[c, t, b:b + 1], v_new[c, t, b:b + 1])
            sets = [fixed[b] | _window(g["tail_desc"][b], int(L[b])) for b in range(B)]
            indptr, phys, logical, masks = _lists_from_tokens(sets, w)
            ref, _, _, _ = orc.selected_decode_attn(q_dec[c, t], host_pool, indptr, phys, logical, L,
                                                    plan_token_masks=masks)
            assert_close(got_d[c, t], ref, what=f"cycle {c} step {t} decode")
            assert gu.normalised_error(got_d[c, t], ref) <= 2e-2
        n_pages = (L.astype(np.int64) + P - 1) // P
        v_indptr = np.concatenate([[0], np.cumsum(n_pages)]).astype(np.int32)
        v_pages = np.concatenate([w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b] + n_pages[b]] for b in range(B)])
        ref, _, _, _ = orc.verify_attn(q_ver[c], np.arange(0, B * k + 1, k), host_pool, v_indptr, v_pages, L)
        assert_close(got_v[c], ref, what=f"cycle {c} verify")
        assert gu.normalised_error(got_v[c], ref) <= 2e-2
        r_top3, r_m, r_next = brute.top3_accept(logits[c], row_indptr, proposed[c])
        np.testing.assert_array_equal(acc[c].cpu().numpy(), r_m)
        np.testing.assert_array_equal(nxt[c].cpu().numpy(), r_next)
        L = (L - (k - r_m)).astype(np.int32)                 # commit: rejected drafts leave the context
        n_rejected += int((k - r_m).sum())
    assert n_rejected > 0                                   # the roll-back really happened
    np.testing.assert_array_equal(dev.ctx.cpu().numpy(), L)
    np.testing.assert_array_equal(eager[2], L)
    dev.ws.close(); ws_v.close()
