"""Growing plans on the GPU: a plan compiled once, kept valid by kap_refresh_recent while the
context grows token by token ("append K/V -> refresh the recent entries -> selected-KV decode
attention", all steps in ONE CUDA graph).  Every step is compared with the oracle's masked
attention over the token set that the oracle's Algorithm 1 compiles afresh at that step's length
(for sequences flagged as moving with the length: over fixed part + window)."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from helpers import assert_close
from oracle import brute
from oracle import kap_oracle as orc
from paper_2607_24260_b200 import kap, synth
from test_host_growing_plan import _fresh, _grow, _tokens, _window

pytestmark = pytest.mark.gpu
P = 16


def _lists_from_tokens(token_sets, w):
    """oracle inputs (indptr, phys, logical, masks) listing exactly the given tokens"""
    indptr, phys, logical, masks = [0], [], [], []
    for b, S in enumerate(token_sets):
        bt = w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b + 1]]
        pages = sorted({t // P for t in S})
        logical += pages
        phys += [int(bt[p]) for p in pages]
        masks += [sum(1 << (t - p * P) for t in S if t // P == p) for p in pages]
        indptr.append(len(logical))
    return (np.asarray(indptr, np.int32), np.asarray(phys, np.int32), np.asarray(logical, np.int32),
            np.asarray(masks, np.uint16))


class _Device:
    def __init__(self, w, g, pool_bits):
        self.pool = gu.bits_to_dev(pool_bits)
        self.indptr = gu.i32(g["plan_indptr"])
        self.phys = gu.i32(g["plan_phys_pages"])
        self.logical = gu.i32(g["plan_logical_pages"])
        self.masks = gu.u16(g["plan_token_masks"])
        self.tail = gu.i32(g["tail_desc"])
        self.bt_indptr, self.bt_pages = gu.i32(w.bt_indptr), gu.i32(w.bt_pages)
        self.ctx = gu.i32(w.ctx_len)
        self.ws = kap.Workspace(max_rows_per_item=w.num_q_heads // w.num_kv_heads, max_batch=w.batch)
        self.ws.schedule(np.diff(g["plan_indptr"]), None, w.num_q_heads, w.num_kv_heads)
        self.n_pool = w.num_pool_pages

    def refresh(self):
        kap.refresh_recent(self.indptr, self.logical, self.phys, self.masks, self.tail, self.bt_indptr,
                           self.bt_pages, self.ctx, self.n_pool, ws=self.ws)

    def decode(self, q, out):
        kap.selected_decode_attn(q, self.pool, self.indptr, self.phys, self.logical, self.ctx, out,
                                 self.ws, plan_token_masks=self.masks)

    def listed_tokens(self, b):
        """(list of tokens with repeats) that the device arrays of sequence b list now"""
        ip = self.indptr.cpu().numpy()
        lg = self.logical.cpu().numpy()[ip[b]:ip[b + 1]]
        mk = self.masks.cpu().numpy().view(np.uint16)[ip[b]:ip[b + 1]]
        return [int(p) * P + t for p, m in zip(lg, mk) for t in range(P) if (int(m) >> t) & 1]


@pytest.mark.parametrize("seed,steps", [(1, 40), (3, 24), (4, 17)])
def test_growth_loop_in_one_graph(seed, steps):
    w = synth.growing_random(seed, batch=5, max_doc=900, growth=steps)
    B, Hq, Hkv, d = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim
    g = _grow(w, steps)
    fixed = []
    for b in range(B):
        lo, hi = g["plan_indptr"][b], g["plan_indptr"][b + 1] - g["tail_desc"][b, 0]
        fixed.append(_tokens(g["plan_logical_pages"][lo:hi], g["plan_token_masks"][lo:hi]))
    moves = (g["plan_flags"] & kap.PLAN_MOVES_WITH_LENGTH) != 0
    assert moves.any() and not moves.all()
    rng = synth.rng_for(seed, "growth-loop")
    # two attention calls per step (two "layers" on the same pool): the first launch after a
    # refresh is an ordinary one, the second overlaps it through programmatic dependent launch
    q_bits, pool_bits = synth.host_qkv(w, seed, q_rows=(steps + 1) * 2 * B, q_std=4.0)
    q_bits = q_bits.reshape(steps + 1, 2, B, Hq, d)
    k_new = synth.normal_bf16((steps, B, Hkv, d), 0.5, rng)
    v_new = synth.normal_bf16((steps, B, Hkv, d), 0.5, rng)
    dev = _Device(w, g, pool_bits)
    d_q, d_k, d_v = gu.bits_to_dev(q_bits), gu.bits_to_dev(k_new), gu.bits_to_dev(v_new)
    d_out = torch.zeros_like(d_q)
    status = torch.zeros(1, dtype=torch.int32, device=gu.DEV)

    def run():
        dev.refresh()                                       # step 0: the length the plan was compiled at
        dev.decode(d_q[0, 0], d_out[0, 0])
        dev.decode(d_q[0, 1], d_out[0, 1])
        for t in range(steps):
            kap.append_kv(d_k[t], d_v[t], dev.pool, dev.bt_indptr, dev.bt_pages, dev.ctx, advance=True,
                          device_status=status)
            dev.refresh()
            dev.decode(d_q[t + 1, 0], d_out[t + 1, 0])
            dev.decode(d_q[t + 1, 1], d_out[t + 1, 1])

    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        run()
    stream.synchronize()
    eager = gu.dev_bf16_to_f64(d_out)
    dev.pool.copy_(gu.bits_to_dev(pool_bits))
    dev.ctx.copy_(gu.i32(w.ctx_len))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        run()
    dev.pool.copy_(gu.bits_to_dev(pool_bits))
    dev.ctx.copy_(gu.i32(w.ctx_len))
    d_out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    dev.ws.check()
    assert int(status.item()) == 0
    got = gu.dev_bf16_to_f64(d_out)
    np.testing.assert_array_equal(got, eager)               # graph replay == eager, bit for bit

    host_pool = pool_bits.copy()
    L = w.ctx_len.copy()
    for t in range(steps + 1):
        if t > 0:
            for b in range(B):
                bt = w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b + 1]]
                L[b] = brute.append_kv(host_pool, bt, int(L[b]), k_new[t - 1, b:b + 1], v_new[t - 1, b:b + 1])
        sets = []
        for b in range(B):
            S = fixed[b] | _window(g["tail_desc"][b], int(L[b]))
            if not moves[b]:
                assert S == _fresh(w, b, int(L[b]))[0], (t, b)      # == Algorithm 1 at this length
            sets.append(S)
        indptr, phys, logical, masks = _lists_from_tokens(sets, w)
        for layer in range(2):
            ref, _, _, _ = orc.selected_decode_attn(q_bits[t, layer], host_pool, indptr, phys, logical, L,
                                                    plan_token_masks=masks)
            assert_close(got[t, layer], ref, what=f"step {t} call {layer}")
            assert gu.normalised_error(got[t, layer], ref) <= 2e-2
    # after the last step the device arrays list exactly that token set, no token twice
    for b in range(B):
        listed = dev.listed_tokens(b)
        assert len(listed) == len(set(listed))
        assert set(listed) == sets[b]
    np.testing.assert_array_equal(dev.ctx.cpu().numpy(), w.ctx_len + steps)
    dev.ws.close()


def test_refresh_reports_outgrown_reservation_and_missing_pages():
    w = synth.growing_random(5, batch=3, growth=64, overlap_every=0)
    w.force_full[:] = [1, 0, 0]
    w.n_recent[2] = 30
    w.ctx_len[2] = max(int(w.ctx_len[2]), 64)
    g = _grow(w, 8)                                         # the full plan may grow by 8 tokens only
    _, pool_bits = synth.host_qkv(w, 5, q_rows=3)
    dev = _Device(w, g, pool_bits)
    dev.refresh()
    torch.cuda.synchronize()
    dev.ws.check()                                          # fine at the compiled length
    dev.ctx.copy_(gu.i32(w.ctx_len + np.array([8, 40, 40], np.int32)))
    dev.refresh()
    dev.ws.check()                                          # 8 more tokens (and any growth of the others) fit
    dev.ctx.copy_(gu.i32(w.ctx_len + np.array([64, 0, 0], np.int32)))
    dev.refresh()
    with pytest.raises(kap.KapError) as e:
        dev.ws.check()
    assert e.value.code == kap.ERR_DEVICE_INDEX
    # a window page without a valid block-table entry: reported, that entry stays empty
    dev.ctx.copy_(gu.i32(w.ctx_len))
    L2 = int(w.ctx_len[2])
    first_window_page = (L2 - 30) // P                      # n_recent[2] = 30: the window spans >= 2 pages
    assert first_window_page < (L2 - 1) // P
    holes = w.bt_pages.copy()
    holes[w.bt_indptr[2] + first_window_page] = -1
    status = torch.zeros(1, dtype=torch.int32, device=gu.DEV)
    kap.refresh_recent(dev.indptr, dev.logical, dev.phys, dev.masks, dev.tail, dev.bt_indptr, gu.i32(holes),
                       dev.ctx, dev.n_pool, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1 << kap.ERR_DEVICE_INDEX
    lst = dev.listed_tokens(2)
    assert (L2 - 1) in lst and not any(t // P == first_window_page and t >= L2 - 30 for t in lst)
    # the page of the last token itself is missing: reported
    short = w.bt_indptr.copy()
    short[3] = short[2] + (L2 - 1) // P
    status.zero_()
    kap.refresh_recent(dev.indptr, dev.logical, dev.phys, dev.masks, dev.tail, gu.i32(short), dev.bt_pages,
                       dev.ctx, dev.n_pool, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1 << kap.ERR_DEVICE_INDEX
    dev.ws.close()
