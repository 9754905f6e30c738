"""kap_verify_attn through the tcgen05 kernel (kap_set_verify_kernel(1)): the same parity bar as the
default kernel - element by element against the fp64 oracle - on shapes that reach its corners:
every group size whose rows fit (1 .. 32 rows per KV head), ragged lengths with partial last pages
and contexts shorter than the row count allows, lists shorter than one batch of four pages, one
CTA per list (no merge pass) and many, the token-major pool layout, reuse under a CUDA graph, and
the fallback to the split kernel when a sequence has more than 32 rows."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from helpers import assert_close
from paper_2607_24260_b200 import kap, synth

pytestmark = pytest.mark.gpu
NORM_TOL = 2e-2


@pytest.fixture(autouse=True)
def tcgen05_kernel():
    kap.set_verify_kernel(1)
    yield
    kap.set_verify_kernel(0)


def _check(w, seed, what, Hq=32, Hkv=8, q_std=1.0, **kw):
    q_bits, pool_bits = synth.host_qkv(w, seed, q_std=q_std)
    pool = gu.bits_to_dev(pool_bits)
    out, lse = gu.run_verify(q_bits, w.n_q, pool, w.bt_indptr, w.bt_pages, w.ctx_len, Hq=Hq, Hkv=Hkv, **kw)
    r_out, r_lse = gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len)
    assert not np.isnan(out).any(), what
    assert_close(out, r_out, what=f"{what} out")
    assert gu.normalised_error(out, r_out) <= NORM_TOL, what
    assert_close(lse, r_lse, atol=1e-2, rtol=1e-3, what=f"{what} lse")


def _ragged(seed, batch, max_len, nq):
    w = synth.tiny_random(seed, batch=batch, max_len=max_len, max_spans=6)
    rng = synth.rng_for(seed, "tcgen05-nq")
    w.n_q = np.minimum(rng.choice(np.asarray(nq), size=batch), w.ctx_len).astype(np.int32)
    return w


def test_config1():
    _check(synth.CONFIGS["c1"](0), 0, "c1")


@pytest.mark.parametrize("seed,batch,max_len,nq", [
    (1, 5, 700, (1, 2, 3, 4)), (2, 7, 3000, (4, 5, 8)), (3, 3, 6000, (7, 8)), (4, 9, 60, (1, 4, 8)),
])
def test_ragged_batches(seed, batch, max_len, nq):
    _check(_ragged(seed, batch, max_len, nq), seed, f"ragged {seed}")


@pytest.mark.parametrize("L,nq", [(1, 1), (3, 3), (16, 8), (17, 8), (63, 4), (64, 8), (65, 5), (129, 8)])
def test_tiny_contexts(L, nq):
    """Lists of one to nine pages: shorter than, equal to and just past one batch of four; n_q == L."""
    w = synth.tiny_random(11, batch=1, max_len=8)
    w.ctx_len = np.array([L], dtype=np.int32)
    w.n_q = np.array([nq], dtype=np.int32)
    w.bt_indptr, w.bt_pages, w.num_pool_pages = synth.block_tables([L], "shuffled", 11, "tinyctx", spare_pages=2)
    _check(w, L, f"L={L} n_q={nq}")


@pytest.mark.parametrize("Hq,Hkv,nq", [(8, 8, 8), (16, 8, 8), (32, 8, 8), (64, 8, 4), (32, 4, 4), (32, 2, 2)])
def test_group_sizes(Hq, Hkv, nq):
    """G = 1, 2, 4, 8, 8, 16 with row counts up to the kernel's 32."""
    w = _ragged(21, 3, 900, (nq,))
    w.num_q_heads, w.num_kv_heads = Hq, Hkv
    _check(w, 21, f"heads {Hq}/{Hkv}", Hq=Hq, Hkv=Hkv)


def test_peaky_scores_force_rescales():
    """Q x 8: the running maximum moves by more than the lazy threshold many times."""
    w = synth.config2(5, batch=2, L=6000 - 3, layers=1)
    w.n_q[:] = 8
    _check(w, 5, "peaky", q_std=8.0)


def test_more_than_32_rows_fall_back_to_the_split_kernel():
    w = _ragged(9, 3, 2000, (8, 16, 12))
    assert int(w.n_q.max()) * 4 > 32
    _check(w, 9, "fallback")


def test_token_major_pool():
    w = _ragged(12, 4, 3000, (4, 8))
    q_bits, pool_bits = synth.host_qkv(w, 12)
    nhd = np.ascontiguousarray(pool_bits.reshape(pool_bits.shape[0], 2, 8, 16, 128).transpose(0, 1, 3, 2, 4))
    out, lse = gu.run_verify(q_bits, w.n_q, gu.bits_to_dev(nhd), w.bt_indptr, w.bt_pages, w.ctx_len, kv_layout=kap.KV_NHD)
    r_out, r_lse = gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len)
    assert_close(out, r_out, what="nhd out")
    assert_close(lse, r_lse, atol=1e-2, rtol=1e-3, what="nhd lse")


def test_graph_replays_are_bit_identical():
    w = synth.config2(3, batch=2, L=8192, layers=1)
    w.n_q[:] = 8
    q_bits, pool_bits = synth.host_qkv(w, 3)
    pool, q = gu.bits_to_dev(pool_bits), gu.bits_to_dev(q_bits)
    ws = kap.Workspace(max_rows_per_item=32, max_batch=2)
    info = ws.schedule((w.ctx_len.astype(np.int64) + 15) // 16, w.n_q, 32, 8)
    assert info["ctas_per_wave"] == 2 * torch.cuda.get_device_properties(0).multi_processor_count
    out = torch.zeros_like(q)
    args = (q, gu.i32(w.q_indptr), pool, gu.i32(w.bt_indptr), gu.i32(w.bt_pages), gu.i32(w.ctx_len), out, ws)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        kap.verify_attn(*args)
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        for _ in range(3):
            kap.verify_attn(*args)
    results = []
    for _ in range(3):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        results.append(out.view(torch.int16).cpu().numpy().copy())
    ws.check()
    ws.close()
    assert np.array_equal(results[0], results[1]) and np.array_equal(results[0], results[2])
    r_out, _ = gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len)
    assert_close(gu.dev_bf16_to_f64(out), r_out, what="graph")
