"""The token-major pool layout [page][2][P][Hkv][d] on the GPU: the same values as the head-major
pool, permuted on the host; results must equal the head-major run bit for bit and match the oracle
(which is layout-free: it is given the head-major bits)."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from oracle import brute
from paper_2607_24260_b200 import kap, synth
from test_gpu_parity import _check_pair, _decode_rows, _ragged_workload, _workload_case

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed,batch,max_len,nq", [(1, 5, 700, (1, 2, 4)), (2, 6, 3000, (4, 5, 8)), (3, 3, 6000, (9, 16))])
def test_nhd_equals_hnd_and_the_oracle(seed, batch, max_len, nq):
    w = _ragged_workload(seed, batch, max_len, nq)
    q_bits, pool_bits, pool = _workload_case(w, seed)
    pool_nhd = gu.bits_to_dev(gu.to_nhd(pool_bits))
    plan = kap.compile_workload(w)
    qd = _decode_rows(w, q_bits)
    masks = plan["plan_token_masks"]
    for chunk in (0, 2):
        hnd = gu.run_decode(qd, pool, plan, w.ctx_len, max_chunk_pages=chunk, masks=masks)
        nhd = gu.run_decode(qd, pool_nhd, plan, w.ctx_len, max_chunk_pages=chunk, masks=masks,
                            kv_layout=kap.KV_NHD)
        np.testing.assert_array_equal(nhd[0], hnd[0])
        np.testing.assert_array_equal(nhd[1], hnd[1])
        _check_pair(nhd, gu.oracle_decode(qd, pool_bits, plan, w.ctx_len, masks=masks), f"nhd decode {seed}")
        hnd = gu.run_verify(q_bits, w.n_q, pool, w.bt_indptr, w.bt_pages, w.ctx_len, max_chunk_pages=chunk)
        nhd = gu.run_verify(q_bits, w.n_q, pool_nhd, w.bt_indptr, w.bt_pages, w.ctx_len,
                            max_chunk_pages=chunk, kv_layout=kap.KV_NHD)
        np.testing.assert_array_equal(nhd[0], hnd[0])
        np.testing.assert_array_equal(nhd[1], hnd[1])
    _check_pair(nhd, gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len),
                f"nhd verify {seed}")


@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (16, 2), (16, 1)])
def test_nhd_group_sizes(Hq, Hkv):
    w = _ragged_workload(21, 3, 900, (1, 3, 4))
    w.num_q_heads, w.num_kv_heads = Hq, Hkv
    q_bits, pool_bits, pool = _workload_case(w, 21)
    pool_nhd = gu.bits_to_dev(gu.to_nhd(pool_bits))
    plan = kap.compile_workload(w)
    qd = _decode_rows(w, q_bits)
    _check_pair(gu.run_decode(qd, pool_nhd, plan, w.ctx_len, Hq, Hkv, kv_layout=kap.KV_NHD),
                gu.oracle_decode(qd, pool_bits, plan, w.ctx_len), f"nhd G={Hq // Hkv} decode")
    _check_pair(gu.run_verify(q_bits, w.n_q, pool_nhd, w.bt_indptr, w.bt_pages, w.ctx_len, Hq, Hkv,
                              kv_layout=kap.KV_NHD),
                gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len),
                f"nhd G={Hq // Hkv} verify")


def test_nhd_append_writes_the_token_major_slots():
    w = _ragged_workload(4, 3, 500, (1,))
    end = w.ctx_len + 5
    w.bt_indptr, w.bt_pages, w.num_pool_pages = synth.block_tables(end, "shuffled", 4, "nhd-append", spare_pages=2)
    _, pool_bits = synth.host_qkv(w, 4, q_rows=1)
    rng = synth.rng_for(4, "nhd-append")
    n_new = np.array([5, 1, 3], dtype=np.int32)
    indptr = np.concatenate([[0], np.cumsum(n_new)]).astype(np.int32)
    k_new = synth.normal_bf16((int(n_new.sum()), w.num_kv_heads, w.head_dim), 0.5, rng)
    v_new = synth.normal_bf16((int(n_new.sum()), w.num_kv_heads, w.head_dim), 0.5, rng)
    pool_nhd = gu.bits_to_dev(gu.to_nhd(pool_bits))
    ctx = gu.i32(w.ctx_len)
    status = torch.zeros(1, dtype=torch.int32, device=gu.DEV)
    kap.append_kv(gu.bits_to_dev(k_new), gu.bits_to_dev(v_new), pool_nhd, gu.i32(w.bt_indptr), gu.i32(w.bt_pages),
                  ctx, new_indptr=gu.i32(indptr), advance=True, device_status=status, kv_layout=kap.KV_NHD)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    host = pool_bits.copy()
    for b in range(w.batch):
        bt = w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b + 1]]
        brute.append_kv(host, bt, int(w.ctx_len[b]), k_new[indptr[b]:indptr[b + 1]], v_new[indptr[b]:indptr[b + 1]])
    np.testing.assert_array_equal(gu.dev_to_bits(pool_nhd), gu.to_nhd(host))
    np.testing.assert_array_equal(ctx.cpu().numpy(), w.ctx_len + n_new)


def test_layout_argument_is_checked():
    ws = kap.Workspace()
    with pytest.raises(kap.KapError) as e:
        ws.set_kv_layout(7)
    assert e.value.code == kap.ERR_INVALID_ARG
    ws.close()
