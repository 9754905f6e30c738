"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element on
the same seeded inputs.  Tolerance for attention: |gpu - ref| <= 1e-2 + 1e-2 |ref| (bf16 inputs,
fp32 accumulation), plus a normalised bound max|d| / max|ref| <= 2e-2 because the absolute
tolerance alone is loose when thousands of tokens are averaged.  Page lists are bit-exact."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from helpers import ATOL, RTOL, assert_close, assert_same_up_to_rounding
from oracle import kap_oracle as orc
from paper_2607_24260_b200 import kap, synth

pytestmark = pytest.mark.gpu
NORM_TOL = 2e-2
LSE_ATOL = 1e-2


def _check_pair(got, ref, what):
    out, lse = got
    r_out, r_lse = ref
    assert not np.isnan(out).any(), f"{what}: NaN in output"
    assert_close(out, r_out, what=f"{what} out")
    assert gu.normalised_error(out, r_out) <= NORM_TOL, f"{what}: normalised error"
    assert_close(lse, r_lse, atol=LSE_ATOL, rtol=1e-3, what=f"{what} lse")


def _workload_case(w, seed, kv_std=0.5, q_std=1.0):
    q_bits, pool_bits = synth.host_qkv(w, seed, kv_std=kv_std, q_std=q_std)
    return q_bits, pool_bits, gu.bits_to_dev(pool_bits)


def _decode_rows(w, q_bits):
    """one decode query row per sequence: the last verification row of each sequence"""
    return q_bits[w.q_indptr[1:] - 1]


# ------------------------------------------------------------------------------ configuration 1
@pytest.mark.parametrize("name", ["c1", "c1b"])
def test_config1_decode_and_verify(name):
    w = synth.CONFIGS[name](0)
    q_bits, pool_bits, pool = _workload_case(w, 0)
    plan = kap.compile_workload(w)
    ref_plan = orc.compile_workload(w)
    for k in ("plan_indptr", "plan_logical_pages", "plan_phys_pages", "plan_flags", "selected_tokens"):
        np.testing.assert_array_equal(plan[k], ref_plan[k])
    qd = _decode_rows(w, q_bits)
    _check_pair(gu.run_decode(qd, pool, plan, w.ctx_len), gu.oracle_decode(qd, pool_bits, ref_plan, w.ctx_len),
                f"{name} decode")
    _check_pair(gu.run_verify(q_bits, w.n_q, pool, w.bt_indptr, w.bt_pages, w.ctx_len),
                gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len),
                f"{name} verify k=4")


# ------------------------------------------------------------ ragged batches, shuffled block tables
def _ragged_workload(seed, batch, max_len, nq_choices):
    """tiny_random's adversarial span mix scaled to a few thousand tokens."""
    w = synth.tiny_random(seed, batch=batch, max_len=max_len, max_spans=12)
    rng = synth.rng_for(seed, "ragged-nq")
    w.n_q = np.minimum(rng.choice(np.asarray(nq_choices), size=batch), w.ctx_len).astype(np.int32)
    return w


@pytest.mark.parametrize("seed,batch,max_len,nq", [
    (1, 5, 700, (1, 2, 3, 4)), (2, 7, 3000, (4, 5, 8)), (3, 3, 6000, (7, 8, 9)),
    (4, 9, 300, (1, 4, 6, 8)), (5, 4, 2500, (13, 16)),
])
def test_ragged_batches(seed, batch, max_len, nq):
    w = _ragged_workload(seed, batch, max_len, nq)
    q_bits, pool_bits, pool = _workload_case(w, seed)
    plan = kap.compile_workload(w)
    ref_plan = orc.compile_workload(w)
    np.testing.assert_array_equal(plan["plan_logical_pages"], ref_plan["plan_logical_pages"])
    np.testing.assert_array_equal(plan["plan_phys_pages"], ref_plan["plan_phys_pages"])
    qd = _decode_rows(w, q_bits)
    ref_d = gu.oracle_decode(qd, pool_bits, ref_plan, w.ctx_len)
    ref_v = gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len)
    for chunk in (0, 1, 3):           # default split, one page per CTA, three pages per CTA
        _check_pair(gu.run_decode(qd, pool, plan, w.ctx_len, max_chunk_pages=chunk), ref_d,
                    f"ragged{seed} decode chunk={chunk}")
        _check_pair(gu.run_verify(q_bits, w.n_q, pool, w.bt_indptr, w.bt_pages, w.ctx_len,
                                  max_chunk_pages=chunk), ref_v, f"ragged{seed} verify chunk={chunk}")


@pytest.mark.parametrize("L,nq", [(1, 1), (2, 2), (15, 4), (16, 4), (17, 8), (33, 9), (64, 1), (65, 16)])
def test_tiny_contexts(L, nq):
    """single page, exactly one page, one token over, n_q == L"""
    w = synth.tiny_random(11, batch=1, max_len=8)
    w.ctx_len = np.array([L], dtype=np.int32)
    w.n_q = np.array([nq], dtype=np.int32)
    w.bt_indptr, w.bt_pages, w.num_pool_pages = synth.block_tables([L], "shuffled", 11, "tinyctx", spare_pages=2)
    w.span_indptr = np.array([0, 0], dtype=np.int32)
    w.span_start = w.span_len = np.zeros(0, dtype=np.int32)
    w.span_score = np.zeros(0, dtype=np.float32)
    w.budget_tokens = np.array([L], dtype=np.int32)
    w.force_full = np.array([1], dtype=np.uint8)
    q_bits, pool_bits, pool = _workload_case(w, L)
    plan = kap.compile_workload(w)
    qd = _decode_rows(w, q_bits)
    _check_pair(gu.run_decode(qd, pool, plan, w.ctx_len), gu.oracle_decode(qd, pool_bits, plan, w.ctx_len),
                f"L={L} decode")
    _check_pair(gu.run_verify(q_bits, w.n_q, pool, w.bt_indptr, w.bt_pages, w.ctx_len),
                gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len),
                f"L={L} verify n_q={nq}")


@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (16, 8), (32, 8), (16, 2), (16, 1)])
def test_group_sizes(Hq, Hkv):
    """G = 1, 2, 4, 8, 16 query heads per KV head"""
    w = _ragged_workload(21, 3, 900, (1, 3, 4))
    w.num_q_heads, w.num_kv_heads = Hq, Hkv
    if 4 * (Hq // Hkv) > 64:
        w.n_q = np.minimum(w.n_q, 64 // (Hq // Hkv)).astype(np.int32)
    q_bits, pool_bits, pool = _workload_case(w, 21)
    plan = kap.compile_workload(w)
    qd = _decode_rows(w, q_bits)
    _check_pair(gu.run_decode(qd, pool, plan, w.ctx_len, Hq, Hkv),
                gu.oracle_decode(qd, pool_bits, plan, w.ctx_len), f"G={Hq // Hkv} decode")
    _check_pair(gu.run_verify(q_bits, w.n_q, pool, w.bt_indptr, w.bt_pages, w.ctx_len, Hq, Hkv),
                gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len),
                f"G={Hq // Hkv} verify")


# ----------------------------------------------------------------- scaled-down configurations 2-5
@pytest.mark.parametrize("name,kwargs,peaky", [
    ("c2", dict(batch=2, L=16384, layers=1), False),
    ("c3", dict(batch=2, L=8192, layers=1, bt_mode="shuffled"), True),
    ("c4", dict(batch=1, L=32768, layers=1, bt_mode="shuffled"), False),
    ("c5", dict(batch=6, layers=1, lo=512, hi=16384), False),
])
def test_scaled_configs(name, kwargs, peaky):
    """The generators of configurations 2-5 at sizes the oracle finishes in seconds: same span
    structure, budgets, fallback mix, ragged shuffled block tables.  `peaky` multiplies Q by 8 so
    the softmax is sharp and the outputs are O(0.3)."""
    w = synth.CONFIGS[name](0, **kwargs)
    q_bits, pool_bits, pool = _workload_case(w, 3, q_std=8.0 if peaky else 1.0)
    plan = kap.compile_workload(w)
    ref_plan = orc.compile_workload(w)
    for k in ("plan_indptr", "plan_logical_pages", "plan_phys_pages", "plan_flags", "selected_tokens"):
        np.testing.assert_array_equal(plan[k], ref_plan[k])
    qd = _decode_rows(w, q_bits)
    if name == "c3":
        # configuration 3 plants keys with a +2 sigma affinity to the queries inside the selected
        # pages; the oracle gets the pool's bits back after planting
        per_seq = [plan["plan_phys_pages"][plan["plan_indptr"][b]:plan["plan_indptr"][b + 1]] for b in range(w.batch)]
        n = synth.plant_affinity_keys_(pool, gu.bits_to_dev(qd), w, per_seq, seed=3, layer=0, q_std=8.0)
        assert n > 0
        pool_bits = gu.dev_to_bits(pool)
    _check_pair(gu.run_decode(qd, pool, plan, w.ctx_len), gu.oracle_decode(qd, pool_bits, ref_plan, w.ctx_len),
                f"{name} scaled decode")
    _check_pair(gu.run_verify(q_bits, w.n_q, pool, w.bt_indptr, w.bt_pages, w.ctx_len),
                gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len),
                f"{name} scaled verify")


# --------------------------------------------------------------------------- closed-form probes
def _probe_setup(L=5000, seed=31, spare=9):
    w = synth.tiny_random(seed, batch=1, max_len=8)
    w.ctx_len = np.array([L], dtype=np.int32)
    w.bt_indptr, w.bt_pages, w.num_pool_pages = synth.block_tables([L], "shuffled", seed, "probe", spare_pages=spare)
    rng = synth.rng_for(seed, "probe")
    n_pages = (L + 15) // 16
    keep = rng.random(n_pages) < 0.3
    keep[-1] = True
    logical = np.nonzero(keep)[0].astype(np.int32)
    plan = dict(plan_indptr=np.array([0, len(logical)], dtype=np.int32), plan_logical_pages=logical,
                plan_phys_pages=w.bt_pages[logical].astype(np.int32))
    q_bits, pool_bits = synth.host_qkv(w, seed, q_rows=8)
    return w, plan, q_bits, pool_bits, n_pages


def test_probe_uniform_attention_counts_tokens():
    """q = 0: out = mean of the visible value rows, lse = ln(n_visible): checks the visible count
    to one part in n, far below the mandated tolerance."""
    w, plan, q_bits, pool_bits, n_pages = _probe_setup()
    L = int(w.ctx_len[0])
    q0 = np.zeros_like(q_bits[:1])
    out, lse = gu.run_decode(q0, gu.bits_to_dev(pool_bits), plan, w.ctx_len)
    n_vis = sum(min(16, L - int(p) * 16) for p in plan["plan_logical_pages"])
    np.testing.assert_allclose(lse, np.log(n_vis), atol=2e-5)
    r_out, _ = gu.oracle_decode(q0, pool_bits, plan, w.ctx_len)
    assert gu.normalised_error(out, r_out) <= 6e-3           # bf16 rounding of the output only


def test_probe_page_coverage_logical_and_physical():
    """q = 0, V[t, j] = 1 iff key(page of t) mod 128 == j: out[j] = visible tokens per residue /
    n_visible.  A dropped, duplicated or wrong page moves a known coordinate by >= 16 / n_visible."""
    w, plan, q_bits, pool_bits, n_pages = _probe_setup(L=7001)
    L = int(w.ctx_len[0])
    one = synth.f32_to_bf16_bits(np.array([1.0], dtype=np.float32))[0]
    q0 = np.zeros_like(q_bits[:1])
    for keyed_by in ("logical", "physical"):
        pool = pool_bits.copy()
        pool[:, 1] = 0
        for lp in range(n_pages):
            key = lp if keyed_by == "logical" else int(w.bt_pages[lp])
            pool[w.bt_pages[lp], 1, :, :, key % 128] = one
        out, _ = gu.run_decode(q0, gu.bits_to_dev(pool), plan, w.ctx_len, max_chunk_pages=5)
        expect = np.zeros(128)
        for lp in plan["plan_logical_pages"]:
            key = int(lp) if keyed_by == "logical" else int(w.bt_pages[lp])
            expect[key % 128] += min(16, L - int(lp) * 16)
        expect /= expect.sum()
        # bf16 output rounding only: relative 2^-9
        np.testing.assert_allclose(out[0], np.broadcast_to(expect, out[0].shape), rtol=5e-3, atol=1e-7)


def _plant(pool_bits, w, token, q_row_bits, head, margin=40.0, G=4):
    q = synth.bf16_bits_to_f64(q_row_bits[head])
    k = q * (margin * np.sqrt(128.0) / (q @ q))
    lp, s = divmod(token, 16)
    pool_bits[w.bt_pages[lp], 0, head // G, s] = synth.f32_to_bf16_bits(k.astype(np.float32))


def test_probe_one_hot_key_and_invisible_key():
    w, plan, q_bits, pool_bits, n_pages = _probe_setup(L=4000, seed=33)
    head = 13
    vis_page = int(plan["plan_logical_pages"][len(plan["plan_logical_pages"]) // 2])
    hidden = next(p for p in range(n_pages) if p not in set(plan["plan_logical_pages"].tolist()))
    qd = q_bits[:1]
    base, base_lse = gu.run_decode(qd, gu.bits_to_dev(pool_bits), plan, w.ctx_len)
    pool = pool_bits.copy()
    _plant(pool, w, vis_page * 16 + 5, qd[0], head)
    out, lse = gu.run_decode(qd, gu.bits_to_dev(pool), plan, w.ctx_len)
    v = synth.bf16_bits_to_f64(pool[w.bt_pages[vis_page], 1, head // 4, 5])
    np.testing.assert_allclose(out[0, head], v, atol=1e-6)           # the weight is 1 to ~e-30
    assert abs(lse[0, head] - 40.0) < 0.3
    others = [h for h in range(32) if h // 4 != head // 4]
    assert_same_up_to_rounding(out[0, others], base[0, others], "other heads")
    pool = pool_bits.copy()
    _plant(pool, w, hidden * 16 + 5, qd[0], head)
    out2, lse2 = gu.run_decode(qd, gu.bits_to_dev(pool), plan, w.ctx_len)
    assert_same_up_to_rounding(out2, base, "invisible key")
    np.testing.assert_allclose(lse2, base_lse, atol=1e-5)


@pytest.mark.parametrize("nq", [4, 8, 7])
def test_probe_verify_causality(nq):
    """A dominant key at position p_j + 1: rows <= j ignore it, rows > j return its value row."""
    L = 3000 + nq
    w, _, q_bits, pool_bits, n_pages = _probe_setup(L=L, seed=35)
    head, j = 6, nq // 2 - 1
    q = np.repeat(q_bits[:1], nq, axis=0)
    base, _ = gu.run_verify(q, [nq], gu.bits_to_dev(pool_bits), w.bt_indptr, w.bt_pages, w.ctx_len)
    pool = pool_bits.copy()
    tok = L - nq + j + 1
    _plant(pool, w, tok, q[0], head)
    out, _ = gu.run_verify(q, [nq], gu.bits_to_dev(pool), w.bt_indptr, w.bt_pages, w.ctx_len)
    lp, s = divmod(tok, 16)
    v = synth.bf16_bits_to_f64(pool[w.bt_pages[lp], 1, head // 4, s])
    for r in range(nq):
        if r <= j:
            assert_same_up_to_rounding(out[r, head], base[r, head], f"row {r}")
        else:
            np.testing.assert_allclose(out[r, head], v, atol=1e-6)


def test_verify_last_row_equals_identity_plan_decode():
    w, _, q_bits, pool_bits, n_pages = _probe_setup(L=2777, seed=37)
    pool = gu.bits_to_dev(pool_bits)
    v_out, v_lse = gu.run_verify(q_bits[:8], [8], pool, w.bt_indptr, w.bt_pages, w.ctx_len)
    ident = dict(plan_indptr=np.array([0, n_pages], dtype=np.int32),
                 plan_logical_pages=np.arange(n_pages, dtype=np.int32),
                 plan_phys_pages=w.bt_pages[:n_pages].astype(np.int32))
    d_out, d_lse = gu.run_decode(q_bits[7:8], pool, ident, w.ctx_len)
    d2_out, d2_lse = gu.run_decode(q_bits[7:8], pool, ident, w.ctx_len, logical=False)
    assert_same_up_to_rounding(d_out, d2_out, "NULL logical list == identity positions")
    np.testing.assert_allclose(v_out[7], d_out[0], atol=2e-3, rtol=1e-2)
    np.testing.assert_allclose(v_lse[7], d_lse[0], atol=1e-4)


def test_garbage_beyond_context_is_ignored():
    """The slots of the last page past ctx_len may hold anything, NaN included."""
    w, plan, q_bits, pool_bits, n_pages = _probe_setup(L=1003, seed=39)
    L = 1003
    clean = gu.run_decode(q_bits[:1], gu.bits_to_dev(pool_bits), plan, w.ctx_len)
    dirty_bits = pool_bits.copy()
    dirty_bits[w.bt_pages[n_pages - 1], :, :, L % 16:, :] = 0x7FC0     # NaN
    dirty = gu.run_decode(q_bits[:1], gu.bits_to_dev(dirty_bits), plan, w.ctx_len)
    assert_same_up_to_rounding(clean[0], dirty[0], "decode with NaN tail")
    np.testing.assert_allclose(clean[1], dirty[1], atol=1e-5)
    v_clean = gu.run_verify(q_bits[:4], [4], gu.bits_to_dev(pool_bits), w.bt_indptr, w.bt_pages, w.ctx_len)
    v_dirty = gu.run_verify(q_bits[:4], [4], gu.bits_to_dev(dirty_bits), w.bt_indptr, w.bt_pages, w.ctx_len)
    assert_same_up_to_rounding(v_clean[0], v_dirty[0], "verify with NaN tail")


# ------------------------------------------------------------- split / launch-option invariance
def test_split_and_launch_option_invariance():
    w = synth.config2(0, batch=2, L=8192, layers=1)
    q_bits, pool_bits, pool = _workload_case(w, 5)
    plan = kap.compile_workload(w)
    qd = _decode_rows(w, q_bits)
    ref = gu.oracle_decode(qd, pool_bits, plan, w.ctx_len)
    ref_v = gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len)
    try:
        kap.set_launch_options(1, 1, -1, 1)
        one_split = gu.run_decode(qd, pool, plan, w.ctx_len, max_chunk_pages=512)
        for pdl, early in ((0, 0), (1, 0), (1, 1)):
            for cluster in (1, 2, 3, 8, 16):
                kap.set_launch_options(pdl, early, -1, cluster)
                for chunk in (0, 1, 7):
                    got = gu.run_decode(qd, pool, plan, w.ctx_len, max_chunk_pages=chunk)
                    _check_pair(got, ref, f"pdl={pdl} early={early} cluster={cluster} chunk={chunk}")
                    # splits only reorder fp32 sums: far tighter than the oracle tolerance
                    np.testing.assert_allclose(got[0], one_split[0], atol=2e-3, rtol=1e-2)
                    # (lse: the row sums are sums of bf16-rounded weights, and which way a weight rounds
                    # depends on the slice's own running maximum: about 1e-4 between slicings)
                    np.testing.assert_allclose(got[1], one_split[1], atol=3e-4)
                got = gu.run_verify(q_bits, w.n_q, pool, w.bt_indptr, w.bt_pages, w.ctx_len)
                _check_pair(got, ref_v, f"verify pdl={pdl} early={early} cluster={cluster}")
    finally:
        kap.set_launch_options(1, 1, 0, 16, 8)


def test_one_long_sequence_many_partial_states():
    """One sequence of 30 000 tokens: 8 lists cut into about 55 slices each, so the merge pass runs
    its eight-threads-per-cell form (lists with 24 or more partial states); rows 5 per KV-head
    group, the last page partial."""
    w = synth.config2(3, batch=1, L=30000 - 7, layers=1)
    w.n_q = np.array([5], dtype=np.int32)
    q_bits, pool_bits, pool = _workload_case(w, 11)
    ws = kap.Workspace(max_rows_per_item=5 * 4, max_batch=1)
    got = gu.run_verify(q_bits, w.n_q, pool, w.bt_indptr, w.bt_pages, w.ctx_len, ws=ws)
    info = ws.info()
    assert info["n_items"] // 8 >= 24 and info["n_merge_groups"] == 8
    ws.close()
    _check_pair(got, gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len), "long verify")
    # the proposal path over the identity plan, at most 8 pages per CTA: 235 states per list
    w.force_full = np.ones(1, dtype=np.uint8)
    plan = kap.compile_workload(w)
    assert plan["plan_flags"][0] & kap.PLAN_FULL
    qd = _decode_rows(w, q_bits)
    _check_pair(gu.run_decode(qd, pool, plan, w.ctx_len, max_chunk_pages=8),
                gu.oracle_decode(qd, pool_bits, plan, w.ctx_len), "long decode, 8 pages per CTA")


@pytest.mark.parametrize("cluster", [1, 2, 5, 8, 13, 16])
@pytest.mark.parametrize("cps,ring", [(1, 8), (2, 12), (0, 24), (0, 8)])
def test_cluster_sizes_on_ragged_batches(cluster, cps, ring):
    """Every cluster size on ragged batches with all row-tile counts (n_q 1..16), including lists
    shorter than the cluster (some CTAs of a cluster get no page at all)."""
    try:
        kap.set_launch_options(1, 1, cps, cluster, ring)
        for seed, batch, max_len, nq in ((1, 5, 700, (1, 2, 3, 4)), (3, 3, 6000, (7, 8, 9)),
                                         (5, 4, 2500, (13, 16)), (6, 6, 40, (1, 2))):
            w = _ragged_workload(seed, batch, max_len, nq)
            q_bits, pool_bits, pool = _workload_case(w, seed)
            plan = kap.compile_workload(w)
            qd = _decode_rows(w, q_bits)
            _check_pair(gu.run_decode(qd, pool, plan, w.ctx_len),
                        gu.oracle_decode(qd, pool_bits, plan, w.ctx_len), f"cluster {cluster} decode {seed}")
            _check_pair(gu.run_verify(q_bits, w.n_q, pool, w.bt_indptr, w.bt_pages, w.ctx_len),
                        gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len),
                        f"cluster {cluster} verify {seed}")
    finally:
        kap.set_launch_options(1, 1, 0, 16, 8)


def test_repeated_calls_and_workspace_reuse():
    """One workspace, one schedule, many calls (the per-layer loop): pages are dealt to warps in a
    fixed order, so results are bit-identical run to run."""
    w = synth.config2(0, batch=2, L=4096, layers=1)
    q_bits, pool_bits, pool = _workload_case(w, 6)
    plan = kap.compile_workload(w)
    qd = _decode_rows(w, q_bits)
    ws = kap.Workspace(max_rows_per_item=4, max_batch=2)
    try:
        first = gu.run_decode(qd, pool, plan, w.ctx_len, ws=ws, max_chunk_pages=4)
        for _ in range(3):
            again = gu.run_decode(qd, pool, plan, w.ctx_len, ws=ws, max_chunk_pages=4)
            np.testing.assert_array_equal(first[0], again[0])
            np.testing.assert_array_equal(first[1], again[1])
    finally:
        ws.close()


def test_cuda_graph_capture_of_layer_loop():
    """The attention calls only enqueue kernels: a loop over layers captures into one CUDA graph
    and replays with the same results."""
    w = synth.config2(0, batch=2, L=4096, layers=3)
    plan = kap.compile_workload(w)
    ws = kap.Workspace(max_rows_per_item=4, max_batch=2)
    ws.schedule(np.diff(plan["plan_indptr"]), None, 32, 8)
    pools, qs, outs, refs = [], [], [], []
    for layer in range(w.layers):
        q_bits, pool_bits = synth.host_qkv(w, 7, layer=layer)
        qd = _decode_rows(w, q_bits)
        pools.append(gu.bits_to_dev(pool_bits))
        qs.append(gu.bits_to_dev(qd))
        outs.append(torch.zeros_like(qs[-1]))
        refs.append(gu.oracle_decode(qd, pool_bits, plan, w.ctx_len)[0])
    args = (gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"]), gu.i32(plan["plan_logical_pages"]),
            gu.i32(w.ctx_len))
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        for layer in range(w.layers):      # warm-up outside capture (tensor maps, attributes)
            kap.selected_decode_attn(qs[layer], pools[layer], *args, outs[layer], ws)
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        for layer in range(w.layers):
            kap.selected_decode_attn(qs[layer], pools[layer], *args, outs[layer], ws)
    for o in outs:
        o.zero_()
    graph.replay()
    torch.cuda.synchronize()
    ws.check()
    for layer in range(w.layers):
        assert_close(gu.dev_bf16_to_f64(outs[layer]), refs[layer], what=f"graph layer {layer}")
    ws.close()


# ------------------------------------------------------------------------------- error behaviour
def test_attention_argument_errors_enqueue_nothing():
    w = synth.config2(0, batch=2, L=1024, layers=1)
    q_bits, pool_bits, pool = _workload_case(w, 8)
    plan = kap.compile_workload(w)
    qd = gu.bits_to_dev(_decode_rows(w, q_bits))
    out = torch.zeros_like(qd)
    ws = kap.Workspace(max_rows_per_item=4, max_batch=2)
    ws.schedule(np.diff(plan["plan_indptr"]), None, 32, 8)
    a = (gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"]), gu.i32(plan["plan_logical_pages"]),
         gu.i32(w.ctx_len))
    before = kap.launch_count()
    with pytest.raises(kap.KapError) as e:          # batch differs from the schedule
        kap.selected_decode_attn(qd[:1], pool, *a, out[:1], ws)
    assert e.value.code == kap.ERR_INVALID_ARG
    with pytest.raises(kap.KapError) as e:          # unsupported head_dim
        kap.selected_decode_attn(qd[:, :, :64].contiguous(), pool[..., :64].contiguous(), *a, out, ws)
    assert e.value.code == kap.ERR_UNSUPPORTED
    with pytest.raises(kap.KapError) as e:          # verification on a proposal-path schedule
        kap.verify_attn(qd, gu.i32([0, 1, 2]), pool, gu.i32(w.bt_indptr), gu.i32(w.bt_pages), a[3], out, ws)
    assert e.value.code == kap.ERR_INVALID_ARG
    with pytest.raises(kap.KapError) as e:          # rows beyond what the workspace was made for
        ws.schedule([4, 4], [8, 8], 32, 8)
    assert e.value.code == kap.ERR_CAPACITY
    assert kap.launch_count() == before
    ws.close()


def test_out_of_range_page_is_reported_not_dereferenced():
    w = synth.config2(0, batch=1, L=1024, layers=1)
    q_bits, pool_bits, pool = _workload_case(w, 9)
    plan = kap.compile_workload(w)
    bad = dict(plan)
    bad["plan_phys_pages"] = plan["plan_phys_pages"].copy()
    bad["plan_phys_pages"][3] = w.num_pool_pages + 1000
    with pytest.raises(kap.KapError) as e:
        gu.run_decode(_decode_rows(w, q_bits), pool, bad, w.ctx_len)
    assert e.value.code == kap.ERR_DEVICE_INDEX
    # the context is still usable and the status word was cleared
    good = gu.run_decode(_decode_rows(w, q_bits), pool, plan, w.ctx_len)
    _check_pair(good, gu.oracle_decode(_decode_rows(w, q_bits), pool_bits, plan, w.ctx_len), "after error")


def test_failed_schedule_leaves_the_previous_one_in_force():
    """A kap_schedule call that fails (more rows than the workspace holds; a changed ring size on
    top, which a half-applied update would have kept) changes nothing: the attention call that
    follows runs on the previous schedule and still matches the oracle."""
    w = synth.config2(3, batch=2, L=3000, layers=1)
    q_bits, pool_bits, pool = _workload_case(w, 3)
    plan = kap.compile_workload(w)
    ws = kap.Workspace(max_rows_per_item=4, max_batch=2)
    first = ws.schedule(np.diff(plan["plan_indptr"]), None, 32, 8)
    kap.set_launch_options(-1, -1, -1, -1, 12)               # another ring size for the next schedule
    try:
        with pytest.raises(kap.KapError) as e:
            ws.schedule(np.diff(plan["plan_indptr"]), [8, 8], 32, 8)      # 32 rows > 4
        assert e.value.code == kap.ERR_CAPACITY
    finally:
        kap.set_launch_options(-1, -1, -1, -1, 8)
    assert ws.info() == first
    qd = gu.bits_to_dev(_decode_rows(w, q_bits))
    out = torch.full_like(qd, float("nan"))
    kap.selected_decode_attn(qd, pool, gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"]),
                             gu.i32(plan["plan_logical_pages"]), gu.i32(w.ctx_len), out, ws)
    ws.check()
    ref = gu.oracle_decode(_decode_rows(w, q_bits), pool_bits, plan, w.ctx_len)
    assert_close(gu.dev_bf16_to_f64(out), ref[0], what="decode on the schedule that stayed in force")
    ws.close()


def test_workspace_calls_keep_the_callers_device_and_attention_checks_it():
    """kap_workspace_create / kap_schedule put the calling thread's current device back; an
    attention call made while another device is current is refused (one-GPU machines: only the first
    half can run)."""
    before = torch.cuda.current_device()
    ws = kap.Workspace(device=0, max_rows_per_item=4, max_batch=1)
    ws.schedule([8], None, 32, 8)
    assert torch.cuda.current_device() == before
    if torch.cuda.device_count() > 1:
        w = synth.config2(0, batch=1, L=128, layers=1)
        q_bits, pool_bits, pool = _workload_case(w, 1)
        plan = kap.compile_workload(w)
        ws.schedule(np.diff(plan["plan_indptr"]), None, 32, 8)
        qd = gu.bits_to_dev(_decode_rows(w, q_bits))
        out = torch.zeros_like(qd)
        with torch.cuda.device(1):
            with pytest.raises(kap.KapError) as e:
                kap.selected_decode_attn(qd, pool, gu.i32(plan["plan_indptr"]), gu.i32(plan["plan_phys_pages"]),
                                         gu.i32(plan["plan_logical_pages"]), gu.i32(w.ctx_len), out, ws)
            assert e.value.code == kap.ERR_INVALID_ARG
    ws.close()
