"""GPU parity for token-granular visibility (the plan's visibility mask at token level): the
proposal-path kernel with per-page 16-bit masks against the oracle, same tolerances as the
page-granular tests."""
import numpy as np
import pytest

import gpu_util as gu
from helpers import assert_close
from oracle import kap_oracle as orc
from paper_2607_24260_b200 import kap, synth
from test_gpu_parity import _check_pair, _decode_rows, _ragged_workload, _workload_case

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed,batch,max_len", [(1, 5, 700), (2, 7, 3000), (3, 3, 6000), (4, 9, 300)])
def test_plan_masks_on_ragged_batches(seed, batch, max_len):
    w = _ragged_workload(seed, batch, max_len, (1,))
    q_bits, pool_bits, pool = _workload_case(w, seed)
    plan, ref_plan = kap.compile_workload(w), orc.compile_workload(w)
    np.testing.assert_array_equal(plan["plan_token_masks"], ref_plan["plan_token_masks"])
    qd = _decode_rows(w, q_bits)
    ref = gu.oracle_decode(qd, pool_bits, ref_plan, w.ctx_len, masks=ref_plan["plan_token_masks"])
    for chunk in (0, 1, 3):
        got = gu.run_decode(qd, pool, plan, w.ctx_len, max_chunk_pages=chunk,
                            masks=plan["plan_token_masks"])
        _check_pair(got, ref, f"masked ragged{seed} chunk={chunk}")


@pytest.mark.parametrize("name,kwargs,partial_pages", [
    ("c2", dict(batch=2, L=16384, layers=1), True),
    ("c4", dict(batch=1, L=32768, layers=1, bt_mode="shuffled"), False),   # page-aligned chunks
    ("c5", dict(batch=6, layers=1, lo=512, hi=16384), True),
])
def test_plan_masks_on_scaled_configs(name, kwargs, partial_pages):
    """Configurations 2, 4 and 5 scaled down, Q multiplied by 8 so that single tokens carry
    weight.  The token-granular result must match the oracle and, where spans do not end on page
    boundaries, must differ from the page-granular one, so the masks are really applied."""
    w = synth.CONFIGS[name](0, **kwargs)
    q_bits, pool_bits, pool = _workload_case(w, 5, q_std=8.0)
    plan, ref_plan = kap.compile_workload(w), orc.compile_workload(w)
    masks = plan["plan_token_masks"]
    np.testing.assert_array_equal(masks, ref_plan["plan_token_masks"])
    assert np.any(masks != 0xFFFF) == partial_pages
    qd = _decode_rows(w, q_bits)
    got = gu.run_decode(qd, pool, plan, w.ctx_len, masks=masks)
    _check_pair(got, gu.oracle_decode(qd, pool_bits, ref_plan, w.ctx_len, masks=masks), f"masked {name}")
    page_granular = gu.run_decode(qd, pool, plan, w.ctx_len)
    if not partial_pages:
        np.testing.assert_array_equal(page_granular[0], got[0])
        return
    assert np.max(np.abs(page_granular[1] - got[1])) > 1e-3      # lse drops when tokens are hidden
    assert np.all(got[1] <= page_granular[1] + 1e-5)


def test_all_ones_masks_change_nothing():
    w = _ragged_workload(6, 4, 2000, (1,))
    q_bits, pool_bits, pool = _workload_case(w, 6)
    plan = kap.compile_workload(w)
    qd = _decode_rows(w, q_bits)
    ones = np.full(len(plan["plan_logical_pages"]), 0xFFFF, dtype=np.uint16)
    a = gu.run_decode(qd, pool, plan, w.ctx_len)
    b = gu.run_decode(qd, pool, plan, w.ctx_len, masks=ones)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])


def test_random_masks_with_hidden_pages_and_hidden_sequences():
    """Arbitrary masks, not only unions of spans: sparse bits, pages with no visible token, one
    sequence with nothing visible at all (out = 0, lse = -inf on both sides), bits set past the
    end of the context (ignored)."""
    w = _ragged_workload(7, 6, 1500, (1,))
    q_bits, pool_bits, pool = _workload_case(w, 7, q_std=4.0)
    plan = kap.compile_workload(w)
    rng = synth.rng_for(7, "random-masks")
    n = len(plan["plan_logical_pages"])
    masks = rng.integers(0, 1 << 16, size=n).astype(np.uint16)
    masks[rng.random(n) < 0.3] = 0                                  # hidden pages
    masks[rng.random(n) < 0.2] &= np.uint16(0x0101)                 # one or two tokens
    lo, hi = plan["plan_indptr"][2], plan["plan_indptr"][3]
    masks[lo:hi] = 0                                                # sequence 2 sees nothing
    last = plan["plan_indptr"][1:] - 1
    masks[last[[0, 1]]] = 0xFFFF                                    # bits beyond ctx_len set
    qd = _decode_rows(w, q_bits)
    ref = gu.oracle_decode(qd, pool_bits, plan, w.ctx_len, masks=masks)
    for chunk in (0, 2):
        out, lse = gu.run_decode(qd, pool, plan, w.ctx_len, max_chunk_pages=chunk, masks=masks)
        assert np.all(out[2] == 0.0) and np.all(np.isneginf(lse[2]))
        assert np.all(ref[0][2] == 0.0) and np.all(np.isneginf(ref[1][2]))
        keep = np.arange(w.batch) != 2
        _check_pair((out[keep], lse[keep]), (ref[0][keep], ref[1][keep]), f"random masks chunk={chunk}")


def test_masks_with_a_context_shorter_than_the_plan():
    """A plan compiled for the end of a proposal cycle, used while the last tokens are not yet
    appended: bits of tokens >= ctx_len are set in the masks but stay invisible."""
    w = _ragged_workload(8, 4, 1200, (1,))
    q_bits, pool_bits, pool = _workload_case(w, 8)
    plan = kap.compile_workload(w)
    qd = _decode_rows(w, q_bits)
    short = np.maximum(w.ctx_len - np.array([0, 3, 17, 40], dtype=np.int32), 1).astype(np.int32)
    masks = plan["plan_token_masks"]
    got = gu.run_decode(qd, pool, plan, short, masks=masks)
    # the oracle takes only pages that exist at the shorter length: trim the plan for it
    keep = np.concatenate([
        plan["plan_logical_pages"][lo:hi].astype(np.int64) * 16 < L
        for lo, hi, L in zip(plan["plan_indptr"][:-1], plan["plan_indptr"][1:], short)])
    seq_of = np.repeat(np.arange(w.batch), np.diff(plan["plan_indptr"]))
    trimmed = dict(plan_indptr=np.concatenate([[0], np.cumsum(np.bincount(seq_of[keep], minlength=w.batch))]),
                   plan_phys_pages=plan["plan_phys_pages"][keep],
                   plan_logical_pages=plan["plan_logical_pages"][keep])
    assert not keep.all()
    ref = gu.oracle_decode(qd, pool_bits, trimmed, short, masks=masks[keep])
    finite = np.isfinite(ref[1]).all(axis=1)
    assert finite.any()
    _check_pair((got[0][finite], got[1][finite]), (ref[0][finite], ref[1][finite]), "short ctx")
    assert_close(got[0][~finite], ref[0][~finite], what="short ctx hidden rows")
