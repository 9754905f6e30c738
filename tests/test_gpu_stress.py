"""Randomised sweep over shapes and launch options on the GPU: ragged batches, every row count,
page-granular and token-granular visibility (plan masks and arbitrary masks with hidden pages), both
pool layouts, cluster sizes 1..16, ring sizes, with and without programmatic dependent launch, forced
chunk sizes.  Every case must match the oracle and must reproduce itself bit for bit when it is
run again (the work split is static; a race would show up as a difference between the runs)."""
import numpy as np
import pytest

import gpu_util as gu
from paper_2607_24260_b200 import kap, synth

pytestmark = pytest.mark.gpu


def _within(got, ref):
    return bool(np.all(np.abs(got - ref) <= 1e-2 + 1e-2 * np.abs(ref)) and not np.isnan(got).any())


@pytest.mark.parametrize("seed", [101, 102, 103])
def test_random_shapes_and_launch_options(seed):
    rng = np.random.default_rng(seed)
    try:
        done = 0
        for case in range(14):
            batch = int(rng.integers(1, 12))
            max_len = int(rng.choice([60, 400, 3000, 9000]))
            w = synth.tiny_random(int(rng.integers(1 << 30)), batch=batch, max_len=max_len, max_spans=12)
            w.n_q = np.minimum(rng.choice([1, 2, 4, 5, 8, 9, 16], size=batch), w.ctx_len).astype(np.int32)
            q_bits, pool_bits = synth.host_qkv(w, case)
            plan = kap.compile_workload(w)
            qd = q_bits[w.q_indptr[1:] - 1]
            opts = (int(rng.integers(0, 2)), int(rng.integers(0, 2)), int(rng.choice([0, 1, 2, 3])),
                    int(rng.choice([1, 2, 3, 5, 8, 16])), int(rng.choice([8, 12, 24])))
            chunk = int(rng.choice([0, 1, 2, 7, 64]))
            layout = int(rng.integers(0, 2))
            masks = plan["plan_token_masks"] if rng.integers(0, 2) else None
            if masks is not None and rng.integers(0, 2):
                masks = rng.integers(0, 1 << 16, size=len(masks)).astype(np.uint16)
                masks[rng.random(len(masks)) < 0.2] = 0
                masks[plan["plan_indptr"][1:] - 1] |= 1          # something stays visible everywhere
            pool = gu.bits_to_dev(gu.to_nhd(pool_bits) if layout else pool_bits)
            kap.set_launch_options(*opts)
            what = f"seed {seed} case {case}: options {opts}, chunk {chunk}, layout {layout}, n_q {w.n_q.tolist()}"
            try:
                runs = [(gu.run_decode(qd, pool, plan, w.ctx_len, max_chunk_pages=chunk, masks=masks, kv_layout=layout),
                         gu.run_verify(q_bits, w.n_q, pool, w.bt_indptr, w.bt_pages, w.ctx_len,
                                       max_chunk_pages=chunk, kv_layout=layout)) for _ in range(3)]
            except kap.KapError as e:
                if e.code == kap.ERR_CAPACITY:                   # a forced chunk of 1-2 pages on long lists
                    continue
                raise
            ref_d = gu.oracle_decode(qd, pool_bits, plan, w.ctx_len, masks=masks)
            ref_v = gu.oracle_verify(q_bits, w.n_q, pool_bits, w.bt_indptr, w.bt_pages, w.ctx_len)
            for d, v in runs:
                assert _within(d[0], ref_d[0]), what + " (decode)"
                assert _within(v[0], ref_v[0]), what + " (verify)"
                np.testing.assert_array_equal(d[0], runs[0][0][0], err_msg=what)
                np.testing.assert_array_equal(v[0], runs[0][1][0], err_msg=what)
            done += 1
        assert done >= 8
    finally:
        kap.set_launch_options(1, 1, 0, 16, 8)
