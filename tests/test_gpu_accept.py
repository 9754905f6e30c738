"""kap_top3_accept on the GPU against the oracle: integer results, bit-exact."""
import numpy as np
import pytest
import torch

import gpu_util as gu
from oracle import brute
from paper_2607_24260_b200 import kap, synth

pytestmark = pytest.mark.gpu


def _run(logits_np, indptr, proposed, stride_pad=0):
    rows, V = logits_np.shape
    buf = torch.zeros((rows, V + stride_pad), dtype=torch.float32, device=gu.DEV)
    buf[:, :V] = torch.from_numpy(logits_np.copy()).to(gu.DEV)
    logits = buf[:, :V]
    top3 = torch.full((rows, 3), -7, dtype=torch.int32, device=gu.DEV)
    acc = torch.full((len(indptr) - 1,), -7, dtype=torch.int32, device=gu.DEV)
    nxt = torch.full((len(indptr) - 1,), -7, dtype=torch.int32, device=gu.DEV)
    ctx = gu.i32(1000 + 10 * np.arange(len(indptr) - 1))
    kap.top3_accept(logits, gu.i32(indptr), gu.i32(proposed), top3, acc, nxt, ctx_len=ctx)
    torch.cuda.synchronize()
    # the commit step: every rejected proposal leaves the context
    k = np.maximum(np.diff(indptr) - 1, 0)          # a window without rows commits nothing
    np.testing.assert_array_equal(ctx.cpu().numpy(), 1000 + 10 * np.arange(len(k)) - (k - acc.cpu().numpy()))
    return top3.cpu().numpy(), acc.cpu().numpy(), nxt.cpu().numpy()


@pytest.mark.parametrize("V,pad", [(3, 0), (7, 1), (1000, 3), (32000, 0), (128256, 0), (151937, 5)])
def test_top3_accept_matches_oracle(V, pad):
    rng = synth.rng_for(V, "accept")
    k_per_seq = [4, 8, 6, 0, 4]
    indptr = np.concatenate([[0], np.cumsum([k + 1 for k in k_per_seq])]).astype(np.int32)
    rows = int(indptr[-1])
    x = rng.standard_normal((rows, V)).astype(np.float32)
    x[1, : min(V, 5)] = x[1].max() + 1.0                      # a tie at the top
    if V > 10:
        x[2, rng.integers(0, V, size=V // 10)] = np.nan        # NaNs rank last
        x[3, :] = -np.inf                                      # a fully masked row
        x[3, V - 1] = 0.0
        x[4, :] = np.nan                                        # NaN, -inf and signed zeros together
        x[4, 5:9] = [-np.inf, -0.0, 0.0, -np.inf]
    ref_top3, _, _ = brute.top3_accept(x, indptr, np.zeros(rows, dtype=np.int32))
    # proposals: mostly inside the top 3, a few outside, so prefixes of every length appear
    proposed = ref_top3[np.arange(rows), rng.integers(0, 3, size=rows)].astype(np.int32)
    bad = rng.random(rows) < 0.15
    proposed[bad] = (ref_top3[bad, 0] + 1 + ref_top3[bad, 1]) % V
    ref = brute.top3_accept(x, indptr, proposed)
    got = _run(x, indptr, proposed, pad)
    for g, r, name in zip(got, ref, ("top3", "accepted", "next_token")):
        np.testing.assert_array_equal(g, r, err_msg=name)


@pytest.mark.parametrize("V", [7, 32000])
def test_top3_accept_empty_windows(V):
    """Windows without any row - first, in the middle and last in the batch - accept nothing, carry
    -1, leave ctx_len alone and do not look at a neighbour's rows."""
    rng = synth.rng_for(V, "accept-empty")
    rows_per_seq = [0, 5, 0, 1, 3, 0]
    indptr = np.concatenate([[0], np.cumsum(rows_per_seq)]).astype(np.int32)
    rows = int(indptr[-1])
    x = rng.standard_normal((rows, V)).astype(np.float32)
    ref_top3, _, _ = brute.top3_accept(x, indptr, np.zeros(rows, dtype=np.int32))
    proposed = ref_top3[:, 1].astype(np.int32)               # every proposal is acceptable
    ref = brute.top3_accept(x, indptr, proposed)
    assert ref[1].tolist() == [0, 4, 0, 0, 2, 0] and ref[2][[0, 2, 5]].tolist() == [-1, -1, -1]
    got = _run(x, indptr, proposed)
    for g, r, name in zip(got, ref, ("top3", "accepted", "next_token")):
        np.testing.assert_array_equal(g, r, err_msg=name)


def test_top3_accept_argument_errors():
    x = torch.zeros((2, 2), dtype=torch.float32, device=gu.DEV)
    z = torch.zeros(6, dtype=torch.int32, device=gu.DEV)
    with pytest.raises(kap.KapError) as e:                     # vocab < 3
        kap.top3_accept(x, gu.i32([0, 2]), z, z, z, z)
    assert e.value.code == kap.ERR_INVALID_ARG
