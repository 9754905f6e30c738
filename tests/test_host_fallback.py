"""kap_fallback_decide (host) against the oracle's rule: decisions and reason masks bit-exact,
the fp64 quantities to rounding; argument errors."""
import numpy as np
import pytest

from oracle import brute
from paper_2607_24260_b200 import kap


def test_fallback_decide_matches_oracle_on_random_batches():
    rng = np.random.default_rng(7)
    fired = 0
    for trial in range(300):
        B = int(rng.integers(1, 9))
        prop = rng.integers(0, 60, size=B)
        acc = (prop * rng.random(B)).astype(np.int64)
        s = np.where(rng.random(B) < 0.1, 0.0, rng.random(B) * 0.7)
        kv = np.where(rng.random(B) < 0.1, 0.0, rng.random(B) * 100)
        kw = dict(w_main=float(rng.random() * 3) * (trial % 2), w_prop=float(rng.random() * 3) * (trial % 2),
                  min_proposed=int(rng.integers(0, 20)), h_prior=float(rng.random()),
                  h_min=float(rng.random() * 0.6), s_max=float(0.3 + rng.random()),
                  confidence_min=0.5)
        flags = rng.integers(0, 16, size=B).astype(np.int32) if trial % 3 else None
        rt = rng.integers(0, 4, size=B).astype(np.int32) if trial % 4 else None
        conf = rng.random(B) if trial % 5 else None
        got = kap.fallback_decide(acc, prop, s, kv, plan_flags=flags, runtime_flags=rt, confidence=conf, **kw)
        ref = brute.fallback_decide(acc, prop, kw["min_proposed"], kw["h_prior"], s, kv, kw["w_main"], kw["w_prop"],
                                    kw["h_min"], kw["s_max"], plan_flags=flags, runtime_flags=rt,
                                    confidence=conf, confidence_min=0.5)
        for b in range(B):
            assert int(got["force_full"][b]) == ref[b]["force_full"], (trial, b)
            assert int(got["reasons"][b]) == ref[b]["reasons"], (trial, b)
            assert got["h"][b] == ref[b]["h"]
            np.testing.assert_allclose(got["slack"][b], ref[b]["slack"], rtol=1e-13, atol=1e-13)
            np.testing.assert_allclose(got["budget_scale"][b], ref[b]["budget_scale"], rtol=1e-12)
            fired |= int(got["reasons"][b])
    assert fired == 127                                      # every reason occurred somewhere


def test_fallback_constants_agree_with_the_oracle():
    assert (kap.FALLBACK_CAPACITY, kap.FALLBACK_METADATA, kap.FALLBACK_CONFIDENCE, kap.FALLBACK_S_HIGH,
            kap.FALLBACK_H_LOW, kap.FALLBACK_NO_MARGIN, kap.FALLBACK_SLACK) == \
        (brute.FB_CAPACITY, brute.FB_METADATA, brute.FB_CONFIDENCE, brute.FB_S_HIGH, brute.FB_H_LOW,
         brute.FB_NO_MARGIN, brute.FB_SLACK)
    assert (kap.RUNTIME_OVER_CAPACITY, kap.RUNTIME_UNSTABLE_METADATA) == \
        (brute.RT_OVER_CAPACITY, brute.RT_UNSTABLE_METADATA)


@pytest.mark.parametrize("bad", [
    dict(accepted_sum=[5], proposed_sum=[4]), dict(accepted_sum=[-1], proposed_sum=[4]),
    dict(s=[-0.1]), dict(kv=[float("nan")]), dict(h_prior=1.5), dict(w_main=-1.0),
    dict(confidence=[float("nan")]), dict(h_min=float("nan")),
])
def test_fallback_decide_rejects_bad_input(bad):
    args = dict(accepted_sum=[3], proposed_sum=[4], s=[0.1], kv=[10.0])
    args.update(bad)
    with pytest.raises(kap.KapError) as e:
        kap.fallback_decide(**args)
    assert e.value.code == kap.ERR_INVALID_ARG
