"""Pins for the oracle's fallback rule (Section 3.2 "Runtime stability and fallback", Section 4.2):
the paper's own algebra and the values its Table 5 prints, not the oracle's formula retyped."""
import math

import numpy as np
import pytest

from helpers import GOLDEN
from oracle import brute


def _one(h, s, kv, w=0.0, w_prop=None, n=1000, **kw):
    w_prop = w if w_prop is None else w_prop
    acc = int(round(h * n))
    r = brute.fallback_decide([acc], [n], kw.pop("min_proposed", 1), kw.pop("h_prior", 1.0), [s], [kv], w, w_prop,
                              kw.pop("h_min", 0.0), kw.pop("s_max", 1.0), **kw)[0]
    return r


def _table5():
    rows = []
    with open(f"{GOLDEN}/phase_table5.txt") as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                c = line.split()
                rows.append((c[0], float(c[1]), float(c[2]), float(c[3]), float(c[4])))
    return rows


def test_paper_table5_rows_keep_their_plans():
    """Every row the paper reports (s, h at 4K ... 128K, speed-up > 1) has h > s and, at the KV /
    weight ratio its own speed-up implies, a positive slack: the rule keeps all six plans."""
    for name, s, h, margin, speedup in _table5():
        assert abs((h - s) - margin) < 2e-3
        # Cost_base / Cost_plan = speedup (Eqs. 6, 7; k = 6, W_prop = W_main = 1) solved for KV
        k = 6.0
        kv = (speedup * (k + 1) - (1 + k * h)) / ((1 + k * h) - speedup * (k * s + 1))
        assert kv > 0
        r = _one(h, s, kv, w=1.0, n=100000)
        assert r["force_full"] == 0 and r["reasons"] == 0, name
        # the slack is (h - s) KV - (1 - h) W for self-speculation (Section 4.2)
        assert r["slack"] == pytest.approx((h - s) * kv - (1 - h) * 1.0, abs=1e-9)


def test_slack_sign_is_the_cycle_cost_comparison_and_k_cancels():
    """Eq. 13's sign equals the sign of Cost_base - Cost_plan (Eqs. 6, 7) for every k."""
    rng = np.random.default_rng(0)
    for _ in range(300):
        h, s = rng.random(), rng.random()
        kv, w, wp = rng.random() * 10, rng.random() * 3, rng.random() * 3
        r = _one(h, s, kv, w=w, w_prop=wp, n=10 ** 6)
        h_used = r["h"]
        for k in (1, 4, 9):
            gain = (1 + k * h_used) * (w + kv) - (k * (wp + s * kv) + (w + kv))
            assert gain == pytest.approx(k * r["slack"], rel=1e-9, abs=1e-9)
            if abs(gain) > 1e-9:
                assert bool(r["reasons"] & brute.FB_SLACK) == (gain <= 0)


def test_no_margin_means_fallback_at_any_context_length():
    """h <= s (Eq. 11 violated): growing KV never rescues the plan under self-speculation."""
    for kv in (1.0, 1e3, 1e9):
        r = _one(0.30, 0.30, kv, w=1.0)
        assert r["force_full"] == 1 and r["reasons"] & brute.FB_NO_MARGIN and r["reasons"] & brute.FB_SLACK
        r = _one(0.20, 0.35, kv, w=0.0)
        assert r["force_full"] == 1 and r["reasons"] & brute.FB_NO_MARGIN


def test_break_even_kv_scale_of_the_paper():
    """Eq. 12: with h > s the slack changes sign at KV_crit = (1 - h) W / (h - s)."""
    h, s, w = 0.9, 0.25, 2.0
    kv_crit = (1 - h) * w / (h - s)
    assert _one(h, s, kv_crit * 1.001, w=w)["force_full"] == 0
    below = _one(h, s, kv_crit * 0.999, w=w)
    assert below["force_full"] == 1 and below["reasons"] == brute.FB_SLACK
    assert abs(_one(h, s, kv_crit, w=w)["slack"]) < 1e-12


def test_budget_scale_is_where_the_slack_vanishes():
    rng = np.random.default_rng(1)
    for _ in range(200):
        h, s = 0.2 + 0.8 * rng.random(), 0.02 + 0.5 * rng.random()
        kv, w = 1 + rng.random() * 50, rng.random() * 2
        r = _one(h, s, kv, w=w, n=10 ** 6)
        if r["budget_scale"] == 0.0:
            assert r["h"] * (w + kv) - w <= 0
            continue
        again = _one(h, s * r["budget_scale"], kv, w=w, n=10 ** 6)
        assert abs(again["slack"]) < 1e-9 * (w + kv)
        assert (r["budget_scale"] > 1) == (r["slack"] > 0)
    assert _one(0.5, 0.0, 10.0)["budget_scale"] == math.inf


def test_each_trigger_on_its_own():
    ok = dict(h=0.9, s=0.1, kv=100.0, w=1.0)
    assert _one(**ok)["reasons"] == 0
    assert _one(**ok, runtime_flags=[brute.RT_OVER_CAPACITY])["reasons"] == brute.FB_CAPACITY
    assert _one(**ok, runtime_flags=[brute.RT_UNSTABLE_METADATA])["reasons"] == brute.FB_METADATA
    assert _one(**ok, confidence=[0.2], confidence_min=0.5)["reasons"] == brute.FB_CONFIDENCE
    assert _one(**ok, confidence=[0.5], confidence_min=0.5)["reasons"] == 0
    assert _one(**ok, s_max=0.05)["reasons"] == brute.FB_S_HIGH
    assert _one(**ok, plan_flags=[4])["reasons"] == brute.FB_S_HIGH
    assert _one(**ok, plan_flags=[1 | 2 | 8])["reasons"] == 0
    assert _one(**ok, h_min=0.95)["reasons"] == brute.FB_H_LOW
    assert _one(**ok, h_min=0.9)["reasons"] == 0             # "low" means below the floor, not at it
    for r in (_one(**ok, s_max=0.05), _one(**ok, h_min=0.95)):
        assert r["force_full"] == 1


def test_acceptance_is_observed_only_after_enough_proposals():
    """Eq. 5 on the running counts; before min_proposed verified proposals the prior stands in."""
    kw = dict(s=[0.1], kv=[100.0], w_main=0.0, w_prop=0.0, h_min=0.5, s_max=1.0)
    r = brute.fallback_decide([0], [7], 8, 0.9, **kw)[0]
    assert r["h"] == 0.9 and r["force_full"] == 0
    r = brute.fallback_decide([0], [8], 8, 0.9, **kw)[0]
    assert r["h"] == 0.0 and r["reasons"] == brute.FB_H_LOW | brute.FB_NO_MARGIN | brute.FB_SLACK
    r = brute.fallback_decide([6], [8], 8, 0.0, **kw)[0]
    assert r["h"] == 0.75 and r["force_full"] == 0
    # sequences are independent
    rs = brute.fallback_decide([6, 1], [8, 8], 8, 0.9, [0.1, 0.1], [100.0, 100.0], 0.0, 0.0, 0.5, 1.0)
    assert [x["force_full"] for x in rs] == [0, 1]
