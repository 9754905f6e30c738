"""Shared test helpers (fixture parsing, tolerances).  No method arithmetic."""
from __future__ import annotations

import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")

# spec tolerance for bf16 inputs with fp32 accumulation
ATOL, RTOL = 1e-2, 1e-2


def read_plan_fixture(name):
    spans, out = [], {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            if key == "span":
                spans.append((int(vals[0]), int(vals[1]), float(vals[2])))
            elif key in ("block_table", "expect_logical", "expect_phys"):
                out[key] = [int(v) for v in vals]
            else:
                out[key] = int(vals[0])
    out["spans"] = spans
    return out


def assert_close(got, ref, atol=ATOL, rtol=RTOL, what=""):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    err = np.abs(got - ref)
    bound = atol + rtol * np.abs(ref)
    bad = ~(err <= bound)
    if bad.any():
        i = np.unravel_index(np.argmax(np.where(bad, err - bound, -np.inf)), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outside |d|<={atol}+{rtol}|ref|; "
                             f"worst at {i}: got {got[i]!r} ref {ref[i]!r}")


def assert_same_up_to_rounding(a, b, what=""):
    """Two runs of the library on inputs whose differences must not matter: equal up to the order
    of the fp32 sums, i.e. within two bf16 ulps of the largest magnitude (pages are handed out
    dynamically, so the summation order is not fixed)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    scale = max(float(np.max(np.abs(b))), 1e-30)
    err = float(np.max(np.abs(a - b)))
    assert err <= 2.0 ** -7 * scale, f"{what}: max diff {err} vs scale {scale}"
