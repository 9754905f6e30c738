"""Host side of growing plans, no GPU: kap_compile_growing_plan's fixed part plus the recent
window, taken at any later length, must be the token set the oracle's Algorithm 1 compiles afresh
at that length (whenever the plan is not flagged as moving with the length)."""
import numpy as np
import pytest

from oracle import kap_oracle as orc
from paper_2607_24260_b200 import kap, synth

P = 16


def _tokens(logical, masks):
    return {int(p) * P + t for p, m in zip(logical, masks) for t in range(P) if (int(m) >> t) & 1}


def _fresh(w, b, L):
    """oracle plan of sequence b compiled at length L: (token set, flags)"""
    lo, hi = w.span_indptr[b], w.span_indptr[b + 1]
    r = orc.compile_plan([L], [0, hi - lo], w.span_start[lo:hi], w.span_len[lo:hi],
                         w.span_score[lo:hi], [w.budget_tokens[b]], [w.n_sink[b]], [w.n_recent[b]],
                         force_full=[w.force_full[b]])
    return _tokens(r["plan_logical_pages"], r["plan_token_masks"]), int(r["plan_flags"][0])


def _grow(w, growth):
    return kap.compile_growing_plan(w.ctx_len, w.span_indptr, w.span_start, w.span_len, w.span_score,
                                    w.budget_tokens, w.n_sink, w.n_recent, w.bt_indptr, w.bt_pages,
                                    force_full=w.force_full, max_growth=growth)


def _window(b_desc, L):
    reserved, window, start = (int(x) for x in b_desc)
    return set(range(max(L - window, start, 0), L))


@pytest.mark.parametrize("seed", range(40))
def test_fixed_part_plus_window_is_a_fresh_compile_at_every_later_length(seed):
    growth = 40
    w = synth.growing_random(seed, batch=4, growth=growth)
    g = _grow(w, growth)
    exact = 0
    for b in range(w.batch):
        lo, hi = g["plan_indptr"][b], g["plan_indptr"][b + 1]
        reserved = int(g["tail_desc"][b, 0])
        fixed = _tokens(g["plan_logical_pages"][lo:hi - reserved], g["plan_token_masks"][lo:hi - reserved])
        # reserved entries start out empty
        assert np.all(g["plan_token_masks"][hi - reserved:hi] == 0)
        assert np.all(np.diff(g["plan_logical_pages"][lo:hi - reserved]) > 0)
        L0 = int(w.ctx_len[b])
        moves = bool(g["plan_flags"][b] & kap.PLAN_MOVES_WITH_LENGTH)
        for L in [L0] + sorted(set(int(x) for x in synth.rng_for(seed, b).integers(L0, L0 + growth + 1, 6))):
            got = fixed | _window(g["tail_desc"][b], L)
            want, flags = _fresh(w, b, L)
            if L == L0:
                assert got == want, (seed, b)                       # always: it is the same union
                assert (g["plan_flags"][b] & ~kap.PLAN_MOVES_WITH_LENGTH) == flags
                assert int(g["selected_tokens"][b]) == len(want)
            elif not moves:
                assert got == want, (seed, b, L)
            # the reservation holds the window's pages at every length
            win = _window(g["tail_desc"][b], L)
            assert len({t // P for t in win}) <= reserved
        exact += not moves
        # physical pages through the block table
        bt = w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b + 1]]
        np.testing.assert_array_equal(g["plan_phys_pages"][lo:hi - reserved],
                                      bt[g["plan_logical_pages"][lo:hi - reserved]])
    assert exact >= 2


def test_flag_is_set_exactly_when_a_span_or_the_sink_reaches_the_window():
    base = dict(span_indptr=[0, 1], span_score=[1.0], budget_tokens=[200], n_sink=[4], n_recent=[16],
                bt_indptr=[0, 20], bt_pages=np.arange(20))
    def flag(L, start, length, **kw):
        a = dict(base, **kw)
        g = kap.compile_growing_plan([L], a["span_indptr"], [start], [length], a["span_score"],
                                     a["budget_tokens"], a["n_sink"], a["n_recent"], a["bt_indptr"],
                                     a["bt_pages"])
        return bool(g["plan_flags"][0] & kap.PLAN_MOVES_WITH_LENGTH)
    assert not flag(200, 100, 84)            # span ends exactly where the window starts
    assert flag(200, 100, 85)                # one token inside the window
    assert flag(200, 250, 10)                # span beyond the end becomes visible later
    assert not flag(200, 100, 0)             # empty span
    assert not flag(200, -30, 20)            # clipped away entirely
    assert flag(18, 100, 0, n_sink=[4])      # sink and window overlap at this length
    assert not flag(20, 100, 0, n_sink=[4])
    assert not flag(200, 100, 50, n_recent=[0])     # window = the last token only
    assert flag(200, 100, 100, n_recent=[0])


def test_full_plan_reserves_for_growth_and_errors():
    bt = np.arange(40)
    g = kap.compile_growing_plan([100], [0, 0], [], [], [], [10], [4], [8], [0, 40], bt,
                                 force_full=[1], max_growth=50)
    assert g["plan_flags"][0] == kap.PLAN_FULL
    reserved, window, start = g["tail_desc"][0]
    assert (window, start) == (2**31 - 1, 100)
    assert reserved == (149 // 16) - (100 // 16) + 1
    n = g["plan_indptr"][1]
    assert n == 7 + reserved
    assert _tokens(g["plan_logical_pages"][:7], g["plan_token_masks"][:7]) == set(range(100))
    g0 = kap.compile_growing_plan([100], [0, 0], [], [], [], [10], [4], [8], [0, 40], bt,
                                  force_full=[1], max_growth=0)
    assert g0["tail_desc"][0, 0] == 0
    with pytest.raises(kap.KapError) as e:
        kap.compile_growing_plan([100], [0, 0], [], [], [], [10], [4], [8], [0, 40], bt, max_growth=-1)
    assert e.value.code == kap.ERR_INVALID_ARG
    with pytest.raises(kap.KapError) as e:       # capacity: the reserved entries count too
        kap.compile_growing_plan([100], [0, 0], [], [], [], [10], [4], [8], [0, 40], bt, capacity=2)
    assert e.value.code == kap.ERR_CAPACITY
