"""Host logic of the library, no GPU: kap_compile_plan against the oracle (bit-exact page lists),
its error behaviour, and the hand-worked fixture."""
import numpy as np
import pytest

from helpers import read_plan_fixture
from oracle import kap_oracle as orc
from paper_2607_24260_b200 import kap, synth

KEYS = ("plan_indptr", "plan_logical_pages", "plan_phys_pages", "plan_flags", "selected_tokens",
        "plan_token_masks")


def _same(a, b, msg=""):
    if a is None or b is None:
        assert a is None and b is None, msg
    else:
        assert a.dtype == b.dtype, msg
        np.testing.assert_array_equal(a, b, err_msg=msg)


def test_fixture_through_the_library():
    fx = read_plan_fixture("plan_worked_example.txt")
    s = fx["spans"]
    r = kap.compile_plan([fx["ctx_len"]], [0, len(s)], [x[0] for x in s], [x[1] for x in s],
                         [x[2] for x in s], [fx["budget"]], [fx["n_sink"]], [fx["n_recent"]],
                         bt_indptr=[0, len(fx["block_table"])], bt_pages=fx["block_table"],
                         page_size=fx["page_size"])
    assert r["plan_logical_pages"].tolist() == fx["expect_logical"]
    assert r["plan_phys_pages"].tolist() == fx["expect_phys"]
    assert int(r["selected_tokens"][0]) == fx["expect_selected_tokens"]
    assert int(r["plan_flags"][0]) == fx["expect_flags"]


def test_library_equals_oracle_on_random_tiny_cases():
    for seed in range(1500):
        w = synth.tiny_random(seed, batch=4, max_len=260, max_spans=14,
                              page_size=(16, 4, 1, 32)[seed % 4])
        a, b = kap.compile_workload(w), orc.compile_workload(w)
        for k in KEYS:
            _same(a[k], b[k], f"seed {seed} {k}")
        assert (a["plan_token_masks"] is None) == (w.page_size > 16)


@pytest.mark.parametrize("name", ["c1", "c1b", "c2", "c3", "c4", "c5"])
def test_library_equals_oracle_on_the_named_configs(name):
    w = synth.CONFIGS[name](0)
    a, b = kap.compile_workload(w), orc.compile_workload(w)
    for k in KEYS:
        _same(a[k], b[k], k)
    # the masks count exactly the selected tokens
    bits = np.array([bin(int(m)).count("1") for m in a["plan_token_masks"]])
    per_seq = np.add.reduceat(bits, a["plan_indptr"][:-1])
    np.testing.assert_array_equal(per_seq, a["selected_tokens"])
    # retained ratio s (Eq. 4, in pages) lands near the stated budgets
    s = np.diff(a["plan_indptr"]) / ((w.ctx_len + 15) // 16)
    if name == "c4":
        assert np.all((s > 0.05) & (s < 0.06))
    if name == "c2":
        assert np.all((s > 0.09) & (s < 0.12))
    if name == "c5":
        full = w.force_full.astype(bool)
        assert full.sum() == 3 and np.all(s[full] == 1.0)
        assert np.all(a["plan_flags"][full] & kap.PLAN_FULL)


def test_s_max_and_flags():
    w = synth.config2(0, batch=2, L=2048, layers=1)
    w.s_max = 0.05
    a, b = kap.compile_workload(w), orc.compile_workload(w)
    assert np.all(a["plan_flags"] & kap.PLAN_S_HIGH)
    np.testing.assert_array_equal(a["plan_flags"], b["plan_flags"])


def _args(**kw):
    base = dict(ctx_len=[64], span_indptr=[0, 1], span_start=[0], span_len=[4], span_score=[1.0],
                budget_tokens=[64], n_sink=[1], n_recent=[1])
    base.update(kw)
    return base


@pytest.mark.parametrize("kw", [
    dict(ctx_len=[0]), dict(ctx_len=[-3]), dict(budget_tokens=[-1]), dict(span_len=[-1]),
    dict(span_score=[float("nan")]), dict(n_sink=[-1]), dict(n_recent=[-1]),
    dict(span_indptr=[0, -1]), dict(span_indptr=[1, 1]), dict(page_size=0),
    dict(bt_indptr=[0, 3], bt_pages=[0, 1, 2]),           # 64 tokens need 4 pages
    dict(bt_indptr=[0, 4], bt_pages=[0, 1, -2, 3]),
])
def test_invalid_arguments_leave_outputs_untouched(kw):
    with pytest.raises(kap.KapError) as e:
        kap.compile_plan(**_args(**kw))
    assert e.value.code == kap.ERR_INVALID_ARG
    assert kap.lib().kap_last_error()            # a message was recorded


def test_capacity_error_and_untouched_outputs():
    import ctypes as C
    ctx = np.array([64, 64], dtype=np.int32)
    z = np.zeros(2, dtype=np.int32)
    indptr = np.full(3, -7, dtype=np.int32)
    pages = np.full(4, -7, dtype=np.int32)
    flags = np.full(2, -7, dtype=np.int32)
    p = lambda a, t=C.c_int32: a.ctypes.data_as(C.POINTER(t))
    sink = np.array([64, 64], dtype=np.int32)
    bud = np.array([64, 64], dtype=np.int32)
    rc = kap.lib().kap_compile_plan(2, 16, p(ctx), p(np.zeros(3, dtype=np.int32)), None, None, None,
                                    p(bud), p(sink), p(z), None, 1.0, None, None, 4, p(indptr),
                                    p(pages), None, p(flags), None, None)
    assert rc == kap.ERR_CAPACITY                  # 8 pages needed, 4 offered
    assert np.all(indptr == -7) and np.all(pages == -7) and np.all(flags == -7)
    pages = np.full(8, -7, dtype=np.int32)
    rc = kap.lib().kap_compile_plan(2, 16, p(ctx), p(np.zeros(3, dtype=np.int32)), None, None, None,
                                    p(bud), p(sink), p(z), None, 1.0, None, None, 8, p(indptr),
                                    p(pages), None, p(flags), None, None)
    assert rc == kap.OK and indptr.tolist() == [0, 4, 8] and pages.tolist() == [0, 1, 2, 3] * 2


def test_empty_batch():
    r = kap.compile_plan(np.zeros(0, np.int32), [0], [], [], [], [], [], [])
    assert r["plan_indptr"].tolist() == [0]
