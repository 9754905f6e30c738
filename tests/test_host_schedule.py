"""The split-K schedule (host, no GPU): every page of every (sequence, KV head) is covered exactly
once, partial slots are unique and contiguous per group, chunk sizes respect the cap, and the work
fits whole waves when it can."""
import numpy as np
import pytest

from paper_2607_24260_b200 import kap, synth


PROPOSAL_CAP, VERIFY_CAP = 512, 1536      # pages per CTA: plan lists (ids + logical + masks) / plain lists


def _verify_schedule(list_len, n_q, items, Hkv, cap, cluster=1):
    B = len(list_len)
    cover = [[np.zeros(int(list_len[b]), dtype=np.int32) for _ in range(Hkv)] for b in range(B)]
    slots = set()
    by_group = {}
    sizes = items[:, 3] - items[:, 2]
    assert np.all(sizes >= 1) and np.all(-(-sizes // cluster) <= cap)
    assert np.all(np.diff(sizes) <= 0), "items must be sorted longest first"
    for seq, g, p0, p1, group, slot, n_splits, nq in items.tolist():
        cover[seq][g][p0:p1] += 1
        assert slot not in slots
        slots.add(slot)
        by_group.setdefault(group, []).append((p0, slot, n_splits, seq, g))
        assert nq == (1 if n_q is None else int(n_q[seq]))
    for b in range(B):
        for g in range(Hkv):
            assert np.all(cover[b][g] == 1)
    assert len(by_group) == B * Hkv
    for group, parts in by_group.items():
        parts.sort()
        assert all(p[2] == len(parts) for p in parts)
        s = [p[1] for p in parts]
        assert s == list(range(s[0], s[0] + len(parts))), "a group's slots are contiguous in page order"
        assert len({(p[3], p[4]) for p in parts}) == 1
    assert slots == set(range(len(items)))


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4", "c5"])
def test_named_configs_schedules(name):
    w = synth.CONFIGS[name](0)
    plan = kap.compile_workload(w)
    n = np.diff(plan["plan_indptr"])
    slots = 296
    items, n_merge, max_chunk = kap.schedule_host(n, None, 32, 8, slots)
    _verify_schedule(n, None, items, 8, 512)
    assert max_chunk == (items[:, 3] - items[:, 2]).max()
    if name in ("c2", "c3", "c4"):
        # uniform batches fit one wave; inside a (sequence, KV head) chunks differ by <= 1 page
        assert len(items) <= slots
        sizes = items[:, 3] - items[:, 2]
        for group in np.unique(items[:, 4]):
            sz = sizes[items[:, 4] == group]
            assert sz.max() - sz.min() <= 1
        feasible = lambda t: int(np.sum(-(-n // t)) * 8) <= slots
        assert feasible(max_chunk) and not feasible(max_chunk - 1)
    pages = (w.ctx_len + 15) // 16
    items, n_merge, max_chunk = kap.schedule_host(pages, w.n_q, 32, 8, slots)
    _verify_schedule(pages, w.n_q, items, 8, VERIFY_CAP)


def test_random_shapes_and_caps():
    rng = synth.rng_for(0, "sched")
    for _ in range(200):
        B = int(rng.integers(1, 20))
        n = rng.integers(1, 3000, size=B).astype(np.int32)
        nq = rng.integers(1, 9, size=B).astype(np.int32) if rng.random() < 0.5 else None
        Hkv = int(rng.choice([1, 2, 8]))
        cap = int(rng.choice([0, 1, 3, 64, 512, 100000]))
        slots = int(rng.choice([4, 148, 296]))
        items, _, _ = kap.schedule_host(n, nq, Hkv * 4, Hkv, slots, cap, max_items=200000)
        hard = PROPOSAL_CAP if nq is None else VERIFY_CAP
        _verify_schedule(n, nq, items, Hkv, hard if cap <= 0 else min(cap, hard))


def test_single_wave_is_minimal_makespan():
    # one wave: the longest chunk is the smallest t with sum ceil(n / t) * Hkv <= slots
    n = np.array([100, 37, 512, 4], dtype=np.int32)
    items, _, max_chunk = kap.schedule_host(n, None, 32, 8, 296)
    feasible = lambda t: int(np.sum(-(-n // t)) * 8) <= 296
    assert len(items) <= 296 and feasible(max_chunk) and not feasible(max_chunk - 1)


def test_schedule_errors():
    for args in (([0], None), ([-1], None), ([4], [0])):
        with pytest.raises(kap.KapError) as e:
            kap.schedule_host(args[0], args[1], 32, 8, 296)
        assert e.value.code == kap.ERR_INVALID_ARG
    with pytest.raises(kap.KapError) as e:          # 17 rows * 4 heads > 64 rows
        kap.schedule_host([4], [17], 32, 8, 296)
    assert e.value.code == kap.ERR_UNSUPPORTED
    with pytest.raises(kap.KapError) as e:          # group size 3 does not divide 16
        kap.schedule_host([4], None, 24, 8, 296)
    assert e.value.code == kap.ERR_UNSUPPORTED
    with pytest.raises(kap.KapError) as e:          # 10 groups cannot fit 4 items
        kap.schedule_host([4] * 10, None, 4, 1, 296, 0, max_items=4)
    assert e.value.code == kap.ERR_CAPACITY


def test_cluster_schedules():
    """With clusters allowed the uniform configurations fit one cluster per (sequence, KV head):
    no merge pass, and the per-CTA chunk is the cluster's share."""
    for name, want_cluster in (("c2", 4), ("c3", 2)):
        w = synth.CONFIGS[name](0)
        n = np.diff(kap.compile_workload(w)["plan_indptr"])
        items, n_merge, max_chunk, cluster = kap.schedule_host(n, None, 32, 8, 296, max_cluster=16)
        _verify_schedule(n, None, items, 8, 512, cluster)
        assert cluster == want_cluster and n_merge == 0 and len(items) == w.batch * 8
        assert max_chunk == -(-int(n.max()) // cluster)
    rng = synth.rng_for(1, "sched-cluster")
    for _ in range(100):
        B = int(rng.integers(1, 40))
        n = rng.integers(1, 9000, size=B).astype(np.int32)
        nq = rng.integers(1, 9, size=B).astype(np.int32) if rng.random() < 0.5 else None
        mc = int(rng.choice([2, 3, 4, 8, 13, 16]))
        items, n_merge, max_chunk, cluster = kap.schedule_host(n, nq, 32, 8, int(rng.choice([296, 444])),
                                                               max_items=100000, max_cluster=mc)
        assert 1 <= cluster <= mc
        _verify_schedule(n, nq, items, 8, PROPOSAL_CAP if nq is None else VERIFY_CAP, cluster)


def test_short_lists_are_not_cut_into_single_pages():
    """One 4K sequence (45 selected pages per KV head, 256 for verification): a CTA per page plus a
    merge pass over dozens of partial states costs more than it spreads.  The candidates include
    launches that fill a half or a quarter of a wave and the merge pass is charged per batch of 16
    partial states, so the choice is a cluster per list (no merge pass) or a few pages per CTA."""
    items, n_merge, max_chunk, cluster = kap.schedule_host([45], None, 32, 8, 444, max_cluster=16)
    ctas = len(items) * cluster
    assert ctas <= 148 and max_chunk >= 3
    assert n_merge == 0 or max(items[:, 6]) <= 16
    items, n_merge, max_chunk = kap.schedule_host([256], [4], 32, 8, 444)
    assert len(items) <= 222 and max_chunk >= 8 and max(items[:, 6]) <= 32
    # long lists still fill the wave
    items, n_merge, max_chunk = kap.schedule_host([8192] * 4, [4] * 4, 32, 8, 444)
    assert len(items) >= 432
