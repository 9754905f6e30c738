"""Pins for the CPU oracle: what the paper's algorithm and the mathematics fix, checked against
something other than the oracle itself (a hand-worked fixture, closed forms, scipy's softmax and
logsumexp, a set-based / dense numpy brute force).  No GPU needed."""
import numpy as np
import pytest
import scipy.special

from helpers import read_plan_fixture
from oracle import brute
from oracle import kap_oracle as orc
from paper_2607_24260_b200 import synth

P = 16


# ------------------------------------------------------------------------------------------ plan
def _compile_one(L, spans, budget, sink, recent, bt=None, force=0, s_max=1.0, page=P):
    n = len(spans)
    st = [s[0] for s in spans]
    ln = [s[1] for s in spans]
    sc = [s[2] for s in spans]
    kw = {}
    if bt is not None:
        kw = dict(bt_indptr=[0, len(bt)], bt_pages=bt)
    return orc.compile_plan([L], [0, n], st, ln, sc, [budget], [sink], [recent],
                            force_full=[force], s_max=s_max, page_size=page, **kw)


def test_plan_hand_worked_fixture():
    fx = read_plan_fixture("plan_worked_example.txt")
    r = _compile_one(fx["ctx_len"], fx["spans"], fx["budget"], fx["n_sink"], fx["n_recent"],
                     bt=fx["block_table"], page=fx["page_size"])
    assert r["plan_logical_pages"].tolist() == fx["expect_logical"]
    assert r["plan_phys_pages"].tolist() == fx["expect_phys"]
    assert int(r["selected_tokens"][0]) == fx["expect_selected_tokens"]
    assert int(r["plan_flags"][0]) == fx["expect_flags"]
    L, ps = fx["ctx_len"], fx["page_size"]
    visible = sum(min(ps, L - p * ps) for p in r["plan_logical_pages"])
    assert visible == fx["expect_visible_tokens"]


def test_plan_fixture_variants_change_the_answer():
    """Plausible mistakes must move the fixture's answer: stopping at the first misfit, truncating
    a span, ranking ties by index instead of start."""
    fx = read_plan_fixture("plan_worked_example.txt")
    spans = fx["spans"]
    # stop-at-first-misfit would drop F (70-74) and so page 4
    assert 4 in _compile_one(100, spans, 48, 4, 8)["plan_logical_pages"]
    # C and B tie on score; swapping the input order must not change the result (start decides)
    swapped = [spans[0], spans[2], spans[1]] + spans[3:]
    a = _compile_one(100, spans, 48, 4, 8)
    b = _compile_one(100, swapped, 48, 4, 8)
    assert a["plan_logical_pages"].tolist() == b["plan_logical_pages"].tolist()
    # with one more token of budget nothing changes; with 51 C fits instead of F's partner set
    assert _compile_one(100, spans, 49, 4, 8)["selected_tokens"][0] == 44
    r51 = _compile_one(100, spans, 51, 4, 8)
    assert r51["selected_tokens"][0] == 51 and 3 in r51["plan_logical_pages"]


def test_plan_special_cases():
    L = 1000
    n_pages = (L + P - 1) // P
    # one span covering everything and an open budget: every page
    r = _compile_one(L, [(0, L, 1.0)], L, 0, 0)
    assert r["plan_logical_pages"].tolist() == list(range(n_pages))
    assert r["selected_tokens"][0] == L
    # nothing selected: exactly the page of the last token
    r = _compile_one(L, [], L, 0, 0)
    assert r["plan_logical_pages"].tolist() == [n_pages - 1]
    assert r["selected_tokens"][0] == 1
    # mandatory set alone exceeds the budget: flagged, spans ignored, mandatory kept
    r = _compile_one(L, [(500, 10, 9.0)], 10, 32, 32)
    assert r["plan_flags"][0] & orc.PLAN_OVER_BUDGET
    assert r["plan_logical_pages"].tolist() == [0, 1, 60, 61, 62]
    assert r["selected_tokens"][0] == 64
    # fallback: all pages, FULL flag
    r = _compile_one(L, [(3, 5, 1.0)], 50, 4, 4, force=1)
    assert r["plan_flags"][0] & orc.PLAN_FULL
    assert r["plan_logical_pages"].tolist() == list(range(n_pages))
    # retained ratio s (Eq. 4) above s_max raises S_HIGH; below it does not
    r = _compile_one(L, [(0, 512, 1.0)], L, 0, 0, s_max=0.5)       # 32 + last page = 33/63
    assert r["plan_flags"][0] & orc.PLAN_S_HIGH
    r = _compile_one(L, [(0, 256, 1.0)], L, 0, 0, s_max=0.5)
    assert not (r["plan_flags"][0] & orc.PLAN_S_HIGH)
    # sink and recent overlapping in a short context are counted once
    r = _compile_one(10, [], 100, 8, 8)
    assert r["selected_tokens"][0] == 10 and r["plan_logical_pages"].tolist() == [0]


def test_plan_rejects_bad_input():
    for kw in (dict(L=0), dict(budget=-1), dict(spans=[(0, -1, 1.0)]),
               dict(spans=[(0, 5, float("nan"))]), dict(sink=-1), dict(recent=-2)):
        args = dict(L=64, spans=[(0, 4, 1.0)], budget=64, sink=1, recent=1)
        args.update(kw)
        with pytest.raises(orc.OracleError) as e:
            _compile_one(args["L"], args["spans"], args["budget"], args["sink"], args["recent"])
        assert e.value.code == orc.INVALID
    with pytest.raises(orc.OracleError) as e:
        orc.compile_plan([64], [0, 0], [], [], [], [64], [64], [0], capacity=2)
    assert e.value.code == orc.CAPACITY


def test_plan_invariants_and_bruteforce_random():
    """>= 10^4 random tiny sequences: C oracle == set-based brute force, plus structural
    invariants (ascending unique pages in range, budget respected, last page present,
    lower-ranked additions never remove higher-ranked pages)."""
    n_seq = 0
    for seed in range(3400):
        w = synth.tiny_random(seed, batch=3, max_len=200, max_spans=12)
        r = orc.compile_workload(w)
        for b in range(w.batch):
            L = int(w.ctx_len[b])
            lo, hi = w.span_indptr[b], w.span_indptr[b + 1]
            spans = list(zip(w.span_start[lo:hi].tolist(), w.span_len[lo:hi].tolist(),
                             w.span_score[lo:hi].tolist()))
            pages, n_tok, over = brute.plan_pages(L, spans, int(w.budget_tokens[b]),
                                                  int(w.n_sink[b]), int(w.n_recent[b]),
                                                  w.page_size, bool(w.force_full[b]))
            got = r["plan_logical_pages"][r["plan_indptr"][b]:r["plan_indptr"][b + 1]]
            assert got.tolist() == pages, (seed, b)
            assert int(r["selected_tokens"][b]) == n_tok
            assert bool(r["plan_flags"][b] & orc.PLAN_OVER_BUDGET) == over
            n_pages = (L + w.page_size - 1) // w.page_size
            assert np.all(np.diff(got) > 0) and got[0] >= 0 and got[-1] == n_pages - 1
            if not over and not w.force_full[b]:
                assert n_tok <= w.budget_tokens[b]
            phys = r["plan_phys_pages"][r["plan_indptr"][b]:r["plan_indptr"][b + 1]]
            bt = w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b + 1]]
            assert phys.tolist() == bt[got].tolist()
            # token masks: bit t of page p <=> token p*P + t is in the brute-force union U
            tokens = (set(range(L)) if w.force_full[b] else
                      brute.plan_tokens(L, spans, int(w.budget_tokens[b]), int(w.n_sink[b]),
                                        int(w.n_recent[b]))[0])
            masks = r["plan_token_masks"][r["plan_indptr"][b]:r["plan_indptr"][b + 1]]
            from_masks = {int(pg) * w.page_size + t for pg, m in zip(got, masks)
                          for t in range(w.page_size) if (int(m) >> t) & 1}
            assert from_masks == tokens, (seed, b)
            assert np.all(masks != 0)
            n_seq += 1
    assert n_seq >= 10_000


def test_plan_lower_ranked_span_never_evicts():
    for seed in range(300):
        rng = synth.rng_for(seed, "evict")
        L = int(rng.integers(50, 400))
        n = int(rng.integers(1, 10))
        spans = [(int(rng.integers(0, L)), int(rng.integers(1, 60)), float(10 + n - i))
                 for i in range(n)]
        budget = int(rng.integers(20, L))
        base = set(_compile_one(L, spans, budget, 4, 8)["plan_logical_pages"].tolist())
        extra = spans + [(int(rng.integers(0, L)), int(rng.integers(1, 60)), 1.0)]
        more = set(_compile_one(L, extra, budget, 4, 8)["plan_logical_pages"].tolist())
        assert base <= more


# ------------------------------------------------------------------------------------- attention
def _small_case(seed, L=150, n_q=3, Hq=8, Hkv=2, d=32, spare=5, q_std=1.0, kv_std=0.5):
    rng = synth.rng_for(seed, "attn-small")
    n_pages = (L + P - 1) // P
    pool_pages = n_pages + spare
    bt = rng.permutation(pool_pages)[:n_pages].astype(np.int32)
    pool = synth.normal_bf16((pool_pages, 2, Hkv, P, d), kv_std, rng)
    q = synth.normal_bf16((n_q, Hq, d), q_std, rng)
    return dict(L=L, n_q=n_q, Hq=Hq, Hkv=Hkv, d=d, n_pages=n_pages, bt=bt, pool=pool, q=q,
                rng=rng)


def _decode(c, logical, q=None, pool=None, L=None, masks=None):
    logical = np.asarray(logical, dtype=np.int32)
    q = c["q"][-1:] if q is None else q
    return orc.selected_decode_attn(q, c["pool"] if pool is None else pool, [0, len(logical)],
                                    c["bt"][logical], logical, [c["L"] if L is None else L],
                                    plan_token_masks=masks)


def _verify(c, q=None, pool=None):
    q = c["q"] if q is None else q
    return orc.verify_attn(q, [0, q.shape[0]], c["pool"] if pool is None else pool,
                           [0, c["n_pages"]], c["bt"], [c["L"]])


def test_attention_matches_scipy_softmax_on_full_context():
    """All-pages plan == textbook attention computed with scipy's softmax / logsumexp."""
    c = _small_case(1)
    out, lse, ws, nv = _decode(c, np.arange(c["n_pages"]))
    q = synth.bf16_bits_to_f64(c["q"][-1])
    pool = synth.bf16_bits_to_f64(c["pool"])
    G = c["Hq"] // c["Hkv"]
    for h in range(c["Hq"]):
        K = pool[c["bt"], 0, h // G].reshape(-1, c["d"])[:c["L"]]
        V = pool[c["bt"], 1, h // G].reshape(-1, c["d"])[:c["L"]]
        z = (K @ q[h]) / np.sqrt(c["d"])
        np.testing.assert_allclose(out[0, h], scipy.special.softmax(z) @ V, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(lse[0, h], scipy.special.logsumexp(z), rtol=1e-12)
    assert np.all(nv == c["L"])
    np.testing.assert_allclose(ws, 1.0, rtol=1e-12)


@pytest.mark.parametrize("seed", range(6))
def test_selected_view_equals_masked_full_attention(seed):
    """Selected-view attention == full attention with the unselected logits at -inf (dense numpy
    brute force), for decode and for every verification row; weights sum to one."""
    c = _small_case(10 + seed, L=int(synth.rng_for(seed, "L").integers(20, 260)),
                    n_q=int(synth.rng_for(seed, "nq").integers(1, 9)))
    rng = c["rng"]
    keep = rng.random(c["n_pages"]) < 0.4
    keep[-1] = True
    logical = np.nonzero(keep)[0]
    out, lse, ws, nv = _decode(c, logical)
    b_out, b_lse, b_w = brute.dense_attention(c["q"][-1:], c["pool"], c["bt"], c["L"], logical, 1)
    np.testing.assert_allclose(out, b_out, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse, b_lse, rtol=1e-11)
    np.testing.assert_allclose(ws, 1.0, rtol=1e-12)
    assert np.all(nv[0] == np.count_nonzero(b_w[0, 0]))
    # weights outside the plan are exactly zero in the brute force
    tok_page = np.arange(c["L"]) // P
    assert np.all(b_w[0][:, ~keep[tok_page]] == 0.0)
    # verification: all pages, causal among the rows
    v_out, v_lse, v_ws, v_nv = _verify(c)
    b_out, b_lse, b_w = brute.dense_attention(c["q"], c["pool"], c["bt"], c["L"],
                                              range(c["n_pages"]), c["n_q"])
    np.testing.assert_allclose(v_out, b_out, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(v_lse, b_lse, rtol=1e-11)
    for j in range(c["n_q"]):
        assert np.all(v_nv[j] == c["L"] - c["n_q"] + j + 1)


def _random_token_masks(c, logical, rng, density=0.5):
    """Per listed page a random non-empty 16-bit mask; returns (masks, set of visible tokens)."""
    masks = np.zeros(len(logical), dtype=np.uint16)
    tokens = set()
    for i, lp in enumerate(logical):
        bits = rng.random(P) < density
        bits[int(rng.integers(0, min(P, c["L"] - lp * P)))] = True
        masks[i] = sum(1 << t for t in range(P) if bits[t])
        tokens |= {int(lp) * P + t for t in range(P) if bits[t] and lp * P + t < c["L"]}
    return masks, tokens


@pytest.mark.parametrize("seed", range(6))
def test_token_masked_view_equals_dense_attention_over_the_token_set(seed):
    """Token-granular visibility: the masked page-list attention equals dense attention in which
    exactly the tokens whose bit is set may be seen (numpy brute force over token positions);
    bits beyond the context end are ignored; an all-ones mask changes nothing."""
    c = _small_case(40 + seed, L=int(synth.rng_for(seed, "Lm").integers(20, 260)))
    rng = c["rng"]
    keep = rng.random(c["n_pages"]) < 0.5
    keep[-1] = True
    logical = np.nonzero(keep)[0]
    masks, tokens = _random_token_masks(c, logical, rng)
    out, lse, ws, nv = _decode(c, logical, masks=masks)
    b_out, b_lse, b_w = brute.dense_attention(c["q"][-1:], c["pool"], c["bt"], c["L"], logical, 1,
                                              visible_tokens=tokens)
    np.testing.assert_allclose(out, b_out, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse, b_lse, rtol=1e-11)
    np.testing.assert_allclose(ws, 1.0, rtol=1e-12)
    assert np.all(nv == len(tokens))
    hidden = np.ones(c["L"], dtype=bool)
    hidden[sorted(tokens)] = False
    assert np.all(b_w[0][:, hidden] == 0.0)
    full = _decode(c, logical, masks=np.full(len(logical), 0xFFFF, dtype=np.uint16))
    plain = _decode(c, logical)
    for a, b in zip(full, plain):
        assert np.array_equal(a, b)


def test_token_mask_closed_form_and_planted_key():
    """q = 0 under a token mask: lse = ln(#set bits inside the context) and out = mean of exactly
    those value rows.  A dominant key at a token whose bit is clear leaves the result unchanged;
    setting the bit makes the output that token's value row."""
    c = _small_case(5, L=203)
    logical = np.array([0, 2, 3, 7, c["n_pages"] - 1])
    masks = np.array([0x0001, 0x8000, 0x0F0F, 0xFFFE, 0xFFFF], dtype=np.uint16)
    tokens = [lp * P + t for lp, m in zip(logical, masks) for t in range(P)
              if (int(m) >> t) & 1 and lp * P + t < c["L"]]
    q0 = np.zeros_like(c["q"][-1:])
    out, lse, _, nv = _decode(c, logical, q=q0, masks=masks)
    assert np.all(nv == len(tokens))
    np.testing.assert_allclose(lse, np.log(len(tokens)), rtol=1e-14)
    pool = synth.bf16_bits_to_f64(c["pool"])
    G = c["Hq"] // c["Hkv"]
    for h in range(c["Hq"]):
        rows = np.stack([pool[c["bt"][t // P], 1, h // G, t % P] for t in tokens])
        np.testing.assert_allclose(out[0, h], rows.mean(0), rtol=1e-12, atol=1e-14)
    # planted key at token 7*P + 0 (bit 0 of mask 0xFFFE is clear)
    head, token = 3, 7 * P
    planted = c["pool"].copy()
    _plant_key(c, planted, token, c["q"][-1], head)
    base = _decode(c, logical, masks=masks)
    hidden = _decode(c, logical, pool=planted, masks=masks)
    np.testing.assert_array_equal(hidden[0][0, head], base[0][0, head])
    masks_on = masks.copy()
    masks_on[3] = 0xFFFF
    seen = _decode(c, logical, pool=planted, masks=masks_on)
    v_row = synth.bf16_bits_to_f64(planted)[c["bt"][7], 1, head // G, 0]
    np.testing.assert_allclose(seen[0][0, head], v_row, atol=1e-9)


def test_uniform_attention_closed_form():
    """q = 0: out is the mean of the visible value rows and lse = ln(n_visible), exactly."""
    c = _small_case(3, L=203)
    logical = np.array([0, 2, 3, 7, c["n_pages"] - 1])
    q0 = np.zeros_like(c["q"][-1:])
    out, lse, _, nv = _decode(c, logical, q=q0)
    n_vis = 4 * P + (c["L"] - (c["n_pages"] - 1) * P)
    assert np.all(nv == n_vis)
    np.testing.assert_allclose(lse, np.log(n_vis), rtol=1e-14)
    pool = synth.bf16_bits_to_f64(c["pool"])
    G = c["Hq"] // c["Hkv"]
    for h in range(c["Hq"]):
        rows = [pool[c["bt"][p], 1, h // G, :min(P, c["L"] - p * P)] for p in logical]
        np.testing.assert_allclose(out[0, h], np.concatenate(rows).mean(0), rtol=1e-12, atol=1e-14)


def test_page_coverage_probe():
    """q = 0 and V[t, j] = 1 iff (page of t) mod d == j: out[j] counts the visible tokens per
    page residue, so a dropped / duplicated / wrong page shows in a known coordinate.  Keyed once
    by logical page (checks the page list) and once by physical page (checks the block table)."""
    c = _small_case(4, L=500, d=32)
    logical = np.array([1, 2, 9, 17, 30, c["n_pages"] - 1])
    q0 = np.zeros_like(c["q"][-1:])
    one = synth.f32_to_bf16_bits(np.array([1.0], dtype=np.float32))[0]
    for keyed_by in ("logical", "physical"):
        pool = c["pool"].copy()
        pool[:, 1] = 0
        for lp in range(c["n_pages"]):
            key = lp if keyed_by == "logical" else int(c["bt"][lp])
            pool[c["bt"][lp], 1, :, :, key % c["d"]] = one
        out, _, _, nv = _decode(c, logical, q=q0, pool=pool)
        expect = np.zeros(c["d"])
        for lp in logical:
            key = lp if keyed_by == "logical" else int(c["bt"][lp])
            expect[key % c["d"]] += min(P, c["L"] - lp * P)
        expect /= expect.sum()
        for h in range(c["Hq"]):
            np.testing.assert_allclose(out[0, h], expect, rtol=1e-13, atol=1e-15)


def _plant_key(c, pool, token, q_row, head, margin=60.0):
    """Make token's key (in the KV head of `head`) score `margin` (scaled logit) for q_row/head."""
    G = c["Hq"] // c["Hkv"]
    q = synth.bf16_bits_to_f64(q_row[head])
    k = q * (margin * np.sqrt(c["d"]) / (q @ q))
    lp, s = divmod(token, P)
    pool[c["bt"][lp], 0, head // G, s] = synth.f32_to_bf16_bits(k.astype(np.float32))


def test_one_hot_key_visible_and_invisible():
    c = _small_case(5, L=300)
    head = 5
    G = c["Hq"] // c["Hkv"]
    logical = np.array([0, 4, 11, c["n_pages"] - 1])
    base, base_lse, _, _ = _decode(c, logical)
    # a dominant key inside the plan: the output is that token's value row
    pool = c["pool"].copy()
    tok = 4 * P + 7
    _plant_key(c, pool, tok, c["q"][-1], head)
    out, lse, _, _ = _decode(c, logical, pool=pool)
    v = synth.bf16_bits_to_f64(pool[c["bt"][4], 1, head // G, 7])
    np.testing.assert_allclose(out[0, head], v, atol=1e-9)
    assert abs(lse[0, head] - 60.0) < 0.5
    # the same key in a page outside the plan changes nothing
    pool = c["pool"].copy()
    _plant_key(c, pool, 5 * P + 3, c["q"][-1], head)
    out2, lse2, _, _ = _decode(c, logical, pool=pool)
    np.testing.assert_array_equal(out2, base)
    np.testing.assert_array_equal(lse2, base_lse)


def test_verify_causality_with_planted_key():
    """A dominant key at position p_j + 1 is ignored by rows <= j and wins rows > j."""
    c = _small_case(6, L=211, n_q=6)
    head, G = 2, c["Hq"] // c["Hkv"]
    j = 2
    tok = c["L"] - c["n_q"] + j + 1
    pool = c["pool"].copy()
    # the same q vector in every row so that one key dominates all of them
    q = np.repeat(c["q"][:1], c["n_q"], axis=0)
    _plant_key(c, pool, tok, q[0], head)
    base, _, _, _ = _verify(c, q=q)
    out, _, _, _ = _verify(c, q=q, pool=pool)
    lp, s = divmod(tok, P)
    v = synth.bf16_bits_to_f64(pool[c["bt"][lp], 1, head // G, s])
    for r in range(c["n_q"]):
        if r <= j:
            np.testing.assert_array_equal(out[r, head], base[r, head])
        else:
            np.testing.assert_allclose(out[r, head], v, atol=1e-9)


def test_verify_last_row_equals_identity_plan_decode():
    c = _small_case(7, L=190, n_q=5)
    v_out, v_lse, _, _ = _verify(c)
    d_out, d_lse, _, _ = _decode(c, np.arange(c["n_pages"]))
    np.testing.assert_allclose(v_out[-1], d_out[0], rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(v_lse[-1], d_lse[0], rtol=1e-13)
    # row j of an n_q-row verification == decode of a context truncated to that row's position
    for j in range(c["n_q"] - 1):
        Lj = c["L"] - c["n_q"] + j + 1
        npg = (Lj + P - 1) // P
        o, l, _, _ = _decode(c, np.arange(npg), q=c["q"][j:j + 1], L=Lj)
        np.testing.assert_allclose(v_out[j], o[0], rtol=1e-13, atol=1e-15)


def test_page_list_order_and_gqa_mapping():
    c = _small_case(8, L=260)
    logical = np.array([0, 3, 5, 8, 12, c["n_pages"] - 1])
    a, al, _, _ = _decode(c, logical)
    perm = c["rng"].permutation(len(logical))
    b, bl, _, _ = _decode(c, logical[perm])
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(al, bl, rtol=1e-13)
    # V of KV head g constant g+1: every query head of group g returns g+1
    pool = c["pool"].copy()
    for g in range(c["Hkv"]):
        pool[:, 1, g] = synth.f32_to_bf16_bits(np.array([g + 1.0], dtype=np.float32))[0]
    out, _, _, _ = _decode(c, logical, pool=pool)
    G = c["Hq"] // c["Hkv"]
    for h in range(c["Hq"]):
        np.testing.assert_allclose(out[0, h], h // G + 1.0, rtol=1e-13)


def test_scale_argument_and_batching():
    """scale is applied to the logits (doubling it == doubling q for power-of-two exact bf16
    scaling), and sequences in a batch are independent of each other."""
    c = _small_case(9, L=120, n_q=2)
    logical = np.arange(c["n_pages"])
    q2 = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(c["q"][-1:]) * 2.0)
    s = 1.0 / np.sqrt(c["d"])
    a = orc.selected_decode_attn(q2, c["pool"], [0, len(logical)], c["bt"][logical], logical,
                                 [c["L"]], scale=s)
    b = orc.selected_decode_attn(c["q"][-1:], c["pool"], [0, len(logical)], c["bt"][logical],
                                 logical, [c["L"]], scale=2 * s)
    np.testing.assert_allclose(a[0], b[0], rtol=1e-12, atol=1e-14)
    # two copies of the sequence in one batch, second with a shorter plan
    qq = np.concatenate([c["q"][-1:], c["q"][-1:]])
    short = logical[::2] if logical[-1] in logical[::2] else np.append(logical[::2], logical[-1])
    both = orc.selected_decode_attn(qq, c["pool"], [0, len(logical), len(logical) + len(short)],
                                    np.concatenate([c["bt"][logical], c["bt"][short]]),
                                    np.concatenate([logical, short]), [c["L"], c["L"]])
    one = _decode(c, short)
    np.testing.assert_array_equal(both[0][1], one[0][0])
    np.testing.assert_array_equal(both[0][0], _decode(c, logical)[0][0])


def test_append_then_attend_equals_attention_over_the_longer_context():
    """Slot-mapping pin: appending tokens one by one and decoding after each append equals the
    dense brute force over a pool that held those tokens from the start."""
    c = _small_case(12, L=90, n_q=1, spare=4)
    rng = c["rng"]
    k_steps = 5
    n_pages_end = (c["L"] + k_steps + P - 1) // P
    extra = n_pages_end - c["n_pages"]
    free = [p for p in range(c["pool"].shape[0]) if p not in set(c["bt"].tolist())]
    bt = np.concatenate([c["bt"], np.asarray(free[:extra], dtype=np.int32)])
    k_new = synth.normal_bf16((k_steps, c["Hkv"], c["d"]), 0.5, rng)
    v_new = synth.normal_bf16((k_steps, c["Hkv"], c["d"]), 0.5, rng)
    q = synth.normal_bf16((k_steps, c["Hq"], c["d"]), 1.0, rng)
    final = c["pool"].copy()
    brute.append_kv(final, bt, c["L"], k_new, v_new)
    pool, L = c["pool"].copy(), c["L"]
    for t in range(k_steps):
        L = brute.append_kv(pool, bt, L, k_new[t:t + 1], v_new[t:t + 1])
        n_pages = (L + P - 1) // P
        logical = np.arange(n_pages, dtype=np.int32)
        out, lse, _, nv = orc.selected_decode_attn(q[t:t + 1], pool, [0, n_pages], bt[logical], logical, [L])
        b_out, b_lse, _ = brute.dense_attention(q[t:t + 1], final, bt, L, range(n_pages), 1)
        np.testing.assert_allclose(out, b_out, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(lse, b_lse, rtol=1e-11)
        assert np.all(nv == L)


def test_append_kv_writes_exactly_the_slot_the_mapping_names():
    """Slot mapping by direct indexing (Section 3.1: token at logical position pos lives in page
    block_table[pos // P], slot pos % P): after one append of a K row and a different V row, exactly
    those two (page, K|V, :, slot) strips changed, they hold K and V respectively, and every other
    word of the pool is untouched.  Crosses a page boundary (L % 16 in {0, 15}) and appends
    several tokens at once."""
    c = _small_case(21, L=95, n_q=1, spare=6)
    free = [p for p in range(c["pool"].shape[0]) if p not in set(c["bt"].tolist())]
    bt = np.concatenate([c["bt"], np.asarray(free[:2], dtype=np.int32)])
    for L, n_new in ((95, 1), (96, 1), (90, 3), (94, 5)):
        k_new = np.empty((n_new, c["Hkv"], c["d"]), dtype=np.uint16)
        v_new = np.empty_like(k_new)
        for j in range(n_new):                   # distinctive words no random bf16 draw produces
            k_new[j] = 0x4100 + 2 * j + np.arange(c["Hkv"])[:, None] * 16
            v_new[j] = 0xC200 + 2 * j + np.arange(c["Hkv"])[:, None] * 16 + 1
        before = c["pool"].copy()
        pool = c["pool"].copy()
        assert brute.append_kv(pool, bt, L, k_new, v_new) == L + n_new
        changed = np.zeros(pool.shape, dtype=bool)
        for j in range(n_new):
            pos = L + j
            page, slot = int(bt[pos // P]), pos % P
            np.testing.assert_array_equal(pool[page, 0, :, slot, :], k_new[j])
            np.testing.assert_array_equal(pool[page, 1, :, slot, :], v_new[j])
            changed[page, :, :, slot, :] = True
        np.testing.assert_array_equal(pool[~changed], before[~changed])
        assert changed.sum() == n_new * 2 * c["Hkv"] * c["d"]


@pytest.mark.parametrize("L", [95, 96, 111, 112])
def test_append_kv_then_decode_returns_the_appended_value(L):
    """Closed form through the C oracle: append a key that dominates the softmax (scaled logit 60)
    together with a known value row; full-context decode at L + 1 must return that value row for
    the planted head.  A K/V swap, a wrong slot or a wrong page fails it."""
    c = _small_case(22, L=L, n_q=1, spare=6)
    free = [p for p in range(c["pool"].shape[0]) if p not in set(c["bt"].tolist())]
    bt = np.concatenate([c["bt"], np.asarray(free[:1], dtype=np.int32)])
    head, G = 3, c["Hq"] // c["Hkv"]
    q = synth.bf16_bits_to_f64(c["q"][-1][head])
    k_row = synth.normal_bf16((1, c["Hkv"], c["d"]), 0.5, c["rng"])
    k_row[0, head // G] = synth.f32_to_bf16_bits((q * (60.0 * np.sqrt(c["d"]) / (q @ q))).astype(np.float32))
    v_row = synth.f32_to_bf16_bits(np.linspace(-3.0, 3.0, c["Hkv"] * c["d"], dtype=np.float32)
                                   ).reshape(1, c["Hkv"], c["d"])
    pool = c["pool"].copy()
    L1 = brute.append_kv(pool, bt, L, k_row, v_row)
    assert L1 == L + 1
    n_pages = (L1 + P - 1) // P
    logical = np.arange(n_pages, dtype=np.int32)
    out, lse, _, nv = orc.selected_decode_attn(c["q"][-1:], pool, [0, n_pages], bt[logical], logical, [L1])
    np.testing.assert_allclose(out[0, head], synth.bf16_bits_to_f64(v_row[0, head // G]), atol=1e-9)
    assert abs(lse[0, head] - 60.0) < 0.5 and np.all(nv == L1)
    # one token short of the append the key is not there yet
    out0, lse0, _, _ = orc.selected_decode_attn(c["q"][-1:], pool, [0, (L + P - 1) // P],
                                                bt[:(L + P - 1) // P], logical[:(L + P - 1) // P], [L])
    assert lse0[0, head] < 30.0


def test_materialize_view_hand_worked():
    """The compact copy on a pool worked by hand: five pages, page p filled with the constant
    100 + p, plan [3, 0, 3] -> compact pages hold 103, 100, 103 and are numbered 0, 1, 2; the
    source pool is not modified and the copy does not alias it."""
    pool = np.empty((5, 2, 2, P, 4), dtype=np.uint16)
    for p in range(5):
        pool[p] = 100 + p
    pool[3, 1] = 203                              # V half of page 3 differs from its K half
    keep = pool.copy()
    compact, ids = brute.materialize_view(pool, [3, 0, 3])
    assert compact.shape == (3, 2, 2, P, 4) and ids.tolist() == [0, 1, 2]
    assert np.all(compact[0, 0] == 103) and np.all(compact[0, 1] == 203)
    assert np.all(compact[1] == 100)
    assert np.all(compact[2, 0] == 103) and np.all(compact[2, 1] == 203)
    compact[0] = 7
    np.testing.assert_array_equal(pool, keep)
    empty, ids0 = brute.materialize_view(pool, [])
    assert empty.shape[0] == 0 and len(ids0) == 0


# --------------------------------------------------------------------------- Top-3 acceptance
def test_top3_accept_hand_cases():
    """Eq. 2 with the Top-3 rule on a window worked by hand (k = 3, vocab 6)."""
    logits = np.array([
        [0.1, 2.0, 0.3, 1.5, 1.0, -1.0],     # top3 = 1, 3, 4
        [5.0, 5.0, 5.0, 5.0, 0.0, 0.0],      # ties: lowest indices first -> 0, 1, 2
        [0.0, np.nan, 3.0, 1.0, 2.0, np.nan],  # NaN ranks last -> 2, 4, 3
        [9.0, 0.0, 0.0, 0.0, 0.0, 8.0],      # bonus row -> 0, 5, 1
    ], dtype=np.float32)
    cases = [
        ([4, 2, 3, 0], 3, 0),     # all three accepted (3rd-best, tie-ranked 3rd, 3rd-best) -> bonus row's best
        ([4, 3, 3, 0], 1, 0),     # second proposal (3) is the 4th of the tie -> m = 1, carry = best of row 1
        ([0, 0, 2, 0], 0, 1),     # first proposal outside the top 3 -> m = 0, carry = best of row 0
        ([1, 1, 1, 0], 2, 2),     # NaN-valued token 1 is not a candidate of row 2 -> m = 2, carry = 2
    ]
    # NaN ranks below -inf, signed zeros tie (lower index first)
    edge = np.array([[np.nan, -np.inf, -0.0, 0.0, np.nan, -np.inf]], dtype=np.float32)
    assert brute.top3_accept(edge, [0, 1], [0])[0].tolist() == [[2, 3, 1]]
    edge2 = np.array([[np.nan, -np.inf, np.nan, np.nan]], dtype=np.float32)
    assert brute.top3_accept(edge2, [0, 1], [0])[0].tolist() == [[1, 0, 2]]
    for proposed, want_m, want_next in cases:
        top3, m, nxt = brute.top3_accept(logits, [0, 4], proposed)
        assert top3.tolist() == [[1, 3, 4], [0, 1, 2], [2, 4, 3], [0, 5, 1]]
        assert (int(m[0]), int(nxt[0])) == (want_m, want_next), proposed


def test_top3_matches_argsort_and_prefix_definition():
    rng = synth.rng_for(0, "top3")
    x = rng.standard_normal((12, 1000)).astype(np.float32)
    indptr = [0, 5, 5, 12]                       # one empty window in the middle
    top3, m, nxt = brute.top3_accept(x, indptr, rng.integers(0, 1000, size=12))
    np.testing.assert_array_equal(top3, np.argsort(-x, axis=1, kind="stable")[:, :3])
    # proposing the 2nd-best token everywhere accepts everything; carry = best of the bonus row
    prop = top3[:, 1].copy()
    _, m, nxt = brute.top3_accept(x, indptr, prop)
    assert m.tolist() == [4, 0, 6] and nxt[0] == top3[4, 0] and nxt[2] == top3[11, 0]
    assert nxt[1] == -1                          # a window without rows has no carry to give
    prop[6] = int(np.argsort(x[6])[0])           # the worst token at the 2nd position of window 3 (rows 5..11)
    _, m, nxt = brute.top3_accept(x, indptr, prop)
    assert m.tolist() == [4, 0, 1] and nxt[2] == top3[6, 0]


def test_top3_empty_windows_accept_nothing_and_carry_minus_one():
    """A window with no row at all - first, in the middle, last - yields accepted = 0 and
    next = -1 and never reads a neighbour's row."""
    x = np.zeros((3, 8), dtype=np.float32)
    x[0, 5] = x[1, 6] = x[2, 7] = 1.0
    top3, m, nxt = brute.top3_accept(x, [0, 0, 2, 2, 3, 3], [5, 0, 0])
    assert m.tolist() == [0, 1, 0, 0, 0]
    assert nxt.tolist() == [-1, 6, -1, 7, -1]
