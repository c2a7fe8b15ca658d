"""Randomised invariants of the fp64 oracle (CPU only): properties that hold for any sizes and any mode."""
import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import CitrusOracle, SHARED, INDIVIDUAL, STANDARD, select_topk, intersection_ratio, rope


@settings(max_examples=60, deadline=None)
@given(st.integers(1, 60), st.integers(1, 70), st.integers(0, 2 ** 31 - 1), st.booleans())
def test_select_topk_keeps_exactly_the_largest_with_lower_index_winning_ties(n, k, seed, coarse):
    rng = np.random.default_rng(seed)
    s = rng.integers(0, 4, n).astype(np.float64) if coarse else rng.normal(size=n)     # coarse: many exact ties
    idx = select_topk(s, k)
    kept = min(n, k)
    assert idx.shape == (kept,) and np.all(np.diff(idx) > 0)
    if kept < n:
        out = np.setdiff1d(np.arange(n), idx)
        assert s[idx].min() >= s[out].max()
        t = s[idx].min()                                   # among candidates equal to the threshold the lowest indices stay
        eq_in, eq_out = idx[s[idx] == t], out[s[out] == t]
        assert eq_out.size == 0 or eq_in.max() < eq_out.min()


@settings(max_examples=25, deadline=None)
@given(st.sampled_from([SHARED, INDIVIDUAL, STANDARD]), st.integers(2, 12), st.integers(1, 9), st.integers(0, 2 ** 31 - 1),
       st.booleans(), st.booleans(), st.lists(st.integers(1, 9), min_size=1, max_size=6))
def test_cache_invariants_for_any_mode_budget_and_chunk_lengths(mode, k, w, seed, accumulate, deferred, lengths):
    rng = np.random.default_rng(seed)
    Hq, Hkv, D, nI = 4, 2, 4, 3
    deferred = deferred and mode != SHARED
    orc = CitrusOracle(Hq, Hkv, D, k, mode, lm_window=w, accumulate=accumulate, deferred_lm=deferred)
    ls = max(lengths)
    seen, rows0 = 0, 0
    K_doc, V_doc = [], []
    for i, L in enumerate(lengths):
        Q, K, V = rng.normal(size=(L, Hq, D)), rng.normal(size=(L, Hkv, D)), rng.normal(size=(L, Hkv, D))
        K_doc.append(K); V_doc.append(V)
        with_instr = mode != STANDARD or i == len(lengths) - 1
        res = orc.process_chunk(Q, K, V, rng.normal(size=(nI, Hq, D)) if with_instr else None)
        lm_scored = mode == INDIVIDUAL or (mode == STANDARD and not with_instr)
        rows0 = (min(rows0, k) + L) if (deferred and lm_scored) else min(rows0 + L, k)
        seen += L
        Kd, Vd = np.concatenate(K_doc), np.concatenate(V_doc)
        # attention rows are convex combinations of value rows: inside their per-dimension range
        assert np.all(res.out <= Vd.max() + 1e-9) and np.all(res.out >= Vd.min() - 1e-9)
        for cid, c in enumerate(orc.caches):
            expect = rows0 if cid == 0 else min(seen, k)
            assert c.K.shape[1] == c.V.shape[1] == c.pos.shape[1] == expect
            for g in range(Hkv):
                p = c.pos[g]
                assert np.all(np.diff(p) > 0) and p.min() >= 0 and p.max() < seen
                assert np.array_equal(c.K[g], Kd[p, g]) and np.array_equal(c.V[g], Vd[p, g])
            if accumulate:
                assert c.acc.shape == c.pos.shape and np.all(c.acc >= 0)
        for cid, S in res.scores.items():
            assert np.all(S >= 0)
            if not accumulate:                           # every scoring query spends one unit of attention per head
                rows = nI if (cid == 1 or not lm_scored) else min(w, L)
                assert np.allclose(S.sum(axis=1), rows * (Hq // Hkv), rtol=1e-9)
    if mode == INDIVIDUAL:
        r = intersection_ratio(orc.caches[0].pos, orc.caches[1].pos)
        assert np.all((0 <= r) & (r <= 1))


@settings(max_examples=25, deadline=None)
@given(st.integers(0, 2 ** 31 - 1), st.integers(1, 5), st.integers(1, 8), st.sampled_from([4, 8, 16]))
def test_position_shift_without_eviction_equals_up_front_embedding(seed, n_chunks, ls, D):
    rng = np.random.default_rng(seed)
    Hq, Hkv, nI, N = 2, 1, 2, n_chunks * ls
    Q, K, V, Qi = (rng.normal(size=s) for s in [(N, Hq, D), (N, Hkv, D), (N, Hkv, D), (nI, Hq, D)])
    a = CitrusOracle(Hq, Hkv, D, N + 1, SHARED, rope_shift=True, rope_base=100.0)
    b = CitrusOracle(Hq, Hkv, D, N + 1, SHARED)
    pos = np.arange(N)[:, None]
    Qr, Kr = rope(Q, pos, 100.0), rope(K, pos, 100.0)
    for c in range(0, N, ls):
        ra = a.process_chunk(Q[c:c + ls], K[c:c + ls], V[c:c + ls], Qi)
        rb = b.process_chunk(Qr[c:c + ls], Kr[c:c + ls], V[c:c + ls], rope(Qi, (c + ls + np.arange(nI))[:, None], 100.0))
        assert np.allclose(ra.out, rb.out, atol=1e-11) and np.allclose(ra.scores[0], rb.scores[0], atol=1e-11)
