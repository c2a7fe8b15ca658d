"""Pins for the fp64 oracle: closed forms, invariants, library special cases and
brute force on tiny inputs.  None of these re-type the oracle's formulas with
numpy; they use pure-Python loops, torch's library attention, or facts the
paper and the mathematics fix."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import CitrusOracle, SHARED, INDIVIDUAL, STANDARD
from paper_2406_12018_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand(rng, *shape):
    return rng.standard_normal(shape)


# ---------------------------------------------------------------- brute force
def brute_attention_row(q, keys, vals, visible):
    """One query row, pure Python floats."""
    D = len(q)
    logit = []
    for j in range(len(keys)):
        if not visible[j]:
            logit.append(None)
            continue
        acc = 0.0
        for d in range(D):
            acc += q[d] * keys[j][d]
        logit.append(acc / math.sqrt(D))
    mx = max(x for x in logit if x is not None)
    e = [0.0 if x is None else math.exp(x - mx) for x in logit]
    z = sum(e)
    p = [x / z for x in e]
    o = [sum(p[j] * vals[j][d] for j in range(len(keys))) for d in range(len(vals[0]))]
    return p, o


@pytest.mark.parametrize("Hq,Hkv,D,m,L", [(2, 1, 4, 3, 5), (4, 2, 4, 0, 6), (2, 2, 8, 7, 1)])
def test_a1_brute_force(Hq, Hkv, D, m, L):
    rng = np.random.default_rng(10 + m)
    Qc, Kc, Vc = rand(rng, L, Hq, D), rand(rng, L, Hkv, D), rand(rng, L, Hkv, D)
    Kcache, Vcache = rand(rng, Hkv, m, D), rand(rng, Hkv, m, D)
    w = min(2, L)
    out, s_lm = oracle.chunk_attention(Qc, Kcache, Vcache, Kc, Vc, lm_window=w)
    G = Hq // Hkv
    ref_lm = [[0.0] * (m + L) for _ in range(Hkv)]
    for h in range(Hq):
        g = h // G
        keys = [list(Kcache[g, j]) for j in range(m)] + [list(Kc[u, g]) for u in range(L)]
        vals = [list(Vcache[g, j]) for j in range(m)] + [list(Vc[u, g]) for u in range(L)]
        for t in range(L):
            visible = [True] * m + [u <= t for u in range(L)]
            p, o = brute_attention_row(list(Qc[t, h]), keys, vals, visible)
            assert np.allclose(out[t, h], o, rtol=0, atol=1e-12)
            if t >= L - w:
                for j in range(m + L):
                    ref_lm[g][j] += p[j]
    assert np.allclose(s_lm, np.array(ref_lm), rtol=0, atol=1e-12)


def test_a2_brute_force_and_rowsum():
    rng = np.random.default_rng(3)
    Hq, Hkv, D, m, L, nI = 4, 2, 4, 5, 3, 3
    Qi, Kc, Kcache = rand(rng, nI, Hq, D), rand(rng, L, Hkv, D), rand(rng, Hkv, m, D)
    S = oracle.importance_sum(Qi, Kcache, Kc)
    G = Hq // Hkv
    ref = [[0.0] * (m + L) for _ in range(Hkv)]
    for h in range(Hq):
        g = h // G
        keys = [list(Kcache[g, j]) for j in range(m)] + [list(Kc[u, g]) for u in range(L)]
        for i in range(nI):
            p, _ = brute_attention_row(list(Qi[i, h]), keys, keys, [True] * (m + L))
            assert abs(sum(p) - 1.0) < 1e-12
            for j in range(m + L):
                ref[g][j] += p[j]
    assert np.allclose(S, np.array(ref), rtol=0, atol=1e-12)
    # every (instruction token, head) distributes exactly one unit of attention
    assert np.allclose(S.sum(axis=1), nI * G, rtol=0, atol=1e-12)


# ------------------------------------------------------------- closed forms
def test_a2_zero_query_uniform_and_dominant_key():
    rng = np.random.default_rng(4)
    Hq, Hkv, D, m, L = 2, 1, 8, 6, 4
    Kc, Kcache = rand(rng, L, Hkv, D), rand(rng, Hkv, m, D)
    S = oracle.importance_sum(np.zeros((1, Hq, D)), Kcache, Kc)
    assert np.allclose(S, Hq / (m + L), atol=1e-15)             # q = 0 -> uniform 1/n per head
    # a key aligned with every query and 200x longer takes all of the mass
    Qi = np.abs(rand(rng, 5, Hq, D)) + 0.5
    Kc2 = Kc.copy()
    Kc2[2, 0] = 200.0 * np.ones(D)
    S2 = oracle.importance_sum(Qi, Kcache, Kc2)
    assert abs(S2[0, m + 2] - 5 * Hq) < 1e-9
    assert S2[0].sum() == pytest.approx(5 * Hq, abs=1e-12)


def test_a2_scale_is_inverse_sqrt_d():
    # two keys, one query: p0/p1 = exp((q.k0 - q.k1)/sqrt(D)) exactly
    D = 16
    q = np.zeros((1, 1, D)); q[0, 0, 0] = 2.0
    Kc = np.zeros((2, 1, D)); Kc[0, 0, 0] = 3.0; Kc[1, 0, 0] = 1.0
    S = oracle.importance_sum(q, np.zeros((1, 0, D)), Kc)
    assert S[0, 0] / S[0, 1] == pytest.approx(math.exp((6.0 - 2.0) / 4.0), rel=1e-13)


# ------------------------------------------------ library special case (a1)
def sdpa_full_causal(Q, K, V):
    """torch's library attention over the whole document, fp64, GQA by head repetition."""
    G = Q.shape[1] // K.shape[1]
    q = torch.from_numpy(Q).permute(1, 0, 2)[None]
    k = torch.from_numpy(np.repeat(K, G, axis=1)).permute(1, 0, 2)[None]
    v = torch.from_numpy(np.repeat(V, G, axis=1)).permute(1, 0, 2)[None]
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)
    return o[0].permute(1, 0, 2).numpy()


@pytest.mark.parametrize("mode", [SHARED, INDIVIDUAL])
def test_no_eviction_equals_full_causal_attention(mode):
    rng = np.random.default_rng(5)
    N, Hq, Hkv, D, ls = 50, 4, 2, 8, 16
    Q, K, V, Qi = rand(rng, N, Hq, D), rand(rng, N, Hkv, D), rand(rng, N, Hkv, D), rand(rng, 3, Hq, D)
    orc = CitrusOracle(Hq, Hkv, D, budget_k=N, mode=mode)
    outs = []
    for s in range(0, N, ls):
        outs.append(orc.process_chunk(Q[s:s + ls], K[s:s + ls], V[s:s + ls], Qi).out)
    got = np.concatenate(outs, axis=0)
    assert np.allclose(got, sdpa_full_causal(Q, K, V), rtol=0, atol=1e-12)
    for c in orc.caches:                                  # nothing evicted, order kept
        assert c.K.shape[1] == N
        assert np.array_equal(c.pos, np.broadcast_to(np.arange(N), (Hkv, N)))
        assert np.array_equal(c.K, K.transpose(1, 0, 2))
        assert np.array_equal(c.V, V.transpose(1, 0, 2))


def test_gqa_equals_mha_with_repeated_kv_heads():
    rng = np.random.default_rng(6)
    L, Hq, Hkv, D, m = 7, 4, 2, 8, 5
    G = Hq // Hkv
    Qc, Kc, Vc = rand(rng, L, Hq, D), rand(rng, L, Hkv, D), rand(rng, L, Hkv, D)
    Kca, Vca = rand(rng, Hkv, m, D), rand(rng, Hkv, m, D)
    o1, _ = oracle.chunk_attention(Qc, Kca, Vca, Kc, Vc)
    o2, _ = oracle.chunk_attention(Qc, np.repeat(Kca, G, 0), np.repeat(Vca, G, 0),
                                   np.repeat(Kc, G, 1), np.repeat(Vc, G, 1))
    assert np.array_equal(o1, o2)


# ------------------------------------------------------------- a2-L / TOVA
def test_lm_scores_window_one_is_last_row_and_tova():
    rng = np.random.default_rng(7)
    Hq, Hkv, D, m = 2, 2, 8, 6
    Kca, Vca = rand(rng, Hkv, m, D), rand(rng, Hkv, m, D)
    Qc, Kc, Vc = rand(rng, 1, Hq, D), rand(rng, 1, Hkv, D), rand(rng, 1, Hkv, D)
    _, s_lm = oracle.chunk_attention(Qc, Kca, Vca, Kc, Vc, lm_window=1)
    for g in range(Hkv):
        keys = [list(Kca[g, j]) for j in range(m)] + [list(Kc[0, g])]
        p, _ = brute_attention_row(list(Qc[0, g]), keys, keys, [True] * (m + 1))
        assert np.allclose(s_lm[g], p, atol=1e-13)
        # chunk of one token and budget n-1: the state dropped is the one the
        # last token attends to least (the token-by-token policy the paper
        # names as the l_s = 1 case of chunked eviction)
        kept = oracle.select_topk(s_lm[g], m)
        dropped = set(range(m + 1)) - set(kept.tolist())
        assert dropped == {int(np.argmin(p))}


def test_lm_scores_mass():
    rng = np.random.default_rng(8)
    L, Hq, Hkv, D, m, w = 9, 4, 2, 4, 3, 4
    _, s_lm = oracle.chunk_attention(rand(rng, L, Hq, D), rand(rng, Hkv, m, D), rand(rng, Hkv, m, D),
                                     rand(rng, L, Hkv, D), rand(rng, L, Hkv, D), lm_window=w)
    assert np.allclose(s_lm.sum(axis=1), w * (Hq // Hkv), atol=1e-12)
    # causal: the last chunk row is seen only by the last query, row L-w-1.. by all w voters
    assert np.all(s_lm[:, -1] <= (Hq // Hkv) + 1e-12)


# -------------------------------------------------------------------- a3
def test_select_bruteforce_and_ties():
    rng = np.random.default_rng(9)
    for n, k in [(1, 1), (5, 5), (5, 7), (17, 4), (64, 63), (200, 64)]:
        score = rng.integers(0, 6, size=n).astype(np.float64)          # many exact ties
        got = oracle.select_topk(score, k).tolist()
        ref = sorted(sorted(range(n), key=lambda j: (-score[j], j))[:k])
        assert got == ref
    s = np.array([0.5, 0.9, 0.5, 0.5, 0.1])
    assert oracle.select_topk(s, 3).tolist() == [0, 1, 2]              # lower index wins the tie
    assert oracle.kth_gap(s, 3) == (0.5, 0.5)
    assert oracle.kth_gap(s, 5) == (None, None)


def test_single_chunk_selection_is_direct_topk():
    rng = np.random.default_rng(11)
    N, Hq, Hkv, D, k, nI = 40, 4, 2, 8, 10, 5
    Q, K, V, Qi = rand(rng, N, Hq, D), rand(rng, N, Hkv, D), rand(rng, N, Hkv, D), rand(rng, nI, Hq, D)
    orc = CitrusOracle(Hq, Hkv, D, k, SHARED)
    res = orc.process_chunk(Q, K, V, Qi)
    # direct definition over the whole document, written with scipy-free torch softmax
    G = Hq // Hkv
    for g in range(Hkv):
        tot = torch.zeros(N, dtype=torch.float64)
        for h in range(g * G, (g + 1) * G):
            logits = torch.from_numpy(Qi[:, h]) @ torch.from_numpy(K[:, g]).T / math.sqrt(D)
            tot += torch.softmax(logits, dim=1).sum(0)
        ref = torch.topk(tot, k).indices.sort().values.numpy()
        assert np.array_equal(res.idx[0][g], ref)
        assert np.array_equal(orc.caches[0].pos[g], ref)


def test_duplicate_keys_keep_lower_positions():
    rng = np.random.default_rng(12)
    N, Hq, Hkv, D, k = 12, 2, 1, 4, 5
    K = np.tile(rand(rng, 1, Hkv, D), (N, 1, 1))                       # all keys identical -> all scores tie
    orc = CitrusOracle(Hq, Hkv, D, k, SHARED)
    orc.process_chunk(rand(rng, N, Hq, D), K, rand(rng, N, Hkv, D), rand(rng, 3, Hq, D))
    assert orc.caches[0].pos[0].tolist() == [0, 1, 2, 3, 4]


# -------------------------------------------------------------------- a4
def test_compact_is_plain_gather():
    rng = np.random.default_rng(13)
    Kg, Vg, Kc, Vc = rand(rng, 4, 3), rand(rng, 4, 3), rand(rng, 2, 3), rand(rng, 2, 3)
    pos = np.array([1, 5, 6, 9]); cpos = np.array([10, 11])
    k2, v2, p2 = oracle.compact(Kg, Vg, pos, Kc, Vc, cpos, np.array([0, 3, 5]))
    assert p2.tolist() == [1, 9, 11]
    assert k2[0].tolist() == Kg[0].tolist() and k2[1].tolist() == Kg[3].tolist() and k2[2].tolist() == Kc[1].tolist()
    assert v2[2].tolist() == Vc[1].tolist()


# ----------------------------------------------------------- whole loop
def _run(orc, doc, ls):
    Q, K, V, Qi = (wl.to_f64(t) for t in (doc.Q, doc.K, doc.V, doc.Q_instr))
    res = []
    for s in range(0, Q.shape[0], ls):
        res.append(orc.process_chunk(Q[s:s + ls], K[s:s + ls], V[s:s + ls], Qi))
    return res


def test_rotated_loop_equals_paper_order():
    w = wl.scaled(wl.CONFIGS["tiny_fp32"], doc_tokens=300, chunk_s=64, budget_k=48, n_planted=4)
    doc = wl.make_document(w)
    orc = CitrusOracle(w.q_heads, w.kv_heads, w.head_dim, w.budget_k, SHARED)
    res = _run(orc, doc, w.chunk_s)
    outs, cache = oracle.run_paper_order_shared(wl.to_f64(doc.Q), wl.to_f64(doc.K), wl.to_f64(doc.V),
                                                wl.to_f64(doc.Q_instr), w.budget_k, w.chunk_s)
    assert np.array_equal(cache.pos, orc.caches[0].pos)
    assert np.array_equal(cache.K, orc.caches[0].K) and np.array_equal(cache.V, orc.caches[0].V)
    for a, b in zip(outs, res):
        assert np.allclose(a, b.out, rtol=0, atol=1e-13)


def test_cache_size_arithmetic_from_paper():
    # golden: the paper's main setting and its footnote on resident states
    vals = {}
    with open(os.path.join(GOLDEN, "cache_sizes.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, v = line.split("=")
            vals[key.strip()] = int(v)
    k, ls = vals["k"], vals["l_s"]
    assert k + ls == vals["resident_shared"] and 2 * (k + ls) == vals["resident_individual"]
    rng = np.random.default_rng(14)
    Hq, Hkv, D = 2, 1, 4
    for mode, expect in [(SHARED, vals["resident_shared"]), (INDIVIDUAL, vals["resident_individual"])]:
        orc = CitrusOracle(Hq, Hkv, D, k, mode, lm_window=8)
        peak = 0
        for c in range(5):
            resident_before = sum(cs.K.shape[1] + ls for cs in orc.caches)   # cache rows + the chunk's states
            peak = max(peak, resident_before)
            orc.process_chunk(rand(rng, ls, Hq, D), rand(rng, ls, Hkv, D), rand(rng, ls, Hkv, D), rand(rng, 2, Hq, D))
            for cs in orc.caches:
                assert cs.K.shape[1] == min(k, orc.tokens_seen) == vals["k_generation"] or orc.tokens_seen < k
                assert np.all(np.diff(cs.pos, axis=1) > 0)
        assert peak == expect


@pytest.mark.parametrize("mode", [SHARED, INDIVIDUAL])
def test_planted_keys_and_sinks_survive(mode):
    w = wl.scaled(wl.CONFIGS["mistral7b_layer"], q_heads=4, kv_heads=2, head_dim=32, budget_k=48, chunk_s=32,
                  doc_tokens=400, n_instr=8, n_planted=6, n_sinks=1, mode=mode)
    doc = wl.make_document(w)
    orc = CitrusOracle(w.q_heads, w.kv_heads, w.head_dim, w.budget_k, mode, lm_window=8)
    _run(orc, doc, w.chunk_s)
    inst = orc.caches[-1]                       # the instruction-aware cache
    for g in range(w.kv_heads):
        kept = set(inst.pos[g].tolist())
        assert set(doc.planted.tolist()) <= kept
        assert set(doc.sinks.tolist()) <= kept
    if mode == INDIVIDUAL:                      # sinks also survive in the LM cache
        for g in range(w.kv_heads):
            assert set(doc.sinks.tolist()) <= set(orc.caches[0].pos[g].tolist())


def test_selection_invariant_to_positive_rescaling_and_layerwise():
    rng = np.random.default_rng(15)
    s = rng.random(50)
    assert np.array_equal(oracle.select_topk(s, 7), oracle.select_topk(s / 37.0, 7))   # mean vs sum form
    # layer-wise granularity: every head gets the index set of the head-summed score
    N, Hq, Hkv, D, k = 30, 4, 2, 4, 6
    Q, K, V, Qi = rand(rng, N, Hq, D), rand(rng, N, Hkv, D), rand(rng, N, Hkv, D), rand(rng, 3, Hq, D)
    orc = CitrusOracle(Hq, Hkv, D, k, SHARED, layerwise=True)
    res = orc.process_chunk(Q, K, V, Qi)
    tot = res.scores[0].sum(axis=0)
    ref = sorted(sorted(range(N), key=lambda j: (-tot[j], j))[:k])
    assert res.idx[0][0].tolist() == ref and res.idx[0][1].tolist() == ref


def test_standard_mode_scores_by_the_chunk_and_by_the_instruction_when_given():
    rng = np.random.default_rng(17)
    Hq, Hkv, D, k, ls, w = 4, 2, 4, 6, 5, 3
    G = Hq // Hkv
    orc = CitrusOracle(Hq, Hkv, D, k, oracle.STANDARD, lm_window=w)
    chunks = [(rand(rng, ls, Hq, D), rand(rng, ls, Hkv, D), rand(rng, ls, Hkv, D)) for _ in range(3)]
    Qi = rand(rng, 2, Hq, D)
    for c, (Q, K, V) in enumerate(chunks):
        cache = orc.caches[0]
        m = cache.K.shape[1]
        last = c == len(chunks) - 1
        res = orc.process_chunk(Q, K, V, Qi if last else None)
        # brute force: votes of the scoring rows on every candidate
        ref = [[0.0] * (m + ls) for _ in range(Hkv)]
        for h in range(Hq):
            g = h // G
            keys = [list(cache.K[g, j]) for j in range(m)] + [list(K[u, g]) for u in range(ls)]
            rows = range(Qi.shape[0]) if last else range(ls - w, ls)
            for t in rows:
                q = list(Qi[t, h]) if last else list(Q[t, h])
                visible = [True] * (m + ls) if last else [True] * m + [u <= t for u in range(ls)]
                p, _ = brute_attention_row(q, keys, keys, visible)
                for j in range(m + ls):
                    ref[g][j] += p[j]
        assert np.allclose(res.scores[0], np.array(ref), rtol=0, atol=1e-12)
        for g in range(Hkv):
            want = sorted(sorted(range(m + ls), key=lambda j: (-ref[g][j], j))[:k])
            got = res.idx[0][g].tolist()
            # brute-force and numpy sums may differ in the last bit: only compare when the cut is clear
            srt = sorted(ref[g], reverse=True)
            if m + ls <= k or srt[k - 1] - srt[k] > 1e-9:
                assert got == want
    assert len(orc.caches) == 1 and orc.caches[0].K.shape[1] == k


def test_start_size_keeps_initial_tokens_and_fills_the_rest_by_score():
    rng = np.random.default_rng(18)
    N, Hq, Hkv, D, k, ls, s0 = 60, 2, 1, 4, 10, 20, 4
    Q, K, V, Qi = rand(rng, N, Hq, D), rand(rng, N, Hkv, D), rand(rng, N, Hkv, D), rand(rng, 3, Hq, D)
    K[:s0] *= 0.01                                        # make the initial tokens unattractive on purpose
    orc = CitrusOracle(Hq, Hkv, D, k, SHARED, start_size=s0)
    for c in range(0, N, ls):
        before = orc.caches[0].pos[0].tolist()
        res = orc.process_chunk(Q[c:c + ls], K[c:c + ls], V[c:c + ls], Qi)
        kept = orc.caches[0].pos[0].tolist()
        assert kept[:s0] == [0, 1, 2, 3]
        # the other k - s0 places go to the best-scoring remaining candidates (plain definition, pure Python)
        cand_pos = before + list(range(c, c + ls))
        sc = res.scores[0][0]
        rest = [j for j in range(len(cand_pos)) if cand_pos[j] >= s0]
        best = sorted(sorted(rest, key=lambda j: (-sc[j], j))[:k - s0])
        assert kept[s0:] == [cand_pos[j] for j in best]


def test_intersection_ratio_on_a_worked_example_and_its_limits():
    from oracle import intersection_ratio
    ctx = np.array([[0, 2, 4, 6, 8, 10], [1, 3, 5, 7, 9, 11]])
    ins = np.array([[0, 1, 2, 3, 4, 5], [0, 2, 4, 6, 8, 10]])
    # head 0 shares {0, 2, 4}; head 1 shares nothing
    assert intersection_ratio(ctx, ins).tolist() == [0.5, 0.0]
    assert intersection_ratio(ins, ins).tolist() == [1.0, 1.0]
    rng = np.random.default_rng(3)
    a = np.sort(rng.choice(1000, size=(3, 200), replace=False) if False else np.stack([rng.choice(1000, 200, replace=False) for _ in range(3)]), axis=1)
    b = np.stack([np.sort(rng.choice(1000, 200, replace=False)) for _ in range(3)])
    r = intersection_ratio(a, b)
    for g in range(3):
        assert r[g] == sum(int(x in set(a[g].tolist())) for x in b[g].tolist()) / 200   # counted one by one


def test_accumulated_scores_without_eviction_are_the_sum_of_every_steps_attention():
    # budget larger than the document: nothing is evicted, so after the last chunk the carried importance of token j
    # is the attention it received from the instruction at every step it was a candidate, over the prefix seen so far
    import math
    rng = np.random.default_rng(21)
    N, Hq, Hkv, D, ls = 24, 2, 1, 4, 8
    Q, K, V, Qi = rand(rng, N, Hq, D), rand(rng, N, Hkv, D), rand(rng, N, Hkv, D), rand(rng, 3, Hq, D)
    orc = CitrusOracle(Hq, Hkv, D, 100, SHARED, accumulate=True)
    for c in range(0, N, ls):
        orc.process_chunk(Q[c:c + ls], K[c:c + ls], V[c:c + ls], Qi)
    expect = [0.0] * N
    for n_t in range(ls, N + 1, ls):                      # candidates of the step: tokens 0 .. n_t - 1
        for h in range(Hq):
            for i in range(Qi.shape[0]):
                logits = [sum(Qi[i, h, d] * K[j, 0, d] for d in range(D)) / math.sqrt(D) for j in range(n_t)]
                mx = max(logits)
                den = sum(math.exp(x - mx) for x in logits)
                for j in range(n_t):
                    expect[j] += math.exp(logits[j] - mx) / den
    assert orc.caches[0].pos[0].tolist() == list(range(N))
    assert np.allclose(orc.caches[0].acc[0], expect, rtol=1e-12, atol=1e-14)


def test_accumulated_scores_change_what_is_kept():
    # a state that one step rates just below the cut survives when its earlier steps' importance counts
    rng = np.random.default_rng(22)
    N, Hq, Hkv, D, k, ls = 96, 2, 1, 8, 12, 16
    Q, K, V, Qi = rand(rng, N, Hq, D), rand(rng, N, Hkv, D), rand(rng, N, Hkv, D), rand(rng, 4, Hq, D)
    plain, acc = CitrusOracle(Hq, Hkv, D, k, SHARED), CitrusOracle(Hq, Hkv, D, k, SHARED, accumulate=True)
    differ = False
    for c in range(0, N, ls):
        a = plain.process_chunk(Q[c:c + ls], K[c:c + ls], V[c:c + ls], Qi)
        b = acc.process_chunk(Q[c:c + ls], K[c:c + ls], V[c:c + ls], Qi)
        # the carried part only ever adds: accumulated scores dominate the step's own
        m_b = b.m_before
        assert np.all(b.scores[0][:, m_b:] >= 0) and b.scores[0].shape == (Hkv, m_b + ls)
        differ |= plain.caches[0].pos[0].tolist() != acc.caches[0].pos[0].tolist()
        # what is carried forward is exactly the kept candidates' accumulated score
        assert np.array_equal(acc.caches[0].acc[0], b.scores[0][0][b.applied[0][0]])
    assert differ


def test_deferred_lm_eviction_follows_the_three_steps_of_standard_cse():
    # Section 4.1 in plain Python: C starts as the first chunk; for every later chunk s: encode s against [C ; s],
    # keep the k states of C that s attends to most (summed over s's queries and the group's heads), put all of s in.
    import math
    rng = np.random.default_rng(31)
    N, Hq, Hkv, D, k, ls = 70, 2, 1, 4, 9, 10
    Q, K, V = rand(rng, N, Hq, D), rand(rng, N, Hkv, D), rand(rng, N, Hkv, D)
    orc = CitrusOracle(Hq, Hkv, D, k, STANDARD, deferred_lm=True)
    cache = []                                            # original positions held by C
    for c in range(0, N, ls):
        orc.process_chunk(Q[c:c + ls], K[c:c + ls], V[c:c + ls], None)
        chunk = list(range(c, c + ls))
        if len(cache) > k:
            score = {j: 0.0 for j in cache}
            for t in chunk:                               # every query of the chunk, causal over the chunk itself
                keys = cache + [u for u in chunk if u <= t]
                for h in range(Hq):
                    logits = [sum(Q[t, h, d] * K[j, 0, d] for d in range(D)) / math.sqrt(D) for j in keys]
                    mx = max(logits)
                    den = sum(math.exp(x - mx) for x in logits)
                    for j, x in zip(keys, logits):
                        if j in score:
                            score[j] += math.exp(x - mx) / den
            cache = sorted(sorted(cache, key=lambda j: (-score[j], j))[:k])
        cache = cache + chunk
        assert orc.caches[0].pos[0].tolist() == cache
        assert len(cache) == min(c + ls, k + ls)


def test_deferred_lm_eviction_with_unit_chunks_is_tova():
    # Baselines section: TOVA is standard CSE with l_s = 1 - the newest token's attention over the cache (itself
    # included) drops the one state it attends to least
    rng = np.random.default_rng(32)
    N, Hq, Hkv, D, k = 30, 1, 1, 6, 7
    Q, K, V = rand(rng, N, Hq, D), rand(rng, N, Hkv, D), rand(rng, N, Hkv, D)
    orc = CitrusOracle(Hq, Hkv, D, k, STANDARD, deferred_lm=True)
    held = []
    for t in range(N):
        orc.process_chunk(Q[t:t + 1], K[t:t + 1], V[t:t + 1], None)
        if len(held) > k:
            keys = held + [t]
            logits = np.array([Q[t, 0] @ K[j, 0] for j in keys]) / np.sqrt(D)
            p = np.exp(logits - logits.max()); p /= p.sum()
            drop = min(range(len(held)), key=lambda i: (p[i], -held[i]))   # least attended; the later position on a tie
            held = held[:drop] + held[drop + 1:]
        held = held + [t]
        assert orc.caches[0].pos[0].tolist() == held


def test_rope_is_a_rotation_of_complex_pairs_and_depends_on_relative_position_only():
    from oracle import rope
    rng = np.random.default_rng(41)
    D = 16
    q, k = rng.normal(size=D), rng.normal(size=D)
    theta = 10000.0 ** (-2.0 * np.arange(D // 2) / D)
    for a, b in [(0, 0), (3, 3), (5, 2), (1000, 977), (7, 40)]:
        # complex form: pair (x_d, x_{d+D/2}) is the number x_d + i x_{d+D/2}, turned by exp(i pos theta_d)
        qa = (q[:D // 2] + 1j * q[D // 2:]) * np.exp(1j * a * theta)
        kb = (k[:D // 2] + 1j * k[D // 2:]) * np.exp(1j * b * theta)
        assert np.allclose(rope(q, np.array(a)), np.concatenate([qa.real, qa.imag]), atol=1e-12)
        dot = float(rope(q, np.array(a)) @ rope(k, np.array(b)))
        assert abs(dot - float(np.real(np.sum(qa * np.conj(kb))))) < 1e-10
        assert abs(dot - float(rope(q, np.array(a - b)) @ k)) < 1e-9          # relative position only
    assert np.allclose(rope(q, np.array(0)), q)
    assert abs(np.linalg.norm(rope(q, np.array(123))) - np.linalg.norm(q)) < 1e-12


def test_round_bf16_is_round_to_nearest_even_on_the_upper_sixteen_bits():
    from oracle import round_bf16
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, 1.0 + 3 * 2.0 ** -8, -0.3, 3.0e-40, 65504.0])
    r = round_bf16(x)
    # 1 + 2^-8 is half way between 1 and 1 + 2^-7: ties go to the even mantissa (1.0); just above goes up;
    # 1 + 3 * 2^-8 is half way between 1 + 2^-7 and 1 + 2^-6: the even one is 1 + 2^-6
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2.0 ** -7 and r[3] == 1.0 + 2.0 ** -6
    assert np.array_equal(r, torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy())


def test_position_shift_without_eviction_is_ordinary_rope_by_document_position():
    # budget larger than the document: every state keeps its place, so cache slot = document position and the shifted
    # run must equal a plain run on inputs that were embedded up front
    from oracle import rope
    rng = np.random.default_rng(42)
    N, Hq, Hkv, D, ls, nI = 48, 4, 2, 8, 16, 5
    Q, K, V, Qi = rand(rng, N, Hq, D), rand(rng, N, Hkv, D), rand(rng, N, Hkv, D), rand(rng, nI, Hq, D)
    shifted = CitrusOracle(Hq, Hkv, D, 1000, SHARED, rope_shift=True)
    plain = CitrusOracle(Hq, Hkv, D, 1000, SHARED)
    pos = np.arange(N)[:, None]
    Qr, Kr = rope(Q, pos), rope(K, pos)
    for c in range(0, N, ls):
        a = shifted.process_chunk(Q[c:c + ls], K[c:c + ls], V[c:c + ls], Qi)
        Qir = rope(Qi, (c + ls + np.arange(nI))[:, None])           # the instruction follows what has been read
        b = plain.process_chunk(Qr[c:c + ls], Kr[c:c + ls], V[c:c + ls], Qir)
        assert np.allclose(a.out, b.out, atol=1e-12) and np.allclose(a.scores[0], b.scores[0], atol=1e-12)
    assert np.array_equal(shifted.caches[0].K, np.transpose(K, (1, 0, 2)))     # the cache keeps un-rotated keys


def test_position_shift_with_eviction_embeds_by_cache_slot():
    # after eviction a kept state sits in a lower slot and is embedded by that slot: brute force for one query
    import math
    from oracle import rope
    rng = np.random.default_rng(43)
    N, Hq, Hkv, D, k, ls = 40, 1, 1, 8, 6, 8
    Q, K, V, Qi = rand(rng, N, Hq, D), rand(rng, N, Hkv, D), rand(rng, N, Hkv, D), rand(rng, 2, Hq, D)
    orc = CitrusOracle(Hq, Hkv, D, k, SHARED, rope_shift=True)
    for c in range(0, N, ls):
        held = orc.caches[0].pos[0].tolist()
        res = orc.process_chunk(Q[c:c + ls], K[c:c + ls], V[c:c + ls], Qi)
        m = len(held)
        t = ls - 1                                            # last token of the chunk sees everything
        keys = [rope(K[p, 0], np.array(slot)) for slot, p in enumerate(held)] + \
               [rope(K[c + i, 0], np.array(m + i)) for i in range(ls)]
        vals = [V[p, 0] for p in held] + [V[c + i, 0] for i in range(ls)]
        qv = rope(Q[c + t, 0], np.array(m + t))
        logits = [float(qv @ kk) / math.sqrt(D) for kk in keys]
        mx = max(logits); w = [math.exp(x - mx) for x in logits]; den = sum(w)
        expect = sum(wi / den * v for wi, v in zip(w, vals))
        assert np.allclose(res.out[t, 0], expect, atol=1e-12)

def _torch_bf16(x):
    """Round with torch's own float32 -> bfloat16 conversion (not the oracle's bit arithmetic)."""
    return torch.tensor(np.asarray(x), dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()


def test_bf16_embedding_branch_rounds_queries_and_keys_once_and_nothing_else():
    # A bf16 model holds its rotary-embedded queries and keys as bf16 tensors.  With a budget larger than the document
    # nothing moves, so the shifted run with embedded_dtype="bf16" must equal a plain run on inputs that were embedded
    # up front and rounded by torch: the chunk's queries and keys and the instruction queries are rounded, V is not,
    # and the cache keeps the un-rotated, un-rounded keys.
    from oracle import rope
    rng = np.random.default_rng(44)
    N, Hq, Hkv, D, ls, nI = 48, 4, 2, 8, 16, 5
    # inputs exactly representable in bf16, as the library receives them
    Q, K, V, Qi = (_torch_bf16(rand(rng, *s)) for s in ((N, Hq, D), (N, Hkv, D), (N, Hkv, D), (nI, Hq, D)))
    shifted = CitrusOracle(Hq, Hkv, D, 1000, SHARED, rope_shift=True, embedded_dtype="bf16")
    plain = CitrusOracle(Hq, Hkv, D, 1000, SHARED)
    pos = np.arange(N)[:, None]
    Qr, Kr = _torch_bf16(rope(Q, pos)), _torch_bf16(rope(K, pos))
    unrounded = CitrusOracle(Hq, Hkv, D, 1000, SHARED, rope_shift=True)
    differs = False
    for c in range(0, N, ls):
        a = shifted.process_chunk(Q[c:c + ls], K[c:c + ls], V[c:c + ls], Qi)
        Qir = _torch_bf16(rope(Qi, (c + ls + np.arange(nI))[:, None]))
        b = plain.process_chunk(Qr[c:c + ls], Kr[c:c + ls], V[c:c + ls], Qir)
        assert np.allclose(a.out, b.out, rtol=0, atol=1e-12)
        assert np.allclose(a.scores[0], b.scores[0], rtol=0, atol=1e-12)
        u = unrounded.process_chunk(Q[c:c + ls], K[c:c + ls], V[c:c + ls], Qi)
        differs = differs or np.abs(a.out - u.out).max() > 1e-6
    assert differs                                                  # the rounding is really applied
    assert np.array_equal(shifted.caches[0].K, np.transpose(K, (1, 0, 2)))      # stored keys: un-rotated, un-rounded
    assert np.array_equal(shifted.caches[0].V, np.transpose(V, (1, 0, 2)))


def test_bf16_embedding_branch_after_eviction_rounds_the_keys_embedded_by_slot():
    # After eviction every kept key is embedded again from its stored (un-rotated) value at its new slot and rounded
    # once; the query likewise.  One query row by plain loops, rounding with torch.
    import math
    from oracle import rope
    rng = np.random.default_rng(45)
    N, Hq, Hkv, D, k, ls = 40, 1, 1, 8, 6, 8
    Q, K, V, Qi = (_torch_bf16(rand(rng, *s)) for s in ((N, Hq, D), (N, Hkv, D), (N, Hkv, D), (3, Hq, D)))
    orc = CitrusOracle(Hq, Hkv, D, k, SHARED, rope_shift=True, embedded_dtype="bf16")
    for c in range(0, N, ls):
        held = orc.caches[0].pos[0].tolist()
        res = orc.process_chunk(Q[c:c + ls], K[c:c + ls], V[c:c + ls], Qi)
        m = len(held)
        keys = [_torch_bf16(rope(K[p, 0], np.array(slot))) for slot, p in enumerate(held)] + \
               [_torch_bf16(rope(K[c + i, 0], np.array(m + i))) for i in range(ls)]
        vals = [V[p, 0] for p in held] + [V[c + i, 0] for i in range(ls)]
        t = ls - 1
        qv = _torch_bf16(rope(Q[c + t, 0], np.array(m + t)))
        logits = [float(qv @ kk) / math.sqrt(D) for kk in keys]
        mx = max(logits); w = [math.exp(x - mx) for x in logits]; den = sum(w)
        assert np.allclose(res.out[t, 0], sum(wi / den * v for wi, v in zip(w, vals)), rtol=0, atol=1e-12)
        # instruction scores (Eq. 1, s = I): instruction token i sits at slot m + L + i
        score = [0.0] * len(keys)
        for i in range(Qi.shape[0]):
            qi = _torch_bf16(rope(Qi[i, 0], np.array(m + ls + i)))
            lg = [float(qi @ kk) / math.sqrt(D) for kk in keys]
            mx = max(lg); den = sum(math.exp(x - mx) for x in lg)
            for j, x in enumerate(lg):
                score[j] += math.exp(x - mx) / den
        assert np.allclose(res.scores[0][0], score, rtol=0, atol=1e-12)


def test_individual_caches_follow_the_two_eviction_rules_in_plain_python():
    # Section 4.2, individual cache (Eq. 4-5): the language-modelling cache C is evicted by the chunk's own attention,
    # the instruction cache C^I by the instruction's attention over C^I's OWN states plus the chunk; the chunk is
    # encoded against C only.  Plain loops over original positions; K/V are looked up in the document by position.
    import math
    rng = np.random.default_rng(46)
    N, Hq, Hkv, D, k, ls, nI, w = 60, 4, 2, 4, 7, 10, 3, 4
    G = Hq // Hkv
    Q, K, V, Qi = rand(rng, N, Hq, D), rand(rng, N, Hkv, D), rand(rng, N, Hkv, D), rand(rng, nI, Hq, D)
    orc = CitrusOracle(Hq, Hkv, D, k, INDIVIDUAL, lm_window=w)

    def softmax_over(qvec, g, keys):
        lg = [sum(qvec[d] * K[j, g, d] for d in range(D)) / math.sqrt(D) for j in keys]
        mx = max(lg); e = [math.exp(x - mx) for x in lg]; den = sum(e)
        return [x / den for x in e]

    C = [[] for _ in range(Hkv)]        # positions held by the language-modelling cache, per KV head
    CI = [[] for _ in range(Hkv)]       # positions held by the instruction cache
    caches_differ = False
    for c in range(0, N, ls):
        chunk = list(range(c, c + ls))
        res = orc.process_chunk(Q[c:c + ls], K[c:c + ls], V[c:c + ls], Qi)
        for g in range(Hkv):
            cand_lm, cand_in = C[g] + chunk, CI[g] + chunk
            s_lm = {j: 0.0 for j in cand_lm}
            s_in = {j: 0.0 for j in cand_in}
            for h in range(g * G, (g + 1) * G):
                for t in chunk:
                    keys = C[g] + [u for u in chunk if u <= t]
                    p = softmax_over(Q[t, h], g, keys)
                    # the output comes from the language-modelling cache
                    expect = [sum(pj * V[j, g, d] for pj, j in zip(p, keys)) for d in range(D)]
                    assert np.allclose(res.out[t - c, h], expect, rtol=0, atol=1e-12)
                    if t >= c + ls - w:                       # the last w queries of the chunk vote on C
                        for pj, j in zip(p, keys):
                            s_lm[j] += pj
                for i in range(nI):                           # every instruction token votes on C^I, unmasked
                    for pj, j in zip(softmax_over(Qi[i, h], g, cand_in), cand_in):
                        s_in[j] += pj
            assert np.allclose(res.scores[0][g], [s_lm[j] for j in cand_lm], rtol=0, atol=1e-12)
            assert np.allclose(res.scores[1][g], [s_in[j] for j in cand_in], rtol=0, atol=1e-12)
            C[g] = sorted(sorted(cand_lm, key=lambda j: (-s_lm[j], j))[:k])
            CI[g] = sorted(sorted(cand_in, key=lambda j: (-s_in[j], j))[:k])
            assert orc.caches[0].pos[g].tolist() == C[g]
            assert orc.caches[1].pos[g].tolist() == CI[g]
            assert np.array_equal(orc.caches[1].K[g], K[CI[g], g]) and np.array_equal(orc.caches[1].V[g], V[CI[g], g])
            caches_differ = caches_differ or C[g] != CI[g]
    assert caches_differ                # otherwise scoring C^I with C's keys would go unnoticed


def test_forced_selection_is_adopted():
    rng = np.random.default_rng(16)
    N, Hq, Hkv, D, k = 10, 2, 1, 4, 3
    orc = CitrusOracle(Hq, Hkv, D, k, SHARED)
    forced = {0: np.array([[1, 4, 7]])}
    res = orc.process_chunk(rand(rng, N, Hq, D), rand(rng, N, Hkv, D), rand(rng, N, Hkv, D), rand(rng, 2, Hq, D), forced)
    assert orc.caches[0].pos[0].tolist() == [1, 4, 7]
    assert res.applied[0].tolist() == [[1, 4, 7]]


def test_workload_generator_is_deterministic_and_shaped():
    w = wl.scaled(wl.CONFIGS["long_doc_stress"], doc_tokens=600, n_planted=5)
    a, b = wl.make_document(w), wl.make_document(w)
    assert torch.equal(a.K, b.K) and torch.equal(a.Q_instr, b.Q_instr)
    assert a.Q.shape == (600, 32, 128) and a.K.dtype == torch.bfloat16
    assert a.sinks.tolist() == [0, 1, 2, 3] and len(set(a.planted.tolist())) == 5
    lens = wl.sequence_lengths(wl.CONFIGS["serving_mix"])
    assert len(lens) == 16 and all(4096 <= x <= 32768 for x in lens) and lens == wl.sequence_lengths(wl.CONFIGS["serving_mix"])
