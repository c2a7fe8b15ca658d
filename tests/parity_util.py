"""Drives the CUDA library and the fp64 oracle through the same chunk sequence
and applies the parity rules:

  * attention output and normalised scores: absolute tolerance 2e-2 (bf16) /
    1e-4 (fp32);
  * kept index sets: equal to the oracle's, except pairs whose oracle scores
    differ by at most 1e-5 relative (the oracle then adopts the library's set so
    one permitted flip does not cascade);
  * compaction: bit-exact against gathering the inputs with the library's own
    indices; positions strictly ascending; row count min(k, tokens seen).
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import CitrusOracle, CacheState
from paper_2406_12018_b200 import workloads as wl
from paper_2406_12018_b200.binding import Citrus

TOL = {"bf16": 2e-2, "fp32": 1e-4}
SWAP_REL = 1e-5


def make_pair(w: wl.Workload, layers=1, layerwise=False):
    ctx = Citrus(layers, w.q_heads, w.kv_heads, w.head_dim, w.budget_k, w.chunk_s, mode=w.mode, dtype=w.dtype,
                 lm_window=w.lm_window, layerwise=layerwise, n_seqs=w.n_seqs, start_size=w.start_size,
                 accumulate=w.accumulate, deferred_lm=w.deferred_lm, position_shift=w.position_shift,
                 rope_base=w.rope_base if w.position_shift else None)
    return ctx


def make_oracle(w: wl.Workload, layerwise=False, unrounded=False):
    """unrounded: keep the rotary-embedded queries and keys in fp64 (the oracle then models no bf16 rounding of the
    embedded tensors, so it is a yardstick the library's position-shift path cannot have been fitted to)."""
    return CitrusOracle(w.q_heads, w.kv_heads, w.head_dim, w.budget_k, w.mode,
                        lm_window=(w.lm_window or None), layerwise=layerwise, start_size=w.start_size,
                        accumulate=w.accumulate, deferred_lm=w.deferred_lm, rope_shift=w.position_shift,
                        rope_base=w.rope_base,
                        embedded_dtype="bf16" if (w.position_shift and w.dtype == "bf16" and not unrounded) else None)


def check_index_rule(own, gpu, scores, n, k):
    """own/gpu [H_kv, kept]; scores [H_kv, n] oracle scores the selection used."""
    flips = 0
    for g in range(own.shape[0]):
        gi = gpu[g]
        assert np.all(np.diff(gi) > 0), "kept indices must be strictly ascending"
        assert gi[0] >= 0 and gi[-1] < n
        a, b = set(own[g].tolist()), set(gi.tolist())
        if a == b:
            continue
        only_o, only_g = sorted(a - b), sorted(b - a)
        assert len(only_o) == len(only_g)
        for i in only_o:
            for j in only_g:
                si, sj = scores[g][i], scores[g][j]
                assert abs(si - sj) <= SWAP_REL * max(si, sj), \
                    f"head {g}: swap of candidates {i} (oracle) and {j} (library) outside the tie band: {si} vs {sj}"
        flips += len(only_o)
    return flips


def load_oracle_from_library(orc: CitrusOracle, ctx: Citrus, layer: int, slot: int, tokens_seen: int):
    """Teacher-force the oracle with the library's current caches."""
    for cid in range(len(orc.caches)):
        K, V, P = ctx.cache_view(layer, cid, slot)
        torch.cuda.synchronize()
        orc.caches[cid] = CacheState(K.to(torch.float64).cpu().numpy(), V.to(torch.float64).cpu().numpy(),
                                     P.cpu().numpy().astype(np.int64))
    orc.tokens_seen = tokens_seen


def check_cache_properties(ctx: Citrus, doc: wl.Document, layer: int, slot: int, tokens_seen: int, Kdev, Vdev,
                           expected_rows=None):
    """Properties that hold at any size: row count, ascending positions, rows are the
    document's rows at those positions (bit-exact)."""
    n_caches = 2 if ctx.individual else 1
    for cid in range(n_caches):
        K, V, P = ctx.cache_view(layer, cid, slot)
        if expected_rows is not None:
            assert K.shape[1] == expected_rows[cid]
        else:
            assert K.shape[1] == min(ctx.budget_k, tokens_seen)
        if P.shape[1] > 1:
            assert bool((P[:, 1:] > P[:, :-1]).all())
        assert int(P.min()) >= 0 and int(P.max()) < tokens_seen
        for g in range(ctx.kv_heads):
            p = P[g].long()
            bits = torch.int16 if K.dtype == torch.bfloat16 else torch.int32
            assert torch.equal(K[g].view(bits), Kdev[p, g].view(bits))
            assert torch.equal(V[g].view(bits), Vdev[p, g].view(bits))


def run_document(w: wl.Workload, ctx: Citrus, layer=0, slot=0, seq=0, n_tokens=None, oracle_chunks="all",
                 layerwise=False, chunk_lengths=None, stats=None, unrounded=False, index_rule=True, out_tol=None):
    """Process one document through the library; compare with the oracle on `oracle_chunks`
    ("all" or a set of chunk numbers); property-check the cache after every chunk.
    index_rule=False: the kept sets are not compared (the oracle adopts the library's), only outputs, scores and the
    bit-exact compaction are."""
    doc = wl.make_document(w, layer=layer, seq=seq, n_tokens=n_tokens)
    N = doc.Q.shape[0]
    tol = TOL[w.dtype]
    Qd, Kd, Vd, Qid = doc.Q.cuda(), doc.K.cuda(), doc.V.cuda(), doc.Q_instr.cuda()
    Q64 = K64 = V64 = None
    Qi64 = wl.to_f64(doc.Q_instr)
    orc = make_oracle(w, layerwise, unrounded)
    G = w.q_heads // w.kv_heads
    bounds = []
    s = 0
    if chunk_lengths is None:
        while s < N:
            bounds.append((s, min(N, s + w.chunk_s))); s += w.chunk_s
    else:
        for Lc in chunk_lengths:
            bounds.append((s, s + Lc)); s += Lc
        assert s == N
    st = stats if stats is not None else {}
    st.setdefault("max_out_err", 0.0); st.setdefault("max_score_err", 0.0)
    st.setdefault("max_score_rel", 0.0); st.setdefault("flips", 0); st.setdefault("checked_chunks", 0)
    tokens_seen = 0
    rows = [0, 0]            # expected rows of each cache (tracked here only for deferred eviction)
    oracle_synced = True     # oracle's caches equal the library's
    for ci, (a, b) in enumerate(bounds):
        L = b - a
        use_oracle = oracle_chunks == "all" or ci in oracle_chunks
        if use_oracle and not oracle_synced:
            load_oracle_from_library(orc, ctx, layer, slot, tokens_seen)
            oracle_synced = True
        # standard chunked eviction: chunks score their own eviction; the last call passes the instruction
        # queries (the paper's final eviction with the instruction text)
        with_instr = w.mode != "standard" or ci == len(bounds) - 1
        out = ctx.process_chunk(layer, Qd[a:b], Kd[a:b], Vd[a:b], Qid if with_instr else None, slot=slot)
        torch.cuda.synchronize()
        tokens_seen += L
        n_caches = 2 if ctx.individual else 1
        views = [ctx.step_view(layer, cid, slot) for cid in range(n_caches)]
        if use_oracle:
            forced = {cid: views[cid][1].cpu().numpy().astype(np.int64) for cid in range(n_caches)}
            res = orc.process_chunk(wl.to_f64(doc.Q[a:b]), wl.to_f64(doc.K[a:b]), wl.to_f64(doc.V[a:b]),
                                    Qi64 if with_instr else None, forced)
            err = float(np.abs(out.to(torch.float64).cpu().numpy() - res.out).max())
            st["max_out_err"] = max(st["max_out_err"], err)
            assert err <= (tol if out_tol is None else out_tol), f"chunk {ci}: attention output error {err}"
            for cid in range(n_caches):
                S_gpu = views[cid][0].to(torch.float64).cpu().numpy()
                assert views[cid][2] == res.m_by_cache[cid]
                n = res.m_by_cache[cid] + L
                S_or = res.scores[cid]
                if (ctx.individual and cid == 0) or not with_instr:
                    wrows = L if not w.lm_window else min(w.lm_window, L)
                else:
                    wrows = w.n_instr
                norm = wrows * G
                # every scoring query spends exactly one unit of attention (accumulated scores also carry earlier steps)
                if not w.accumulate:
                    assert np.allclose(S_gpu.sum(axis=1), norm, rtol=2e-3 if w.dtype == "bf16" else 1e-4)
                serr = float(np.abs(S_gpu - S_or).max()) / norm
                st["max_score_err"] = max(st["max_score_err"], serr)
                assert serr <= tol, f"chunk {ci} cache {cid}: score error {serr}"
                big = S_or > norm / (10.0 * n)
                if big.any():
                    st["max_score_rel"] = max(st["max_score_rel"], float((np.abs(S_gpu - S_or)[big] / S_or[big]).max()))
                S_sel = S_or
                if layerwise:
                    S_sel = np.broadcast_to(S_or.sum(axis=0, keepdims=True), S_or.shape)
                if index_rule:
                    st["flips"] += check_index_rule(res.idx[cid], forced[cid], S_sel, n, w.budget_k)
                # compaction bit-exact given the library's indices (oracle applied them to the exact inputs)
                K, V, P = ctx.cache_view(layer, cid, slot)
                oc = orc.caches[cid]
                assert np.array_equal(P.cpu().numpy().astype(np.int64), oc.pos)
                assert np.array_equal(K.to(torch.float64).cpu().numpy(), oc.K)
                assert np.array_equal(V.to(torch.float64).cpu().numpy(), oc.V)
            st["checked_chunks"] += 1
        else:
            oracle_synced = False
        expected = None
        if w.deferred_lm:
            lm_scored = w.mode == "individual" or not with_instr
            rows[0] = (min(rows[0], w.budget_k) + L) if lm_scored else min(rows[0] + L, w.budget_k)
            rows[1] = min(rows[1] + L, w.budget_k)
            expected = list(rows)
        check_cache_properties(ctx, doc, layer, slot, tokens_seen, Kd, Vd, expected)
    return doc, st
