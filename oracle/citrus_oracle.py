"""Slow fp64 CPU oracle for chunked instruction-aware state eviction (CItruS).

TEST INFRASTRUCTURE ONLY.  This module is the yardstick the CUDA library is
checked against; it is never on the product path.  It is written from the
paper's definitions in plain numpy fp64, one step after another, with no
blocking, fusion or reordering.  It imports nothing from the CUDA package.

What is pinned (see tests/test_oracle_pins.py):
  * chunk_attention      -- brute-force loops on tiny shapes; equality with a
                            library full-causal attention when nothing is evicted.
  * importance_sum       -- rows sum to one; zero query -> uniform; dominant key.
  * lm_importance_sum    -- w = 1 gives the last attention row; column mass = w*G.
  * select_topk          -- brute-force stable sort; constructed exact ties.
  * compact              -- plain gather; positions ascending.
  * whole loop           -- paper-order (evict, encode, append, final eviction)
                            equals the rotated order used by the library.
Numeric values: parity unpinned by any printed number -- the paper prints no
worked example of Eq. 1; only invariants, closed forms, special cases and brute
force pin the arithmetic.

Notation follows the paper (Section 4.1-4.3): chunk s of length l_s, cache C,
instruction I, budget k, Imp(s, c) of Eq. 1.  Tensors are token-major:
Q [tokens, H_q, D], K/V [tokens, H_kv, D]; query head h reads KV head
g = h // G with G = H_q // H_kv.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

SHARED = "shared"
INDIVIDUAL = "individual"
STANDARD = "standard"     # standard chunked eviction (Section 4.1): one cache, scored by the chunk itself


# --------------------------------------------------------------------------
# Step a1 -- attention of the chunk over [retained cache ; chunk]
# (Section 4.1, step 1 of the chunked eviction loop; softmax of Eq. 1's inner
# term with the usual causal mask inside the chunk.)
# --------------------------------------------------------------------------
def attention_probabilities(q_rows: np.ndarray, keys: np.ndarray, m: int, causal: bool) -> np.ndarray:
    """softmax_j( q_t . k_j / sqrt(d_k) ) for one query head.

    q_rows [L, D]; keys [n, D] = m cache rows followed by the chunk's rows.
    With causal=True chunk row t may look at every cache row and at chunk rows
    u <= t (candidate index m + u); masked entries get probability exactly 0.
    Max-subtracted for stability; scale is exactly 1/sqrt(D) (Eq. 1).
    """
    L, D = q_rows.shape
    n = keys.shape[0]
    logits = (q_rows @ keys.T) / np.sqrt(float(D))            # [L, n]
    if causal:
        t = np.arange(L)[:, None]
        j = np.arange(n)[None, :]
        visible = j <= (m + t)
        logits = np.where(visible, logits, -np.inf)
    logits = logits - logits.max(axis=1, keepdims=True)
    e = np.exp(logits)
    return e / e.sum(axis=1, keepdims=True)


def chunk_attention(Qc, Kcache, Vcache, Kc, Vc, lm_window: int = 0):
    """Step a1 for all heads, plus (optionally) step a2-L's column sums.

    Qc [L,H_q,D]; Kcache,Vcache [H_kv,m,D]; Kc,Vc [L,H_kv,D].
    Returns out [L,H_q,D] and, when lm_window = w > 0, the language-modelling
    importance  S_LM[g][j] = sum_{h in g} sum_{t in last w chunk rows} P[t,h,j]
    (Eq. 1 with s = the chunk itself, sum instead of mean).
    """
    L, Hq, D = Qc.shape
    Hkv = Kc.shape[1]
    G = Hq // Hkv
    m = Kcache.shape[1]
    n = m + L
    out = np.zeros((L, Hq, D), dtype=np.float64)
    s_lm = np.zeros((Hkv, n), dtype=np.float64) if lm_window > 0 else None
    for h in range(Hq):
        g = h // G
        keys = np.concatenate([Kcache[g], Kc[:, g, :]], axis=0)
        vals = np.concatenate([Vcache[g], Vc[:, g, :]], axis=0)
        P = attention_probabilities(Qc[:, h, :], keys, m, causal=True)
        out[:, h, :] = P @ vals
        if lm_window > 0:
            t0 = max(0, L - lm_window)
            s_lm[g] += P[t0:, :].sum(axis=0)
    return out, s_lm


# --------------------------------------------------------------------------
# Step a2-I -- Eq. 1 with s = the instruction text I
# --------------------------------------------------------------------------
def importance_sum(Qs, Kcache, Kc):
    """S[g][j] = sum_{h in g} sum_{t in s} softmax_j(Q_t K_j^T / sqrt(d_k)).

    This is |s| * G times Eq. 1's mean -- a positive constant that does not
    change which k states are largest.  The softmax runs over exactly the
    candidates [cache rows ; chunk rows] (the set C of Eq. 1); the instruction
    follows the whole document, so nothing is masked.
    Qs [n_s,H_q,D]; Kcache [H_kv,m,D]; Kc [L,H_kv,D] -> [H_kv, m+L].
    """
    n_s, Hq, D = Qs.shape
    Hkv = Kc.shape[1]
    G = Hq // Hkv
    m = Kcache.shape[1]
    S = np.zeros((Hkv, m + Kc.shape[0]), dtype=np.float64)
    for h in range(Hq):
        g = h // G
        keys = np.concatenate([Kcache[g], Kc[:, g, :]], axis=0)
        P = attention_probabilities(Qs[:, h, :], keys, m, causal=False)
        S[g] += P.sum(axis=0)
    return S


# --------------------------------------------------------------------------
# Step a3 -- Eq. 2-3 (and Eq. 4-5 for the instruction cache): keep the k
# states with the highest importance.
# --------------------------------------------------------------------------
def select_topk(score: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest scores, ties to the lower index, ascending.

    If there are at most k candidates every one is kept.
    """
    n = score.shape[0]
    if n <= k:
        return np.arange(n, dtype=np.int64)
    # primary key: score descending; secondary: index ascending
    order = np.lexsort((np.arange(n), -score))
    return np.sort(order[:k]).astype(np.int64)


def kth_gap(score: np.ndarray, k: int):
    """(k-th largest, (k+1)-th largest) score, or (None, None) if n <= k."""
    if score.shape[0] <= k:
        return None, None
    s = np.sort(score)[::-1]
    return float(s[k - 1]), float(s[k])


# --------------------------------------------------------------------------
# Position shift (Section "Hyperparameters": positional embeddings follow the place in the cache, not the place in
# the document).  Rotary embedding in the half-split layout of the Llama / Mistral backbones: element d pairs with
# element d + D/2 and the pair turns by pos * base^(-2d/D).
# --------------------------------------------------------------------------
def rope(x: np.ndarray, pos: np.ndarray, base: float = 10000.0) -> np.ndarray:
    """x [..., D]; pos broadcastable to x.shape[:-1]."""
    D = x.shape[-1]
    half = D // 2
    theta = base ** (-2.0 * np.arange(half, dtype=np.float64) / D)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * theta
    c, s_ = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s_, x2 * c + x1 * s_], axis=-1)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even), returned as fp64: the precision in which a bf16 model holds
    its rotary-embedded queries and keys."""
    b = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    b = ((b + 0x7FFF + ((b >> 16) & 1)) & 0xFFFF0000).astype(np.uint32)
    return b.view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------
# Diagnostic of the appendix "Details for the Intersection Probing Experiments":
# |C_context  intersect  C_instruction| / |C_instruction| for two sets of retained states
# --------------------------------------------------------------------------
def intersection_ratio(pos_context: np.ndarray, pos_instruction: np.ndarray) -> np.ndarray:
    """pos_* [H_kv, rows] original token positions of two caches; ratio per head."""
    out = np.zeros(pos_instruction.shape[0], dtype=np.float64)
    for g in range(pos_instruction.shape[0]):
        a, b = set(pos_context[g].tolist()), set(pos_instruction[g].tolist())
        out[g] = len(a & b) / len(b)
    return out


# --------------------------------------------------------------------------
# Step a4 -- the evicted cache C-hat of Eq. 3 with the chunk's states put in
# --------------------------------------------------------------------------
def compact(Kcache_g, Vcache_g, pos_g, Kc_g, Vc_g, chunk_pos, idx):
    """Rows idx (ascending) of the candidate list [cache ; chunk] for one head."""
    keys = np.concatenate([Kcache_g, Kc_g], axis=0)
    vals = np.concatenate([Vcache_g, Vc_g], axis=0)
    pos = np.concatenate([pos_g, chunk_pos], axis=0)
    return keys[idx], vals[idx], pos[idx]


# --------------------------------------------------------------------------
# The loop
# --------------------------------------------------------------------------
@dataclass
class CacheState:
    K: np.ndarray      # [H_kv, m, D]
    V: np.ndarray      # [H_kv, m, D]
    pos: np.ndarray    # [H_kv, m] original token positions, ascending per head
    acc: Optional[np.ndarray] = None   # [H_kv, m] importance carried over from earlier steps (accumulate policy)


@dataclass
class StepResult:
    out: np.ndarray                                   # [L, H_q, D]
    scores: Dict[int, np.ndarray]                     # cache id -> [H_kv, n] (sum form)
    idx: Dict[int, np.ndarray]                        # cache id -> [H_kv, kept] the oracle's own choice
    applied: Dict[int, np.ndarray]                    # cache id -> indices actually applied
    gap: Dict[int, list] = field(default_factory=dict)  # cache id -> per head (kth, k+1th)
    m_before: int = 0                                  # rows of cache 0 before the step
    m_by_cache: Dict[int, int] = field(default_factory=dict)   # rows of every cache before the step


class CitrusOracle:
    """One decoder layer's cache state driven chunk by chunk.

    Cache 0 is the language-modelling side (the shared cache in shared mode);
    cache 1 exists only in individual mode and is the instruction-aware cache
    C^I of Eq. 4-5.  One call = encode the chunk over [cache 0 ; chunk]
    (a1), score all n = m + L candidates (a2), keep the top k (a3), compact
    (a4).  In shared mode this is the paper's evict -> encode -> append loop
    cut one phase later, so the paper's final eviction by I is the last call's
    own a2-a4 (checked by run_paper_order_shared).
    """

    def __init__(self, q_heads, kv_heads, head_dim, budget_k, mode=SHARED,
                 lm_window: Optional[int] = None, layerwise: bool = False, start_size: int = 0,
                 accumulate: bool = False, deferred_lm: bool = False, rope_shift: bool = False,
                 rope_base: float = 10000.0, embedded_dtype: Optional[str] = None):
        assert q_heads % kv_heads == 0
        self.Hq, self.Hkv, self.D, self.k = q_heads, kv_heads, head_dim, budget_k
        self.mode = mode
        self.lm_window = lm_window          # None -> every chunk query votes (Eq. 1)
        self.layerwise = layerwise
        self.start_size = start_size        # initial tokens that are always preserved (appendix on initial tokens)
        # accumulative score policy (the "H2O + Shared Cache" variant of the Baselines section): a retained state's
        # importance is the sum of what it received at every eviction step since it entered the cache
        self.accumulate = accumulate
        # Standard CSE exactly as Section 4.1 orders it (individual and standard modes): the language-modelling cache
        # C holds k states plus the previous chunk; the current chunk is encoded against all of them, its attention
        # evicts C down to k, then ALL of the chunk's states are put in.  Without the flag the chunk's own states
        # compete for the k places at once.
        self.deferred_lm = deferred_lm
        assert not deferred_lm or mode in (INDIVIDUAL, STANDARD)
        # position shift: Q, K and the instruction queries arrive without rotary embedding; every step embeds them by
        # their place in [cache ; chunk ; instruction] (cache row r -> r, chunk token i -> m + i, instruction token
        # i -> m + L + i).  The caches keep the un-rotated keys.
        self.rope_shift = rope_shift
        self.rope_base = rope_base
        # "bf16": the embedded queries and keys exist as bf16 tensors (one rounding of the fp64 rotation), as they do
        # in a bf16 model; None keeps them in fp64
        self.embedded_dtype = embedded_dtype
        assert not (rope_shift and deferred_lm)
        self.tokens_seen = 0
        n_caches = 2 if mode == INDIVIDUAL else 1
        self.caches = [CacheState(np.zeros((kv_heads, 0, head_dim)),
                                  np.zeros((kv_heads, 0, head_dim)),
                                  np.zeros((kv_heads, 0), dtype=np.int64))
                       for _ in range(n_caches)]

    def process_chunk(self, Qc, Kc, Vc, Qi, forced: Optional[Dict[int, np.ndarray]] = None) -> StepResult:
        Qc = np.asarray(Qc, dtype=np.float64)
        Kc = np.asarray(Kc, dtype=np.float64)
        Vc = np.asarray(Vc, dtype=np.float64)
        Qi = None if Qi is None else np.asarray(Qi, dtype=np.float64)
        L = Qc.shape[0]
        c0 = self.caches[0]
        m = c0.K.shape[1]
        chunk_pos = self.tokens_seen + np.arange(L, dtype=np.int64)

        raw_Kc = Kc
        cacheK = {cid: st.K for cid, st in enumerate(self.caches)}
        if self.rope_shift:
            b = self.rope_base
            Qc = rope(Qc, (m + np.arange(L))[:, None], b)
            Kc = rope(Kc, (m + np.arange(L))[:, None], b)
            if Qi is not None:
                Qi = rope(Qi, (m + L + np.arange(Qi.shape[0]))[:, None], b)
            cacheK = {cid: rope(st.K, np.arange(st.K.shape[1])[None, :], b) for cid, st in enumerate(self.caches)}
            if self.embedded_dtype == "bf16":
                Qc, Kc = round_bf16(Qc), round_bf16(Kc)
                Qi = None if Qi is None else round_bf16(Qi)
                cacheK = {cid: round_bf16(x) for cid, x in cacheK.items()}
        c0K = cacheK[0]

        scores: Dict[int, np.ndarray] = {}
        if self.mode == STANDARD and Qi is None:
            # Eq. 1 with s = the chunk: its last w queries vote on [cache ; chunk]
            w = L if self.lm_window is None else min(self.lm_window, L)
            out, s_lm = chunk_attention(Qc, c0K, c0.V, Kc, Vc, lm_window=w)
            scores[0] = s_lm
        elif self.mode in (SHARED, STANDARD):
            out, _ = chunk_attention(Qc, c0K, c0.V, Kc, Vc, lm_window=0)
            scores[0] = importance_sum(Qi, c0K, Kc)
        else:
            w = L if self.lm_window is None else min(self.lm_window, L)
            out, s_lm = chunk_attention(Qc, c0K, c0.V, Kc, Vc, lm_window=w)
            scores[0] = s_lm
            scores[1] = importance_sum(Qi, cacheK[1], Kc)

        rows = {cid: self.caches[cid].K.shape[1] for cid in scores}
        lm_scored = self.mode == INDIVIDUAL or (self.mode == STANDARD and Qi is None)   # cache 0 scored by the chunk
        if self.accumulate:
            for cid in list(scores):
                prev = self.caches[cid].acc
                carried = np.zeros((self.Hkv, rows[cid])) if prev is None else prev
                scores[cid] = scores[cid] + np.concatenate([carried, np.zeros((self.Hkv, L))], axis=1)
        res = StepResult(out=out, scores=scores, idx={}, applied={}, m_before=m, m_by_cache=rows)
        for cid, S in scores.items():
            S_total = S
            budget = self.k
            if self.deferred_lm and cid == 0 and lm_scored:
                # only C's own rows are candidates for eviction; the chunk's states all enter
                S = S.copy()
                S[:, m:] = np.inf
                budget = min(m, self.k) + L
            if self.layerwise:
                # one score vector for the whole layer (paper's stated granularity):
                # heads are aggregated before the top-k.
                S = np.broadcast_to(S.sum(axis=0, keepdims=True), S.shape)
            if self.start_size > 0:
                # the first start_size tokens of the document are never evicted: give them an unbeatable score
                S = S.copy()
                for g in range(self.Hkv):
                    cand_pos = np.concatenate([self.caches[cid].pos[g], chunk_pos])
                    S[g][cand_pos < self.start_size] = np.inf
            own = np.stack([select_topk(S[g], budget) for g in range(self.Hkv)])
            res.idx[cid] = own
            res.gap[cid] = [kth_gap(S[g], budget) for g in range(self.Hkv)]
            use = own if forced is None or cid not in forced else np.asarray(forced[cid], dtype=np.int64)
            res.applied[cid] = use
            c = self.caches[cid]
            newK, newV, newP = [], [], []
            for g in range(self.Hkv):
                kk, vv, pp = compact(c.K[g], c.V[g], c.pos[g], raw_Kc[:, g, :], Vc[:, g, :], chunk_pos, use[g])
                newK.append(kk); newV.append(vv); newP.append(pp)
            new_acc = np.stack([S_total[g][use[g]] for g in range(self.Hkv)]) if self.accumulate else None
            self.caches[cid] = CacheState(np.stack(newK), np.stack(newV), np.stack(newP), new_acc)
        self.tokens_seen += L
        return res


def run_paper_order_shared(Q_doc, K_doc, V_doc, Qi, budget_k, chunk_s):
    """Shared-cache CItruS in the order the paper states it (Section 4.1-4.3).

    Put the first chunk into the cache; for every later chunk: evict the cache to
    k states by Imp(I, c), encode the chunk against the evicted cache, put the
    chunk's states in; after the document, evict once more by Imp(I, c).
    Returns (outs per chunk, final CacheState).  Used only to check that the
    rotated loop of CitrusOracle performs the same operations.
    """
    Q_doc = np.asarray(Q_doc, dtype=np.float64); K_doc = np.asarray(K_doc, dtype=np.float64)
    V_doc = np.asarray(V_doc, dtype=np.float64); Qi = np.asarray(Qi, dtype=np.float64)
    N, Hq, D = Q_doc.shape
    Hkv = K_doc.shape[1]
    empty = np.zeros((Hkv, 0, D))
    cache = CacheState(empty.copy(), empty.copy(), np.zeros((Hkv, 0), dtype=np.int64))
    outs = []

    def evict(cache):
        no_chunk = np.zeros((0, Hkv, D))
        S = importance_sum(Qi, cache.K, no_chunk)
        Ks, Vs, Ps = [], [], []
        for g in range(Hkv):
            idx = select_topk(S[g], budget_k)
            Ks.append(cache.K[g][idx]); Vs.append(cache.V[g][idx]); Ps.append(cache.pos[g][idx])
        return CacheState(np.stack(Ks), np.stack(Vs), np.stack(Ps))

    for start in range(0, N, chunk_s):
        stop = min(N, start + chunk_s)
        if start > 0:
            cache = evict(cache)
        out, _ = chunk_attention(Q_doc[start:stop], cache.K, cache.V, K_doc[start:stop], V_doc[start:stop])
        outs.append(out)
        pos = np.broadcast_to(np.arange(start, stop, dtype=np.int64), (Hkv, stop - start))
        cache = CacheState(np.concatenate([cache.K, K_doc[start:stop].transpose(1, 0, 2)], axis=1),
                           np.concatenate([cache.V, V_doc[start:stop].transpose(1, 0, 2)], axis=1),
                           np.concatenate([cache.pos, pos], axis=1))
    cache = evict(cache)
    return outs, cache
