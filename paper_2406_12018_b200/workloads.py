"""Seeded synthetic Q/K/V documents shaped like 7B decoder layers.

This module only draws inputs.  It holds none of the eviction method's
arithmetic and is the one piece shared by the CPU oracle's tests and the CUDA
library's tests and benchmark, so that both sides see bit-identical tensors.

Recipe (all entries i.i.d. z ~ N(0,1) unless stated; the 1/sqrt(D) of the
softmax makes logits unit-variance):
  * per KV group g an orthonormal pair (u_g, v_g);
  * instruction queries  q^I = z + 3 v_g  (a "topic" direction);
  * planted relevant keys at seeded distinct document positions:
        k_p = 3 sqrt(D) m_g,  m_g = unit mean of the group's instruction queries,
    so instruction logits on them are about 9 while document logits stay N(0,9);
  * sink keys (when the workload has them) k_s = 4 sqrt(D) u_g at the first
    positions, and every query (document and instruction) gets + 2 u_g, so each
    query's logit on a sink is about 8;
  * heavy-tailed keys: Student-t(nu=3) / sqrt(3) (unit variance) before planting.
Values are generated in fp32 and rounded once to the storage dtype.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import List, Optional

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    layers: int
    q_heads: int
    kv_heads: int
    head_dim: int
    budget_k: int
    chunk_s: int
    doc_tokens: int            # per sequence (max for ragged)
    n_instr: int
    dtype: str                 # "bf16" | "fp32"
    mode: str                  # "shared" | "individual"
    lm_window: int = 0         # 0 -> every chunk query scores the LM cache
    n_planted: int = 0
    n_sinks: int = 0
    heavy_tail: bool = False
    n_seqs: int = 1
    min_tokens: int = 0        # ragged: lengths ~ U{min_tokens..doc_tokens}
    start_size: int = 0        # initial tokens that are never evicted (paper's appendix variant: 4)
    accumulate: bool = False   # accumulative score policy: importance carried across steps
    deferred_lm: bool = False  # language-modelling cache evicted by the next chunk (Section 4.1 order)
    position_shift: bool = False   # inputs without rotary embedding; embedded by cache slot every step
    rope_base: float = 10000.0
    layerwise: bool = False    # one kept set per layer from head-summed scores (the paper's stated granularity)

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32


CONFIGS = {
    # Tiny fp32, 4 chunks, shared cache.
    "tiny_fp32": Workload("tiny_fp32", 0, 1, 8, 2, 64, 64, 128, 512, 16, "fp32", "shared", n_planted=8),
    # Mistral-7B-shaped single layer, shared cache, sink at position 0.
    "mistral7b_layer": Workload("mistral7b_layer", 2, 1, 32, 8, 128, 768, 512, 16384, 64, "bf16", "shared",
                                n_planted=32, n_sinks=1),
    # Llama-2-7B-shaped 32-layer stack, individual caches, LM window 64.
    "llama2_7b_stack": Workload("llama2_7b_stack", 3, 32, 32, 32, 128, 1024, 1024, 32768, 128, "bf16",
                                "individual", lm_window=64),
    # Ragged serving mix of 16 sequences, 4K-32K tokens, shared cache.
    "serving_mix": Workload("serving_mix", 4, 1, 32, 8, 128, 2048, 2048, 32768, 128, "bf16", "shared",
                            n_seqs=16, min_tokens=4096),
    # 131072-token heavy-tailed stress, individual caches.
    "long_doc_stress": Workload("long_doc_stress", 5, 1, 32, 8, 128, 4096, 4096, 131072, 256, "bf16",
                                "individual", n_planted=256, n_sinks=4, heavy_tail=True),
}


# The paper's own setting (Section "Hyperparameters": k = 768, l_s = 256, cache of 1024 while reading) on the head
# geometries of its backbone models; one decoder layer each, shared cache.
PAPER_SHAPES = {
    "paper_mistral7b": Workload("paper_mistral7b", 11, 1, 32, 8, 128, 768, 256, 16384, 64, "bf16", "shared",
                                n_planted=32, n_sinks=1),
    # the same with the position shift the paper applies (inputs without rotary embedding, embedded by cache slot)
    "paper_mistral7b_shift": Workload("paper_mistral7b_shift", 11, 1, 32, 8, 128, 768, 256, 16384, 64, "bf16", "shared",
                                      n_planted=32, n_sinks=1, position_shift=True),
    "paper_llama2_13b": Workload("paper_llama2_13b", 12, 1, 40, 40, 128, 768, 256, 16384, 64, "bf16", "shared",
                                 n_planted=32, n_sinks=1),
    "paper_llama3_8b": Workload("paper_llama3_8b", 13, 1, 32, 8, 128, 768, 256, 16384, 64, "bf16", "individual",
                                lm_window=64, n_planted=32, n_sinks=1),
}


# The other eviction policies of Section 4.1 on the Mistral-7B-shaped layer: standard chunked eviction (one cache,
# scored by the chunk's own last 64 queries; the instruction only evicts in the last call) and the layer-wise
# granularity (scores summed over the KV heads, one kept set for the whole layer).
VARIANTS = {
    "mistral7b_standard": Workload("mistral7b_standard", 2, 1, 32, 8, 128, 768, 512, 16384, 64, "bf16", "standard",
                                   lm_window=64, n_planted=32, n_sinks=1),
    "mistral7b_layerwise": Workload("mistral7b_layerwise", 2, 1, 32, 8, 128, 768, 512, 16384, 64, "bf16", "shared",
                                    n_planted=32, n_sinks=1, layerwise=True),
}


def scaled(w: Workload, **kw) -> Workload:
    """A smaller or altered copy of a workload (for tests)."""
    return replace(w, **kw)


def sequence_lengths(w: Workload) -> List[int]:
    """Document length of every sequence slot (ragged workloads draw them uniformly)."""
    if w.n_seqs == 1 or w.min_tokens == 0:
        return [w.doc_tokens] * w.n_seqs
    rng = np.random.Generator(np.random.Philox(key=[w.seed, 0xA11CE]))
    return [int(x) for x in rng.integers(w.min_tokens, w.doc_tokens + 1, size=w.n_seqs)]


@dataclass
class Document:
    Q: torch.Tensor            # [N, H_q, D]   document queries
    K: torch.Tensor            # [N, H_kv, D]
    V: torch.Tensor            # [N, H_kv, D]
    Q_instr: torch.Tensor      # [n_I, H_q, D]
    planted: np.ndarray        # [n_planted] positions
    sinks: np.ndarray          # [n_sinks] positions


def _orthonormal_pair(rng, D):
    a = rng.standard_normal(D)
    b = rng.standard_normal(D)
    a /= np.linalg.norm(a)
    b -= a * (a @ b)
    b /= np.linalg.norm(b)
    return a.astype(np.float32), b.astype(np.float32)


def make_document(w: Workload, layer: int = 0, seq: int = 0, n_tokens: Optional[int] = None) -> Document:
    """Draw one (layer, sequence) document of workload w on the CPU."""
    if n_tokens is not None:
        N = n_tokens
    else:
        lens = sequence_lengths(w)
        N = lens[seq] if seq < len(lens) else w.doc_tokens      # further sequences of a fixed-length workload
    Hq, Hkv, D = w.q_heads, w.kv_heads, w.head_dim
    G = Hq // Hkv
    rng = np.random.Generator(np.random.Philox(key=[w.seed * 1000 + layer, seq]))

    pairs = [_orthonormal_pair(rng, D) for _ in range(Hkv)]
    U = np.stack([p[0] for p in pairs])            # [Hkv, D] sink direction
    Vdir = np.stack([p[1] for p in pairs])         # [Hkv, D] topic direction
    Uq = np.repeat(U, G, axis=0)                   # per query head
    Vq = np.repeat(Vdir, G, axis=0)

    Q = rng.standard_normal((N, Hq, D), dtype=np.float32)
    Qi = rng.standard_normal((w.n_instr, Hq, D), dtype=np.float32) + 3.0 * Vq[None]
    if w.heavy_tail:
        K = (rng.standard_t(3.0, size=(N, Hkv, D)) / np.sqrt(3.0)).astype(np.float32)
    else:
        K = rng.standard_normal((N, Hkv, D), dtype=np.float32)
    Vv = rng.standard_normal((N, Hkv, D), dtype=np.float32)

    sinks = np.arange(min(w.n_sinks, N), dtype=np.int64)
    if len(sinks):
        Q += 2.0 * Uq[None]
        Qi += 2.0 * Uq[None]
        K[sinks] = 4.0 * np.sqrt(D) * U[None]

    n_pl = min(w.n_planted, max(0, N - len(sinks)))
    planted = np.zeros(0, dtype=np.int64)
    if n_pl:
        planted = np.sort(rng.choice(np.arange(len(sinks), N), size=n_pl, replace=False)).astype(np.int64)
        mean_q = Qi.reshape(w.n_instr, Hkv, G, D).mean(axis=(0, 2))          # [Hkv, D]
        mean_q /= np.linalg.norm(mean_q, axis=1, keepdims=True)
        K[planted] = 3.0 * np.sqrt(D) * mean_q[None]

    dt = w.torch_dtype
    return Document(torch.from_numpy(Q).to(dt), torch.from_numpy(K).to(dt), torch.from_numpy(Vv).to(dt),
                    torch.from_numpy(Qi).to(dt), planted, sinks)


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact fp64 value of a stored bf16/fp32 tensor (what both sides compute on)."""
    return t.to(torch.float64).numpy()
