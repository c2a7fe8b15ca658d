"""fp64 CPU oracle (test infrastructure; never imported by the CUDA package)."""
from .citrus_oracle import (CitrusOracle, CacheState, StepResult, SHARED, INDIVIDUAL, STANDARD,
                            attention_probabilities, chunk_attention, importance_sum,
                            select_topk, kth_gap, compact, run_paper_order_shared, intersection_ratio, rope, round_bf16)
