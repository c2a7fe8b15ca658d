// Internal declarations shared by the host API and the kernel translation units.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace citrus {

// Where the n = m + L candidate states of one call live.  Candidate j < m is row
// j of the retained cache [kv_heads, cap, D]; candidate j >= m is row j - m of
// the caller's token-major chunk tensor [L, kv_heads, D].
struct Candidates {
    const void* cacheK;
    const void* cacheV;
    const void* chunkK;
    const void* chunkV;
    int m;        // retained rows
    int L;        // chunk rows
    int cap;      // row capacity of the cache buffers (= budget_k)
    int kv_heads;
};

// A block of scoring / attending query rows, token-major [rows, q_heads, D].
struct QueryRows {
    const void* Q;
    int rows;
    int q_heads;
    int causal;   // 1: row r sees chunk candidates u <= t0 + r only
    int t0;       // chunk index of row 0 (causal only)
};

// ---- SIMT (true fp32 arithmetic) path ------------------------------------
// out may be null (log-sum-exp only).  lse2 [q_heads, lse_stride] receives
// log2(sum_j exp(logit_j)) of every row (logits scaled by 1/sqrt(D)).
cudaError_t simt_attention(bool is_fp32, int D, const QueryRows& q, const Candidates& c,
                           void* out, float* lse2, int lse_stride, cudaStream_t s);
// scores [kv_heads, score_stride]: column sums of exp2(logit2 - lse2) over rows and group heads.
cudaError_t simt_colsum(bool is_fp32, int D, const QueryRows& q, const Candidates& c,
                        const float* lse2, int lse_stride, float* scores, int score_stride, cudaStream_t s);

// ---- tensor-core (tcgen05 / TMEM / TMA) path: bf16, D = 128 ----------------
cudaError_t tc_init();   // resolves the driver entry point for tensor-map encoding
cudaError_t tc_attention(const QueryRows& q, const Candidates& c, void* out, float* lse2, int lse_stride,
                         int* status, cudaStream_t s);
cudaError_t tc_score_lse(const QueryRows& q, const Candidates& c, float* lse2, int lse_stride,
                         int* status, cudaStream_t s);
cudaError_t tc_colsum(const QueryRows& q, const Candidates& c, const float* lse2, int lse_stride,
                      float* scores, int score_stride, int* status, cudaStream_t s);

// ---- select (a3) and compaction (a4) ---------------------------------------
struct SelectJob {            // one per cache handled by the launch
    const float* scores;      // [kv_heads, score_stride]
    int* idx;                 // [kv_heads, budget_k]
    int score_stride;
};
// n candidates, keep min(k, n); layerwise: sum scores over heads first and give every head the same set.
cudaError_t select_topk(const SelectJob* jobs, int n_jobs, int kv_heads, int n, int k, int layerwise, cudaStream_t s);

struct CompactJob {
    const void* srcK; const void* srcV; const int* srcPos;   // old cache buffers
    void* dstK; void* dstV; int* dstPos;                      // new cache buffers
    const int* idx;                                           // [kv_heads, budget_k]
    int m;                                                    // rows in the old cache
};
cudaError_t compact_kv(const CompactJob* jobs, int n_jobs, const void* chunkK, const void* chunkV,
                       int kv_heads, int cap, int row_bytes, int kept, int chunk_pos0, cudaStream_t s);
}  // namespace citrus
