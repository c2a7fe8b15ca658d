// Internal declarations shared by the host API and the kernel translation units.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

// Optional cycle stamps of one CTA's roles (build with -DCITRUS_TRACE; compiled out otherwise).
// Every translation unit that stamps keeps its own buffer and exports its own reader.
#ifdef CITRUS_TRACE
static __device__ unsigned long long g_citrus_trace[256];
#define CITRUS_TR(i) do { if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && (threadIdx.x & 31) == 0) \
                              g_citrus_trace[(i)] = clock64(); } while (0)
#define CITRUS_TRACE_EXPORT(suffix) \
    extern "C" int citrus_trace_read##suffix(unsigned long long* out) { return (int)cudaMemcpyFromSymbol(out, g_citrus_trace, sizeof(g_citrus_trace)); } \
    extern "C" int citrus_trace_clear##suffix() { static unsigned long long z[256]; return (int)cudaMemcpyToSymbol(g_citrus_trace, z, sizeof(z)); }
#else
#define CITRUS_TR(i) do { } while (0)
#define CITRUS_TRACE_EXPORT(suffix)
#endif

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

// One-time set-up that is per DEVICE (a kernel's shared-memory limit, the address of a __device__ symbol): which
// devices of this process have had it.  Host bookkeeping only; the caller holds its own mutex around a
// needs_setup / mark pair.
struct DeviceOnce {
    static constexpr int kMaxDevices = 64;
    bool done[kMaxDevices] = {};
    bool needs_setup(int dev) const { return dev < 0 || dev >= kMaxDevices || !done[dev]; }
    void mark(int dev) { if (dev >= 0 && dev < kMaxDevices) done[dev] = true; }
};
// Streaming multiprocessors of the current device (cached per device).
int sm_count();

// Called by every launcher immediately before its kernel launch: when per-launch timing is on, this is where the
// start event is recorded, so that host-side preparation (tensor-map encoding) is not counted as kernel time.
void before_launch(cudaStream_t s);

// A block of scoring / attending query rows, token-major [rows, q_heads, D].
struct QueryRows {
    const void* Q;
    int rows;
    int q_heads;
    int causal;   // 1: row r sees chunk candidates u <= t0 + r only
    int t0;       // chunk index of row 0 (causal only)
    int produced; // 1: Q and the chunk's keys were written by a kernel earlier in the stream (position shift), so a
                  // kernel launched with programmatic serialization must wait for its predecessors before ANY load
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
cudaError_t tc_init();   // resolves the driver entry point for tensor-map encoding; raises the kernels' shared-memory limits on the current device
// Test aid: one warp waits limit_ns on an mbarrier nobody arms, raises *status and returns.
cudaError_t tc_expire_wait(int* status, unsigned long long limit_ns, cudaStream_t s);
// Number of key splits for pass 1 of a2-I (1 = the pass writes final log-sum-exp values).
int tc_lse_splits(int n_rows, int q_heads, int kv_heads, int m, int L, int n_attn_items);
constexpr int kTcMaxLseSplits = 8;
constexpr int kTcMaxBatch = 32;            // sequences of one batched launch

// The tensors of one launch as its tensor maps see them: the packed token-major tensors of every sequence of the call
// and the cache tensors of all slots.  A sequence's rows and its cache's heads are offsets inside them.
struct TcTensors {
    const void* Q; void* out; int q_rows;          // chunk queries / attention output [q_rows, q_heads, D]
    const void* K; const void* V; int kv_rows;     // chunk keys / values [kv_rows, kv_heads, D]
    const void* Qi; int qi_rows;                   // instruction queries [qi_rows, q_heads, D]
    const void* cacheK[2]; const void* cacheV[2];  // cache id 0 (LM side / shared) and 1 (instruction): [cache_heads, cap, D]
    int cap[2], cache_heads[2];
    int q_heads, kv_heads;
};
// One sequence's step inside such a launch.
struct TcSeqStep {
    int L, q_row0, kv_row0;                // chunk rows; row offset of the sequence in Q / out and in K / V
    int nI, qi_row0;                       // instruction rows (0: none) and their offset in Qi
    int m[2], chead[2];                    // rows retained, and head offset inside the cache tensor, per cache id
    int ic;                                // cache that the instruction scores (0 shared design, 1 individual design)
    int w;                                 // chunk rows that score the LM-side cache (the last w), 0: none
    float* lse_chunk;                      // row log-sum-exp of a1 [q_heads, lse_chunk_stride], or null when nothing reads it
    float* lse_instr; float* part;         // pass 1 of a2-I: [q_heads, lse_instr_stride] / (max, sum) pairs per key split
    int splits;
    float* scores[2]; int score_stride;    // per cache id: [kv_heads, score_stride]
    int produced;                          // 1: wait for the preceding kernels before the first load of Q / K / Qi
};
// One launch: a1 (chunk over [cache 0 ; chunk] -> out, optional row log-sum-exp) and pass 1 of a2-I of every sequence.
// t.out == nullptr: pass 1 of a2-I alone; nI == 0 everywhere: a1 alone.
cudaError_t tc_attention_lse(const TcTensors& t, const TcSeqStep* seq, int n, int lse_chunk_stride, int lse_instr_stride,
                             int* status, cudaStream_t s);
// The column sums, one launch for both scorings and all sequences.  do_lm: the chunk's last w rows score cache 0's
// candidates with a1's probabilities; do_instr: the instruction rows score cache ic's candidates.
cudaError_t tc_colsum(const TcTensors& t, const TcSeqStep* seq, int n, bool do_lm, bool do_instr, int lse_chunk_stride,
                      int lse_instr_stride, int* status, cudaStream_t s);

// ---- select (a3) and compaction (a4) ---------------------------------------
struct SelectJob {            // one per cache handled by the launch
    float* scores;            // [kv_heads, score_stride]; with `carried` set, rewritten as score + carried
    int* idx;                 // [kv_heads, budget_k]
    int score_stride;
    // forced keeps ("start size"): candidates whose original position is below `start` are always selected
    const int* pos;           // positions of the old cache rows [kv_heads, pos_stride]
    int pos_stride, m, chunk_pos0, start;
    // accumulative policy: importance carried by the old cache rows [kv_heads, pos_stride], or null
    const float* carried;
    // sizes of this cache's step: n candidates, keep min(k, n); idx rows are idx_stride apart; candidates
    // j >= forced_from always stay (deferred eviction: the chunk's own states), n when there are none
    int n, k, idx_stride, forced_from;
};
// layerwise: sum scores over heads first and give every head the same set.
cudaError_t select_topk(const SelectJob* jobs, int n_jobs, int kv_heads, int layerwise, cudaStream_t s);

struct CompactJob {
    const void* srcK; const void* srcV; const int* srcPos;   // old cache buffers
    void* dstK; void* dstV; int* dstPos;                      // new cache buffers
    const int* idx;                                           // [kv_heads, budget_k]
    int m;                                                    // rows in the old cache
    // accumulative policy: the kept candidates' accumulated scores become the new cache's carried importance
    const float* totals; int score_stride; float* dstCarried;  // null when the policy is off
    int cap;                                                  // row capacity of this cache's buffers (old and new)
    int kept;                                                 // rows of the new cache
    // position shift: the un-rotated keys are what is gathered (old raw cache, caller's chunk K) and kept in
    // dstKraw; dstK receives them embedded by their new slot.  Null when the mode is off.
    const void* srcKraw; void* dstKraw;
    // the chunk's rows of this job's sequence: token-major [L, kv_heads, D] (un-rotated keys), and the original
    // position of its first token
    const void* chunkK; const void* chunkV; int chunk_pos0;
};
// Rotary embedding in the half-split layout: element d pairs with d + D/2, the pair turns by pos * theta[d].
struct RopeTable { double theta[64]; };
// One tensor of the embedding pre-pass: token-major [rows, heads, D], row i embedded at position pos0 + i.
struct RopeRows { const void* in; void* out; int rows, heads, pos0; };
cudaError_t rope_rows(const RopeRows* jobs, int n_jobs, int D, int elt, const RopeTable& table, cudaStream_t s);
// rope: table of the position shift, or null (the jobs' raw pointers are then null too); elt = bytes per element.
// Up to 2 * kTcMaxBatch jobs per launch (one per cache of every sequence of a batch).
cudaError_t compact_kv(const CompactJob* jobs, int n_jobs, int kv_heads, int row_bytes, const RopeTable* rope, int elt, cudaStream_t s);
// a3 + a4 in one launch (per-head granularity, no carried importance, no position shift) for small steps: several
// CTAs per (cache, KV head), each staging its share of the candidate rows in shared memory while it selects.
// early_chunk_rows: the chunk's K / V may be read before the preceding kernels have ended (caller inputs, complete).
// layerwise: every head keeps the candidates that the sum of the heads' scores ranks highest.
// select_compact_fits: whether a step of n candidates with rows of row_bytes fits that kernel's shared memory.
bool select_compact_fits(int n, int row_bytes);
cudaError_t select_compact(const SelectJob* sjobs, const CompactJob* cjobs, int n_jobs, int kv_heads, int row_bytes,
                           int elt, int early_chunk_rows, int layerwise, cudaStream_t s);
// ratio[g] = |{positions of a} intersect {positions of b}| / rows_b over two ascending position lists per head
cudaError_t intersection_ratio(const int* pos_a, int stride_a, int rows_a, const int* pos_b, int stride_b, int rows_b,
                               int kv_heads, float* ratio, cudaStream_t s);
}  // namespace citrus
