// Allocation-free importance scoring: Eq. 1 column sums with the log-sum-exp scratch in a
// statically reserved device array instead of memory obtained from cudaMalloc.
#include "../../include/citrus.h"
#include "citrus_internal.h"

#include <mutex>

namespace {

using namespace citrus;

constexpr int kStatusFloats = 64;                                   // first 256 bytes: status word
constexpr int kLseFloats = CITRUS_STATIC_MAX_LSE;                   // log-sum-exp of every (head, scoring row)

// Reserved in every GPU's memory that loads this library, until the process exits.
static __device__ __align__(256) float g_static_scratch[kStatusFloats + kLseFloats];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
float* g_static_ptr[kMaxDevices] = {nullptr};   // device address of g_static_scratch, per device

// The symbol's name is only a host-side handle; kernels need its device address, looked up once
// per device with that device current.
int static_scratch(float** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return CITRUS_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) return CITRUS_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (g_static_ptr[dev] == nullptr) {
        float* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch);
        if (e != cudaSuccess || p == nullptr) { cudaGetLastError(); return CITRUS_ERR_CUDA; }
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return CITRUS_OK;
}

}  // namespace

extern "C" int citrus_importance_static(const void* Q_s, int n_s, const void* K, int n_keys,
                                        int q_heads, int kv_heads, int head_dim, unsigned mode,
                                        float* scores, int score_stride, int* device_status,
                                        citrus_stream_t stream) {
    if (Q_s == nullptr || K == nullptr || scores == nullptr) return CITRUS_ERR_INVALID_ARG;
    if (q_heads < 1 || kv_heads < 1 || n_s < 1 || n_keys < 1 || score_stride < n_keys) return CITRUS_ERR_INVALID_ARG;
    if (mode & ~CITRUS_MODE_FP32) return CITRUS_ERR_INVALID_ARG;
    if (q_heads % kv_heads != 0) return CITRUS_ERR_SHAPE;
    const bool fp32 = (mode & CITRUS_MODE_FP32) != 0;
    if (head_dim != 128 && !(fp32 && head_dim == 64)) return CITRUS_ERR_UNSUPPORTED;
    const int lse_stride = (n_s + 3) & ~3;
    // sizes beyond the static reservation are refused, never truncated
    if (n_s > CITRUS_MAX_INSTR || n_keys > CITRUS_MAX_CANDIDATES) return CITRUS_ERR_SHAPE;
    if ((long long)q_heads * lse_stride > kLseFloats) return CITRUS_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(Q_s) | reinterpret_cast<uintptr_t>(K)) & 15u) return CITRUS_ERR_ALIGN;

    float* scratch = nullptr;
    int rc = static_scratch(&scratch);
    if (rc != CITRUS_OK) return rc;
    if (!fp32 && tc_init() != cudaSuccess) { cudaGetLastError(); return CITRUS_ERR_UNSUPPORTED; }

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int* status = device_status != nullptr ? device_status : reinterpret_cast<int*>(scratch);
    float* lse = scratch + kStatusFloats;
    // the array keeps whatever the previous call left: the status word must start at zero
    if (device_status == nullptr && cudaMemsetAsync(scratch, 0, kStatusFloats * sizeof(float), st) != cudaSuccess) {
        cudaGetLastError();
        return CITRUS_ERR_CUDA;
    }
    // all candidates are "chunk" rows of a token-major tensor; there is no retained cache (m = 0)
    cudaError_t e;
    if (fp32) {
        Candidates cand{K, K, K, K, 0, n_keys, n_keys, kv_heads};
        QueryRows q{Q_s, n_s, q_heads, 0, 0, 1};   // produced = 1: wait for earlier stream work before the first load of Q_s or K
        e = simt_attention(true, head_dim, q, cand, nullptr, lse, lse_stride, st);
        if (e == cudaSuccess) e = simt_colsum(true, head_dim, q, cand, lse, lse_stride, scores, score_stride, st);
    } else {
        TcTensors t{};
        t.q_heads = q_heads; t.kv_heads = kv_heads;
        t.Q = nullptr; t.out = nullptr; t.q_rows = 0;
        t.K = K; t.V = K; t.kv_rows = n_keys;
        t.Qi = Q_s; t.qi_rows = n_s;
        for (int ci = 0; ci < 2; ++ci) { t.cacheK[ci] = K; t.cacheV[ci] = K; t.cap[ci] = n_keys; t.cache_heads[ci] = kv_heads; }   // never read: m = 0
        TcSeqStep q{};
        q.L = n_keys; q.nI = n_s; q.ic = 0; q.splits = 1; q.w = 0;
        q.lse_chunk = nullptr; q.lse_instr = lse; q.part = nullptr;
        q.scores[0] = scores; q.scores[1] = scores; q.score_stride = score_stride;
        q.produced = 1;                            // wait for earlier stream work before the first load of Q_s or K
        e = tc_attention_lse(t, &q, 1, 0, lse_stride, status, st);
        if (e == cudaSuccess) e = tc_colsum(t, &q, 1, false, true, 0, lse_stride, status, st);
    }
    if (e != cudaSuccess) { cudaGetLastError(); return CITRUS_ERR_CUDA; }
    return CITRUS_OK;
}
