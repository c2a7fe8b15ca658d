// True-fp32 CUDA-core path for steps a1 (attention over [cache ; chunk]) and a2
// (Eq. 1 importance column sums).  Used for fp32 tensors, where the 1e-4 tolerance
// rules out reduced-precision tensor-core products.
#include "citrus_internal.h"

namespace citrus {
namespace {

constexpr float kLog2e = 1.4426950408889634f;

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T, int D>
__device__ __forceinline__ const T* key_row(const Candidates& c, const void* cache, const void* chunk, int g, int j) {
    if (j < c.m) return reinterpret_cast<const T*>(cache) + ((size_t)g * c.cap + j) * D;
    return reinterpret_cast<const T*>(chunk) + ((size_t)(j - c.m) * c.kv_heads + g) * D;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

constexpr int kRowsPerCta = 8;    // one warp per query row
constexpr int kKeyTile = 32;      // one key per lane

// One warp per (query row, head): online softmax over key tiles of 32.
template <typename T, int D>
__global__ void __launch_bounds__(kRowsPerCta * 32)
simt_attention_kernel(QueryRows q, Candidates c, T* __restrict__ out, float* __restrict__ lse2, int lse_stride) {
    __shared__ float Ks[kKeyTile][D + 1];
    __shared__ float Vs[kKeyTile][D];
    __shared__ float Qs[kRowsPerCta][D];

    const int h = blockIdx.y;
    const int G = q.q_heads / c.kv_heads;
    const int g = h / G;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row0 = blockIdx.x * kRowsPerCta;
    const int r = row0 + warp;
    const bool row_ok = r < q.rows;
    const int n = c.m + c.L;
    const float scale2 = kLog2e * rsqrtf((float)D);

    const T* Qp = reinterpret_cast<const T*>(q.Q);
    for (int i = threadIdx.x; i < kRowsPerCta * D; i += blockDim.x) {
        int rr = row0 + i / D;
        Qs[i / D][i % D] = rr < q.rows ? to_f<T>(Qp[((size_t)rr * q.q_heads + h) * D + (i % D)]) : 0.f;
    }

    // last candidate any row of this CTA may see
    int last_row = min(row0 + kRowsPerCta, q.rows) - 1;
    int n_cta = q.causal ? min(n, c.m + q.t0 + last_row + 1) : n;
    int n_row = q.causal ? min(n, c.m + q.t0 + r + 1) : n;

    float m_run = -INFINITY, l_run = 0.f;
    float o[D / 32];
#pragma unroll
    for (int i = 0; i < D / 32; ++i) o[i] = 0.f;

    for (int j0 = 0; j0 < n_cta; j0 += kKeyTile) {
        __syncthreads();
        for (int i = threadIdx.x; i < kKeyTile * D; i += blockDim.x) {
            int jj = i / D, d = i % D, j = j0 + jj;
            float kv = 0.f, vv = 0.f;
            if (j < n) {
                kv = to_f<T>(key_row<T, D>(c, c.cacheK, c.chunkK, g, j)[d]);
                if (out != nullptr) vv = to_f<T>(key_row<T, D>(c, c.cacheV, c.chunkV, g, j)[d]);
            }
            Ks[jj][d] = kv;
            Vs[jj][d] = vv;
        }
        __syncthreads();
        float s = 0.f;
#pragma unroll 8
        for (int d = 0; d < D; ++d) s = fmaf(Qs[warp][d], Ks[lane][d], s);
        s *= scale2;
        const int j = j0 + lane;
        if (!row_ok || j >= n_row) s = -INFINITY;
        float tile_max = warp_max(s);
        if (tile_max == -INFINITY) continue;          // nothing visible to this row in the tile (uniform per warp)
        float m_new = fmaxf(m_run, tile_max);
        float corr = exp2f(m_run - m_new);            // 0 on the first visible tile
        float p = exp2f(s - m_new);
        l_run = l_run * corr + warp_sum(p);
        m_run = m_new;
        if (out != nullptr) {
#pragma unroll
            for (int i = 0; i < D / 32; ++i) o[i] *= corr;
            for (int jj = 0; jj < kKeyTile; ++jj) {
                float pj = __shfl_sync(0xffffffffu, p, jj);
#pragma unroll
                for (int i = 0; i < D / 32; ++i) o[i] = fmaf(pj, Vs[jj][lane + 32 * i], o[i]);
            }
        }
    }
    if (row_ok) {
        if (out != nullptr) {
            float inv = 1.f / l_run;
#pragma unroll
            for (int i = 0; i < D / 32; ++i)
                out[((size_t)r * q.q_heads + h) * D + lane + 32 * i] = from_f<T>(o[i] * inv);
        }
        if (lse2 != nullptr && lane == 0) lse2[(size_t)h * lse_stride + r] = m_run + log2f(l_run);
    }
}

constexpr int kColsumKeys = 128;   // one candidate per thread
constexpr int kColsumRows = 16;    // scoring rows staged per step

// Thread j owns candidate j: S[g][j] = sum_{h in g} sum_r exp2(q_{r,h}.k_j * scale2 - lse2[h][r]).
// Fixed (h, r) summation order, so the result is run-to-run identical.
template <typename T, int D>
__global__ void __launch_bounds__(kColsumKeys)
simt_colsum_kernel(QueryRows q, Candidates c, const float* __restrict__ lse2, int lse_stride,
                   float* __restrict__ scores, int score_stride) {
    __shared__ float Qs[kColsumRows][D];
    __shared__ float Ls[kColsumRows];
    const int g = blockIdx.y;
    const int G = q.q_heads / c.kv_heads;
    const int n = c.m + c.L;
    const int j = blockIdx.x * kColsumKeys + threadIdx.x;
    const float scale2 = kLog2e * rsqrtf((float)D);

    float kreg[D];
    {
        const T* kp = key_row<T, D>(c, c.cacheK, c.chunkK, g, min(j, n - 1));
#pragma unroll
        for (int d = 0; d < D; ++d) kreg[d] = to_f<T>(kp[d]);
    }
    // first scoring row that may see this candidate
    const int u = j - c.m;                               // chunk index if j >= m
    const int r_first = (q.causal && u > q.t0) ? (u - q.t0) : 0;
    const T* Qp = reinterpret_cast<const T*>(q.Q);
    float acc = 0.f;
    for (int hh = 0; hh < G; ++hh) {
        const int h = g * G + hh;
        for (int r0 = 0; r0 < q.rows; r0 += kColsumRows) {
            __syncthreads();
            for (int i = threadIdx.x; i < kColsumRows * D; i += blockDim.x) {
                int rr = r0 + i / D;
                Qs[i / D][i % D] = rr < q.rows ? to_f<T>(Qp[((size_t)rr * q.q_heads + h) * D + (i % D)]) : 0.f;
            }
            if (threadIdx.x < kColsumRows) {
                int rr = r0 + threadIdx.x;
                Ls[threadIdx.x] = rr < q.rows ? lse2[(size_t)h * lse_stride + rr] : INFINITY;
            }
            __syncthreads();
            const int rn = min(kColsumRows, q.rows - r0);
            for (int rr = 0; rr < rn; ++rr) {
                float s = 0.f;
#pragma unroll
                for (int d = 0; d < D; ++d) s = fmaf(Qs[rr][d], kreg[d], s);
                float p = exp2f(s * scale2 - Ls[rr]);
                if (r0 + rr >= r_first) acc += p;
            }
        }
    }
    if (j < n) scores[(size_t)g * score_stride + j] = acc;
}

template <typename T, int D>
cudaError_t launch_attention(const QueryRows& q, const Candidates& c, void* out, float* lse2, int lse_stride, cudaStream_t s) {
    dim3 grid((q.rows + kRowsPerCta - 1) / kRowsPerCta, q.q_heads);
    before_launch(s);
    simt_attention_kernel<T, D><<<grid, kRowsPerCta * 32, 0, s>>>(q, c, reinterpret_cast<T*>(out), lse2, lse_stride);
    return cudaGetLastError();
}
template <typename T, int D>
cudaError_t launch_colsum(const QueryRows& q, const Candidates& c, const float* lse2, int lse_stride,
                          float* scores, int score_stride, cudaStream_t s) {
    int n = c.m + c.L;
    dim3 grid((n + kColsumKeys - 1) / kColsumKeys, c.kv_heads);
    before_launch(s);
    simt_colsum_kernel<T, D><<<grid, kColsumKeys, 0, s>>>(q, c, lse2, lse_stride, scores, score_stride);
    return cudaGetLastError();
}

}  // namespace

cudaError_t simt_attention(bool is_fp32, int D, const QueryRows& q, const Candidates& c,
                           void* out, float* lse2, int lse_stride, cudaStream_t s) {
    if (is_fp32) return D == 64 ? launch_attention<float, 64>(q, c, out, lse2, lse_stride, s)
                                : launch_attention<float, 128>(q, c, out, lse2, lse_stride, s);
    return D == 64 ? launch_attention<__nv_bfloat16, 64>(q, c, out, lse2, lse_stride, s)
                   : launch_attention<__nv_bfloat16, 128>(q, c, out, lse2, lse_stride, s);
}

cudaError_t simt_colsum(bool is_fp32, int D, const QueryRows& q, const Candidates& c,
                        const float* lse2, int lse_stride, float* scores, int score_stride, cudaStream_t s) {
    if (is_fp32) return D == 64 ? launch_colsum<float, 64>(q, c, lse2, lse_stride, scores, score_stride, s)
                                : launch_colsum<float, 128>(q, c, lse2, lse_stride, scores, score_stride, s);
    return D == 64 ? launch_colsum<__nv_bfloat16, 64>(q, c, lse2, lse_stride, scores, score_stride, s)
                   : launch_colsum<__nv_bfloat16, 128>(q, c, lse2, lse_stride, scores, score_stride, s);
}

}  // namespace citrus
