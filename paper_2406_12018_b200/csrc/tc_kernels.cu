// Tensor-core path (bf16, head_dim 128) for steps a1 and a2 on sm_100a:
// TMA (cp.async.bulk.tensor) stages 128-byte-swizzled tiles in shared memory,
// tcgen05.mma accumulates in tensor memory, and the softmax / column-sum warps read
// the accumulators back with tcgen05.ld.  Three kernels share the machinery:
//
//   attn_lse_kernel     one launch of attn_body items:
//     attn_body<true,*>   a1: causal attention of the chunk over [cache ; chunk] (+ row LSE)
//     attn_body<false,*>  a2 pass 1: row log-sum-exp of the scoring queries over (a split of) the candidates
//   colsum_kernel       a2 pass 2: S^T = K Q^T with the candidates on the accumulator's rows,
//                       so the column sum of Eq. 1 over scoring rows is a per-thread sum
//
// Every wait on an mbarrier is bounded; a wait that expires raises the status word,
// the CTA drains and returns (tensor memory is always released).
#include "citrus_internal.h"

#include <cuda.h>

#include <mutex>
#include <utility>

CITRUS_TRACE_EXPORT()

namespace citrus {
namespace {

constexpr int kTile = 128;              // rows of every staged tile (queries, keys)
constexpr int kD = 128;                 // head dimension
constexpr int kHalfBytes = kTile * 128; // one [128 rows][64 bf16] swizzle-128B sub-tile
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint64_t kWaitLimitNs = 1000000000ull;   // a bounded wait gives up after about one second

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One arrival for the whole warp: every lane's earlier work (ordered by its own fences) is published by lane 0.
// 32 per-thread arrivals on one barrier word are 32 serialised shared-memory atomics; this is one.
__device__ __forceinline__ void mbar_arrive_warp(uint32_t bar) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false (and the status word raised) if the phase never completes.
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, int* status, uint64_t limit_ns = kWaitLimitNs) {
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < limit_ns) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try(bar, parity)) return true;
        __nanosleep(128);
    }
    atomicExch(status, 1);
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* status, uint64_t limit_ns = kWaitLimitNs) {
    for (int i = 0; i < 512; ++i)
        if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, status, limit_ns);
}
// Same, with one outcome for the whole warp (the callers go on to warp-collective instructions).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, int* status, uint64_t limit_ns = kWaitLimitNs) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, status, limit_ns));
}

// One lane of a converged warp.  Loop control, addresses and descriptors are computed by the whole
// warp (so they stay warp-uniform); only the issuing instruction itself is predicated on the leader.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
    return pred != 0;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d), "r"(a), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp gets lane (base + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
          "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// Two fp32 values in one 64-bit register pair for the packed fp32 instructions.
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Shared-memory matrix descriptors (sm_100 format: version 1 at bit 46, 128-byte swizzle = 2 at bit 61).
// K-major operand tile [rows][64 bf16]: 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// MN-major operand (V as B of P.V): [keys][64 bf16] sub-tiles; 8-key groups 1024 B apart (stride offset),
// the two 64-wide halves of the head dimension kHalfBytes apart (leading offset).
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(kHalfBytes >> 4) << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}

// ------------------------------------------------------------------ parameters
struct TcParams {
    int rows;        // query rows in the block
    int row0;        // row offset of the block inside the Q tensor map (and of its output rows inside the out map)
    int krow0;       // row offset of this sequence's chunk keys / values inside the chunk K / V maps
    int chead;       // head offset of this sequence's retained cache inside the cache maps
    int q_heads, kv_heads;
    int m, L;        // retained rows, chunk rows
    int causal, t0;  // row r sees chunk keys u <= t0 + r
    void* out;       // [rows, q_heads, 128] bf16 or null
    float* lse2;     // [q_heads, lse_stride]
    int lse_stride;
    float2* part;    // a2 pass 1 with key splits: (max, sum) of every (split, head, row), [splits, q_heads, lse_stride]
    int splits;      // number of key splits (1: lse2 / lse_in hold final log-sum-exp values)
    int pack;        // a2 pass 1: heads of one KV group sharing a 128-row tile (short instruction texts), 1 = none
    int pack_rows;   // rows per head in a packed tile (= rows)
    const float* lse_in;   // colsum: log-sum-exp of the scoring rows
    float* scores;   // colsum: [kv_heads, score_stride]
    int score_stride;
    int* status;
    int dep_first;   // the queries and the chunk's keys come from a preceding kernel: wait for it before the first load
};

// Load one 128x128 bf16 tile as two swizzled halves.  token_major: coordinates (d, head, row);
// otherwise (cache layout) (d, row, head).
// Called by a converged warp; one elected lane arms the barrier and issues the two copies.
__device__ __forceinline__ void load_tile(uint32_t dst, const CUtensorMap* map, uint32_t bar, int row, int head, bool token_major) {
    const int y = token_major ? head : row, z = token_major ? row : head;
    if (elect_one()) {
        mbar_expect_tx(bar, kTileBytes);
        tma_load_3d(dst, map, bar, 0, y, z);
        tma_load_3d(dst + kHalfBytes, map, bar, 64, y, z);
    }
    __syncwarp();
}

// S[128 x n_cols] = A_tile . B_tile^T over the 128-wide head dimension (8 steps of 16).
// Called by a converged warp; bar1/bar2 (0 = none) receive a commit after the eight MMAs.
__device__ __forceinline__ void issue_qk(uint32_t tmem_d, uint32_t a_smem, uint32_t b_smem, uint32_t idesc,
                                         uint32_t bar1, uint32_t bar2) {
    const uint64_t a0 = desc_kmajor(a_smem), b0 = desc_kmajor(b_smem);
    if (elect_one()) {
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            const uint64_t off = (uint64_t)(((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4);   // start-address field units
            mma_ss(tmem_d, a0 + off, b0 + off, idesc, kk > 0);
        }
        if (bar1) mma_commit(bar1);
        if (bar2) mma_commit(bar2);
    }
    __syncwarp();
}
// O (+)= P . V for one key tile: P (bf16) in tensor memory, V tile MN-major in shared memory.
__device__ __forceinline__ void issue_pv(uint32_t tmem_o, uint32_t tmem_p, uint32_t v_smem, uint32_t idesc, bool first,
                                         uint32_t bar1, uint32_t bar2) {
    const uint64_t b0 = desc_mnmajor(v_smem);
    if (elect_one()) {
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)     // 16 keys per step: P columns 8*kk.., V rows 16*kk.. (2048 B apart)
            mma_ts(tmem_o, tmem_p + kk * 8, b0 + (uint64_t)((kk * 2048) >> 4), idesc, !(first && kk == 0));
        mma_commit(bar1);
        mma_commit(bar2);
    }
    __syncwarp();
}

constexpr int kStagesK = 2;             // K ring
constexpr int kStagesV = 2;             // V ring
constexpr int kVStageBytes = kTileBytes + kHalfBytes;   // a V tile and, right behind it, a [128 keys][64] block of ones
constexpr int kAttnThreads = 352;       // 8 softmax warps, K-TMA warp, MMA warp, V-TMA warp
constexpr int kColGroups = 4;           // column-sum warp groups (four warps each), one S^T accumulator per group
constexpr int kColThreads = (kColGroups * 4 + 2) * 32;   // the groups, 1 TMA warp, 1 MMA warp
constexpr int kTmemCols = 512;
constexpr uint32_t kTmemO = 256;        // O accumulator: 128 output columns + 16 columns that all hold the row sum of P
constexpr uint32_t kTmemL = kTmemO + 128;
constexpr uint32_t kTmemP = 400;        // P (bf16 pairs), 64 columns
constexpr int kOCols = 144;
constexpr int kMaxLseSplits = 8;
constexpr float kRescaleTau = 8.f;      // rescale O only when the row max grows by more than 2^8

// Bulk tensor store shared -> global (rows past the tensor map's extent are clipped).
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

struct AttnSmem {
    uint64_t q_full, k_full[kStagesK], k_empty[kStagesK], v_full[kStagesV], v_empty[kStagesV];
    uint64_t s_full[2], s_free[2], p_full, o_done[2], xch, out_ready[2], drain;
    uint32_t tmem_base;
    float lsum[2][kTile];               // fp32 row sums of the two column halves, exchanged once at the end
};
constexpr int kAttnSmemBytes = 1024 /*align slack*/ + kTileBytes * (1 + kStagesK) + kVStageBytes * kStagesV + 4096;

// grid: (ceil(rows / 128), q_heads).  One CTA = 128 query rows of one head.
// WITH_PV: accumulate O = P.V and write `out`; NEED_LSE: keep the fp32 row sum and write the row log-sum-exp.
//
// Tensor memory: S[0], S[1] (128 fp32 columns each, Q.K^T of alternating key tiles), O (128 + 16 columns),
// P (64 columns of bf16 pairs).  S is double-buffered and P has a place of its own, so Q.K^T of tile j+2 is issued
// as soon as the softmax warps have read S of tile j into registers; the tensor pipe never waits for the
// exponentials of the tile it is about to overwrite, only P.V of tile j waits for P of tile j.
//
// Softmax: eight warps; warps w and w+4 share rows 32 (w & 3) .. +31, thread (w, lane) owns columns
// 64 (w >> 2) .. +63 of its row.  Both threads of a row read all 128 columns once to take the same row maximum
// (so they agree on the exponent reference and on every rescale without exchanging anything) and keep only their
// own half for the exponentials.  The row sum of the bf16-rounded probabilities - the normaliser that makes
// out = sum(p~ v) / sum(p~) a convex combination of V rows - comes from the tensor core itself: the V operand of
// P.V is 144 columns wide, the last 16 read from a block of ones, so columns 128..143 of O accumulate sum(p~)
// in the same fp32 arithmetic as the output columns, and are rescaled with them.
template <bool WITH_PV, bool NEED_LSE>
__device__ __forceinline__ void attn_body(const CUtensorMap& mapQ, const CUtensorMap& mapCK, const CUtensorMap& mapCV,
                                          const CUtensorMap& mapSK, const CUtensorMap& mapSV, const CUtensorMap& mapO,
                                          const TcParams& p, const int qt, const int h, const int tile_begin, int tile_end,
                                          const int split, uint8_t* smem_raw) {
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = base;
    const uint32_t sK = sQ + kTileBytes;
    const uint32_t sV = sK + kStagesK * kTileBytes;
    uint8_t* const gQ = smem_raw + (sQ - smem_u32(smem_raw));         // generic pointer to the Q tile / output staging
    AttnSmem* bars = reinterpret_cast<AttnSmem*>(smem_raw + (sV + kStagesV * kVStageBytes - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = h / (p.q_heads / p.kv_heads);
    if (WITH_PV && warp == 0) CITRUS_TR(0);
    const int q_row0 = qt * kTile;                                  // first row of this tile inside the block
    const int n_cache_tiles = (p.m + kTile - 1) / kTile;
    // chunk key tiles this query tile may see
    int n_chunk_tiles = (p.L + kTile - 1) / kTile;
    if (p.causal) {
        int last_t = p.t0 + min(q_row0 + kTile, p.rows) - 1;         // highest chunk index among the rows
        n_chunk_tiles = min(n_chunk_tiles, last_t / kTile + 1);
    }
    // this CTA sweeps key tiles [tile_begin, tile_end) of the candidate list; j below is local to that range
    tile_end = min(tile_end, n_cache_tiles + n_chunk_tiles);
    const int nt = max(0, tile_end - tile_begin);

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars->q_full), 1);
        for (int s = 0; s < kStagesK; ++s) { mbar_init(smem_u32(&bars->k_full[s]), 1); mbar_init(smem_u32(&bars->k_empty[s]), 1); }
        for (int s = 0; s < kStagesV; ++s) { mbar_init(smem_u32(&bars->v_full[s]), 1); mbar_init(smem_u32(&bars->v_empty[s]), 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bars->s_full[b]), 1); mbar_init(smem_u32(&bars->s_free[b]), 8);
            mbar_init(smem_u32(&bars->o_done[b]), 1); mbar_init(smem_u32(&bars->out_ready[b]), 4);
        }
        mbar_init(smem_u32(&bars->p_full), 8);
        mbar_init(smem_u32(&bars->xch), 8);
        mbar_init(smem_u32(&bars->drain), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (WITH_PV) {
        // the blocks of ones behind the V stages (bf16 1.0 everywhere, so the swizzle does not matter)
        constexpr int kVec = kHalfBytes / 16;
        for (int i = threadIdx.x; i < kStagesV * kVec; i += kAttnThreads) {
            uint8_t* dst = smem_raw + (sV + (i / kVec) * kVStageBytes + kTileBytes - smem_u32(smem_raw)) + (i % kVec) * 16;
            *reinterpret_cast<uint4*>(dst) = make_uint4(0x3f803f80u, 0x3f803f80u, 0x3f803f80u, 0x3f803f80u);
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == 9) tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // Programmatic dependent launch: this kernel may run while its predecessor (the previous chunk's compaction)
    // still does.  The chunk's own tiles come first in the sweep and need nothing from it, so only two things
    // wait for the predecessor (griddepcontrol.wait): the first load of a retained-cache tile, and the
    // log-sum-exp writes of the epilogue (the previous chunk's column-sum kernel may still be reading them).
    // Exception (p.dep_first): with the position shift the queries and the chunk's keys are written by the
    // embedding pre-pass launched just before, so the Q/K producer waits before its first load.
    // Sweep order: tile index jg(j) = chunk tiles first, then cache tiles.
    auto sweep_tile = [&](int j) {
        const int t = tile_begin + j;
        return t < n_chunk_tiles ? n_cache_tiles + t : t - n_chunk_tiles;
    };
    const uint32_t tmem = bars->tmem_base;
    auto tmS = [tmem](int b) { return tmem + (uint32_t)b * 128u; };
    // completion of P.V of tile j: phase (j >> 1) of o_done[j & 1]
    auto pv_done = [&](int j) { return mbar_wait_warp(smem_u32(&bars->o_done[j & 1]), (j >> 1) & 1, p.status); };
    if (WITH_PV && warp == 0) CITRUS_TR(1);

    if (warp == 8) {
        // ---------------------------------------------------------------- K (and Q) TMA producer (converged warp)
        bool dep_waited = false;
        if (p.dep_first) { asm volatile("griddepcontrol.wait;" ::: "memory"); dep_waited = true; }
        if (!WITH_PV && p.pack > 1) {
            // several heads' scoring rows side by side in one tile (mapQ's box is pack_rows rows high)
            if (elect_one()) {
                const uint32_t bar = smem_u32(&bars->q_full);
                mbar_expect_tx(bar, (uint32_t)(p.pack * p.pack_rows * 256));
                for (int hh = 0; hh < p.pack; ++hh) {
                    tma_load_3d(sQ + hh * p.pack_rows * 128, &mapQ, bar, 0, h + hh, p.row0);
                    tma_load_3d(sQ + kHalfBytes + hh * p.pack_rows * 128, &mapQ, bar, 64, h + hh, p.row0);
                }
            }
            __syncwarp();
        } else {
            load_tile(sQ, &mapQ, smem_u32(&bars->q_full), p.row0 + q_row0, h, true);
        }
        for (int j = 0; j < nt; ++j) {
            const int s = j % kStagesK, jg = sweep_tile(j);
            const bool from_cache = jg < n_cache_tiles;
            const int row = from_cache ? jg * kTile : p.krow0 + (jg - n_cache_tiles) * kTile;
            if (from_cache && !dep_waited) {
                asm volatile("griddepcontrol.wait;" ::: "memory");
                dep_waited = true;
#ifdef CITRUS_TRACE
                if (WITH_PV && lane == 0) atomicMax(&g_citrus_trace[244], ~global_ns());
#endif
            }
            if (!mbar_wait_warp(smem_u32(&bars->k_empty[s]), ((j / kStagesK) & 1) ^ 1, p.status)) break;
            load_tile(sK + s * kTileBytes, from_cache ? &mapCK : &mapSK, smem_u32(&bars->k_full[s]), row, from_cache ? p.chead + g : g, !from_cache);
        }
    } else if (warp == 10) {
        // ---------------------------------------------------------------- V TMA producer (converged warp)
        if (WITH_PV) {
            bool dep_waited = false;
            for (int j = 0; j < nt; ++j) {
                const int s = j % kStagesV, jg = sweep_tile(j);
                const bool from_cache = jg < n_cache_tiles;
                const int row = from_cache ? jg * kTile : p.krow0 + (jg - n_cache_tiles) * kTile;
                if (from_cache && !dep_waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); dep_waited = true; }
                if (!mbar_wait_warp(smem_u32(&bars->v_empty[s]), ((j / kStagesV) & 1) ^ 1, p.status)) break;
                load_tile(sV + s * kVStageBytes, from_cache ? &mapCV : &mapSV, smem_u32(&bars->v_full[s]), row, from_cache ? p.chead + g : g, !from_cache);
            }
        }
    } else if (warp == 9) {
        // ---------------------------------------------------------------- MMA issuer (converged warp)
        constexpr uint32_t idesc_qk = make_idesc(128, 0);
        constexpr uint32_t idesc_pv = make_idesc(kOCols, 1);
        bool ok = mbar_wait_warp(smem_u32(&bars->q_full), 0, p.status);
        if (WITH_PV) CITRUS_TR(2);
        auto k_ready = [&](int j) { return mbar_wait_warp(smem_u32(&bars->k_full[j % kStagesK]), (j / kStagesK) & 1, p.status); };
        auto qk = [&](int j) {
            const int s = j % kStagesK;
            issue_qk(tmS(j & 1), sQ, sK + s * kTileBytes, idesc_qk, smem_u32(&bars->s_full[j & 1]), smem_u32(&bars->k_empty[s]));
        };
        for (int j = 0; j < 2 && j < nt && ok; ++j) {
            ok = k_ready(j);
            if (ok) { tc_fence_after(); qk(j); }
        }
        for (int j = 0; j < nt && ok; ++j) {
            if (j + 2 < nt) {
                // S[j & 1] is free as soon as every softmax thread holds tile j in registers
                ok = k_ready(j + 2) && mbar_wait_warp(smem_u32(&bars->s_free[j & 1]), (j >> 1) & 1, p.status);
                if (!ok) break;
                tc_fence_after();
                qk(j + 2);
                if (WITH_PV && j + 2 < 12) CITRUS_TR(10 + j + 2);
            }
            if (WITH_PV) {
                const int s = j % kStagesV;
                ok = mbar_wait_warp(smem_u32(&bars->v_full[s]), (j / kStagesV) & 1, p.status) &&
                     mbar_wait_warp(smem_u32(&bars->p_full), j & 1, p.status);
                if (!ok) break;
                tc_fence_after();
                if (j < 10) CITRUS_TR(90 + j);
                issue_pv(tmem + kTmemO, tmem + kTmemP, sV + s * kVStageBytes, idesc_pv, j == 0,
                         smem_u32(&bars->v_empty[s]), smem_u32(&bars->o_done[j & 1]));
                if (j < 10) CITRUS_TR(30 + j);
            }
        }
        // all tensor-core work retired before tensor memory is released
        if (elect_one()) mma_commit(smem_u32(&bars->drain));
        __syncwarp();
        mbar_wait_warp(smem_u32(&bars->drain), 0, p.status);
    } else {
        // ---------------------------------------------------------------- softmax warps 0-7
        const int half = warp >> 2;                                  // which 64 columns of the row this thread keeps
        const int row_in_tile = (warp & 3) * 32 + lane;
        const int r = q_row0 + row_in_tile;                          // row inside the block
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t o_addr = tmem + kTmemO + lane_base;
        const uint32_t p_addr = tmem + kTmemP + lane_base + (uint32_t)half * 32u;
        const float scale2 = kLog2e * rsqrtf((float)kD);
        const uint64_t scale2x2 = pack_f32x2(scale2, scale2);
        float m_ref = -INFINITY, l_run = 0.f;
        bool ok = true;
#pragma unroll 1
        for (int j = 0; j < nt; ++j) {
            const int b = j & 1;
            ok = mbar_wait_warp(smem_u32(&bars->s_full[b]), (j >> 1) & 1, p.status);
            if (!ok) break;
            if (WITH_PV && (warp & 3) == 0 && j < 8) CITRUS_TR((half ? 200 : 50) + 5 * j);
            tc_fence_after();
            // number of visible columns of this tile for this row
            int lim = kTile;
            const int jg = sweep_tile(j);
            if (jg < n_cache_tiles) {
                lim = min(kTile, p.m - jg * kTile);
            } else {
                const int u0 = (jg - n_cache_tiles) * kTile;
                lim = min(kTile, p.L - u0);
                if (p.causal) lim = min(lim, p.t0 + r - u0 + 1);
            }
            const uint32_t s_addr = tmS(b) + lane_base;
            uint32_t own[64], oth[64];
            tmem_ld32(s_addr + (half ^ 1) * 64, oth);
            tmem_ld32(s_addr + (half ^ 1) * 64 + 32, oth + 32);
            tmem_ld32(s_addr + half * 64, own);
            tmem_ld32(s_addr + half * 64 + 32, own + 32);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive_warp(smem_u32(&bars->s_free[b]));
            // ---- row maximum over the visible columns.  A tile that holds hidden columns (future tokens of the chunk,
            // rows past the end of the cache or chunk - zero fill, stale cache rows, or in a packed batch the next
            // sequence's rows) has them set to -inf first, in both halves, so both threads of the row still agree.
            if (lim < kTile) {
                const int lim_own = lim - half * 64, lim_oth = lim - (half ^ 1) * 64;
#pragma unroll
                for (int q = 0; q < 64; ++q) {
                    if (q >= lim_own) own[q] = 0xff800000u;          // -inf
                    if (q >= lim_oth) oth[q] = 0xff800000u;
                }
            }
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int q = 0; q < 64; q += 2) {
                mx4[(q >> 1) & 1] = max3(mx4[(q >> 1) & 1], __uint_as_float(oth[q]), __uint_as_float(oth[q + 1]));
                mx4[2 + ((q >> 1) & 1)] = max3(mx4[2 + ((q >> 1) & 1)], __uint_as_float(own[q]), __uint_as_float(own[q + 1]));
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
            const float m_new = fmaxf(m_ref, mx * scale2);
            if (WITH_PV && (warp & 3) == 0 && j < 8) CITRUS_TR((half ? 201 : 51) + 5 * j);
            if (j == 0) {
                m_ref = m_new;
            } else {
                // both threads of a row see the same values, so they take the same decision
                const bool grow = m_new > m_ref + kRescaleTau;       // also when the row has seen nothing so far (m_ref = -inf)
                if (__any_sync(0xffffffffu, grow)) {
                    // Only the rows that grew change their reference; the others scale by exactly one.  A row's
                    // arithmetic therefore never depends on what the other rows of its warp hold (in a packed batch
                    // the rows past a sequence's end are the next sequence's), and results are the same bits whether
                    // a sequence is stepped alone or inside a batch.
                    const float f = grow ? ex2(m_ref - m_new) : 1.f;
                    if (grow) { l_run *= f; m_ref = m_new; }
                    if (WITH_PV) {
                        // O must be quiescent: P.V of tile j-1 (and with it every earlier one) has retired
                        ok = pv_done(j - 1);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll 1
                        for (int c = 0; c < 2; ++c) {
                            uint32_t oreg[32];
                            tmem_ld32(o_addr + half * 64 + c * 32, oreg);
                            tmem_wait_ld();
#pragma unroll
                            for (int q = 0; q < 32; ++q) oreg[q] = __float_as_uint(__uint_as_float(oreg[q]) * f);
                            tmem_st32(o_addr + half * 64 + c * 32, oreg);
                        }
                        if (half == 0) {
                            uint32_t lreg[16];
                            tmem_ld16(tmem + kTmemL + lane_base, lreg);
                            tmem_wait_ld();
#pragma unroll
                            for (int q = 0; q < 16; ++q) lreg[q] = __float_as_uint(__uint_as_float(lreg[q]) * f);
                            tmem_st16(tmem + kTmemL + lane_base, lreg);
                        }
                    }
                }
            }
            // ---- probabilities of this thread's 64 columns; with NEED_LSE the fp32 values are summed too (that sum
            // feeds the log-sum-exp that the LM scoring pass reuses)
            const float neg_m = m_ref == -INFINITY ? 0.f : -m_ref;
            const uint64_t neg_m2 = pack_f32x2(neg_m, neg_m);
            uint64_t sum2[2] = {0ull, 0ull};
            uint32_t packed[32];
            if (WITH_PV && (warp & 3) == 0 && j < 8) CITRUS_TR((half ? 202 : 52) + 5 * j);
#pragma unroll
            for (int q = 0; q < 32; ++q) {
                float x0, x1;
                unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(own[2 * q]), __uint_as_float(own[2 * q + 1])), scale2x2, neg_m2), x0, x1);
                const float p0 = ex2(x0), p1 = ex2(x1);
                if (NEED_LSE) sum2[q & 1] = add_f32x2(sum2[q & 1], pack_f32x2(p0, p1));
                packed[q] = pack_bf16(p0, p1);
            }
            if (NEED_LSE) {
                float a0, a1, b0, b1;
                unpack_f32x2(sum2[0], a0, a1); unpack_f32x2(sum2[1], b0, b1);
                l_run += (a0 + a1) + (b0 + b1);
            }
            if (WITH_PV && (warp & 3) == 0 && j < 8) CITRUS_TR((half ? 203 : 53) + 5 * j);
            if (WITH_PV) {
                // the single P buffer is free once P.V of the previous tile has read it
                if (j > 0) { ok = pv_done(j - 1); if (!ok) break; }
                tc_fence_after();
                tmem_st16(p_addr, packed);
                tmem_st16(p_addr + 16, packed + 16);
                tmem_wait_st();                                      // also covers a rescale's stores to O
                tc_fence_before();
                mbar_arrive_warp(smem_u32(&bars->p_full));
            }
            if (WITH_PV && (warp & 3) == 0 && j < 8) CITRUS_TR((half ? 204 : 54) + 5 * j);
        }
        // ---- epilogue
        if (ok && WITH_PV && nt > 0) ok = pv_done(nt - 1);
        if (NEED_LSE) {
            bars->lsum[half][row_in_tile] = l_run;
            mbar_arrive_warp(smem_u32(&bars->xch));
            ok = mbar_wait_warp(smem_u32(&bars->xch), 0, p.status) && ok;
        }
        if (ok) {
            tc_fence_after();
            if (warp == 0) CITRUS_TR(110);
            if (WITH_PV && nt > 0) {
                // this thread finishes columns [64 half, 64 half + 64) of its row
                uint32_t lreg[16];
                tmem_ld16(tmem + kTmemL + lane_base, lreg);
                tmem_wait_ld();
                const float inv = 1.f / __uint_as_float(lreg[0]);
                uint8_t* stage = gQ + half * kHalfBytes + row_in_tile * 128;   // [128 rows][64 bf16], 128-byte swizzle
                // A tile that reaches past the block's last row is written row by row (a bulk store would run into the
                // rows of the next sequence of a packed batch); whole tiles go through shared memory and TMA.
                const bool whole_tile = q_row0 + kTile <= p.rows;
                uint4* direct = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) +
                                                         ((size_t)(p.row0 + r) * p.q_heads + h) * kD + half * 64);
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t o0[32];
                    tmem_ld32(o_addr + half * 64 + c * 32, o0);
                    tmem_wait_ld();
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float v[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(o0[8 * q + e]) * inv;
                        uint4 u;
                        u.x = pack_bf16(v[0], v[1]); u.y = pack_bf16(v[2], v[3]);
                        u.z = pack_bf16(v[4], v[5]); u.w = pack_bf16(v[6], v[7]);
                        const int chunk = c * 4 + q;                 // 16-byte chunk inside the 128-byte row
                        if (whole_tile) *reinterpret_cast<uint4*>(stage + ((chunk ^ (row_in_tile & 7)) << 4)) = u;
                        else if (r < p.rows) direct[chunk] = u;
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive_warp(smem_u32(&bars->out_ready[half]));
                if (whole_tile && (warp & 3) == 0) {
                    // one warp per column half stores its 128 x 64 part of the output tile
                    if (mbar_wait_warp(smem_u32(&bars->out_ready[half]), 0, p.status)) {
                        if (elect_one()) {
                            tma_store_3d(&mapO, sQ + half * kHalfBytes, half * 64, h, p.row0 + q_row0);
                            tma_store_wait_read();
                        }
                        __syncwarp();
                    }
                }
            }
            // which (head, row) this thread's tile row stands for
            int oh = h, orow = r;
            bool row_ok = r < p.rows;
            if (!WITH_PV && p.pack > 1) {
                oh = h + row_in_tile / p.pack_rows;
                orow = row_in_tile % p.pack_rows;
                row_ok = row_in_tile < p.pack * p.pack_rows;
            }
            if (NEED_LSE && half == 0) asm volatile("griddepcontrol.wait;" ::: "memory");   // see the note on the sweep order
            if (NEED_LSE && half == 0 && row_ok) {
                const float l = bars->lsum[0][row_in_tile] + bars->lsum[1][row_in_tile];
                if (p.splits > 1) p.part[((size_t)split * p.q_heads + oh) * p.lse_stride + orow] = make_float2(m_ref, l);
                else if (p.lse2 != nullptr) p.lse2[(size_t)oh * p.lse_stride + orow] = m_ref + log2f(l);
            }
        }
    }
    if (WITH_PV && warp == 0) CITRUS_TR(111);
    tc_fence_before();
    __syncthreads();
    if (WITH_PV && warp == 0) CITRUS_TR(112);
    if (warp == 9) { __syncwarp(); tmem_dealloc(tmem, kTmemCols); }
}

// One launch for a1 and for pass 1 of a2-I of every sequence of a batch (CAP = 1: a single sequence).  The grid is
// a list of segments: first the attention items (query tile, head) of sequence 0, 1, ... - each sequence's longest
// sweeps first - then the log-sum-exp items (instruction row tile, head, key split) of sequence 0, 1, ..., which fill
// the SMs that a partial wave of attention items leaves idle.
//   pa[s] / maps Q, CK, CV, SK, SV, O : attention of the chunk over [cache 0 ; chunk]
//   pl[s] / maps QI, CKI, SK          : instruction queries over [instruction-side cache ; chunk]
// The maps cover the packed tensors of the whole batch; a sequence's rows and cache heads are offsets in them.
template <int CAP>
struct AttnBatch {
    int n;                       // sequences
    int seg_end[2 * CAP];        // exclusive end of every segment in the 1-D grid
    TcParams pa[CAP], pl[CAP];
};
template <bool NEED_LSE, int CAP>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_lse_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapCK,
                const __grid_constant__ CUtensorMap mapCV, const __grid_constant__ CUtensorMap mapSK,
                const __grid_constant__ CUtensorMap mapSV, const __grid_constant__ CUtensorMap mapO,
                const __grid_constant__ CUtensorMap mapQI, const __grid_constant__ CUtensorMap mapCKI,
                const __grid_constant__ AttnBatch<CAP> bt) {
    extern __shared__ uint8_t smem_raw[];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int id = blockIdx.x, seg = 0;
    if (CAP > 1) {
        while (seg + 1 < 2 * bt.n && id >= bt.seg_end[seg]) ++seg;
        if (seg > 0) id -= bt.seg_end[seg - 1];
    } else if (id >= bt.seg_end[0]) {
        id -= bt.seg_end[0]; seg = 1;
    }
#ifdef CITRUS_TRACE
    unsigned long long t_start = 0;
    if (threadIdx.x == 0) { t_start = global_ns(); atomicMax(&g_citrus_trace[240], ~t_start); }   // complemented: max = earliest
#endif
    if (seg < bt.n) {
        const TcParams& pa = bt.pa[seg];
        const int n_qt = (pa.rows + kTile - 1) / kTile;
        const int qt = n_qt - 1 - id / pa.q_heads, h = id % pa.q_heads;      // later query tiles see more keys
        attn_body<true, NEED_LSE>(mapQ, mapCK, mapCV, mapSK, mapSV, mapO, pa, qt, h, 0, 1 << 30, 0, smem_raw);
    } else {
        const TcParams& pl = bt.pl[seg - bt.n];
        const int split = id % pl.splits, rest = id / pl.splits;
        const int head_slots = pl.q_heads / pl.pack;
        const int h = (rest % head_slots) * pl.pack, rt = rest / head_slots;
        const int tiles = (pl.m + kTile - 1) / kTile + (pl.L + kTile - 1) / kTile;
        const int t0 = (int)((long long)split * tiles / pl.splits), t1 = (int)((long long)(split + 1) * tiles / pl.splits);
        attn_body<false, true>(mapQI, mapCKI, mapCKI, mapSK, mapSK, mapQI, pl, rt, h, t0, t1, split, smem_raw);
    }
#ifdef CITRUS_TRACE
    if (threadIdx.x == 0) {
        const unsigned long long t_end = global_ns();
        atomicMax(&g_citrus_trace[241], t_end);
        atomicMax(&g_citrus_trace[seg < bt.n ? 242 : 243], t_end - t_start);   // longest attention / log-sum-exp item
    }
#endif
}

// ------------------------------------------------------------------ column sums (a2 pass 2)
constexpr int kColStages = 4;
constexpr int kColTmemCols = 512;         // four S^T accumulators: Q.K^T of four iterations can be in flight
struct ColSmem {
    uint64_t k_full, q_full[kColStages], q_empty[kColStages], s_full[4], s_free[4], lse_full[8], drain;
    uint32_t tmem_base;
    alignas(16) float lse[8][kTile];          // log-sum-exp of the scoring rows of eight consecutive (head, row block)s
    float acc_other[kColGroups - 1][kTile];   // partial column sums of the other warp groups
};
constexpr int kColSmemBytes = 1024 + kTileBytes * (1 + kColStages) + 8192;

// grid: (kv_heads, candidate tiles) - the KV head varies fastest, so CTAs are dispatched in the order of their tile
// index: the retained-cache tiles (which every scoring row sees) first, then the chunk's tiles, whose sweeps get
// shorter and shorter under the causal mask; the short ones fill the tail of the last wave.
// Accumulator rows = 128 candidates, columns = scoring rows of one
// (head, row block); thread i owns candidate i and adds exp2(logit2 - lse2[row]) over its columns.
// One launch serves both scoring passes of a step and every sequence of a batch: blockIdx.y runs over the candidate
// tiles of entry 0, 1, ... (tile_end = exclusive prefix ends).  Entries [0, n_first) are LM scorings (the chunk's last
// w rows over cache 0's candidates: query map Q0, cache map CK0), the others instruction scorings (instruction rows
// over the instruction-side cache's candidates: Q1, CK1).  The LM entries come first: their sweeps are the long ones.
template <int CAP>
struct ColBatch {
    int n_entries, n_first;
    int tile_end[2 * CAP];
    TcParams p[2 * CAP];
};
template <int CAP>
__global__ void __launch_bounds__(kColThreads, 1)
colsum_kernel(const __grid_constant__ CUtensorMap mapQ0, const __grid_constant__ CUtensorMap mapCK0,
              const __grid_constant__ CUtensorMap mapQ1, const __grid_constant__ CUtensorMap mapCK1,
              const __grid_constant__ CUtensorMap mapSK, const __grid_constant__ ColBatch<CAP> bt) {
    extern __shared__ uint8_t smem_raw[];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int entry = 0, kt = blockIdx.y;
    while (entry + 1 < bt.n_entries && kt >= bt.tile_end[entry]) ++entry;
    if (entry > 0) kt -= bt.tile_end[entry - 1];
    const TcParams& p = bt.p[entry];
    const CUtensorMap& mapQ = entry < bt.n_first ? mapQ0 : mapQ1;
    const CUtensorMap& mapCK = entry < bt.n_first ? mapCK0 : mapCK1;
#ifdef CITRUS_TRACE
    if (threadIdx.x == 0) atomicMax(&g_citrus_trace[245], ~global_ns());
#endif
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sK = base;
    const uint32_t sQ = sK + kTileBytes;
    ColSmem* bars = reinterpret_cast<ColSmem*>(smem_raw + (sQ + kColStages * kTileBytes - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = blockIdx.x;
    const int G = p.q_heads / p.kv_heads;
    const int n_cache_tiles = (p.m + kTile - 1) / kTile;
    const bool from_cache = kt < n_cache_tiles;
    if (warp == 0) CITRUS_TR(128);
    const int key_row0 = from_cache ? kt * kTile : (kt - n_cache_tiles) * kTile;   // row in its source
    const int n_rb = (p.rows + kTile - 1) / kTile;
    // first row block that can see any key of this tile
    int rb0 = 0;
    if (p.causal && !from_cache && key_row0 > p.t0) rb0 = (key_row0 - p.t0) / kTile;
    const int rb_per_head = n_rb - rb0;
    const int nb = G * rb_per_head;                   // (head, row block) iterations

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars->k_full), 1);
        for (int s = 0; s < kColStages; ++s) { mbar_init(smem_u32(&bars->q_full[s]), 1); mbar_init(smem_u32(&bars->q_empty[s]), 1); }
        for (int b = 0; b < 4; ++b) {
            mbar_init(smem_u32(&bars->s_full[b]), 1); mbar_init(smem_u32(&bars->s_free[b]), 4);
        }
        for (int b = 0; b < 8; ++b) mbar_init(smem_u32(&bars->lse_full[b]), 4);
        mbar_init(smem_u32(&bars->drain), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    constexpr int kTmaWarp = kColGroups * 4, kMmaWarp = kColGroups * 4 + 1;
    if (warp == kMmaWarp) tmem_alloc(smem_u32(&bars->tmem_base), kColTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // Programmatic dependent launch: the scoring queries and the chunk's keys are the caller's inputs and are loaded
    // at once (unless p.dep_first says that a preceding kernel wrote them: then the producer waits first); what the preceding kernels produce is touched only after griddepcontrol.wait - a retained-cache
    // tile (written by the previous chunk's compaction), the log-sum-exp values of pass 1, and the score vector
    // (still read by the previous chunk's select until that kernel has ended).
    const uint32_t tmem = bars->tmem_base;
    auto tmS = [tmem](int b) { return tmem + (uint32_t)b * 128u; };

    if (warp == kTmaWarp) {
        // TMA producer (converged warp)
        auto load_q = [&](int it) {
            const int s = it % kColStages;
            const int h = g * G + it / rb_per_head;
            const int rb = rb0 + it % rb_per_head;
            if (!mbar_wait_warp(smem_u32(&bars->q_empty[s]), ((it / kColStages) & 1) ^ 1, p.status)) return false;
            load_tile(sQ + s * kTileBytes, &mapQ, smem_u32(&bars->q_full[s]), p.row0 + rb * kTile, h, true);
            return true;
        };
        bool ok = true;
        int it = 0;
        if (p.dep_first) asm volatile("griddepcontrol.wait;" ::: "memory");
        for (; it < nb && it < kColStages && ok; ++it) ok = load_q(it);
        if (from_cache && !p.dep_first) asm volatile("griddepcontrol.wait;" ::: "memory");
        load_tile(sK, from_cache ? &mapCK : &mapSK, smem_u32(&bars->k_full), from_cache ? key_row0 : p.krow0 + key_row0,
                  from_cache ? p.chead + g : g, !from_cache);
        for (; it < nb && ok; ++it) ok = load_q(it);
    } else if (warp == kMmaWarp) {
        // MMA issuer (converged warp)
        bool ok = mbar_wait_warp(smem_u32(&bars->k_full), 0, p.status);
        for (int it = 0; it < nb && ok; ++it) {
            const int s = it % kColStages, b = it & 3;
            const int rb = rb0 + it % rb_per_head;
            const int ncols = min(kTile, ((p.rows - rb * kTile) + 31) & ~31);     // whole 32-column pieces
            ok = mbar_wait_warp(smem_u32(&bars->q_full[s]), (it / kColStages) & 1, p.status);
            if (!ok) break;
            ok = mbar_wait_warp(smem_u32(&bars->s_free[b]), ((it >> 2) & 1) ^ 1, p.status);
            if (!ok) break;
            tc_fence_after();
            CITRUS_TR(140 + 2 * (it & 7));
            issue_qk(tmS(b), sK, sQ + s * kTileBytes, make_idesc(ncols, 0),
                     smem_u32(&bars->s_full[b]), smem_u32(&bars->q_empty[s]));
            CITRUS_TR(141 + 2 * (it & 7));
        }
        if (elect_one()) mma_commit(smem_u32(&bars->drain));
        __syncwarp();
        mbar_wait_warp(smem_u32(&bars->drain), 0, p.status);
    } else {
        asm volatile("griddepcontrol.wait;" ::: "memory");
#ifdef CITRUS_TRACE
        if (threadIdx.x == 0) atomicMax(&g_citrus_trace[246], ~global_ns());
#endif
        // kColGroups groups of four warps: group t takes the (head, row block) iterations it = t (mod kColGroups) and
        // owns accumulator S[t]; thread i of every group owns candidate i of the tile.  With four warps per scheduler the
        // exponentials of one group cover the tensor-memory loads, barrier round trips and Q.K^T latency of the others
        // (two groups left the special-function pipe 40 % idle).
        const int group = warp >> 2;
        const int key_in_tile = (warp & 3) * 32 + lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const float scale2 = kLog2e * rsqrtf((float)kD);
        const uint64_t scale2x2 = pack_f32x2(scale2, scale2);
        const int j = kt < n_cache_tiles ? key_row0 + key_in_tile : p.m + key_row0 + key_in_tile;   // candidate index
        const int n_src = from_cache ? p.m : p.L;
        const bool key_ok = key_row0 + key_in_tile < n_src;
        // first scoring row that may see this candidate
        int r_first = 0;
        if (p.causal && !from_cache) r_first = max(0, key_row0 + key_in_tile - p.t0);
        float acc = 0.f;
        bool ok = true;
        // The log-sum-exp values of iteration `it2` (thread i brings row r0 + i) go to buffer it2 & 7; a group reads
        // only what it published itself.  The global load is issued one iteration of the group before its value is
        // stored to shared memory, so its latency hides behind the exponentials in between.  A thread in iteration
        // `it` publishes the group's next iteration into the buffer the group last read one iteration ago; it has
        // seen the MMA of `it`, which needed s_free of that earlier iteration from all four warps of the group, so
        // everybody has finished reading that buffer.
        auto fetch_lse = [&](int it2) -> float {
            const int h2 = g * G + it2 / rb_per_head;
            const int rr = (rb0 + it2 % rb_per_head) * kTile + key_in_tile;
            float lse = INFINITY;
            if (rr < p.rows) {
                if (p.splits > 1) {                              // merge the key splits of pass 1
                    float2 ml[kMaxLseSplits];
#pragma unroll
                    for (int sp = 0; sp < kMaxLseSplits; ++sp)
                        ml[sp] = sp < p.splits ? __ldg(&p.part[((size_t)sp * p.q_heads + h2) * p.lse_stride + rr])
                                               : make_float2(-INFINITY, 0.f);
                    float M = -INFINITY, l = 0.f;
#pragma unroll
                    for (int sp = 0; sp < kMaxLseSplits; ++sp) M = fmaxf(M, ml[sp].x);
#pragma unroll
                    for (int sp = 0; sp < kMaxLseSplits; ++sp) l += ml[sp].x == -INFINITY ? 0.f : ml[sp].y * ex2(ml[sp].x - M);
                    lse = M + log2f(l);
                } else {
                    lse = __ldg(p.lse_in + (size_t)h2 * p.lse_stride + rr);
                }
            }
            return lse;
        };
        auto publish_lse = [&](int it2, float lse) {
            bars->lse[it2 & 7][key_in_tile] = -lse;              // negated: the exponent is one fused multiply-add
            mbar_arrive_warp(smem_u32(&bars->lse_full[it2 & 7]));
        };
        float lse_next = INFINITY;
        if (nb > group) publish_lse(group, fetch_lse(group));
        if (nb > group + kColGroups) lse_next = fetch_lse(group + kColGroups);
        for (int it = group; it < nb; it += kColGroups) {
            const int b = it & 3;
            const int rb = rb0 + it % rb_per_head;
            const int r0 = rb * kTile;
            const int ncols = min(kTile, p.rows - r0);
            const int lb = it & 7;
            ok = mbar_wait_warp(smem_u32(&bars->s_full[b]), (it >> 2) & 1, p.status);
            if (!ok) break;
            if (warp == 0) CITRUS_TR(160 + 3 * (it & 7));
            if (it + kColGroups < nb) publish_lse(it + kColGroups, lse_next);      // loaded one iteration ago
            if (it + 2 * kColGroups < nb) lse_next = fetch_lse(it + 2 * kColGroups);   // lands during this iteration's exponentials
            ok = mbar_wait_warp(smem_u32(&bars->lse_full[lb]), (it >> 3) & 1, p.status);
            if (!ok) break;
            if (warp == 0) CITRUS_TR(161 + 3 * (it & 7));
            tc_fence_after();
            const float4* nlse4 = reinterpret_cast<const float4*>(bars->lse[lb]);   // -lse (rows past the block end: -inf)
            const int c_lo = max(0, r_first - r0);                 // first column (scoring row) this candidate is visible to
            const int n_pieces = (ncols + 31) >> 5;                // the MMA wrote round_up(ncols, 32) columns
            float part[4] = {0.f, 0.f, 0.f, 0.f};
            uint64_t part2[2] = {0ull, 0ull};
#pragma unroll 1
            for (int c = 0; c < n_pieces; ++c) {
                const int lo = c_lo - c * 32;                      // columns below lo do not see this candidate
                if (__all_sync(0xffffffffu, lo >= 32)) continue;   // a piece that no candidate of the warp sees
                uint32_t v[32];
                tmem_ld32(tmS(b) + lane_base + c * 32, v);
                tmem_wait_ld();
                if (__all_sync(0xffffffffu, lo <= 0)) {
                    // every candidate of the warp sees the whole piece (always so away from the causal diagonal):
                    // packed arithmetic, no predicates
#pragma unroll
                    for (int q = 0; q < 32; q += 4) {
                        const float4 l = nlse4[c * 8 + (q >> 2)];
                        float e0, e1, e2, e3;
                        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(v[q + 0]), __uint_as_float(v[q + 1])), scale2x2, pack_f32x2(l.x, l.y)), e0, e1);
                        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(v[q + 2]), __uint_as_float(v[q + 3])), scale2x2, pack_f32x2(l.z, l.w)), e2, e3);
                        part2[0] = add_f32x2(part2[0], pack_f32x2(ex2(e0), ex2(e1)));
                        part2[1] = add_f32x2(part2[1], pack_f32x2(ex2(e2), ex2(e3)));
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < 32; q += 4) {
                        const float4 l = nlse4[c * 8 + (q >> 2)];
                        float e0 = ex2(fmaf(__uint_as_float(v[q + 0]), scale2, l.x));
                        float e1 = ex2(fmaf(__uint_as_float(v[q + 1]), scale2, l.y));
                        float e2 = ex2(fmaf(__uint_as_float(v[q + 2]), scale2, l.z));
                        float e3 = ex2(fmaf(__uint_as_float(v[q + 3]), scale2, l.w));
                        part[0] += q + 0 >= lo ? e0 : 0.f;
                        part[1] += q + 1 >= lo ? e1 : 0.f;
                        part[2] += q + 2 >= lo ? e2 : 0.f;
                        part[3] += q + 3 >= lo ? e3 : 0.f;
                    }
                }
            }
            {
                float a0, a1, b0, b1;
                unpack_f32x2(part2[0], a0, a1); unpack_f32x2(part2[1], b0, b1);
                part[0] += a0; part[1] += a1; part[2] += b0; part[3] += b1;
            }
            tc_fence_before();
            mbar_arrive_warp(smem_u32(&bars->s_free[b]));
            acc += (part[0] + part[1]) + (part[2] + part[3]);
            if (warp == 0) CITRUS_TR(162 + 3 * (it & 7));
        }
        // all column-sum warps arrive here, also after a wait that gave up; the partial sums are added in group order
        if (group > 0) bars->acc_other[group - 1][key_in_tile] = acc;
        asm volatile("bar.sync 1, %0;" ::"n"(kColGroups * 128) : "memory");
        if (group == 0 && ok && key_ok) {
#pragma unroll
            for (int t = 0; t < kColGroups - 1; ++t) acc += bars->acc_other[t][key_in_tile];
            p.scores[(size_t)g * p.score_stride + j] = acc;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) CITRUS_TR(190);
#ifdef CITRUS_TRACE
    if (threadIdx.x == 0) atomicMax(&g_citrus_trace[247], global_ns());
#endif
    if (warp == kMmaWarp) { __syncwarp(); tmem_dealloc(tmem, kColTmemCols); }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn g_encode = nullptr;
std::mutex g_init_mu;
DeviceOnce g_device_ready;

// Token-major tensor [rows, heads, 128] bf16: coordinates (d, head, row), box 64 x 1 x 128.
bool map_token_major(CUtensorMap* map, const void* ptr, int rows, int heads, int box_rows = kTile) {
    cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)heads, (cuuint64_t)rows};
    cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)heads * kD * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
    cuuint32_t es[3] = {1, 1, 1};
    return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// Cache tensor [heads, cap, 128] bf16: coordinates (d, row, head), box 64 x 128 x 1.
bool map_cache(CUtensorMap* map, const void* ptr, int cap, int heads) {
    cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)cap, (cuuint64_t)heads};
    cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)cap * kD * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)kTile, 1};
    cuuint32_t es[3] = {1, 1, 1};
    return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Launch with programmatic stream serialisation: the kernel may begin (prologue only) before its predecessor
// in the stream has finished; it reads the predecessor's results after griddepcontrol.wait.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, int threads, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = dim3(threads); cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    before_launch(s);
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

}  // namespace

// A wait on an mbarrier that nothing ever arms: the bounded wait runs out after limit_ns, raises the status word and
// the kernel returns normally.  Launched only by citrus_debug_expire_wait (the test of the time-out path).
__global__ void expire_wait_kernel(int* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    mbar_wait_warp(smem_u32(&bar), 0, status, limit_ns);
}

cudaError_t tc_expire_wait(int* status, unsigned long long limit_ns, cudaStream_t s) {
    expire_wait_kernel<<<1, 32, 0, s>>>(status, limit_ns);
    return cudaGetLastError();
}

cudaError_t tc_init() {
    // The driver entry point is per process; the kernels' shared-memory limits are per device.
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lk(g_init_mu);
    if (g_encode == nullptr) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return e;
        if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return cudaErrorNotSupported;
        g_encode = reinterpret_cast<EncodeFn>(fn);
    }
    if (!g_device_ready.needs_setup(dev)) return cudaSuccess;
    e = cudaFuncSetAttribute(attn_lse_kernel<true, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemBytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_lse_kernel<false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemBytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_lse_kernel<true, kTcMaxBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemBytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_lse_kernel<false, kTcMaxBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemBytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(colsum_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kColSmemBytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(colsum_kernel<kTcMaxBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, kColSmemBytes);
    if (e != cudaSuccess) return e;
    g_device_ready.mark(dev);
    return cudaSuccess;
}

// Heads of one KV group whose scoring rows share a 128-row tile in pass 1 of a2-I (1 = one head per tile).
static int lse_pack(int n_rows, int q_heads, int kv_heads) {
    const int G = q_heads / kv_heads;
    if (n_rows > 64 || n_rows % 8 != 0 || kTile % n_rows != 0) return 1;
    int pack = kTile / n_rows;
    while (pack > 1 && (pack > G || G % pack != 0)) pack >>= 1;
    return pack < 1 ? 1 : pack;
}

int tc_lse_splits(int n_rows, int q_heads, int kv_heads, int m, int L, int n_attn_items) {
    // The log-sum-exp items share a launch with the attention items.  When those leave SMs idle (fewer items than
    // SMs), split the key range so that there is about one short item per idle SM; otherwise keep whole sweeps,
    // because every extra item pays a CTA prologue.
    const int kSMs = sm_count();
    const int tiles = (m + kTile - 1) / kTile + (L + kTile - 1) / kTile;
    const int base_items = ((n_rows + kTile - 1) / kTile) * q_heads / lse_pack(n_rows, q_heads, kv_heads);
    const int idle = n_attn_items < kSMs ? kSMs - n_attn_items : 0;
    // several waves of attention items: short log-sum-exp items (about four key tiles each) at the end of the
    // grid fill the ragged tail of the last wave instead of extending it
    int s = n_attn_items < kSMs ? idle / base_items : (tiles + 3) / 4;
    if (s > tiles) s = tiles;
    if (s > kMaxLseSplits) s = kMaxLseSplits;
    return s < 1 ? 1 : s;
}

// Largest pack that every sequence of the batch can use (they share one query map, whose box is pack_rows high).
static int batch_pack(const TcSeqStep* seq, int n, int q_heads, int kv_heads) {
    int rows = 0;
    for (int i = 0; i < n; ++i) {
        if (seq[i].nI <= 0) continue;
        if (rows == 0) rows = seq[i].nI;
        else if (rows != seq[i].nI) return 1;
    }
    return rows > 0 ? lse_pack(rows, q_heads, kv_heads) : 1;
}

template <int CAP>
static cudaError_t launch_attention(const TcTensors& t, const TcSeqStep* seq, int n, int lse_chunk_stride, int lse_instr_stride,
                                    int* status, cudaStream_t s) {
    bool has_attn = false, has_lse = false, need_lse = false;
    for (int i = 0; i < n; ++i) {
        has_attn |= seq[i].L > 0 && t.out != nullptr;
        has_lse |= seq[i].nI > 0;
        need_lse |= seq[i].lse_chunk != nullptr;
    }
    if (!has_attn && !has_lse) return cudaSuccess;
    const int ic = seq[0].ic;
    CUtensorMap mQ{}, mCK{}, mCV{}, mSK{}, mSV{}, mO{}, mQI{}, mCKI{};
    if (!map_token_major(&mSK, t.K, t.kv_rows, t.kv_heads)) return cudaErrorInvalidValue;
    if (has_attn) {
        if (!map_token_major(&mQ, t.Q, t.q_rows, t.q_heads) || !map_token_major(&mO, t.out, t.q_rows, t.q_heads) ||
            !map_token_major(&mSV, t.V, t.kv_rows, t.kv_heads) ||
            !map_cache(&mCK, t.cacheK[0], t.cap[0], t.cache_heads[0]) || !map_cache(&mCV, t.cacheV[0], t.cap[0], t.cache_heads[0]))
            return cudaErrorInvalidValue;
    }
    const int pack = has_lse ? batch_pack(seq, n, t.q_heads, t.kv_heads) : 1;
    int pack_rows = 0;
    if (has_lse) {
        for (int i = 0; i < n; ++i) if (seq[i].nI > 0) pack_rows = seq[i].nI;
        if (!map_token_major(&mQI, t.Qi, t.qi_rows, t.q_heads, pack > 1 ? pack_rows : kTile) ||
            !map_cache(&mCKI, t.cacheK[ic], t.cap[ic], t.cache_heads[ic]))
            return cudaErrorInvalidValue;
    }
    if (!has_attn) { mQ = mQI; mO = mQI; mCK = mCKI; mCV = mCKI; mSV = mSK; }
    if (!has_lse) { mQI = mQ; mCKI = mCK; }
    AttnBatch<CAP> bt{};
    bt.n = n;
    int items = 0;
    for (int i = 0; i < n; ++i) {
        const TcSeqStep& q = seq[i];
        TcParams& pa = bt.pa[i];
        pa.rows = has_attn ? q.L : 0; pa.row0 = q.q_row0; pa.krow0 = q.kv_row0; pa.chead = q.chead[0];
        pa.q_heads = t.q_heads; pa.kv_heads = t.kv_heads; pa.m = q.m[0]; pa.L = q.L; pa.causal = 1; pa.t0 = 0;
        pa.out = t.out; pa.lse2 = q.lse_chunk; pa.lse_stride = lse_chunk_stride; pa.splits = 1; pa.pack = 1; pa.pack_rows = 0;
        pa.status = status; pa.dep_first = q.produced;
        items += ((pa.rows + kTile - 1) / kTile) * t.q_heads;
        bt.seg_end[i] = items;
    }
    for (int i = 0; i < n; ++i) {
        const TcSeqStep& q = seq[i];
        TcParams& pl = bt.pl[i];
        pl.rows = q.nI; pl.row0 = q.qi_row0; pl.krow0 = q.kv_row0; pl.chead = q.chead[ic];
        pl.q_heads = t.q_heads; pl.kv_heads = t.kv_heads; pl.m = q.m[ic]; pl.L = q.L; pl.causal = 0; pl.t0 = 0;
        pl.lse2 = q.lse_instr; pl.part = reinterpret_cast<float2*>(q.part); pl.lse_stride = lse_instr_stride;
        pl.splits = q.splits < 1 ? 1 : q.splits; pl.pack = pack; pl.pack_rows = q.nI;
        pl.status = status; pl.dep_first = q.produced;
        items += ((q.nI + kTile - 1) / kTile) * (t.q_heads / pack) * pl.splits;
        bt.seg_end[n + i] = items;
    }
    if (items == 0) return cudaSuccess;
    dim3 grid(items);
    if (need_lse)
        return launch_pdl(attn_lse_kernel<true, CAP>, grid, kAttnThreads, kAttnSmemBytes, s, mQ, mCK, mCV, mSK, mSV, mO, mQI, mCKI, bt);
    return launch_pdl(attn_lse_kernel<false, CAP>, grid, kAttnThreads, kAttnSmemBytes, s, mQ, mCK, mCV, mSK, mSV, mO, mQI, mCKI, bt);
}

cudaError_t tc_attention_lse(const TcTensors& t, const TcSeqStep* seq, int n, int lse_chunk_stride, int lse_instr_stride,
                             int* status, cudaStream_t s) {
    if (n < 1 || n > kTcMaxBatch) return cudaErrorInvalidValue;
    if (n == 1) return launch_attention<1>(t, seq, n, lse_chunk_stride, lse_instr_stride, status, s);
    return launch_attention<kTcMaxBatch>(t, seq, n, lse_chunk_stride, lse_instr_stride, status, s);
}

// The column sums of a step in one launch: with do_lm the chunk's last w rows score cache 0's candidates with a1's
// probabilities (causal); with do_instr the instruction rows score the instruction-side cache's candidates.
template <int CAP>
static cudaError_t launch_colsum(const TcTensors& t, const TcSeqStep* seq, int n, bool do_lm, bool do_instr,
                                 int lse_chunk_stride, int lse_instr_stride, int* status, cudaStream_t s) {
    const int ic = seq[0].ic;
    CUtensorMap mQ0{}, mCK0{}, mQ1{}, mCK1{}, mSK{};
    if (!map_token_major(&mSK, t.K, t.kv_rows, t.kv_heads)) return cudaErrorInvalidValue;
    if (do_lm && (!map_token_major(&mQ0, t.Q, t.q_rows, t.q_heads) || !map_cache(&mCK0, t.cacheK[0], t.cap[0], t.cache_heads[0])))
        return cudaErrorInvalidValue;
    if (do_instr && (!map_token_major(&mQ1, t.Qi, t.qi_rows, t.q_heads) || !map_cache(&mCK1, t.cacheK[ic], t.cap[ic], t.cache_heads[ic])))
        return cudaErrorInvalidValue;
    if (!do_lm) { mQ0 = mQ1; mCK0 = mCK1; }
    if (!do_instr) { mQ1 = mQ0; mCK1 = mCK0; }
    ColBatch<CAP> bt{};
    int tiles = 0, e = 0;
    for (int which = 0; which < 2; ++which) {
        if (which == 0 ? !do_lm : !do_instr) continue;
        const int ci = which == 0 ? 0 : ic;
        for (int i = 0; i < n; ++i) {
            const TcSeqStep& q = seq[i];
            const int rows = which == 0 ? q.w : q.nI;
            if (rows <= 0) continue;
            TcParams& p = bt.p[e];
            p.rows = rows; p.krow0 = q.kv_row0; p.chead = q.chead[ci];
            p.q_heads = t.q_heads; p.kv_heads = t.kv_heads; p.m = q.m[ci]; p.L = q.L; p.status = status; p.dep_first = q.produced;
            if (which == 0) {
                p.row0 = q.q_row0 + (q.L - q.w); p.causal = 1; p.t0 = q.L - q.w;
                p.lse_in = q.lse_chunk + (q.L - q.w); p.part = nullptr; p.splits = 1; p.lse_stride = lse_chunk_stride;
            } else {
                p.row0 = q.qi_row0; p.causal = 0; p.t0 = 0;
                p.splits = q.splits < 1 ? 1 : q.splits;
                p.lse_in = q.lse_instr; p.part = reinterpret_cast<float2*>(q.part); p.lse_stride = lse_instr_stride;
            }
            p.scores = q.scores[ci]; p.score_stride = q.score_stride;
            tiles += (p.m + kTile - 1) / kTile + (p.L + kTile - 1) / kTile;
            bt.tile_end[e++] = tiles;
        }
        if (which == 0) bt.n_first = e;
    }
    bt.n_entries = e;
    if (tiles == 0) return cudaSuccess;
    dim3 grid(t.kv_heads, tiles);
    return launch_pdl(colsum_kernel<CAP>, grid, kColThreads, kColSmemBytes, s, mQ0, mCK0, mQ1, mCK1, mSK, bt);
}

cudaError_t tc_colsum(const TcTensors& t, const TcSeqStep* seq, int n, bool do_lm, bool do_instr, int lse_chunk_stride,
                      int lse_instr_stride, int* status, cudaStream_t s) {
    if (n < 1 || n > kTcMaxBatch) return cudaErrorInvalidValue;
    if (!do_lm && !do_instr) return cudaSuccess;
    if (n == 1) return launch_colsum<1>(t, seq, n, do_lm, do_instr, lse_chunk_stride, lse_instr_stride, status, s);
    return launch_colsum<kTcMaxBatch>(t, seq, n, do_lm, do_instr, lse_chunk_stride, lse_instr_stride, status, s);
}

}  // namespace citrus
