// Step a3 (exact top-k with lower-index tie-break, ascending output) and step a4
// (ordered gather of K, V and positions into the other ping-pong buffer).
#include "citrus_internal.h"

#include <mutex>

CITRUS_TRACE_EXPORT(_sc)
#ifdef CITRUS_TRACE
static __device__ __forceinline__ unsigned long long trace_ns() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
#define CITRUS_SPAN_MIN(i) do { if (threadIdx.x == 0) atomicMax(&g_citrus_trace[(i)], ~trace_ns()); } while (0)
#define CITRUS_SPAN_MAX(i) do { if (threadIdx.x == 0) atomicMax(&g_citrus_trace[(i)], trace_ns()); } while (0)
#else
#define CITRUS_SPAN_MIN(i) do { } while (0)
#define CITRUS_SPAN_MAX(i) do { } while (0)
#endif

namespace citrus {
namespace {

constexpr int kSelThreads = 1024;
// Jobs of one launch: one per cache of every sequence.  Two capacities, so that a single sequence's launch does not
// carry the parameter block of a whole batch.
constexpr int kJobsSingle = 2;
constexpr int kJobsBatch = 2 * kTcMaxBatch;

template <int CAP> struct SelectArgs { SelectJob job[CAP]; };
template <int CAP> struct CompactArgs { CompactJob job[CAP]; RopeTable rope; int elt; };

// A 16-byte piece of a key row embedded at position `pos`: `mine` holds elements [d0, d0 + E) of one half of the head
// dimension, `other` the same elements of the other half (E = 8 bf16 or 4 fp32); lower: `mine` is the first half.
// first' = first cos - second sin, second' = second cos + first sin, angle = pos * theta[d].
__device__ __forceinline__ uint4 rope_piece(uint4 mine, uint4 other, int pos, int d0, bool lower, const RopeTable& t, int elt) {
    const uint32_t* a = reinterpret_cast<const uint32_t*>(&mine);
    const uint32_t* b = reinterpret_cast<const uint32_t*>(&other);
    uint4 out;
    uint32_t* o = reinterpret_cast<uint32_t*>(&out);
    // fp64 throughout, rounded once at the end: the embedded value is the correctly rounded rotation of the stored
    // one (up to the last bit of sin / cos), whatever the position
    auto turn = [&](float x, float y, int d) {
        double sn, cs;
        sincos((double)pos * t.theta[d], &sn, &cs);
        return (float)(lower ? (double)x * cs - (double)y * sn : (double)x * cs + (double)y * sn);
    };
    if (elt == 2) {
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float x0 = __uint_as_float(a[w] << 16), x1 = __uint_as_float(a[w] & 0xffff0000u);
            const float y0 = __uint_as_float(b[w] << 16), y1 = __uint_as_float(b[w] & 0xffff0000u);
            __nv_bfloat162 r = __floats2bfloat162_rn(turn(x0, y0, d0 + 2 * w), turn(x1, y1, d0 + 2 * w + 1));
            o[w] = *reinterpret_cast<uint32_t*>(&r);
        }
    } else {
#pragma unroll
        for (int w = 0; w < 4; ++w) o[w] = __float_as_uint(turn(__uint_as_float(a[w]), __uint_as_float(b[w]), d0 + w));
    }
    return out;
}

// Order-preserving map from fp32 to uint32 (larger float <=> larger key).
__device__ __forceinline__ uint32_t order_key(float f) {
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// The score vector of one (cache, KV head) - or of the whole layer when layerwise - is staged once in shared memory as
// order keys; a most-significant-digit radix select (8-bit digits; as soon as at most 32 candidates share the prefix
// one warp ranks them directly) finds the k-th largest key T and how many candidates equal to T are kept (the
// lowest-index ones).  Called by all kSelThreads threads of a CTA with n > k.
__device__ __forceinline__ void select_threshold(const SelectJob& job, const int g, int kv_heads, int layerwise,
                                                 uint32_t* keys /* shared, [n] */, uint32_t& T_out, uint32_t& take_eq_out) {
    const int n = job.n, k = job.k;
    __shared__ uint32_t hist[256];
    __shared__ uint32_t s_prefix, s_remaining, s_bin_count, s_n_short;
    __shared__ uint32_t s_short[32];
    __shared__ uint32_t s_wmin[32], s_wmax[32];
    const int tid = threadIdx.x;
    uint32_t kmin = 0xffffffffu, kmax = 0u;        // over this thread's keys; the forced ones (all-ones) stay out of the maximum
    for (int j = tid; j < n; j += kSelThreads) {
        // one head's score of candidate j; with the accumulative policy the importance its cache row carries is
        // added and the sum written back (it is what the compaction hands on, and what the step view shows)
        auto head_score = [&](int gg) {
            float* p = job.scores + (size_t)gg * job.score_stride + j;
            float x = *p;
            if (job.carried != nullptr) {
                if (j < job.m) x += job.carried[(size_t)gg * job.pos_stride + j];
                *p = x;
            }
            return x;
        };
        float v;
        if (layerwise) {
            v = 0.f;
            for (int gg = 0; gg < kv_heads; ++gg) v += head_score(gg);
        } else {
            v = head_score(g);
        }
        uint32_t key = order_key(v);
        if (job.start > 0) {
            // original position of candidate j (layer-wise mode: all heads hold the same positions)
            const int pos = j < job.m ? job.pos[(size_t)(layerwise ? 0 : g) * job.pos_stride + j] : job.chunk_pos0 + (j - job.m);
            if (pos < job.start) key = 0xffffffffu;           // beats every score; ties among them keep index order
        }
        if (j >= job.forced_from) key = 0xffffffffu;          // the chunk's own states all enter (deferred eviction)
        keys[j] = key;
        kmin = min(kmin, key);
        if (key != 0xffffffffu) kmax = max(kmax, key);
    }
    // The scores of one head share their sign and most of their exponent bits, so the leading digits of the raw keys
    // tell nothing.  The keys are rebased to d = key - min (a forced key: range + 1) and shifted up so that the range
    // fills whole 8-bit digits: the order is unchanged, the first digit already spreads the candidates over up to 256
    // bins, and the digits below the range's width need no pass at all.
    kmin = __reduce_min_sync(0xffffffffu, kmin); kmax = __reduce_max_sync(0xffffffffu, kmax);
    if ((tid & 31) == 0) { s_wmin[tid >> 5] = kmin; s_wmax[tid >> 5] = kmax; }
    if (tid == 0) { s_prefix = 0u; s_remaining = (uint32_t)k; s_bin_count = (uint32_t)n; s_n_short = 0u; }
    __syncthreads();
    kmin = __reduce_min_sync(0xffffffffu, s_wmin[tid & 31]); kmax = __reduce_max_sync(0xffffffffu, s_wmax[tid & 31]);
    const uint32_t range = kmax > kmin ? kmax - kmin : 0u;            // of the keys that are not forced
    const uint32_t top = range == 0xffffffffu ? range : range + 1u;   // value given to the forced keys
    const int nbits = 32 - __clz(top | 1u);
    const int width = (nbits + 7) & ~7;                               // digits cover `width` bits
    const int up = width - nbits;
    for (int j = tid; j < n; j += kSelThreads) {
        const uint32_t key = keys[j];
        keys[j] = (key == 0xffffffffu ? top : key - kmin) << up;
    }
    __syncthreads();
    CITRUS_TR(10);

    uint32_t mask = 0u;
    for (int shift = width - 8; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        for (int j0 = 0; j0 < n; j0 += kSelThreads) {            // warp-uniform trip count
            const int j = j0 + tid;
            const uint32_t key = j < n ? keys[j] : 0u;
            const bool act = j < n && (key & mask) == prefix;
            const uint32_t bin = (key >> shift) & 255u;
            // The leading digit (sign and exponent) is the same for nearly every score of a head, later digits are
            // spread out: one atomic for the warp when all its lanes agree, otherwise one per lane.
            int all_same;
            __match_all_sync(0xffffffffu, act ? bin : 256u, &all_same);
            if (all_same) {
                if (act && (tid & 31) == 0) atomicAdd(&hist[bin], 32u);
            } else if (act) {
                atomicAdd(&hist[bin], 1u);
            }
        }
        __syncthreads();
        if (tid < 32) {
            // warp 0 walks the 256 bins from the top: lane l owns bins [8l, 8l+8)
            const uint32_t remaining = s_remaining;
            uint32_t mine = 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) mine += hist[tid * 8 + i];
            uint32_t suffix = mine;                              // inclusive sum over lanes >= tid
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                uint32_t v = __shfl_down_sync(0xffffffffu, suffix, o);
                if (tid + o < 32) suffix += v;
            }
            const uint32_t above = suffix - mine;                // candidates in bins of higher lanes
            if (above < remaining && remaining <= suffix) {      // exactly one lane holds the k-th largest
                uint32_t cum = above;
                int b = tid * 8 + 7;
                for (; b > tid * 8; --b) {
                    if (cum + hist[b] >= remaining) break;
                    cum += hist[b];
                }
                s_remaining = remaining - cum;                   // still to take inside bin b
                s_prefix = prefix | ((uint32_t)b << shift);
                s_bin_count = hist[b];
            }
        }
        mask |= 255u << shift;
        __syncthreads();
        CITRUS_TR(11 + (width - 8 - shift) / 8);
        // Short cut: at most 32 candidates still share the prefix.  One warp ranks them directly instead of
        // walking the remaining digits.
        if (shift > 0 && s_bin_count <= 32u) {
            const uint32_t prefix2 = s_prefix;
            for (int j = tid; j < n; j += kSelThreads) {
                const uint32_t key = keys[j];
                if ((key & mask) == prefix2) s_short[atomicAdd(&s_n_short, 1u)] = key;
            }
            __syncthreads();
            if (tid < 32) {
                const uint32_t c = s_n_short, r = s_remaining;      // r-th largest of the c listed keys (1 <= r <= c)
                const uint32_t mine = tid < (int)c ? s_short[tid] : 0u;
                uint32_t n_gt = 0u, n_ge = 0u;
                for (uint32_t i = 0; i < c; ++i) {
                    const uint32_t other = __shfl_sync(0xffffffffu, mine, (int)i);
                    n_gt += other > mine; n_ge += other >= mine;
                }
                if (tid < (int)c && n_gt < r && r <= n_ge) {        // every lane holding the r-th largest value writes the same
                    s_prefix = mine;
                    s_remaining = r - n_gt;
                }
            }
            __syncthreads();
            break;
        }
    }
    T_out = s_prefix;                              // k-th largest key (in the rebased form that `keys` now holds)
    take_eq_out = s_remaining;                     // candidates equal to T that are kept (lowest indices)
}

// One CTA per (cache, KV head) -- or per cache when layerwise: threshold, then a flagged block scan in index order
// emits the kept indices ascending, taking the lowest-index candidates among those equal to T.
__device__ __forceinline__ void select_body(const SelectJob& job, const int g, int kv_heads, int layerwise,
                                            uint32_t* keys /* shared, [n] */) {
    const int n = job.n, k = job.k, ks = job.idx_stride;
    __shared__ uint32_t warp_gt[32], warp_eq[32];

    const int tid = threadIdx.x;
    const int heads_out = layerwise ? kv_heads : 1;
    int* idx0 = job.idx + (size_t)g * ks;

    if (n <= k) {                                  // nothing to evict: identity
        for (int j = tid; j < n; j += kSelThreads) {
            for (int ho = 0; ho < heads_out; ++ho) idx0[(size_t)ho * ks + j] = j;
            if (job.carried != nullptr && j < job.m) {
                // accumulative policy: the carried importance still has to be added to what is handed on
                for (int ho = 0; ho < heads_out; ++ho) {
                    const int gg = layerwise ? ho : g;
                    job.scores[(size_t)gg * job.score_stride + j] += job.carried[(size_t)gg * job.pos_stride + j];
                }
            }
        }
        return;
    }
    uint32_t T, take_eq;
    select_threshold(job, g, kv_heads, layerwise, keys, T, take_eq);

    // ordered emission: thread t owns the contiguous index range [t*per, (t+1)*per)
    const int per = (n + kSelThreads - 1) / kSelThreads;
    const int lo = min(n, tid * per), hi = min(n, lo + per);
    uint32_t gt = 0u, eq = 0u;
    for (int j = lo; j < hi; ++j) { uint32_t key = keys[j]; gt += key > T; eq += key == T; }
    // block exclusive scan of (gt, eq)
    const int lane = tid & 31, warp = tid >> 5;
    uint32_t sgt = gt, seq = eq;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t a = __shfl_up_sync(0xffffffffu, sgt, o), b = __shfl_up_sync(0xffffffffu, seq, o);
        if (lane >= o) { sgt += a; seq += b; }
    }
    if (lane == 31) { warp_gt[warp] = sgt; warp_eq[warp] = seq; }
    __syncthreads();
    if (warp == 0) {
        uint32_t a = warp_gt[lane], b = warp_eq[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t x = __shfl_up_sync(0xffffffffu, a, o), y = __shfl_up_sync(0xffffffffu, b, o);
            if (lane >= o) { a += x; b += y; }
        }
        warp_gt[lane] = a; warp_eq[lane] = b;      // inclusive over warps
    }
    __syncthreads();
    uint32_t gt_before = sgt - gt + (warp ? warp_gt[warp - 1] : 0u);
    uint32_t eq_before = seq - eq + (warp ? warp_eq[warp - 1] : 0u);
    for (int j = lo; j < hi; ++j) {
        uint32_t key = keys[j];
        bool keep = key > T || (key == T && eq_before < take_eq);
        if (keep) {
            uint32_t p = gt_before + min(eq_before, take_eq);
            for (int ho = 0; ho < heads_out; ++ho) idx0[(size_t)ho * ks + p] = j;
        }
        gt_before += key > T;
        eq_before += key == T;
    }
    CITRUS_TR(15);
}

template <int CAP>
__global__ void __launch_bounds__(kSelThreads)
select_topk_kernel(const __grid_constant__ SelectArgs<CAP> args, int kv_heads, int layerwise) {
    extern __shared__ uint32_t keys[];            // [largest n of the jobs]
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the scores are final after this
    select_body(args.job[blockIdx.y], blockIdx.x, kv_heads, layerwise, keys);
}

// Rows [r_begin, r_end) of one (cache, head) are copied with 128-bit accesses, row_bytes/16 lanes per row.
template <bool SHIFT>
__device__ __forceinline__ void compact_rows_t(const CompactJob& job, const int g, int kv_heads,
                                             int row_vecs, int r_begin, int r_end, const int* idx,
                                             const RopeTable& rope, int elt) {
    const int cap = job.cap;
    const uint4* __restrict__ chunkK = reinterpret_cast<const uint4*>(job.chunkK);
    const uint4* __restrict__ chunkV = reinterpret_cast<const uint4*>(job.chunkV);
    const int chunk_pos0 = job.chunk_pos0;
    constexpr bool shift = SHIFT;                     // position shift: gather un-rotated keys, embed by the new slot
    // idx[r] = candidate kept in row r of this head (global list, or the CTA's slice in shared memory)
    const int rows_per_pass = blockDim.x / row_vecs;
    const int sub = threadIdx.x / row_vecs, v = threadIdx.x % row_vecs;
    const uint4* srcK = reinterpret_cast<const uint4*>(shift ? job.srcKraw : job.srcK);
    const uint4* srcV = reinterpret_cast<const uint4*>(job.srcV);
    uint4* dstK = reinterpret_cast<uint4*>(shift ? job.dstKraw : job.dstK);
    uint4* dstKrot = reinterpret_cast<uint4*>(job.dstK);
    uint4* dstV = reinterpret_cast<uint4*>(job.dstV);
    // four rows per thread in flight: first every index, then every load, then the stores
    constexpr int kInFlight = 4;
    // The trip count is the same for every lane of a warp (the position-shift variant exchanges registers with a
    // full-mask shuffle): the loop runs on the row of the warp's first lane, a lane whose own row lies past the end
    // carries j = -1 and only skips its loads and stores.
    const int sub_first = (int)(threadIdx.x & ~31u) / row_vecs;
    for (int rb_w = r_begin + sub_first; rb_w < r_end; rb_w += kInFlight * rows_per_pass) {
        const int rb = rb_w + (sub - sub_first);
        int j[kInFlight];
        uint4 a[kInFlight], b[kInFlight];
        if (SHIFT) {
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) a[u] = make_uint4(0u, 0u, 0u, 0u);   // rows past the end still take part in the exchange
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const int r = rb + u * rows_per_pass;
            j[u] = r < r_end ? idx[r] : -1;
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            if (j[u] < 0) continue;
            const uint4 *pk, *pv;
            if (j[u] < job.m) {
                size_t off = ((size_t)g * cap + j[u]) * row_vecs + v;
                pk = srcK + off; pv = srcV + off;
            } else {
                size_t off = ((size_t)(j[u] - job.m) * kv_heads + g) * row_vecs + v;
                pk = chunkK + off; pv = chunkV + off;
            }
            a[u] = __ldg(pk); b[u] = __ldg(pv);
        }
        if (shift) {
            // the other half of the head dimension sits half a row away, in a lane of the same warp; every lane
            // takes part in the exchange, rows past the end only skip the store
            const int half_vecs = row_vecs >> 1, per_vec = 16 / elt;
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) {
                uint4 other;
                other.x = __shfl_xor_sync(0xffffffffu, a[u].x, half_vecs); other.y = __shfl_xor_sync(0xffffffffu, a[u].y, half_vecs);
                other.z = __shfl_xor_sync(0xffffffffu, a[u].z, half_vecs); other.w = __shfl_xor_sync(0xffffffffu, a[u].w, half_vecs);
                if (j[u] < 0) continue;
                const int r = rb + u * rows_per_pass;
                dstKrot[((size_t)g * cap + r) * row_vecs + v] =
                    rope_piece(a[u], other, r, (v % half_vecs) * per_vec, v < half_vecs, rope, elt);
            }
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            if (j[u] < 0) continue;
            const int r = rb + u * rows_per_pass;
            size_t doff = ((size_t)g * cap + r) * row_vecs + v;
            dstK[doff] = a[u];
            dstV[doff] = b[u];
            if (v == 0) {
                job.dstPos[(size_t)g * cap + r] = j[u] < job.m ? job.srcPos[(size_t)g * cap + j[u]] : chunk_pos0 + (j[u] - job.m);
                if (job.dstCarried != nullptr) job.dstCarried[(size_t)g * cap + r] = job.totals[(size_t)g * job.score_stride + j[u]];
            }
        }
    }
}

// The position-shift variant is a separate instantiation (and a separate kernel) so that the plain gather stays lean.
// grid: (row tiles, KV heads, caches)
constexpr int kCompactThreads = 256;
constexpr int kCompactRowsPerCta = 64;

template <bool SHIFT, int CAP>
__global__ void __launch_bounds__(kCompactThreads)
compact_kv_kernel(const __grid_constant__ CompactArgs<CAP> args, int kv_heads, int row_vecs) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the index lists are final after this
    const CompactJob& job = args.job[blockIdx.z];
    const int r0 = blockIdx.x * kCompactRowsPerCta;
    if (r0 >= job.kept) return;                              // the grid is sized for the job that keeps most
    compact_rows_t<SHIFT>(job, blockIdx.y, kv_heads, row_vecs,
                          r0, min(job.kept, r0 + kCompactRowsPerCta), job.idx + (size_t)blockIdx.y * job.cap, args.rope, args.elt);
}

// a3 + a4 in one launch, for steps that are small enough to be latency-bound: kFusedParts CTAs per (cache, KV head),
// each responsible for a contiguous share of the CANDIDATES.  A CTA
//   1. starts bulk copies of its share's K and V rows into shared memory (the chunk's rows at once when the caller's
//      inputs are declared complete, the old cache's rows after griddepcontrol.wait), so that the whole load latency
//      hides behind the selection;
//   2. runs the selection on the full score vector (every CTA of the head repeats this small computation instead of
//      waiting for one that does it: no cluster, no hand-over of index lists);
//   3. counts the kept candidates that precede its share, scans its own share (one candidate per thread) and writes
//      its kept rows - consecutive kept candidates are consecutive rows of the new cache - from shared memory.
// grid: (kFusedParts, KV heads, jobs)
constexpr int kFusedParts = 8;
constexpr int kFusedMaxShare = kSelThreads;      // one candidate per thread in the local scan

__device__ __forceinline__ uint32_t sc_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

template <int CAP>
__global__ void __launch_bounds__(kSelThreads)
select_gather_kernel(const __grid_constant__ SelectArgs<CAP> sel, const __grid_constant__ CompactArgs<CAP> cmp,
                     int kv_heads, int n_max, int share_max, int row_bytes, int early_chunk_rows, int layerwise) {
    extern __shared__ __align__(128) uint8_t sg_smem[];
    __shared__ uint64_t rows_bar;
    __shared__ uint32_t w_gt[32], w_eq[32], w_keep[32];
    __shared__ int s_lkept[kFusedMaxShare];          // local candidate index of the CTA's r-th kept candidate
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const SelectJob& sjob = sel.job[blockIdx.z];
    const CompactJob& job = cmp.job[blockIdx.z];
    const int g = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = sjob.n, k = sjob.k, m = job.m, cap = job.cap;
    const int share = (n + kFusedParts - 1) / kFusedParts;
    const int c0 = min(n, (int)blockIdx.x * share), c1 = min(n, c0 + share);
    const int cnt = c1 - c0;
    uint32_t* keys = reinterpret_cast<uint32_t*>(sg_smem);                       // [n_max]
    uint8_t* rowK = sg_smem + (((size_t)n_max * 4 + 127) & ~(size_t)127);        // [share_max][row_bytes]
    uint8_t* rowV = rowK + (size_t)share_max * row_bytes;
    const uint32_t bar = sc_smem_u32(&rows_bar);
    // this CTA's candidates: [c0, cm) are rows of the old cache, [cm, c1) rows of the chunk
    const int cm = min(c1, max(c0, m));
    const uint8_t* srcK = reinterpret_cast<const uint8_t*>(job.srcK);
    const uint8_t* srcV = reinterpret_cast<const uint8_t*>(job.srcV);
    const uint8_t* chunkK = reinterpret_cast<const uint8_t*>(job.chunkK);
    const uint8_t* chunkV = reinterpret_cast<const uint8_t*>(job.chunkV);
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)(2 * cnt * row_bytes)) : "memory");
    }
    __syncthreads();
    auto copy_chunk_rows = [&]() {
        // one copy per row and tensor: chunk rows are kv_heads * row_bytes apart
        for (int j = cm + tid; j < c1; j += kSelThreads) {
            const size_t src = ((size_t)(j - m) * kv_heads + g) * row_bytes;
            bulk_g2s(sc_smem_u32(rowK + (size_t)(j - c0) * row_bytes), chunkK + src, (uint32_t)row_bytes, bar);
            bulk_g2s(sc_smem_u32(rowV + (size_t)(j - c0) * row_bytes), chunkV + src, (uint32_t)row_bytes, bar);
        }
    };
    CITRUS_TR(1);
    if (early_chunk_rows) copy_chunk_rows();
    CITRUS_TR(2);
    asm volatile("griddepcontrol.wait;" ::: "memory");       // scores, the old cache and its positions are final after this
    CITRUS_TR(3);
    if (!early_chunk_rows) copy_chunk_rows();
    if (tid == 0 && cm > c0) {
        // the old cache's rows of the share are contiguous: one copy per tensor (pieces of at most 64 KB)
        const size_t src = ((size_t)g * cap + c0) * row_bytes;
        const uint32_t total = (uint32_t)(cm - c0) * (uint32_t)row_bytes;
        for (uint32_t off = 0; off < total; off += 65536u) {
            const uint32_t piece = min(65536u, total - off);
            bulk_g2s(sc_smem_u32(rowK + off), srcK + src + off, piece, bar);
            bulk_g2s(sc_smem_u32(rowV + off), srcV + src + off, piece, bar);
        }
    }
    // original position of this thread's candidate (thread t <-> candidate c0 + t), fetched before the selection
    const int j_mine = c0 + tid;
    int pos_mine = 0;
    if (tid < cnt) pos_mine = j_mine < m ? __ldg(job.srcPos + (size_t)g * cap + j_mine) : job.chunk_pos0 + (j_mine - m);

    // ---- selection on the whole score vector
    bool keep = false;
    uint32_t p_mine = 0;                                      // place of this thread's candidate in the ascending list
    int p_base = 0, kept_here = 0;
    if (n <= k) {                                             // nothing to evict
        keep = tid < cnt; p_mine = (uint32_t)j_mine; p_base = c0; kept_here = cnt;
        if (keep) s_lkept[tid] = tid;
        __syncthreads();
    } else {
        uint32_t T, take_eq;
        CITRUS_TR(4);
        // (layer-wise granularity: every CTA ranks the sum of the heads' scores, so all heads keep the same candidates)
        select_threshold(sjob, g, kv_heads, layerwise, keys, T, take_eq);
        CITRUS_TR(5);
        // kept candidates and candidates equal to T before the share (all threads count a slice of keys[0, c0))
        uint32_t gt = 0u, eq = 0u;
        for (int j = tid; j < c0; j += kSelThreads) { const uint32_t key = keys[j]; gt += key > T; eq += key == T; }
        const uint32_t key_mine = tid < cnt ? keys[j_mine] : 0u;
        const bool is_gt = tid < cnt && key_mine > T, is_eq = tid < cnt && key_mine == T;
        gt = __reduce_add_sync(0xffffffffu, gt); eq = __reduce_add_sync(0xffffffffu, eq);
        // the share itself, one candidate per thread: ballots give the in-warp ranks
        const uint32_t b_gt = __ballot_sync(0xffffffffu, is_gt), b_eq = __ballot_sync(0xffffffffu, is_eq);
        if (lane == 0) { w_gt[warp] = gt | ((uint32_t)__popc(b_gt) << 16); w_eq[warp] = eq | ((uint32_t)__popc(b_eq) << 16); }
        __syncthreads();
        // every warp adds up: totals before the share (low halves), and the share's counts of the warps before it
        uint32_t v_gt = w_gt[lane], v_eq = w_eq[lane];
        const uint32_t gt_before = __reduce_add_sync(0xffffffffu, v_gt & 0xffffu);
        const uint32_t eq_before = __reduce_add_sync(0xffffffffu, v_eq & 0xffffu);
        const uint32_t gt_warps = __reduce_add_sync(0xffffffffu, lane < warp ? (v_gt >> 16) : 0u);
        const uint32_t eq_warps = __reduce_add_sync(0xffffffffu, lane < warp ? (v_eq >> 16) : 0u);
        const uint32_t lt_mask = (1u << lane) - 1u;
        const uint32_t gt_rank = gt_warps + (uint32_t)__popc(b_gt & lt_mask);       // kept-by-value candidates of the share before mine
        const uint32_t eq_rank = eq_before + eq_warps + (uint32_t)__popc(b_eq & lt_mask);   // equal-to-T candidates before mine, whole vector
        keep = is_gt || (is_eq && eq_rank < take_eq);
        // ties kept before the share, and inside the share before mine
        const uint32_t eq_kept_before = min(eq_before, take_eq);
        const uint32_t eq_kept_rank = min(eq_rank, take_eq) - eq_kept_before;
        p_base = (int)(gt_before + eq_kept_before);
        p_mine = (uint32_t)p_base + gt_rank + eq_kept_rank;
        const uint32_t b_keep = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) w_keep[warp] = (uint32_t)__popc(b_keep);
        if (keep) s_lkept[p_mine - (uint32_t)p_base] = tid;
        __syncthreads();
        kept_here = (int)__reduce_add_sync(0xffffffffu, w_keep[lane]);
    }
    CITRUS_TR(6);
    // ---- index list and positions of the kept candidates of the share
    if (keep) {
        sjob.idx[(size_t)g * sjob.idx_stride + p_mine] = j_mine;
        job.dstPos[(size_t)g * cap + p_mine] = pos_mine;
    }
    // ---- rows: wait for the copies, then shared memory -> new cache, row_vecs lanes per row
    {
        bool landed = false;
        for (int spin = 0; spin < (1 << 22) && !landed; ++spin) {       // bounded: the copies of a few KB take microseconds
            uint32_t ok;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(bar) : "memory");
            landed = ok != 0;
        }
        if (!landed) return;                                            // (never seen; the rows are then left unwritten)
    }
    CITRUS_TR(7);
    const int row_vecs = row_bytes / 16;
    const int rows_per_pass = kSelThreads / row_vecs;
    const int sub = tid / row_vecs, v = tid % row_vecs;
    uint4* dstK = reinterpret_cast<uint4*>(job.dstK);
    uint4* dstV = reinterpret_cast<uint4*>(job.dstV);
    for (int r = sub; r < kept_here; r += rows_per_pass) {
        const int l = s_lkept[r];
        const uint4 a = *reinterpret_cast<const uint4*>(rowK + (size_t)l * row_bytes + (size_t)v * 16);
        const uint4 bb = *reinterpret_cast<const uint4*>(rowV + (size_t)l * row_bytes + (size_t)v * 16);
        const size_t doff = ((size_t)g * cap + p_base + r) * row_vecs + v;
        dstK[doff] = a;
        dstV[doff] = bb;
    }
    CITRUS_TR(8);
}

// One CTA per KV head: thread t looks element t, t + 256, ... of list b up in list a (both strictly ascending) by
// binary search; the hits are counted with a warp reduction and one shared-memory atomic per warp.
__global__ void __launch_bounds__(256)
intersection_kernel(const int* __restrict__ pos_a, int stride_a, int rows_a, const int* __restrict__ pos_b, int stride_b, int rows,
                    float* __restrict__ ratio) {
    __shared__ int hits;
    const int g = blockIdx.x;
    const int* a = pos_a + (size_t)g * stride_a;
    const int* b = pos_b + (size_t)g * stride_b;
    if (threadIdx.x == 0) hits = 0;
    __syncthreads();
    int mine = 0;
    for (int i = threadIdx.x; i < rows; i += blockDim.x) {
        const int x = b[i];
        int lo = 0, hi = rows_a;                  // first index with a[idx] >= x
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (a[mid] < x) lo = mid + 1; else hi = mid;
        }
        mine += lo < rows_a && a[lo] == x;
    }
    mine = __reduce_add_sync(0xffffffffu, mine);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&hits, mine);
    __syncthreads();
    if (threadIdx.x == 0) ratio[g] = (float)hits / (float)rows;
}

constexpr int kMaxRopeJobs = 3;
struct RopeArgs { RopeRows job[kMaxRopeJobs]; RopeTable table; int n_jobs, row_vecs, elt; };

// Embedding pre-pass of the position shift: every 16-byte piece of the listed token-major tensors is turned by the
// position of its row.  grid.y = tensor, grid-stride over its pieces.
__global__ void __launch_bounds__(256)
rope_rows_kernel(const __grid_constant__ RopeArgs args) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // the outputs are scratch that the previous step's kernels may still be reading
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const RopeRows& job = args.job[blockIdx.y];
    const int row_vecs = args.row_vecs, half_vecs = row_vecs >> 1, per_vec = 16 / args.elt;
    const long long total = (long long)job.rows * job.heads * row_vecs;          // a multiple of row_vecs, not always of 32
    const uint4* in = reinterpret_cast<const uint4*>(job.in);
    uint4* out = reinterpret_cast<uint4*>(job.out);
    const int lane = threadIdx.x & 31;
    // warp-uniform trip count (the exchange below is a full-mask shuffle): the loop runs on the warp's first piece
    for (long long i_w = (long long)blockIdx.x * blockDim.x + (threadIdx.x - lane); i_w < total; i_w += (long long)gridDim.x * blockDim.x) {
        const long long i = i_w + lane;
        const bool active = i < total;
        const int v = (int)(i % row_vecs);
        const int row = (int)(i / ((long long)row_vecs * job.heads));
        const uint4 mine = active ? __ldg(in + i) : make_uint4(0u, 0u, 0u, 0u);
        uint4 other;
        other.x = __shfl_xor_sync(0xffffffffu, mine.x, half_vecs); other.y = __shfl_xor_sync(0xffffffffu, mine.y, half_vecs);
        other.z = __shfl_xor_sync(0xffffffffu, mine.z, half_vecs); other.w = __shfl_xor_sync(0xffffffffu, mine.w, half_vecs);
        if (active) out[i] = rope_piece(mine, other, job.pos0 + row, (v % half_vecs) * per_vec, v < half_vecs, args.table, args.elt);
    }
}

// The dynamic shared-memory limit of a kernel is a per-device attribute: raised once on every device that launches.
std::mutex g_attr_mu;
DeviceOnce g_attr_ready;
cudaError_t raise_smem_limits() {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lk(g_attr_mu);
    if (!g_attr_ready.needs_setup(dev)) return cudaSuccess;
    e = cudaFuncSetAttribute(select_topk_kernel<kJobsSingle>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(select_topk_kernel<kJobsBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(select_gather_kernel<kJobsSingle>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(select_gather_kernel<kJobsBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    g_attr_ready.mark(dev);
    return cudaSuccess;
}

}  // namespace

cudaError_t rope_rows(const RopeRows* jobs, int n_jobs, int D, int elt, const RopeTable& table, cudaStream_t s) {
    if (n_jobs < 1 || n_jobs > kMaxRopeJobs) return cudaErrorInvalidValue;
    RopeArgs a;
    a.table = table; a.n_jobs = n_jobs; a.row_vecs = D * elt / 16; a.elt = elt;
    long long most = 0;
    for (int i = 0; i < n_jobs; ++i) {
        a.job[i] = jobs[i];
        const long long t = (long long)jobs[i].rows * jobs[i].heads * a.row_vecs;
        most = t > most ? t : most;
    }
    cudaLaunchConfig_t cfg = {};
    long long blocks = (most + 255) / 256;
    cfg.gridDim = dim3((unsigned)(blocks > 592 ? 592 : (blocks < 1 ? 1 : blocks)), n_jobs);
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    before_launch(s);
    return cudaLaunchKernelEx(&cfg, rope_rows_kernel, a);
}

cudaError_t intersection_ratio(const int* pos_a, int stride_a, int rows_a, const int* pos_b, int stride_b, int rows_b,
                               int kv_heads, float* ratio, cudaStream_t s) {
    intersection_kernel<<<kv_heads, 256, 0, s>>>(pos_a, stride_a, rows_a, pos_b, stride_b, rows_b, ratio);
    return cudaGetLastError();
}

template <int CAP>
static cudaError_t launch_select_topk(const SelectJob* jobs, int n_jobs, int kv_heads, int layerwise, cudaStream_t s) {
    SelectArgs<CAP> a;
    int n = 0;
    for (int i = 0; i < n_jobs; ++i) { a.job[i] = jobs[i]; n = jobs[i].n > n ? jobs[i].n : n; }
    size_t smem = (size_t)n * sizeof(uint32_t);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(layerwise ? 1 : kv_heads, n_jobs);
    cfg.blockDim = dim3(kSelThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    before_launch(s);
    return cudaLaunchKernelEx(&cfg, select_topk_kernel<CAP>, a, kv_heads, layerwise);
}

cudaError_t select_topk(const SelectJob* jobs, int n_jobs, int kv_heads, int layerwise, cudaStream_t s) {
    if (n_jobs < 1 || n_jobs > kJobsBatch) return cudaErrorInvalidValue;
    cudaError_t e = raise_smem_limits();
    if (e != cudaSuccess) return e;
    if (n_jobs <= kJobsSingle) return launch_select_topk<kJobsSingle>(jobs, n_jobs, kv_heads, layerwise, s);
    return launch_select_topk<kJobsBatch>(jobs, n_jobs, kv_heads, layerwise, s);
}

// Shared memory of the fused kernel for a step with at most n candidates per job.
static size_t fused_smem_bytes(int n, int row_bytes) {
    const int share = (n + kFusedParts - 1) / kFusedParts;
    return (((size_t)n * 4 + 127) & ~(size_t)127) + (size_t)2 * share * row_bytes;
}
bool select_compact_fits(int n, int row_bytes) {
    return (n + kFusedParts - 1) / kFusedParts <= kFusedMaxShare && fused_smem_bytes(n, row_bytes) <= 200 * 1024;
}

template <int CAP>
static cudaError_t launch_select_compact(const SelectJob* sjobs, const CompactJob* cjobs, int n_jobs, int kv_heads, int row_bytes,
                                         int elt, int early_chunk_rows, int layerwise, cudaStream_t s) {
    SelectArgs<CAP> sa; CompactArgs<CAP> ca;
    ca.elt = elt;
    int n = 0;
    for (int i = 0; i < n_jobs; ++i) {
        sa.job[i] = sjobs[i]; ca.job[i] = cjobs[i];
        n = sjobs[i].n > n ? sjobs[i].n : n;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kFusedParts, kv_heads, n_jobs);
    cfg.blockDim = dim3(kSelThreads);
    cfg.dynamicSmemBytes = fused_smem_bytes(n, row_bytes);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    before_launch(s);
    return cudaLaunchKernelEx(&cfg, select_gather_kernel<CAP>, sa, ca, kv_heads, n, (n + kFusedParts - 1) / kFusedParts, row_bytes,
                              early_chunk_rows, layerwise);
}

cudaError_t select_compact(const SelectJob* sjobs, const CompactJob* cjobs, int n_jobs, int kv_heads, int row_bytes,
                           int elt, int early_chunk_rows, int layerwise, cudaStream_t s) {
    if (n_jobs < 1 || n_jobs > kJobsBatch) return cudaErrorInvalidValue;
    cudaError_t e = raise_smem_limits();
    if (e != cudaSuccess) return e;
    if (n_jobs <= kJobsSingle) return launch_select_compact<kJobsSingle>(sjobs, cjobs, n_jobs, kv_heads, row_bytes, elt, early_chunk_rows, layerwise, s);
    return launch_select_compact<kJobsBatch>(sjobs, cjobs, n_jobs, kv_heads, row_bytes, elt, early_chunk_rows, layerwise, s);
}

template <int CAP>
static cudaError_t launch_compact_kv(const CompactJob* jobs, int n_jobs, int kv_heads, int row_bytes, const RopeTable* rope, int elt,
                                     cudaStream_t s) {
    CompactArgs<CAP> a;
    a.elt = elt;
    if (rope != nullptr) a.rope = *rope;
    int kept = 0;
    for (int i = 0; i < n_jobs; ++i) { a.job[i] = jobs[i]; kept = jobs[i].kept > kept ? jobs[i].kept : kept; }
    int row_vecs = row_bytes / 16;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((kept + kCompactRowsPerCta - 1) / kCompactRowsPerCta, kv_heads, n_jobs);
    cfg.blockDim = dim3(kCompactThreads);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    before_launch(s);
    if (rope != nullptr) return cudaLaunchKernelEx(&cfg, compact_kv_kernel<true, CAP>, a, kv_heads, row_vecs);
    return cudaLaunchKernelEx(&cfg, compact_kv_kernel<false, CAP>, a, kv_heads, row_vecs);
}

cudaError_t compact_kv(const CompactJob* jobs, int n_jobs, int kv_heads, int row_bytes, const RopeTable* rope, int elt, cudaStream_t s) {
    if (n_jobs < 1 || n_jobs > kJobsBatch) return cudaErrorInvalidValue;
    if (n_jobs <= kJobsSingle) return launch_compact_kv<kJobsSingle>(jobs, n_jobs, kv_heads, row_bytes, rope, elt, s);
    return launch_compact_kv<kJobsBatch>(jobs, n_jobs, kv_heads, row_bytes, rope, elt, s);
}

}  // namespace citrus
