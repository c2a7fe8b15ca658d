// Host side of the C ABI declared in include/citrus.h: context state, argument
// checks, ping-pong cache bookkeeping and the launch sequence of one chunk step.
#include "../../include/citrus.h"
#include "citrus_internal.h"
#include <algorithm>

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <set>
#include <vector>

namespace {

using namespace citrus;

struct CacheBufs {
    void* K[2] = {nullptr, nullptr};
    void* V[2] = {nullptr, nullptr};
    int* pos[2] = {nullptr, nullptr};
    float* carried[2] = {nullptr, nullptr};      // accumulative policy: importance carried by the rows
    void* Kraw[2] = {nullptr, nullptr};          // position shift: the un-rotated keys (K[] then holds them embedded by slot)
    int cur = 0;
};

// The caches of one (layer, cache id) for all sequence slots and both ping-pong halves live in ONE tensor
// [2 x n_slots x kv_heads, cap, D] (positions / carried importance: [2 x n_slots x kv_heads, cap]), so that a single
// tensor map covers them and a batched launch reaches every sequence's cache through a head offset.
struct LayerCache {
    void* K = nullptr; void* V = nullptr; void* Kraw = nullptr; int* pos = nullptr; float* carried = nullptr;
};

struct Unit {                       // one (layer, sequence slot)
    CacheBufs cache[2];
    float* scores = nullptr;        // [n_caches, kv_heads, score_stride]
    int* idx[2] = {nullptr, nullptr};   // per cache [kv_heads, cap]
    float* lse_chunk = nullptr;     // [q_heads, chunk_s]
    float* lse_instr = nullptr;     // [q_heads, CITRUS_MAX_INSTR]
    float* part = nullptr;          // key-split (max, sum) pairs of a2 pass 1 [splits, q_heads, CITRUS_MAX_INSTR] (tensor-core path)
    int m[2] = {0, 0};              // rows retained in each cache
    long long tokens_seen = 0;
    int last_n[2] = {0, 0}, last_kept[2] = {0, 0}, last_m[2] = {0, 0};
    bool has_step = false;
};

}  // namespace

struct citrus_ctx {
    int device = 0;
    int layers = 0, Hq = 0, Hkv = 0, D = 0, k = 0, ls = 0;
    bool individual = false, standard = false, fp32 = false, layerwise = false, use_tc = false;
    int lm_window = 0;
    int start_size = 0;             // initial tokens that are never evicted
    bool accumulate = false;        // scores carried across steps
    bool deferred = false;          // cache 0 holds k states + the previous chunk and is evicted by the next chunk
    int cap[2] = {0, 0};            // row capacity of each cache's buffers
    bool shift = false;             // position shift: rotary embedding by cache slot
    RopeTable rope;                 // its angles per pair
    void *rotQ = nullptr, *rotK = nullptr, *rotQi = nullptr;   // the step's embedded chunk queries / keys / instruction queries
    int elt = 2;
    int n_caches = 1;
    int n_slots = 1;
    int score_stride = 0;
    bool used = false;
    std::vector<Unit> units;        // [layers * n_slots]
    std::vector<LayerCache> layer_cache;   // [layers * 2]
    std::vector<void*> allocs;      // cache buffers and per-unit scratch
    std::vector<void*> misc;        // status word, host-variant staging
    int* status = nullptr;
    // The caller has promised that the inputs of every call are complete before the call's first kernel can start
    // (citrus_set_inputs_ready): the kernels may then load them ahead of griddepcontrol.wait.
    bool inputs_ready = false;
    // position shift: stream of the last step and an event to order a step on another stream behind it (the
    // embedding scratch is one per context)
    cudaStream_t shift_stream = nullptr;
    bool shift_stream_set = false;
    cudaEvent_t shift_done = nullptr;
    // a1 beside a2-a4: when nothing in a2-a4 reads a1's result (shared cache scored by the instruction text), the
    // attention of a step of at most a1_cap items (CTAs) runs on a side stream while the caller's stream runs the
    // chain log-sum-exp -> column sums -> select / gather on the SMs it leaves free; the streams fork at the start of
    // a call and join before it returns.  0 = off.
    int a1_cap = 64;
    cudaStream_t a1_stream = nullptr;
    cudaEvent_t a1_fork = nullptr, a1_done = nullptr;
    // optional per-launch timing: (kernel id, start, stop) event pairs recorded on the launching stream
    bool profiling = false;
    struct Timed { int id; cudaEvent_t a, b; };
    std::vector<Timed> timed;
    // staging of the host-buffer variant
    void *stQ = nullptr, *stK = nullptr, *stV = nullptr, *stQi = nullptr, *stOut = nullptr;
    // whole-document host variant: two staging sets of a few chunks each, two copy streams, events per set
    void *docQ[2] = {nullptr, nullptr}, *docK[2] = {nullptr, nullptr}, *docV[2] = {nullptr, nullptr}, *docOut[2] = {nullptr, nullptr};
    void* docQi = nullptr;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_step[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr}, ev_qi = nullptr;
    // ragged batches of small steps: the sequences of one call are dealt to side streams ("lanes") that fork from the
    // caller's stream and join it again before the call returns, so that the latency chains of different sequences
    // (a step of a few dozen CTAs leaves most SMs idle) overlap.  0 = chosen per call.
    static constexpr int kMaxLanes = 8;
    int lanes_wanted = 0;
    cudaStream_t lane[kMaxLanes] = {};
    cudaEvent_t lane_done[kMaxLanes] = {};
    cudaEvent_t lane_fork = nullptr;
    // position shift: the embedding scratch of a step, one set per lane (the context's own set serves the caller's stream)
    void *laneRotQ[kMaxLanes] = {}, *laneRotK[kMaxLanes] = {}, *laneRotQi[kMaxLanes] = {};
};

namespace {

std::mutex g_mu;
std::set<citrus_ctx*> g_live;
std::set<citrus_ctx*> g_dead;

bool is_live(citrus_ctx* h) {
    std::lock_guard<std::mutex> lk(g_mu);
    return g_live.count(h) != 0;
}

int dev_alloc(citrus_ctx* c, void** p, size_t bytes, bool zero, bool misc = false) {
    cudaError_t e = cudaMalloc(p, bytes);
    if (e != cudaSuccess) { cudaGetLastError(); return e == cudaErrorMemoryAllocation ? CITRUS_ERR_NOMEM : CITRUS_ERR_CUDA; }
    (misc ? c->misc : c->allocs).push_back(*p);
    if (zero) {
        e = cudaMemset(*p, 0, bytes);
        if (e != cudaSuccess) return CITRUS_ERR_CUDA;
    }
    return CITRUS_OK;
}

void free_units(citrus_ctx* c) {
    for (void* p : c->allocs) cudaFree(p);
    c->allocs.clear();
    c->units.clear();
    c->layer_cache.clear();
}
void free_copy_streams(citrus_ctx* c) {
    for (int b = 0; b < 2; ++b) {
        if (c->ev_in[b]) cudaEventDestroy(c->ev_in[b]);
        if (c->ev_step[b]) cudaEventDestroy(c->ev_step[b]);
        if (c->ev_out[b]) cudaEventDestroy(c->ev_out[b]);
    }
    if (c->ev_qi) cudaEventDestroy(c->ev_qi);
    if (c->s_in) cudaStreamDestroy(c->s_in);
    if (c->s_out) cudaStreamDestroy(c->s_out);
    for (int i = 0; i < citrus_ctx::kMaxLanes; ++i) {
        if (c->lane_done[i]) cudaEventDestroy(c->lane_done[i]);
        if (c->lane[i]) cudaStreamDestroy(c->lane[i]);
        c->lane_done[i] = nullptr; c->lane[i] = nullptr;
    }
    if (c->lane_fork) cudaEventDestroy(c->lane_fork);
    c->lane_fork = nullptr;
    if (c->shift_done) cudaEventDestroy(c->shift_done);
    c->shift_done = nullptr;
    if (c->a1_fork) cudaEventDestroy(c->a1_fork);
    if (c->a1_done) cudaEventDestroy(c->a1_done);
    if (c->a1_stream) cudaStreamDestroy(c->a1_stream);
    c->a1_fork = c->a1_done = nullptr; c->a1_stream = nullptr;
}
// Side streams and events of the batch lanes (created once, by citrus_set_batch for more than one slot).
int make_lanes(citrus_ctx* c) {
    cudaError_t e = cudaSuccess;
    if (c->lane_fork == nullptr) e = cudaEventCreateWithFlags(&c->lane_fork, cudaEventDisableTiming);
    for (int i = 0; i < citrus_ctx::kMaxLanes && e == cudaSuccess; ++i) {
        if (c->lane[i] == nullptr) e = cudaStreamCreateWithFlags(&c->lane[i], cudaStreamNonBlocking);
        if (e == cudaSuccess && c->lane_done[i] == nullptr) e = cudaEventCreateWithFlags(&c->lane_done[i], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) { cudaGetLastError(); return CITRUS_ERR_CUDA; }
    if (c->shift) {
        const size_t row = (size_t)c->D * c->elt;
        for (int i = 0; i < citrus_ctx::kMaxLanes; ++i) {
            if (c->laneRotQ[i] != nullptr) continue;
            int rc = dev_alloc(c, &c->laneRotQ[i], (size_t)c->ls * c->Hq * row, false, true);
            if (rc == CITRUS_OK) rc = dev_alloc(c, &c->laneRotK[i], (size_t)c->ls * c->Hkv * row, false, true);
            if (rc == CITRUS_OK) rc = dev_alloc(c, &c->laneRotQi[i], (size_t)CITRUS_MAX_INSTR * c->Hq * row, false, true);
            if (rc != CITRUS_OK) return rc;
        }
    }
    return CITRUS_OK;
}
void free_all(citrus_ctx* c) {
    free_units(c);
    for (void* p : c->misc) cudaFree(p);
    c->misc.clear();
}

int alloc_units(citrus_ctx* c) {
    const size_t row = (size_t)c->D * c->elt;
    c->units.assign((size_t)c->layers * c->n_slots, Unit());
    c->layer_cache.assign((size_t)c->layers * 2, LayerCache());
    int rc;
    for (int layer = 0; layer < c->layers; ++layer) {
        for (int ci = 0; ci < c->n_caches; ++ci) {
            LayerCache& lc = c->layer_cache[(size_t)layer * 2 + ci];
            const size_t heads = (size_t)2 * c->n_slots * c->Hkv;           // ping-pong halves x slots x KV heads
            const size_t kv_bytes = heads * c->cap[ci] * row;
            if ((rc = dev_alloc(c, &lc.K, kv_bytes, true))) return rc;
            if ((rc = dev_alloc(c, &lc.V, kv_bytes, true))) return rc;
            if (c->shift && (rc = dev_alloc(c, &lc.Kraw, kv_bytes, true))) return rc;
            if ((rc = dev_alloc(c, (void**)&lc.pos, heads * c->cap[ci] * sizeof(int), true))) return rc;
            if (c->accumulate && (rc = dev_alloc(c, (void**)&lc.carried, heads * c->cap[ci] * sizeof(float), true))) return rc;
            for (int slot = 0; slot < c->n_slots; ++slot) {
                Unit& u = c->units[(size_t)layer * c->n_slots + slot];
                for (int b = 0; b < 2; ++b) {
                    const size_t first_head = ((size_t)b * c->n_slots + slot) * c->Hkv;
                    const size_t off = first_head * c->cap[ci];
                    u.cache[ci].K[b] = static_cast<char*>(lc.K) + off * row;
                    u.cache[ci].V[b] = static_cast<char*>(lc.V) + off * row;
                    if (c->shift) u.cache[ci].Kraw[b] = static_cast<char*>(lc.Kraw) + off * row;
                    u.cache[ci].pos[b] = lc.pos + off;
                    if (c->accumulate) u.cache[ci].carried[b] = lc.carried + off;
                }
            }
        }
    }
    for (Unit& u : c->units) {
        for (int ci = 0; ci < c->n_caches; ++ci)
            if ((rc = dev_alloc(c, (void**)&u.idx[ci], (size_t)c->Hkv * c->cap[ci] * sizeof(int), true))) return rc;
        if ((rc = dev_alloc(c, (void**)&u.scores, (size_t)c->n_caches * c->Hkv * c->score_stride * sizeof(float), true))) return rc;
        if ((rc = dev_alloc(c, (void**)&u.lse_chunk, (size_t)c->Hq * c->ls * sizeof(float), true))) return rc;
        if ((rc = dev_alloc(c, (void**)&u.lse_instr, (size_t)c->Hq * CITRUS_MAX_INSTR * sizeof(float), true))) return rc;
        if (c->use_tc && (rc = dev_alloc(c, (void**)&u.part, (size_t)kTcMaxLseSplits * c->Hq * CITRUS_MAX_INSTR * 2 * sizeof(float), true))) return rc;
    }
    return CITRUS_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int cuda_rc(cudaError_t e) {
    if (e == cudaSuccess) return CITRUS_OK;
    cudaGetLastError();
    return CITRUS_ERR_CUDA;
}

int check_process_args(citrus_ctx* h, int layer, int slot, const void* Q, const void* K, const void* V, int L,
                       const void* Qi, int nI, const void* out) {
    if (h == nullptr || !is_live(h)) return CITRUS_ERR_INVALID_ARG;
    // standard chunked eviction: a call without instruction queries (n_instr == 0) is scored by the chunk itself
    const bool no_instr = h->standard && nI == 0;
    if (!Q || !K || !V || (!Qi && !no_instr) || !out) return CITRUS_ERR_INVALID_ARG;
    if (layer < 0 || layer >= h->layers) return CITRUS_ERR_LAYER;
    if (slot < 0 || slot >= h->n_slots) return CITRUS_ERR_INVALID_ARG;
    if (L < 1 || L > h->ls || (nI < 1 && !no_instr) || nI > CITRUS_MAX_INSTR) return CITRUS_ERR_SHAPE;
    return CITRUS_OK;
}

thread_local cudaEvent_t t_pending_start = nullptr;      // start event of the launch being prepared, if any

struct LaunchTimer {                 // brackets one kernel launch with events when profiling is on
    citrus_ctx* c; cudaStream_t st; cudaEvent_t a = nullptr, b = nullptr; int id;
    LaunchTimer(citrus_ctx* c_, int id_, cudaStream_t st_) : c(c_), st(st_), id(id_) {
        if (!c->profiling) return;
        if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { a = b = nullptr; cudaGetLastError(); return; }
        t_pending_start = a;         // recorded by before_launch(), right in front of the kernel
    }
    ~LaunchTimer() {
        if (a == nullptr) return;
        if (t_pending_start == a) { cudaEventRecord(a, st); t_pending_start = nullptr; }   // nothing was launched
        cudaEventRecord(b, st);
        c->timed.push_back(citrus_ctx::Timed{id, a, b});
    }
};

// One sequence's chunk as the step launcher takes it; all pointers are device pointers to the sequence's own rows.
struct StepIn {
    int slot;
    const void *Q, *K, *V, *Qi;
    int L, nI;
    void* out;
};
// The tensors that hold every sequence's rows of a batched call (null: a single sequence, its own tensors).
struct PackedIn {
    const void *Q, *K, *V, *Qi;
    void* out;
    int tok_rows, instr_rows;       // rows of Q / K / V / out and of Qi that the call spans
};

// The launch sequence of one chunk step for n sequences of one layer (n > 1: the tensor-core path without position
// shift; every launch then covers all sequences).  The steps of different sequences are independent.
cudaError_t join_a1(citrus_ctx* c, cudaStream_t st) {
    cudaError_t e = cudaEventRecord(c->a1_done, c->a1_stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, c->a1_done, 0);
    return e;
}

int run_steps(citrus_ctx* c, int layer, int n, const StepIn* in, const PackedIn* packed, cudaStream_t st, int lane = -1,
              bool inputs_ordered = false) {
    c->used = true;
    if (n < 1 || n > kTcMaxBatch || (n > 1 && (!c->use_tc || c->shift || packed == nullptr))) return CITRUS_ERR_INVALID_ARG;
    if (c->shift && lane < 0) {
        // One embedding scratch per context: a step on another stream than the last one is ordered behind everything
        // enqueued there so far.  Steps that stay on one stream pay nothing.
        if (c->shift_stream_set && c->shift_stream != st) {
            cudaError_t ee = cudaEventRecord(c->shift_done, c->shift_stream);
            if (ee == cudaSuccess) ee = cudaStreamWaitEvent(st, c->shift_done, 0);
            if (ee != cudaSuccess) return cuda_rc(ee);
        }
        c->shift_stream = st; c->shift_stream_set = true;
    }
    // embedding scratch of this step (position shift): the lane's own set when the step runs on a side stream
    void* const rotQ = lane >= 0 ? c->laneRotQ[lane] : c->rotQ;
    void* const rotK = lane >= 0 ? c->laneRotK[lane] : c->rotK;
    void* const rotQi = lane >= 0 ? c->laneRotQi[lane] : c->rotQi;
    const size_t qrow = (size_t)c->Hq * c->D * c->elt, krow = (size_t)c->Hkv * c->D * c->elt;
    const int ic = c->individual ? 1 : 0;     // the cache scored by the instruction text
    // 1: the kernels wait for their predecessors in the stream before their first load of Q / K / Q_instr.  Needed when
    // the embedding pre-pass wrote them, and whenever the inputs may still be in the making: the call's first
    // kernel is launched with programmatic stream serialisation, so a preceding kernel of the CALLER that signals
    // its dependents early could otherwise still be writing them.
    const int produced = (c->shift || !(c->inputs_ready || inputs_ordered)) ? 1 : 0;

    struct Sizes { int mc[2], nc[2], kept[2], forced_from[2]; bool lm_scoring, instr_scoring; };
    std::vector<Sizes> sz(n);
    std::vector<TcSeqStep> seq(n);
    std::vector<SelectJob> sj;
    std::vector<CompactJob> cj;
    sj.reserve((size_t)n * c->n_caches); cj.reserve((size_t)n * c->n_caches);
    bool any_lm = false, any_instr = false;
    size_t gather_bytes = 0;
    for (int i = 0; i < n; ++i) {
        Unit& u = c->units[(size_t)layer * c->n_slots + in[i].slot];
        const int L = in[i].L, nI = in[i].nI;
        if (u.tokens_seen + L > 0x7fffffffLL) return CITRUS_ERR_SHAPE;
        Sizes& z = sz[i];
        z.lm_scoring = c->individual || (c->standard && nI == 0);   // cache 0 is scored by the chunk's own queries
        z.instr_scoring = nI > 0;
        any_lm |= z.lm_scoring; any_instr |= z.instr_scoring;
        // sizes of each cache's step.  Deferred eviction (cache 0, when the chunk scores it): only the cache's own rows
        // compete for the k places, all of the chunk's rows enter.
        for (int ci = 0; ci < c->n_caches; ++ci) {
            z.mc[ci] = u.m[ci]; z.nc[ci] = z.mc[ci] + L;
            z.forced_from[ci] = z.nc[ci];
            z.kept[ci] = z.nc[ci] < c->k ? z.nc[ci] : c->k;
            if (c->deferred && ci == 0 && z.lm_scoring) {
                z.kept[ci] = (z.mc[ci] < c->k ? z.mc[ci] : c->k) + L;
                z.forced_from[ci] = z.mc[ci];
            }
        }
        if (c->n_caches == 1) { z.mc[1] = z.mc[0]; z.nc[1] = z.nc[0]; z.kept[1] = z.kept[0]; z.forced_from[1] = z.forced_from[0]; }
        TcSeqStep& q = seq[i];
        q = TcSeqStep{};
        q.L = L; q.nI = nI; q.ic = ic; q.produced = produced;
        q.q_row0 = packed ? (int)((static_cast<const char*>(in[i].Q) - static_cast<const char*>(packed->Q)) / qrow) : 0;
        q.kv_row0 = packed ? (int)((static_cast<const char*>(in[i].K) - static_cast<const char*>(packed->K)) / krow) : 0;
        q.qi_row0 = (packed && nI > 0) ? (int)((static_cast<const char*>(in[i].Qi) - static_cast<const char*>(packed->Qi)) / qrow) : 0;
        for (int ci = 0; ci < 2; ++ci) {
            const int cc = ci < c->n_caches ? ci : 0;
            q.m[ci] = z.mc[cc];
            q.chead[ci] = (u.cache[cc].cur * c->n_slots + in[i].slot) * c->Hkv;
            q.scores[ci] = u.scores + (size_t)cc * c->Hkv * c->score_stride;
        }
        q.score_stride = c->score_stride;
        q.w = z.lm_scoring ? ((c->lm_window > 0 && c->lm_window < L) ? c->lm_window : L) : 0;
        q.lse_chunk = z.lm_scoring ? u.lse_chunk : nullptr;           // only a2-L reads a1's row log-sum-exp
        q.lse_instr = u.lse_instr; q.part = u.part;
        q.splits = 1;
        if (c->use_tc && z.instr_scoring)
            // (chosen as for a call of this sequence alone, so that a batched step gives the same bits)
            q.splits = tc_lse_splits(nI, c->Hq, c->Hkv, z.mc[ic], L, ((L + 127) / 128) * c->Hq);
    }
    // a batch shares one kernel template: either every sequence's a1 keeps its row log-sum-exp or none does
    for (int i = 1; i < n; ++i)
        if (sz[i].lm_scoring != sz[0].lm_scoring || sz[i].instr_scoring != sz[0].instr_scoring) return CITRUS_ERR_INVALID_ARG;

    cudaError_t e = cudaSuccess;
    bool beside = false;                                           // a1 runs on the side stream: join before returning
    const void *Qc = in[0].Q, *Kc = in[0].K, *Qi = in[0].Qi;       // single-sequence paths below (n == 1)
    if (c->shift) {
        // position shift: embed the chunk's queries and keys at rows m .. m+L-1 and the instruction queries behind them
        const int m0 = sz[0].mc[0], L = in[0].L, nI = in[0].nI;
        RopeRows jobs[3] = {{Qc, rotQ, L, c->Hq, m0}, {Kc, rotK, L, c->Hkv, m0}, {Qi, rotQi, nI, c->Hq, m0 + L}};
        LaunchTimer t(c, CITRUS_KERNEL_ROPE, st);
        e = rope_rows(jobs, sz[0].instr_scoring ? 3 : 2, c->D, c->elt, c->rope, st);
        if (e != cudaSuccess) return cuda_rc(e);
        Qc = rotQ; Kc = rotK; if (sz[0].instr_scoring) Qi = rotQi;
    }

    if (c->use_tc) {
        TcTensors t{};
        t.q_heads = c->Hq; t.kv_heads = c->Hkv;
        if (packed != nullptr && !c->shift) {
            t.Q = packed->Q; t.out = packed->out; t.q_rows = packed->tok_rows;
            t.K = packed->K; t.V = packed->V; t.kv_rows = packed->tok_rows;
            t.Qi = packed->Qi; t.qi_rows = packed->instr_rows;
        } else {
            t.Q = Qc; t.out = in[0].out; t.q_rows = in[0].L;
            t.K = Kc; t.V = in[0].V; t.kv_rows = in[0].L;
            t.Qi = Qi; t.qi_rows = in[0].nI;
        }
        for (int ci = 0; ci < 2; ++ci) {
            const int cc = ci < c->n_caches ? ci : 0;
            const LayerCache& lc = c->layer_cache[(size_t)layer * 2 + cc];
            t.cacheK[ci] = lc.K; t.cacheV[ci] = lc.V; t.cap[ci] = c->cap[cc]; t.cache_heads[ci] = 2 * c->n_slots * c->Hkv;
        }
        // a1 beside a2-a4 (see a1_cap): one sequence on the caller's stream, nothing downstream reads a1's result,
        // and the attention items leave SMs free for the chain
        const int a1_items = ((in[0].L + 127) / 128) * c->Hq;
        beside = n == 1 && lane < 0 && c->a1_stream != nullptr && !any_lm && any_instr &&
                 in[0].out != nullptr && a1_items <= c->a1_cap;
        if (beside) {
            e = cudaEventRecord(c->a1_fork, st);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(c->a1_stream, c->a1_fork, 0);
            if (e != cudaSuccess) return cuda_rc(e);
            cudaError_t e1, e2;
            {
                // a1 alone, behind everything the caller's stream held at the fork (so its inputs are complete)
                TcSeqStep qa = seq[0];
                qa.nI = 0; qa.produced = 0;
                LaunchTimer tm(c, CITRUS_KERNEL_ATTENTION, c->a1_stream);
                e1 = tc_attention_lse(t, &qa, 1, c->ls, CITRUS_MAX_INSTR, c->status, c->a1_stream);
            }
            {
                // pass 1 of a2-I alone
                TcTensors tl = t;
                tl.out = nullptr;
                LaunchTimer tm(c, CITRUS_KERNEL_SCORE_LSE, st);
                e2 = tc_attention_lse(tl, seq.data(), 1, c->ls, CITRUS_MAX_INSTR, c->status, st);
            }
            if (e1 != cudaSuccess || e2 != cudaSuccess) {
                join_a1(c, st);
                return cuda_rc(e1 != cudaSuccess ? e1 : e2);
            }
        } else {
            // a1 and pass 1 of a2-I (row log-sum-exp of the instruction queries, possibly split over key ranges): one launch
            LaunchTimer tm(c, CITRUS_KERNEL_ATTENTION, st);
            e = tc_attention_lse(t, seq.data(), n, c->ls, CITRUS_MAX_INSTR, c->status, st);
        }
        if (e != cudaSuccess) return cuda_rc(e);
        // a2-L (individual design, standard chunked eviction: votes of the chunk's last w queries on cache 0's
        // candidates) and pass 2 of a2-I (Eq. 1 column sums of the instruction queries over the instruction-side cache's
        // candidates) in one launch: the two are independent, and the short instruction sweeps fill the tail of the LM ones
        if (any_lm || any_instr) {
            LaunchTimer tm(c, CITRUS_KERNEL_COLSUM, st);
            e = tc_colsum(t, seq.data(), n, any_lm, any_instr, c->ls, CITRUS_MAX_INSTR, c->status, st);
            if (e != cudaSuccess) { if (beside) join_a1(c, st); return cuda_rc(e); }
        }
    } else {
        Unit& u = c->units[(size_t)layer * c->n_slots + in[0].slot];
        const Sizes& z = sz[0];
        const int L = in[0].L, nI = in[0].nI;
        Candidates cand[2];
        for (int ci = 0; ci < c->n_caches; ++ci) {
            const CacheBufs& cb = u.cache[ci];
            cand[ci] = Candidates{cb.K[cb.cur], cb.V[cb.cur], Kc, in[0].V, z.mc[ci], L, c->cap[ci], c->Hkv};
        }
        QueryRows q_chunk{Qc, L, c->Hq, 1, 0, produced};
        QueryRows q_instr{Qi, z.instr_scoring ? nI : 0, c->Hq, 0, 0, produced};
        float* scores[2] = {u.scores, u.scores + (size_t)c->Hkv * c->score_stride};
        float* lse_chunk = z.lm_scoring ? u.lse_chunk : nullptr;
        {
            LaunchTimer t(c, CITRUS_KERNEL_ATTENTION, st);
            e = simt_attention(c->fp32, c->D, q_chunk, cand[0], in[0].out, lse_chunk, c->ls, st);
        }
        if (e == cudaSuccess && z.instr_scoring) {
            LaunchTimer t(c, CITRUS_KERNEL_SCORE_LSE, st);
            e = simt_attention(c->fp32, c->D, q_instr, cand[ic], nullptr, u.lse_instr, CITRUS_MAX_INSTR, st);
        }
        if (e != cudaSuccess) return cuda_rc(e);
        if (z.lm_scoring) {
            const int w = seq[0].w;
            const char* q0 = reinterpret_cast<const char*>(Qc) + (size_t)(L - w) * qrow;
            QueryRows q_lm{q0, w, c->Hq, 1, L - w, produced};
            LaunchTimer t(c, CITRUS_KERNEL_COLSUM, st);
            e = simt_colsum(c->fp32, c->D, q_lm, cand[0], u.lse_chunk + (L - w), c->ls, scores[0], c->score_stride, st);
            if (e != cudaSuccess) return cuda_rc(e);
        }
        if (z.instr_scoring) {
            LaunchTimer t(c, CITRUS_KERNEL_COLSUM, st);
            e = simt_colsum(c->fp32, c->D, q_instr, cand[ic], u.lse_instr, CITRUS_MAX_INSTR, scores[ic], c->score_stride, st);
            if (e != cudaSuccess) return cuda_rc(e);
        }
    }

    // a3 + a4 for every cache of every sequence
    for (int i = 0; i < n; ++i) {
        Unit& u = c->units[(size_t)layer * c->n_slots + in[i].slot];
        const Sizes& z = sz[i];
        for (int ci = 0; ci < c->n_caches; ++ci) {
            CacheBufs& cb = u.cache[ci];
            int* idx = u.idx[ci];
            float* scores = u.scores + (size_t)ci * c->Hkv * c->score_stride;
            sj.push_back(SelectJob{scores, idx, c->score_stride, cb.pos[cb.cur], c->cap[ci], z.mc[ci], (int)u.tokens_seen,
                                   c->start_size, c->accumulate ? cb.carried[cb.cur] : nullptr,
                                   z.nc[ci], z.kept[ci], c->cap[ci], z.forced_from[ci]});
            cj.push_back(CompactJob{cb.K[cb.cur], cb.V[cb.cur], cb.pos[cb.cur],
                                    cb.K[cb.cur ^ 1], cb.V[cb.cur ^ 1], cb.pos[cb.cur ^ 1], idx, z.mc[ci],
                                    c->accumulate ? scores : nullptr, c->score_stride,
                                    c->accumulate ? cb.carried[cb.cur ^ 1] : nullptr, c->cap[ci], z.kept[ci],
                                    c->shift ? cb.Kraw[cb.cur] : nullptr, c->shift ? cb.Kraw[cb.cur ^ 1] : nullptr,
                                    in[i].K, in[i].V, (int)u.tokens_seen});       // the un-rotated chunk keys are what is gathered
            gather_bytes += (size_t)c->Hkv * z.kept[ci] * c->D * c->elt * 2;
        }
    }
    const int n_jobs = (int)sj.size();
    // Small steps (a few MB to move) are latency-bound: one cluster launch does a3 and a4.  Large steps want every
    // SM streaming rows, which the clusters (idle while their first CTA selects) cannot give: two launches.
    int n_most = 0;
    for (const SelectJob& j : sj) n_most = j.n > n_most ? j.n : n_most;
    if (!c->shift && !c->accumulate && gather_bytes <= ((size_t)8 << 20) * (size_t)n &&
        select_compact_fits(n_most, c->D * c->elt)) {
        // one launch does both (timed under the compaction id)
        LaunchTimer t(c, CITRUS_KERNEL_COMPACT, st);
        e = select_compact(sj.data(), cj.data(), n_jobs, c->Hkv, c->D * c->elt, c->elt, produced ? 0 : 1, c->layerwise ? 1 : 0, st);
        if (e != cudaSuccess) { if (beside) join_a1(c, st); return cuda_rc(e); }
    } else {
        {
            LaunchTimer t(c, CITRUS_KERNEL_SELECT, st);
            e = select_topk(sj.data(), n_jobs, c->Hkv, c->layerwise ? 1 : 0, st);
        }
        if (e != cudaSuccess) { if (beside) join_a1(c, st); return cuda_rc(e); }
        {
            LaunchTimer t(c, CITRUS_KERNEL_COMPACT, st);
            e = compact_kv(cj.data(), n_jobs, c->Hkv, c->D * c->elt, c->shift ? &c->rope : nullptr, c->elt, st);
        }
        if (e != cudaSuccess) { if (beside) join_a1(c, st); return cuda_rc(e); }
    }
    // the caller's stream continues behind a1: `out` is complete in stream order, and the next step's compaction, which
    // overwrites the cache buffer this a1 reads, comes after it
    if (beside && (e = join_a1(c, st)) != cudaSuccess) return cuda_rc(e);

    for (int i = 0; i < n; ++i) {
        Unit& u = c->units[(size_t)layer * c->n_slots + in[i].slot];
        for (int ci = 0; ci < c->n_caches; ++ci) {
            u.cache[ci].cur ^= 1;
            u.last_n[ci] = sz[i].nc[ci]; u.last_kept[ci] = sz[i].kept[ci]; u.last_m[ci] = sz[i].mc[ci];
            u.m[ci] = sz[i].kept[ci];
        }
        u.has_step = true;
        u.tokens_seen += in[i].L;
    }
    return CITRUS_OK;
}

int run_step(citrus_ctx* c, int layer, int slot, const void* Qc, const void* Kc, const void* Vc, int L,
             const void* Qi, int nI, void* out, cudaStream_t st, int lane = -1, bool inputs_ordered = false) {
    StepIn in{slot, Qc, Kc, Vc, Qi, L, nI, out};
    return run_steps(c, layer, 1, &in, nullptr, st, lane, inputs_ordered);
}

}  // namespace

int citrus::sm_count() {
    static std::mutex mu;
    static int count[DeviceOnce::kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= DeviceOnce::kMaxDevices) { cudaGetLastError(); return 148; }
    std::lock_guard<std::mutex> lk(mu);
    if (count[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) { cudaGetLastError(); n = 148; }
        count[dev] = n;
    }
    return count[dev];
}

void citrus::before_launch(cudaStream_t s) {
    if (t_pending_start != nullptr) {
        cudaEventRecord(t_pending_start, s);
        t_pending_start = nullptr;
    }
}

extern "C" {

int citrus_create(citrus_handle* out, int layers, int q_heads, int kv_heads, int head_dim,
                  int budget_k, int chunk_s, unsigned mode) {
    if (out == nullptr) return CITRUS_ERR_INVALID_ARG;
    *out = nullptr;
    if (layers < 1 || q_heads < 1 || kv_heads < 1 || budget_k < 1 || chunk_s < 1) return CITRUS_ERR_INVALID_ARG;
    if (mode & ~(0xFu | 0xFFFF00u | 0xF000000u | CITRUS_MODE_ACCUMULATE | CITRUS_MODE_DEFERRED_LM | CITRUS_MODE_POSITION_SHIFT)) return CITRUS_ERR_INVALID_ARG;
    if ((mode & CITRUS_MODE_POSITION_SHIFT) && (mode & CITRUS_MODE_DEFERRED_LM)) return CITRUS_ERR_INVALID_ARG;
    if ((mode & CITRUS_MODE_DEFERRED_LM) && !(mode & (CITRUS_MODE_INDIVIDUAL | CITRUS_MODE_STANDARD))) return CITRUS_ERR_INVALID_ARG;
    if ((mode & CITRUS_MODE_STANDARD) && (mode & CITRUS_MODE_INDIVIDUAL)) return CITRUS_ERR_INVALID_ARG;
    if (q_heads % kv_heads != 0) return CITRUS_ERR_SHAPE;
    if (head_dim != 64 && head_dim != 128) return CITRUS_ERR_UNSUPPORTED;
    const bool fp32 = (mode & CITRUS_MODE_FP32) != 0;
    if (!fp32 && head_dim != 128) return CITRUS_ERR_UNSUPPORTED;
    if ((long long)budget_k + chunk_s + ((mode & CITRUS_MODE_DEFERRED_LM) ? chunk_s : 0) > CITRUS_MAX_CANDIDATES) return CITRUS_ERR_UNSUPPORTED;
    if ((int)((mode >> 24) & 0xFu) > budget_k) return CITRUS_ERR_SHAPE;

    citrus_ctx* c = new (std::nothrow) citrus_ctx();
    if (c == nullptr) return CITRUS_ERR_NOMEM;
    if (cudaGetDevice(&c->device) != cudaSuccess) { cudaGetLastError(); delete c; return CITRUS_ERR_CUDA; }
    c->layers = layers; c->Hq = q_heads; c->Hkv = kv_heads; c->D = head_dim; c->k = budget_k; c->ls = chunk_s;
    c->individual = (mode & CITRUS_MODE_INDIVIDUAL) != 0;
    c->standard = (mode & CITRUS_MODE_STANDARD) != 0;
    c->fp32 = fp32;
    c->layerwise = (mode & CITRUS_MODE_LAYERWISE) != 0;
    c->lm_window = (int)((mode >> 8) & 0xFFFFu);
    c->start_size = (int)((mode >> 24) & 0xFu);
    c->accumulate = (mode & CITRUS_MODE_ACCUMULATE) != 0;
    c->deferred = (mode & CITRUS_MODE_DEFERRED_LM) != 0;
    c->shift = (mode & CITRUS_MODE_POSITION_SHIFT) != 0;
    for (int d = 0; d < 64; ++d) c->rope.theta[d] = std::pow(10000.0, -2.0 * d / head_dim);
    c->cap[0] = budget_k + (c->deferred ? chunk_s : 0);
    c->cap[1] = budget_k;
    c->elt = fp32 ? 4 : 2;
    c->n_caches = c->individual ? 2 : 1;
    c->score_stride = (c->cap[0] + chunk_s + 3) & ~3;
    c->use_tc = !fp32 && head_dim == 128;
    int rc = dev_alloc(c, (void**)&c->status, sizeof(int), true, true);
    if (rc == CITRUS_OK && c->use_tc && tc_init() != cudaSuccess) rc = CITRUS_ERR_UNSUPPORTED;
    if (rc == CITRUS_OK && c->shift && cudaEventCreateWithFlags(&c->shift_done, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        rc = CITRUS_ERR_CUDA;
    }
    if (rc == CITRUS_OK && c->use_tc && !c->individual &&
        (cudaStreamCreateWithFlags(&c->a1_stream, cudaStreamNonBlocking) != cudaSuccess ||
         cudaEventCreateWithFlags(&c->a1_fork, cudaEventDisableTiming) != cudaSuccess ||
         cudaEventCreateWithFlags(&c->a1_done, cudaEventDisableTiming) != cudaSuccess)) {
        cudaGetLastError();
        rc = CITRUS_ERR_CUDA;
    }
    if (rc == CITRUS_OK && c->shift) {
        const size_t row = (size_t)head_dim * c->elt;
        rc = dev_alloc(c, &c->rotQ, (size_t)chunk_s * q_heads * row, false, true);
        if (rc == CITRUS_OK) rc = dev_alloc(c, &c->rotK, (size_t)chunk_s * kv_heads * row, false, true);
        if (rc == CITRUS_OK) rc = dev_alloc(c, &c->rotQi, (size_t)CITRUS_MAX_INSTR * q_heads * row, false, true);
    }
    if (rc == CITRUS_OK) rc = alloc_units(c);
    if (rc != CITRUS_OK) { if (c->shift_done) cudaEventDestroy(c->shift_done); free_all(c); delete c; return rc; }
    {
        std::lock_guard<std::mutex> lk(g_mu);
        g_live.insert(c);
        g_dead.erase(c);
    }
    *out = c;
    return CITRUS_OK;
}

int citrus_set_batch(citrus_handle h, int n_seq) {
    if (h == nullptr || !is_live(h)) return CITRUS_ERR_INVALID_ARG;
    if (n_seq < 1) return CITRUS_ERR_INVALID_ARG;
    if (h->used) return CITRUS_ERR_STATE;
    if (n_seq != h->n_slots) {
        const int old = h->n_slots;
        free_units(h);
        h->n_slots = n_seq;
        int rc = alloc_units(h);
        if (rc != CITRUS_OK) {           // fall back to the geometry that worked before
            free_units(h);
            h->n_slots = old;
            if (alloc_units(h) != CITRUS_OK) free_units(h);
            return rc;
        }
    }
    if (h->n_slots > 1) return make_lanes(h);
    return CITRUS_OK;
}

int citrus_set_batch_lanes(citrus_handle h, int n_lanes) {
    if (h == nullptr || !is_live(h)) return CITRUS_ERR_INVALID_ARG;
    if (n_lanes < 0 || n_lanes > citrus_ctx::kMaxLanes) return CITRUS_ERR_INVALID_ARG;
    h->lanes_wanted = n_lanes;
    return CITRUS_OK;
}

int citrus_set_attention_beside(citrus_handle h, int max_ctas) {
    if (h == nullptr || !is_live(h) || max_ctas < 0) return CITRUS_ERR_INVALID_ARG;
    h->a1_cap = max_ctas;
    return CITRUS_OK;
}

int citrus_set_inputs_ready(citrus_handle h, int ready) {
    if (h == nullptr || !is_live(h)) return CITRUS_ERR_INVALID_ARG;
    h->inputs_ready = ready != 0;
    return CITRUS_OK;
}

int citrus_set_rope_base(citrus_handle h, double base) {
    if (h == nullptr || !is_live(h) || !(base > 1.0)) return CITRUS_ERR_INVALID_ARG;
    if (!h->shift || h->used) return CITRUS_ERR_STATE;
    for (int d = 0; d < 64; ++d) h->rope.theta[d] = std::pow(base, -2.0 * d / h->D);
    return CITRUS_OK;
}

int citrus_reset(citrus_handle h) {
    if (h == nullptr || !is_live(h)) return CITRUS_ERR_INVALID_ARG;
    for (Unit& u : h->units) {
        u.tokens_seen = 0; u.has_step = false;
        for (int ci = 0; ci < 2; ++ci) u.m[ci] = u.last_n[ci] = u.last_kept[ci] = u.last_m[ci] = 0;
    }
    return CITRUS_OK;
}

int citrus_process_chunk_slot(citrus_handle h, int layer, int seq_slot,
                              const void* Q_chunk, const void* K_chunk, const void* V_chunk, int n_tokens,
                              const void* Q_instr, int n_instr, void* out, citrus_stream_t stream) {
    int rc = check_process_args(h, layer, seq_slot, Q_chunk, K_chunk, V_chunk, n_tokens, Q_instr, n_instr, out);
    if (rc) return rc;
    if (!aligned16(Q_chunk) || !aligned16(K_chunk) || !aligned16(V_chunk) || !aligned16(Q_instr) || !aligned16(out))
        return CITRUS_ERR_ALIGN;
    return run_step(h, layer, seq_slot, Q_chunk, K_chunk, V_chunk, n_tokens, Q_instr, n_instr, out,
                    reinterpret_cast<cudaStream_t>(stream));
}

int citrus_process_chunk(citrus_handle h, int layer,
                         const void* Q_chunk, const void* K_chunk, const void* V_chunk, int n_tokens,
                         const void* Q_instr, int n_instr, void* out, citrus_stream_t stream) {
    return citrus_process_chunk_slot(h, layer, 0, Q_chunk, K_chunk, V_chunk, n_tokens, Q_instr, n_instr, out, stream);
}

int citrus_process_chunk_batch(citrus_handle h, int layer, int n_active, const int* seq_slot, const int* tok_offset,
                               const void* Q, const void* K, const void* V, const int* instr_offset,
                               const void* Q_instr, void* out, citrus_stream_t stream) {
    if (h == nullptr || !is_live(h)) return CITRUS_ERR_INVALID_ARG;
    if (n_active < 1 || !seq_slot || !tok_offset || !instr_offset || !Q || !K || !V || !Q_instr || !out) return CITRUS_ERR_INVALID_ARG;
    if (layer < 0 || layer >= h->layers) return CITRUS_ERR_LAYER;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(Q_instr) || !aligned16(out)) return CITRUS_ERR_ALIGN;
    std::set<int> seen;
    for (int i = 0; i < n_active; ++i) {
        const int L = tok_offset[i + 1] - tok_offset[i], nI = instr_offset[i + 1] - instr_offset[i];
        if (seq_slot[i] < 0 || seq_slot[i] >= h->n_slots || !seen.insert(seq_slot[i]).second) return CITRUS_ERR_INVALID_ARG;
        if (tok_offset[i] < 0 || instr_offset[i] < 0) return CITRUS_ERR_INVALID_ARG;
        if (L < 1 || L > h->ls || nI < 1 || nI > CITRUS_MAX_INSTR) return CITRUS_ERR_SHAPE;
        const Unit& u = h->units[(size_t)layer * h->n_slots + seq_slot[i]];
        if (u.tokens_seen + L > 0x7fffffffLL) return CITRUS_ERR_SHAPE;
    }
    const size_t qrow = (size_t)h->Hq * h->D * h->elt, krow = (size_t)h->Hkv * h->D * h->elt;   // multiples of 16 bytes
    cudaStream_t caller = reinterpret_cast<cudaStream_t>(stream);
    // One grid over all sequences (tensor-core path, no position shift; unless citrus_set_batch_lanes asked for the
    // per-sequence launches): every kernel of the step is launched once, its work items are those of all sequences -
    // each sequence's longest sweeps first, the longest sequence first - and a sequence's rows and caches are
    // offsets inside the packed tensors and the layer's cache tensors.
    if (n_active > 1 && h->use_tc && !h->shift && h->lanes_wanted == 0) {
        std::vector<int> order(n_active);
        for (int i = 0; i < n_active; ++i) order[i] = i;
        std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
            return tok_offset[a + 1] - tok_offset[a] > tok_offset[b + 1] - tok_offset[b];
        });
        const char* q0 = reinterpret_cast<const char*>(Q) + qrow * tok_offset[0];
        const char* k0 = reinterpret_cast<const char*>(K) + krow * tok_offset[0];
        const char* v0 = reinterpret_cast<const char*>(V) + krow * tok_offset[0];
        const char* qi0 = reinterpret_cast<const char*>(Q_instr) + qrow * instr_offset[0];
        char* o0 = reinterpret_cast<char*>(out) + qrow * tok_offset[0];
        PackedIn packed{q0, k0, v0, qi0, o0, tok_offset[n_active] - tok_offset[0], instr_offset[n_active] - instr_offset[0]};
        for (int first = 0; first < n_active; first += kTcMaxBatch) {
            const int cnt = std::min(kTcMaxBatch, n_active - first);
            std::vector<StepIn> in(cnt);
            for (int j = 0; j < cnt; ++j) {
                const int i = order[first + j];
                in[j] = StepIn{seq_slot[i],
                               reinterpret_cast<const char*>(Q) + qrow * tok_offset[i], reinterpret_cast<const char*>(K) + krow * tok_offset[i],
                               reinterpret_cast<const char*>(V) + krow * tok_offset[i], reinterpret_cast<const char*>(Q_instr) + qrow * instr_offset[i],
                               tok_offset[i + 1] - tok_offset[i], instr_offset[i + 1] - instr_offset[i],
                               reinterpret_cast<char*>(out) + qrow * tok_offset[i]};
            }
            int rc = run_steps(h, layer, cnt, in.data(), &packed, caller);
            if (rc != CITRUS_OK) return rc;                  // only a launch failure can get here; earlier groups have advanced
        }
        return CITRUS_OK;
    }
    // Lanes (position-shift and fp32 contexts, or on request): only where a step is small (its attention items make a
    // few waves over the SMs at most), which is where a sequence's kernels wait for each other more than they compute.
    // Per-launch timing wants one stream, so profiled runs stay in the caller's stream; a position-shift context needs
    // its per-lane embedding scratch.
    int n_lanes = 1;
    if (n_active > 1 && h->lane_fork != nullptr && !h->profiling &&
        (!h->shift || h->laneRotQi[citrus_ctx::kMaxLanes - 1] != nullptr)) {
        int items = 0;
        for (int i = 0; i < n_active; ++i) items = std::max(items, (tok_offset[i + 1] - tok_offset[i] + 127) / 128 * h->Hq);
        // measured: four lanes pay up to one wave of attention items per sequence, two up to about three waves
        n_lanes = h->lanes_wanted > 0 ? h->lanes_wanted : (items <= sm_count() ? 4 : (items <= 3 * sm_count() ? 2 : 1));
        n_lanes = std::min(n_lanes, n_active);
    }
    if (n_lanes > 1) {
        cudaError_t e = cudaEventRecord(h->lane_fork, caller);
        for (int l = 0; l < n_lanes && e == cudaSuccess; ++l) e = cudaStreamWaitEvent(h->lane[l], h->lane_fork, 0);
        if (e != cudaSuccess) return cuda_rc(e);
    }
    int first_rc = CITRUS_OK;
    for (int i = 0; i < n_active; ++i) {
        cudaStream_t st_i = n_lanes > 1 ? h->lane[i % n_lanes] : caller;
        const char* q = reinterpret_cast<const char*>(Q) + qrow * tok_offset[i];
        const char* k = reinterpret_cast<const char*>(K) + krow * tok_offset[i];
        const char* v = reinterpret_cast<const char*>(V) + krow * tok_offset[i];
        const char* qi = reinterpret_cast<const char*>(Q_instr) + qrow * instr_offset[i];
        char* o = reinterpret_cast<char*>(out) + qrow * tok_offset[i];
        int rc = run_step(h, layer, seq_slot[i], q, k, v, tok_offset[i + 1] - tok_offset[i], qi,
                          instr_offset[i + 1] - instr_offset[i], o, st_i, n_lanes > 1 ? i % n_lanes : -1,
                          /*inputs_ordered=*/n_lanes > 1);    // a lane starts behind an event of the caller's stream
        if (rc != CITRUS_OK) { first_rc = rc; break; }   // only a launch failure can get here; earlier sequences have advanced
    }
    if (n_lanes > 1) {
        // the caller's stream continues only after every lane (also after a failure: nothing is left running unjoined)
        for (int l = 0; l < n_lanes; ++l) {
            cudaError_t e = cudaEventRecord(h->lane_done[l], h->lane[l]);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(caller, h->lane_done[l], 0);
            if (e != cudaSuccess && first_rc == CITRUS_OK) first_rc = cuda_rc(e);
        }
    }
    return first_rc;
}

int citrus_process_chunk_host(citrus_handle h, int layer, int seq_slot,
                              const void* Qh, const void* Kh, const void* Vh, int n_tokens,
                              const void* Qih, int n_instr, void* out_h, citrus_stream_t stream) {
    int rc = check_process_args(h, layer, seq_slot, Qh, Kh, Vh, n_tokens, Qih, n_instr, out_h);
    if (rc) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t qrow = (size_t)h->Hq * h->D * h->elt, krow = (size_t)h->Hkv * h->D * h->elt;
    if (h->stQ == nullptr) {
        if ((rc = dev_alloc(h, &h->stQ, qrow * h->ls, false, true))) return rc;
        if ((rc = dev_alloc(h, &h->stOut, qrow * h->ls, false, true))) return rc;
        if ((rc = dev_alloc(h, &h->stK, krow * h->ls, false, true))) return rc;
        if ((rc = dev_alloc(h, &h->stV, krow * h->ls, false, true))) return rc;
        if ((rc = dev_alloc(h, &h->stQi, qrow * CITRUS_MAX_INSTR, false, true))) return rc;
    }
    cudaError_t e;
    if ((e = cudaMemcpyAsync(h->stQ, Qh, qrow * n_tokens, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_rc(e);
    if ((e = cudaMemcpyAsync(h->stK, Kh, krow * n_tokens, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_rc(e);
    if ((e = cudaMemcpyAsync(h->stV, Vh, krow * n_tokens, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_rc(e);
    if (n_instr > 0 && (e = cudaMemcpyAsync(h->stQi, Qih, qrow * n_instr, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_rc(e);
    rc = run_step(h, layer, seq_slot, h->stQ, h->stK, h->stV, n_tokens, h->stQi, n_instr, h->stOut, st, -1, true);
    if (rc) return rc;
    if ((e = cudaMemcpyAsync(out_h, h->stOut, qrow * n_tokens, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return cuda_rc(e);
    return cuda_rc(cudaStreamSynchronize(st));
}

int citrus_process_document_host(citrus_handle h, int layer, int seq_slot,
                                 const void* Qh, const void* Kh, const void* Vh, long long n_tokens,
                                 const void* Qih, int n_instr, void* out_h, citrus_stream_t stream) {
    if (h == nullptr || !is_live(h)) return CITRUS_ERR_INVALID_ARG;
    if (n_tokens < 1 || n_tokens > 0x7fffffffLL) return CITRUS_ERR_SHAPE;
    const int first = (int)(n_tokens < h->ls ? n_tokens : h->ls);
    int rc = check_process_args(h, layer, seq_slot, Qh, Kh, Vh, first, Qih, n_instr, out_h);
    if (rc) return rc;
    if (n_instr < 1) return CITRUS_ERR_SHAPE;
    {
        const Unit& u = h->units[(size_t)layer * h->n_slots + seq_slot];
        if (u.tokens_seen + n_tokens > 0x7fffffffLL) return CITRUS_ERR_SHAPE;
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t qrow = (size_t)h->Hq * h->D * h->elt, krow = (size_t)h->Hkv * h->D * h->elt;
    // Copies move kDocBlock chunks at a time: a few large transfers use the link better than many small ones.
    constexpr int kDocBlock = 4;
    const size_t blk_rows = (size_t)h->ls * kDocBlock;
    cudaError_t e = cudaSuccess;
    if (h->s_in == nullptr) {
        for (int b = 0; b < 2; ++b) {
            if ((rc = dev_alloc(h, &h->docQ[b], qrow * blk_rows, false, true))) return rc;
            if ((rc = dev_alloc(h, &h->docOut[b], qrow * blk_rows, false, true))) return rc;
            if ((rc = dev_alloc(h, &h->docK[b], krow * blk_rows, false, true))) return rc;
            if ((rc = dev_alloc(h, &h->docV[b], krow * blk_rows, false, true))) return rc;
        }
        if ((rc = dev_alloc(h, &h->docQi, qrow * CITRUS_MAX_INSTR, false, true))) return rc;
        e = cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking);
        for (int b = 0; b < 2 && e == cudaSuccess; ++b) {
            e = cudaEventCreateWithFlags(&h->ev_in[b], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_step[b], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_out[b], cudaEventDisableTiming);
        }
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_qi, cudaEventDisableTiming);
        if (e != cudaSuccess) return cuda_rc(e);
    }
    const char *q = reinterpret_cast<const char*>(Qh), *k = reinterpret_cast<const char*>(Kh), *v = reinterpret_cast<const char*>(Vh);
    char* o = reinterpret_cast<char*>(out_h);
    // the copy streams start behind whatever the caller's stream already holds
    if ((e = cudaEventRecord(h->ev_qi, st)) != cudaSuccess) return cuda_rc(e);
    if ((e = cudaStreamWaitEvent(h->s_in, h->ev_qi, 0)) != cudaSuccess) return cuda_rc(e);
    if ((e = cudaStreamWaitEvent(h->s_out, h->ev_qi, 0)) != cudaSuccess) return cuda_rc(e);
    if ((e = cudaMemcpyAsync(h->docQi, Qih, qrow * n_instr, cudaMemcpyHostToDevice, h->s_in)) != cudaSuccess) return cuda_rc(e);
    const long long n_chunks = (n_tokens + h->ls - 1) / h->ls;
    const long long n_blocks = (n_chunks + kDocBlock - 1) / kDocBlock;
    for (long long blk = 0; blk < n_blocks && rc == CITRUS_OK && e == cudaSuccess; ++blk) {
        const int b = (int)(blk & 1);
        const long long t0 = blk * (long long)blk_rows;
        const long long rows = n_tokens - t0 < (long long)blk_rows ? n_tokens - t0 : (long long)blk_rows;
        // inputs of the block into set b, once the steps that last read the set (block blk-2) are done
        if (blk >= 2 && (e = cudaStreamWaitEvent(h->s_in, h->ev_step[b], 0)) != cudaSuccess) break;
        if ((e = cudaMemcpyAsync(h->docQ[b], q + qrow * t0, qrow * rows, cudaMemcpyHostToDevice, h->s_in)) != cudaSuccess) break;
        if ((e = cudaMemcpyAsync(h->docK[b], k + krow * t0, krow * rows, cudaMemcpyHostToDevice, h->s_in)) != cudaSuccess) break;
        if ((e = cudaMemcpyAsync(h->docV[b], v + krow * t0, krow * rows, cudaMemcpyHostToDevice, h->s_in)) != cudaSuccess) break;
        if ((e = cudaEventRecord(h->ev_in[b], h->s_in)) != cudaSuccess) break;
        // the block's steps, once its inputs are there and the set's output buffer has been copied back (block blk-2)
        if ((e = cudaStreamWaitEvent(st, h->ev_in[b], 0)) != cudaSuccess) break;
        if (blk >= 2 && (e = cudaStreamWaitEvent(st, h->ev_out[b], 0)) != cudaSuccess) break;
        for (long long r0 = 0; r0 < rows && rc == CITRUS_OK; r0 += h->ls) {
            const int L = (int)(rows - r0 < h->ls ? rows - r0 : h->ls);
            const bool last = t0 + r0 + L == n_tokens;
            const bool with_instr = !h->standard || last;
            rc = run_step(h, layer, seq_slot, (char*)h->docQ[b] + qrow * r0, (char*)h->docK[b] + krow * r0, (char*)h->docV[b] + krow * r0, L,
                          with_instr ? h->docQi : nullptr, with_instr ? n_instr : 0, (char*)h->docOut[b] + qrow * r0, st, -1, true);
        }
        if (rc != CITRUS_OK) break;
        if ((e = cudaEventRecord(h->ev_step[b], st)) != cudaSuccess) break;
        // its output back to the host
        if ((e = cudaStreamWaitEvent(h->s_out, h->ev_step[b], 0)) != cudaSuccess) break;
        if ((e = cudaMemcpyAsync(o + qrow * t0, h->docOut[b], qrow * rows, cudaMemcpyDeviceToHost, h->s_out)) != cudaSuccess) break;
        if ((e = cudaEventRecord(h->ev_out[b], h->s_out)) != cudaSuccess) break;
    }
    // whatever was enqueued is drained before returning, also after an error
    cudaError_t e1 = cudaStreamSynchronize(h->s_in), e2 = cudaStreamSynchronize(st), e3 = cudaStreamSynchronize(h->s_out);
    if (rc != CITRUS_OK) return rc;
    if (e != cudaSuccess) return cuda_rc(e);
    if (e1 != cudaSuccess) return cuda_rc(e1);
    if (e2 != cudaSuccess) return cuda_rc(e2);
    return cuda_rc(e3);
}

int citrus_cache_view(citrus_handle h, int layer, int which, int seq_slot,
                      const void** K, const void** V, const int** positions, int* n_rows) {
    if (h == nullptr || !is_live(h)) return CITRUS_ERR_INVALID_ARG;
    if (layer < 0 || layer >= h->layers) return CITRUS_ERR_LAYER;
    if (which < 0 || which >= h->n_caches || seq_slot < 0 || seq_slot >= h->n_slots) return CITRUS_ERR_INVALID_ARG;
    if (h->units.empty()) return CITRUS_ERR_STATE;
    const Unit& u = h->units[(size_t)layer * h->n_slots + seq_slot];
    const CacheBufs& cb = u.cache[which];
    if (K) *K = h->shift ? cb.Kraw[cb.cur] : cb.K[cb.cur];
    if (V) *V = cb.V[cb.cur];
    if (positions) *positions = cb.pos[cb.cur];
    if (n_rows) *n_rows = u.m[which];
    return CITRUS_OK;
}

int citrus_intersection_ratio(citrus_handle h, int layer, int seq_slot, float* ratio_dev, citrus_stream_t stream) {
    if (h == nullptr || !is_live(h) || ratio_dev == nullptr) return CITRUS_ERR_INVALID_ARG;
    if (layer < 0 || layer >= h->layers) return CITRUS_ERR_LAYER;
    if (seq_slot < 0 || seq_slot >= h->n_slots) return CITRUS_ERR_INVALID_ARG;
    if (!h->individual || h->units.empty()) return CITRUS_ERR_STATE;
    const Unit& u = h->units[(size_t)layer * h->n_slots + seq_slot];
    if (u.m[0] < 1 || u.m[1] < 1) return CITRUS_ERR_STATE;
    const CacheBufs &lm = u.cache[0], &in = u.cache[1];
    return cuda_rc(intersection_ratio(lm.pos[lm.cur], h->cap[0], u.m[0], in.pos[in.cur], h->cap[1], u.m[1], h->Hkv,
                                      ratio_dev, reinterpret_cast<cudaStream_t>(stream)));
}

int citrus_step_view(citrus_handle h, int layer, int which, int seq_slot,
                     const float** scores, int* score_stride, const int** idx,
                     int* n_candidates, int* n_kept, int* m_before) {
    if (h == nullptr || !is_live(h)) return CITRUS_ERR_INVALID_ARG;
    if (layer < 0 || layer >= h->layers) return CITRUS_ERR_LAYER;
    if (which < 0 || which >= h->n_caches || seq_slot < 0 || seq_slot >= h->n_slots) return CITRUS_ERR_INVALID_ARG;
    if (h->units.empty()) return CITRUS_ERR_STATE;
    const Unit& u = h->units[(size_t)layer * h->n_slots + seq_slot];
    if (!u.has_step) return CITRUS_ERR_STATE;
    if (scores) *scores = u.scores + (size_t)which * h->Hkv * h->score_stride;
    if (score_stride) *score_stride = h->score_stride;
    if (idx) *idx = u.idx[which];
    if (n_candidates) *n_candidates = u.last_n[which];
    if (n_kept) *n_kept = u.last_kept[which];
    if (m_before) *m_before = u.last_m[which];
    return CITRUS_OK;
}

int citrus_profile(citrus_handle h, int enable) {
    if (h == nullptr || !is_live(h)) return CITRUS_ERR_INVALID_ARG;
    h->profiling = enable != 0;
    return CITRUS_OK;
}

int citrus_profile_read(citrus_handle h, double* ms, long long* launches) {
    if (h == nullptr || !is_live(h) || ms == nullptr || launches == nullptr) return CITRUS_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return CITRUS_ERR_CUDA; }
    for (int i = 0; i < CITRUS_N_KERNELS; ++i) { ms[i] = 0.0; launches[i] = 0; }
    for (const citrus_ctx::Timed& t : h->timed) {
        float f = 0.f;
        if (cudaEventElapsedTime(&f, t.a, t.b) == cudaSuccess) { ms[t.id] += f; launches[t.id] += 1; }
        else cudaGetLastError();
        cudaEventDestroy(t.a);
        cudaEventDestroy(t.b);
    }
    h->timed.clear();
    return CITRUS_OK;
}

int citrus_poll_status(citrus_handle h) {
    if (h == nullptr || !is_live(h)) return CITRUS_ERR_INVALID_ARG;
    int v = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return CITRUS_ERR_CUDA; }
    if (cudaMemcpy(&v, h->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return CITRUS_ERR_CUDA; }
    if (v != 0 && cudaMemset(h->status, 0, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return CITRUS_ERR_CUDA; }
    return v == 0 ? CITRUS_OK : CITRUS_ERR_TIMEOUT;
}

int citrus_debug_expire_wait(citrus_handle h, unsigned long long limit_ns, citrus_stream_t stream) {
    if (h == nullptr || !is_live(h)) return CITRUS_ERR_INVALID_ARG;
    if (limit_ns < 1 || limit_ns > 100000000ull) return CITRUS_ERR_INVALID_ARG;       // at most 0.1 s
    return cuda_rc(tc_expire_wait(h->status, limit_ns, reinterpret_cast<cudaStream_t>(stream)));
}

int citrus_destroy(citrus_handle h) {
    if (h == nullptr) return CITRUS_OK;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        if (g_live.count(h) == 0) return g_dead.count(h) ? CITRUS_ERR_STATE : CITRUS_ERR_INVALID_ARG;
        g_live.erase(h);
        g_dead.insert(h);
    }
    cudaDeviceSynchronize();
    for (const citrus_ctx::Timed& t : h->timed) { cudaEventDestroy(t.a); cudaEventDestroy(t.b); }
    free_copy_streams(h);
    free_all(h);
    cudaGetLastError();
    delete h;
    return CITRUS_OK;
}

const char* citrus_strerror(int code) {
    switch (code) {
        case CITRUS_OK: return "ok";
        case CITRUS_ERR_INVALID_ARG: return "invalid argument";
        case CITRUS_ERR_SHAPE: return "size out of range";
        case CITRUS_ERR_ALIGN: return "pointer not 16-byte aligned";
        case CITRUS_ERR_LAYER: return "layer index out of range";
        case CITRUS_ERR_STATE: return "call not valid in this state";
        case CITRUS_ERR_NOMEM: return "out of device memory";
        case CITRUS_ERR_CUDA: return "CUDA runtime error";
        case CITRUS_ERR_TIMEOUT: return "a bounded device wait expired";
        case CITRUS_ERR_UNSUPPORTED: return "configuration not supported";
        default: return "unknown error";
    }
}

}  // extern "C"
