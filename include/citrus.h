/*
 * citrus.h -- C ABI of the chunked instruction-aware state eviction library
 * (CItruS, arXiv 2406.12018) for NVIDIA B200 (sm_100a).
 *
 * One call of citrus_process_chunk performs, for one decoder layer and one
 * document chunk s of L <= l_s tokens, the four steps of the eviction loop:
 *
 *   a1  attention of the chunk's queries over [retained cache ; chunk], causal
 *       inside the chunk (Section 4.1, step 1 of the chunked eviction process);
 *   a2  importance of every candidate state c in [cache ; chunk]:
 *       Imp(s', c) of Eq. 1 -- the softmax attention c receives, summed over the
 *       scoring tokens s' and over the query heads of c's KV group.  The scoring
 *       tokens are the instruction text I for the instruction-aware cache
 *       (Section 4.2) and the chunk's own last w queries for the language-
 *       modelling cache of the individual design (Section 4.1, Eq. 1 with s = chunk);
 *   a3  top-k selection (Eq. 2-3; Eq. 4-5 for the instruction cache): keep the
 *       budget_k candidates with the highest score, the lower position winning
 *       exact ties, kept indices in ascending order;
 *   a4  compaction of K, V and original positions of the kept candidates into
 *       the new cache (the cache C-hat of Eq. 3 with the chunk's states put in).
 *
 * Scores are the SUM form of Eq. 1 (|s'| * G times the printed mean), which
 * selects the same states.  The softmax of a2 runs over exactly the n = m + L
 * candidates (m = rows currently retained).
 *
 * Conventions
 *   - All tensor arguments are DEVICE pointers unless a function says "host".
 *   - Token-major, densely packed: Q [tokens, q_heads, head_dim],
 *     K/V [tokens, kv_heads, head_dim]; query head h uses KV head h / (q_heads/kv_heads).
 *   - Element type is bf16 (default) or fp32 (CITRUS_MODE_FP32).
 *   - Pointers must be 16-byte aligned.  The library never retains caller
 *     pointers after the stream work of the call has completed.
 *   - Every function returns 0 on success or a negative CITRUS_ERR_* code; none
 *     aborts, throws, traps or prints.  A call that fails leaves all cache state
 *     as it was.
 *   - Work is enqueued on the caller's stream; no call synchronises the device
 *     except citrus_create / citrus_destroy / citrus_poll_status and the *_host
 *     variant (which waits for its own copies).
 */
#ifndef CITRUS_H_
#define CITRUS_H_

#ifdef __cplusplus
extern "C" {
#endif

typedef struct citrus_ctx* citrus_handle;
/* Same object as the CUDA runtime's cudaStream_t (NULL = legacy default stream). */
typedef struct CUstream_st* citrus_stream_t;

/* mode bit-field of citrus_create */
#define CITRUS_MODE_SHARED      0u        /* one cache, evicted by Imp(I, c)         (Section 4.2, shared cache)   */
#define CITRUS_MODE_INDIVIDUAL  1u        /* LM cache C + instruction cache C^I       (Section 4.2, Eq. 4-5)        */
#define CITRUS_MODE_FP32        2u        /* tensors are fp32 (default bf16)                                         */
#define CITRUS_MODE_LAYERWISE   4u        /* one index set per layer from head-summed scores (Section 4.1, last par.) */
#define CITRUS_MODE_STANDARD    8u        /* standard chunked eviction: one cache scored by the chunk itself (Section 4.1); a call
                                             that does pass instruction queries is scored by them instead (the final eviction
                                             "with the instruction text as a new chunk") */
#define CITRUS_MODE_START_SIZE(n) (((unsigned)(n) & 0xFu) << 24)   /* always keep the first n tokens (appendix on
                                             initial tokens; the paper's variant uses 4, its main setting 0); n <= budget_k */
#define CITRUS_MODE_LM_WINDOW(w) (((unsigned)(w) & 0xFFFFu) << 8)   /* w scoring queries for C; 0 = whole chunk */
#define CITRUS_MODE_ACCUMULATE  0x20000000u /* accumulative score policy (the "H2O + Shared Cache" variant named in the
                                             Baselines section): a retained state's importance is the sum of the
                                             scores it received at every step since it entered the cache; a chunk's
                                             own states start at this step's score.  citrus_step_view then shows the
                                             accumulated scores. */

#define CITRUS_MODE_DEFERRED_LM  0x40000000u /* with INDIVIDUAL or STANDARD: standard chunked eviction in the order of
                                             Section 4.1 - the language-modelling cache C holds budget_k states plus
                                             the previous chunk (capacity budget_k + chunk_s rows: K, V, positions and
                                             index lists of cache 0 are that wide); a chunk is encoded against all of
                                             them, its attention evicts C's own rows down to budget_k, then all of the
                                             chunk's states enter.  Without the bit the chunk's own states compete for
                                             the budget_k places in the same step.  A STANDARD call that passes
                                             instruction queries (the final eviction) evicts [C ; chunk] to budget_k.
                                             budget_k + 2 chunk_s <= CITRUS_MAX_CANDIDATES. */

#define CITRUS_MODE_POSITION_SHIFT 0x80000000u /* position shift (Section "Hyperparameters"): positional embeddings follow
                                             the place in the cache, not the place in the document.  Q_chunk, K_chunk
                                             and Q_instr are passed WITHOUT rotary embedding; every step embeds them
                                             by their place in [cache ; chunk ; instruction] (cache row r -> r, chunk
                                             token i -> rows + i, instruction token i -> rows + n_tokens + i; half-split
                                             layout: element d pairs with d + head_dim/2 and turns by
                                             pos * base^(-2d/head_dim), base 10000 unless citrus_set_rope_base is
                                             called).  The caches keep the un-rotated keys (that is what
                                             citrus_cache_view shows) next to a copy embedded by slot, which the
                                             compaction rewrites as rows move.  Not together with DEFERRED_LM. */

#define CITRUS_OK                 0
#define CITRUS_ERR_INVALID_ARG   -1
#define CITRUS_ERR_SHAPE         -2
#define CITRUS_ERR_ALIGN         -3
#define CITRUS_ERR_LAYER         -4
#define CITRUS_ERR_STATE         -5
#define CITRUS_ERR_NOMEM         -6
#define CITRUS_ERR_CUDA          -7
#define CITRUS_ERR_TIMEOUT       -8
#define CITRUS_ERR_UNSUPPORTED   -9

#define CITRUS_MAX_INSTR       4096       /* largest n_instr accepted */
#define CITRUS_MAX_CANDIDATES 49152       /* largest budget_k + chunk_s accepted */

/*
 * Allocate a context on the current CUDA device (Sections 4.1-4.3; cache sizes
 * follow the footnote of Section 4.3: budget_k retained rows per cache, plus the
 * caller's chunk of up to chunk_s rows while a call runs).
 * Per layer and per cache (1 shared, 2 individual) it owns two ping-pong buffers
 * K,V [kv_heads, budget_k, head_dim] and positions [kv_heads, budget_k] (int32),
 * plus score / index / log-sum-exp scratch.  Requirements: layers >= 1,
 * q_heads % kv_heads == 0, head_dim in {64, 128} (bf16 needs 128),
 * budget_k >= 1, chunk_s >= 1, budget_k + chunk_s <= CITRUS_MAX_CANDIDATES.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED, NOMEM, CUDA.
 */
int citrus_create(citrus_handle* out, int layers, int q_heads, int kv_heads, int head_dim,
                  int budget_k, int chunk_s, unsigned mode);

/* Number of independent sequence slots sharing the geometry (ragged serving
 * batches); must be called before the first process call. Default 1. */
int citrus_set_batch(citrus_handle h, int n_seq);

/* Side streams used by citrus_process_chunk_batch (Section 4 has no counterpart: the paper processes one document at
 * a time).  n_lanes = 0 (default) lets each call choose (four for the smallest steps, two for medium ones, one otherwise); 1 enqueues every
 * sequence on the caller's stream; up to 8.  May be changed between calls.  Errors: INVALID_ARG. */
int citrus_set_batch_lanes(citrus_handle h, int n_lanes);

/*
 * Ordering of the caller's inputs (no counterpart in the paper; a property of how the kernels are launched).  The
 * kernels of a call are launched with programmatic stream serialisation, which lets a kernel begin while its
 * predecessor in the stream is still running.  By default (ready = 0) every kernel of a call waits for all earlier
 * work in the stream before it first reads Q_chunk / K_chunk / V_chunk / Q_instr or writes `out`, so plain stream
 * order holds whatever produced the inputs - also a kernel of the caller's that signals its dependents early.
 * ready = 1 is the caller's promise that the inputs of every later call are complete before the call's first kernel
 * can start executing (they were produced by copies, by work the stream has been synchronised with, or by kernels
 * that do not signal their dependents early): the chunk's own tiles are then loaded while the previous call's
 * compaction is still running.  The *_host variants order their own copies and always take the fast route.
 * Errors: INVALID_ARG.
 */
int citrus_set_inputs_ready(citrus_handle h, int ready);

/*
 * Attention beside the scoring chain (no counterpart in the paper; a property of how the kernels are launched).  With a
 * shared cache scored by the instruction text (section 4.2, shared cache design) nothing in a2-a4 reads a1's result.
 * For a step with at most max_ctas attention items (128 query rows of one head each: one CTA) the library then runs a1
 * on a stream of its own while the caller's stream runs log-sum-exp -> column sums -> select / gather on the SMs that
 * leaves free; the two fork at the start of the call and join before it returns, so `out`, the caches and stream
 * order look the same to the caller.  max_ctas = 0 switches this off (one launch for a1 and the log-sum-exp pass);
 * the default is 64 (measured on 148 SMs: +20 % for 64 items; 128 items lose 10 % in any split, so they stay in one
 * stream).  Results do not depend on the setting.  Errors: INVALID_ARG.
 */
int citrus_set_attention_beside(citrus_handle h, int max_ctas);

/* Forget every cache of every layer and slot (start a new document). Host-only
 * bookkeeping; enqueues nothing. */
int citrus_reset(citrus_handle h);

/*
 * Steps a1-a4 for (layer, sequence slot 0) on `stream`.
 *   Q_chunk [n_tokens, q_heads, D], K_chunk / V_chunk [n_tokens, kv_heads, D],
 *   Q_instr [n_instr, q_heads, D] (queries of the instruction text I for this
 *   layer), out [n_tokens, q_heads, D] receives the attention output of a1 in the
 *   element type.  With CITRUS_MODE_STANDARD, n_instr == 0 (Q_instr may then be NULL) selects scoring by the chunk.
 *   1 <= n_tokens <= chunk_s (a shorter chunk is allowed anywhere,
 *   cf. "except for the final chunk", Section 4.1); 1 <= n_instr <= CITRUS_MAX_INSTR.
 * Chunks of one (layer, slot) must be submitted in document order on one stream.
 * The caller's K_chunk / V_chunk must stay valid until the stream work is done
 * (the new cache is gathered straight from them).
 * Errors: INVALID_ARG (NULL), LAYER, SHAPE, ALIGN, CUDA (launch failure).
 */
int citrus_process_chunk(citrus_handle h, int layer,
                         const void* Q_chunk, const void* K_chunk, const void* V_chunk, int n_tokens,
                         const void* Q_instr, int n_instr, void* out, citrus_stream_t stream);

/* Same, for sequence slot `seq_slot` (ragged batches submit one call per active
 * sequence; slots are independent and may use different streams).  A CITRUS_MODE_POSITION_SHIFT context has one
 * embedding scratch: a step submitted on another stream than the context's previous step is ordered, by an event,
 * behind everything enqueued on that stream so far (so such steps do not overlap; all of them must then belong to
 * the same stream capture, or to none). */
int citrus_process_chunk_slot(citrus_handle h, int layer, int seq_slot,
                              const void* Q_chunk, const void* K_chunk, const void* V_chunk, int n_tokens,
                              const void* Q_instr, int n_instr, void* out, citrus_stream_t stream);

/*
 * Ragged batch (serving mix): one chunk for each of n_active sequences, packed token-major.  Sequence i uses slot
 * seq_slot[i]; its chunk rows are [tok_offset[i], tok_offset[i+1]) of Q / K / V / out and its instruction rows are
 * [instr_offset[i], instr_offset[i+1]) of Q_instr.  seq_slot, tok_offset and instr_offset are HOST arrays
 * (n_active, n_active + 1 and n_active + 1 ints); the tensors are device pointers as in citrus_process_chunk.
 * Every sequence's chunk obeys the single-call rules (1..chunk_s tokens, 1..CITRUS_MAX_INSTR instruction rows,
 * distinct slots).  All arguments are validated before anything is enqueued; sequences are independent (no state
 * is shared between slots).  Where every sequence's step is small (its attention items make at most about three
 * waves over the SMs) the sequences are dealt to side streams owned by the context, which fork from `stream` when the call starts and join
 * it again before the call returns: to the caller the call is still one piece of work on `stream` (it can be captured
 * in a CUDA graph through `stream`), but the steps of different sequences overlap.  Larger steps and profiled
 * runs are enqueued one after the other on `stream` itself (a position-shift context keeps one embedding scratch per
 * side stream: 8 x (chunk_s + CITRUS_MAX_INSTR) x q_heads rows more, allocated by citrus_set_batch).  See citrus_set_batch_lanes.
 * Errors: as citrus_process_chunk; INVALID_ARG for duplicate slots or non-increasing offsets.
 */
int citrus_process_chunk_batch(citrus_handle h, int layer, int n_active, const int* seq_slot, const int* tok_offset,
                               const void* Q, const void* K, const void* V, const int* instr_offset,
                               const void* Q_instr, void* out, citrus_stream_t stream);

/*
 * End-to-end variant with HOST buffers (pinned memory recommended): copies the
 * four inputs to device staging owned by the context, runs a1-a4, copies `out`
 * back and waits for that copy.  Same argument rules otherwise.
 */
int citrus_process_chunk_host(citrus_handle h, int layer, int seq_slot,
                              const void* Q_chunk_host, const void* K_chunk_host, const void* V_chunk_host,
                              int n_tokens, const void* Q_instr_host, int n_instr, void* out_host,
                              citrus_stream_t stream);

/*
 * A whole document from HOST buffers (pinned memory recommended): Qh / Kh / Vh / out_h hold n_tokens rows
 * (any number: the document is cut into chunks of chunk_s tokens, the last one shorter), Qih the n_instr
 * instruction queries that score every chunk (STANDARD contexts: only the last chunk, as in citrus_process_chunk
 * with n_instr = 0 before it).  The unit continues from its current state (citrus_reset starts a new document).
 * The document moves in blocks of four chunks: the next block's inputs are copied to the device and the previous
 * block's output is copied back while the current block is computed - two staging sets and two copy streams owned
 * by the context, created by the first call (make that call outside any stream capture).  Returns when out_h is complete.  Errors: as citrus_process_chunk; nothing is enqueued if the
 * arguments are rejected.
 */
int citrus_process_document_host(citrus_handle h, int layer, int seq_slot,
                                 const void* Qh, const void* Kh, const void* Vh, long long n_tokens,
                                 const void* Qih, int n_instr, void* out_h, citrus_stream_t stream);

/*
 * Borrowed device pointers into the current cache of (layer, which, seq_slot);
 * which = 0 the language-modelling / shared cache, 1 the instruction cache C^I
 * (individual mode only).  K, V are [kv_heads, cap, D] with rows
 * [0, *n_rows) valid, cap = budget_k (budget_k + chunk_s for cache 0 of a
 * CITRUS_MODE_DEFERRED_LM context); positions [kv_heads, cap] int32 are the original
 * token positions, strictly ascending per head (the order a position-shift
 * caller needs).  *n_rows = min(budget_k, tokens seen) is host bookkeeping, so
 * the call does not synchronise; the contents are final once the stream work of
 * the last process call is done.  Valid until the next process / reset / destroy.
 */
int citrus_cache_view(citrus_handle h, int layer, int which, int seq_slot,
                      const void** K, const void** V, const int** positions, int* n_rows);

/*
 * Borrowed device pointers to what the last process call on (layer, which,
 * seq_slot) computed in a2-a3: scores [kv_heads, *n_candidates] fp32 (row stride
 * *score_stride elements) and kept candidate indices [kv_heads, *n_kept] int32
 * ascending (row stride budget_k).  Candidate j < m_before is old cache row j,
 * otherwise chunk row j - m_before.
 */
int citrus_step_view(citrus_handle h, int layer, int which, int seq_slot,
                     const float** scores, int* score_stride, const int** idx,
                     int* n_candidates, int* n_kept, int* m_before);

/*
 * Measurement aid for the roofline figures (kernel time of a1 / a2 / a3 / a4 taken
 * separately).  While enabled, every kernel launch of a process call is bracketed by
 * CUDA events recorded on the call's stream (do not enable during stream capture).
 * citrus_profile_read synchronises the device, adds up the elapsed milliseconds and
 * the number of launches per kernel id since the last read into ms[CITRUS_N_KERNELS]
 * and launches[CITRUS_N_KERNELS] (host arrays), and clears the record.
 */
#define CITRUS_KERNEL_ATTENTION 0   /* a1 (bf16 path: one launch with the log-sum-exp pass of a2) */
#define CITRUS_KERNEL_SCORE_LSE 1   /* a2, log-sum-exp pass of the instruction queries (fp32 path only) */
#define CITRUS_KERNEL_COLSUM    2   /* a2, column sums (instruction and LM) */
#define CITRUS_KERNEL_SELECT    3   /* a3 (separate launch only with CITRUS_MODE_LAYERWISE) */
#define CITRUS_KERNEL_COMPACT   4   /* a4 (per-head granularity: one launch with a3) */
#define CITRUS_KERNEL_ROPE      5   /* embedding pre-pass of CITRUS_MODE_POSITION_SHIFT */
#define CITRUS_N_KERNELS        6
int citrus_profile(citrus_handle h, int enable);
int citrus_profile_read(citrus_handle h, double* ms, long long* launches);

/*
 * Importance scoring without any allocation.  The paper has no counterpart: this exists for
 * callers that must not (or cannot) allocate device memory -- a serving loop that has handed the
 * whole GPU to its own memory pool so that cudaMalloc fails or stalls every stream with its
 * device-wide synchronisation, a plug-in that is only allowed to launch work on streams it is
 * given, or code that may run while another thread holds an allocator lock.
 *
 * Computes the same quantity as step a2-I of citrus_process_chunk on an empty cache:
 *   scores[g][j] = sum over heads h of KV group g, and over the n_s scoring rows i, of
 *                  softmax_j( Q_s[i,h] . K[j,g] / sqrt(head_dim) ),     j < n_keys,
 * with Q_s [n_s, q_heads, head_dim] and K [n_keys, kv_heads, head_dim] token-major device
 * tensors (bf16, or fp32 with CITRUS_MODE_FP32 as the only accepted mode bit) and scores
 * [kv_heads, score_stride] fp32 device memory, all owned by the caller.  No context is needed.
 *
 * The intermediate log-sum-exp of every (head, row) lives in a fixed array of
 * CITRUS_STATIC_MAX_LSE floats (256 KB, plus a 256-byte status word) that is part of the
 * library image: every GPU that loads the library holds it until the process exits.  Limits:
 * q_heads * round_up(n_s, 4) <= CITRUS_STATIC_MAX_LSE, n_s <= CITRUS_MAX_INSTR,
 * n_keys <= CITRUS_MAX_CANDIDATES; head_dim 128 (bf16) or 64/128 (fp32).  Larger sizes return
 * CITRUS_ERR_SHAPE and launch nothing.  The function never calls cudaMalloc, cudaFree or any
 * allocating routine.
 *
 * The first call on a device looks up the array's device address (and, for bf16, resolves the
 * tensor-map encoder and raises the kernels' shared-memory limits); make that first call
 * outside of any stream capture.  All calls on a device share the one array and overwrite it:
 * two calls whose GPU work overlaps (different streams, or different threads) race; run them
 * on one stream or order them with events.  device_status is a caller-owned device int, zeroed by
 * the caller, set to 1 if a bounded wait inside a kernel expires (the scores are then not valid).
 * It may be NULL: the flag then goes to a word of the shared array that the next call clears and
 * nothing reports, i.e. an expired wait goes unnoticed - pass a status word wherever that matters.
 */
#define CITRUS_STATIC_MAX_LSE 65536
int citrus_importance_static(const void* Q_s, int n_s, const void* K, int n_keys,
                             int q_heads, int kv_heads, int head_dim, unsigned mode,
                             float* scores, int score_stride, int* device_status,
                             citrus_stream_t stream);

/*
 * Intersection ratio of the appendix "Details for the Intersection Probing Experiments":
 *   ratio[g] = | C(g)  intersect  C^I(g) | / | C^I(g) |
 * over the states currently retained for KV head g by the language-modelling cache C (selected by the document
 * context) and by the instruction cache C^I of (layer, seq_slot); states are identified by their original token
 * position.  Individual mode only (CITRUS_ERR_STATE otherwise, and before the first step).  ratio_dev: device,
 * [kv_heads] fp32, caller-owned; written by work enqueued on `stream`, which must be ordered after the last
 * process call of that unit.
 */
int citrus_intersection_ratio(citrus_handle h, int layer, int seq_slot, float* ratio_dev, citrus_stream_t stream);

/* Base of the rotary embedding of a CITRUS_MODE_POSITION_SHIFT context (default 10000; Llama-3 uses 500000).
 * Only before the context's first step (CITRUS_ERR_STATE afterwards); base > 1. */
int citrus_set_rope_base(citrus_handle h, double base);

/* Reads the device status word (0, or CITRUS_ERR_TIMEOUT if a bounded wait in a
 * kernel gave up: every wait on an mbarrier inside the kernels ends after about one second, raises the word, and
 * the kernel drains and returns).  Synchronises the device.  A raised word is cleared by the read; the caches of
 * the steps that ran meanwhile are not valid (citrus_reset starts over). */
int citrus_poll_status(citrus_handle h);

/* Test aid for the time-out path (the paper has no counterpart): enqueues one warp that waits limit_ns nanoseconds
 * (1 .. 100 000 000) on an mbarrier that nothing arms, with the same bounded wait the kernels use; the wait runs
 * out, the kernel raises the context's status word and returns normally.  citrus_poll_status then reports
 * CITRUS_ERR_TIMEOUT once.  Nothing else is touched.  Errors: INVALID_ARG, CUDA. */
int citrus_debug_expire_wait(citrus_handle h, unsigned long long limit_ns, citrus_stream_t stream);

/* Frees everything. NULL is a no-op; a handle that was already destroyed
 * returns CITRUS_ERR_STATE. */
int citrus_destroy(citrus_handle h);

const char* citrus_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* CITRUS_H_ */
