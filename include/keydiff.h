/*
 * keydiff.h -- C ABI of the B200 (sm_100a) KeyDiff eviction-step library.
 *
 * The library implements one operation: the per-KV-head cache eviction step of
 * KeyDiff's block-wise prefill (Sec. 2.3-2.4 and 3.2 of the paper).  After a block of
 * B new keys/values is appended to a cache bounded by a budget of N tokens, every
 * (layer, sequence, KV head) unit independently
 *   1. forms the anchor  mu = (1/n) sum_i k_i/||k_i||  over its n = len + B keys,
 *   2. scores each key   s_i = mu.k_i / max(||mu||*||k_i||, eps)        (App. B.1),
 *   3. keeps the N keys with the LOWEST cosine (Eq. efficient-keydiff:
 *      S = topk(-CosSim(mu, k_i), N)), ties keeping the older token,
 *   4. gathers K' = gather(K,S), V' = gather(V,S) (Eq. keydiff) in original token
 *      order, in place.
 *
 * Conventions
 *   - No exceptions cross this boundary.  Every call returns an int status
 *     (KEYDIFF_OK or a negative KEYDIFF_ERR_*); keydiff_strerror names it.
 *   - "device" pointers are CUDA global-memory addresses on the ctx's device;
 *     "host" pointers are ordinary process memory.
 *   - All work is enqueued on the given stream; nothing here synchronises with the
 *     host unless stated.  keydiff_evict allocates nothing.
 *   - Not thread-safe per ctx: use a ctx from one host thread / one stream at a
 *     time.  Distinct ctxs are independent.
 *   - There is no CPU fallback: on a machine without a usable sm_100 device
 *     keydiff_create fails with KEYDIFF_ERR_CUDA / KEYDIFF_ERR_UNSUPPORTED.
 *   - The environment is read once, by keydiff_create, for four launch-tuning aids (integers; unset =
 *     automatic): KEYDIFF_CLUSTER_SIZE (CTAs per cluster of the fused kernels, 1..16), KEYDIFF_MAX_CLUSTERS
 *     (upper limit on the clusters the ordered fused kernel launches), KEYDIFF_STAGGER_NS and
 *     KEYDIFF_LATE_NS (start-up delays between clusters, nanoseconds).  They change launch shapes
 *     only, never results; no other call looks at the environment.
 *   - Accuracy of the scores (fp32 storage, fp64 oracle): a score is (mu.k)/(||mu|| ||k||).  The
 *     dot product is accumulated in double precision above chains of four fp32 products, so its error
 *     is about 1e-8 of the SIZE OF ITS TERMS, kappa = sum_c |mu_c k_c| / (||mu|| ||k||) <= 1; the norms
 *     and the division add about 4e-7 RELATIVE to the score.  Hence |e_gpu - e| <~ 4e-7 |e| + 3e-8
 *     kappa: within 1e-5 relative for |e| >= 1e-2 whatever the data; for a score nearer to zero (a
 *     cancelling sum) the error is bounded by the size of the terms, not by the score.
 *
 * Tensor layouts (bf16, contiguous, row = token):
 *   k_cache, v_cache : [n_layers][batch][n_kv_heads][budget N][head_dim]
 *                      rows [0, len) of every unit are valid
 *   new_k,  new_v    : [n_layers][batch][n_kv_heads][block B][head_dim]
 *   All four base pointers must be 16-byte aligned.  The caches and the blocks
 *   must not overlap.
 */
#ifndef KEYDIFF_H_
#define KEYDIFF_H_

#include <stdint.h>

#if defined(__GNUC__)
#define KEYDIFF_API __attribute__((visibility("default")))
#else
#define KEYDIFF_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct keydiff_ctx keydiff_ctx; /* opaque; owns only its scratch memory */

enum {
    KEYDIFF_OK = 0,
    KEYDIFF_ERR_INVALID_ARG = -1, /* NULL / misaligned pointer, value out of range, mismatch with ctx */
    KEYDIFF_ERR_UNSUPPORTED = -2, /* valid request this build cannot serve (dtype, head_dim, size, device) */
    KEYDIFF_ERR_ALLOC = -3,       /* scratch allocation failed in keydiff_create */
    KEYDIFF_ERR_CUDA = -4,        /* a CUDA runtime call failed; see keydiff_last_cuda_error */
    KEYDIFF_ERR_STATE = -5,       /* call not valid in the ctx's current state */
    KEYDIFF_ERR_TIMEOUT = -6,     /* a bounded device-side wait expired (reported in the status word) */
    KEYDIFF_ERR_TOO_LARGE = -7,   /* keydiff_evict_static: the request does not fit the built-in scratch */
    KEYDIFF_ERR_INTERNAL = -8     /* status word only, debug-checks build only: a kernel computed a row index outside
                                     its tensor; the store was skipped */
};

enum { KEYDIFF_BF16 = 0 };

/* The anchor of Eq. (efficient-keydiff).  The equation and App. B.1 use the mean of the normalised
 * keys; the text that follows the equation says the mean of the keys themselves serves as well.  Both
 * are built; the score formula s_i = mu.k_i / max(||mu|| ||k_i||, eps) is the same. */
enum {
    KEYDIFF_ANCHOR_NORMALISED = 0,  /* mu = (1/n) sum_i k_i/||k_i||   (default) */
    KEYDIFF_ANCHOR_RAW_MEAN = 1     /* mu = (1/n) sum_i k_i */
};

/* Where the kept rows end up.  Eq. (keydiff) gathers them, K' = gather(K,S), without fixing their
 * order (attention does not depend on the order of the cached pairs; positions are already rotated
 * into the keys).  Both layouts are built. */
enum {
    KEYDIFF_COMPACT_ORDERED = 0,    /* kept rows in original token order, compacted to the front (default) */
    KEYDIFF_COMPACT_SLOT_REUSE = 1  /* kept cache rows stay in their slots; the kept block rows take the
                                       freed slots: at most block_B rows per tensor are written.  The fused
                                       path serves it with a streaming kernel for max_block <= 1024; larger
                                       blocks go to the staged kernels (KEYDIFF_PATH_FUSED then fails with
                                       KEYDIFF_ERR_UNSUPPORTED) */
};

/* Which kernels serve keydiff_evict. */
enum {
    KEYDIFF_PATH_AUTO = 0,    /* fused cluster kernel when a unit fits, else the staged kernels */
    KEYDIFF_PATH_STAGED = 1,  /* four launches: anchor partials, scores, select, compaction */
    KEYDIFF_PATH_FUSED = 2    /* one launch, one thread-block cluster per unit; create fails
                                 with KEYDIFF_ERR_UNSUPPORTED if a unit cannot fit */
};

typedef struct {
    int32_t n_layers;      /* >= 1 */
    int32_t batch;         /* >= 1, independent sequences */
    int32_t n_kv_heads;    /* >= 1, KV heads per layer (GQA groups share one KV head) */
    int32_t head_dim;      /* 128 (the only value built) */
    int32_t budget;        /* N, cache budget in tokens (Sec. 2.3), >= 1 */
    int32_t max_block;     /* largest B ever passed to keydiff_evict (Sec. 2.4), >= 1 */
    int32_t dtype;         /* KEYDIFF_BF16 */
    int32_t path;          /* KEYDIFF_PATH_* */
    float   eps;           /* eps of App. B.1's max(.,eps); 0 selects the default 1e-8 */
    int32_t device;        /* CUDA device ordinal */
    int32_t anchor_mode;   /* KEYDIFF_ANCHOR_*: which mean is the anchor (Sec. 3.2) */
    int32_t recent_window; /* w >= 0 most recent tokens that are never evicted (Sec. 3.2, "KeyDiff with
                              sliding window"); 0 = plain KeyDiff; w <= budget */
    int32_t compaction;    /* KEYDIFF_COMPACT_*: layout of the kept rows */
} keydiff_config;

/*
 * keydiff_create -- allocate a context and its device scratch for U = n_layers*batch*
 * n_kv_heads units (scores U*(N+max_block) fp32, kept-index list U*N int32, anchor
 * partials, per-unit counters, one status word).  Synchronous.  *out is set only on
 * KEYDIFF_OK.  The initial cache length is 0 (C_0 = empty, Eq. block_processing).
 * Errors: INVALID_ARG (NULL, non-positive sizes, unknown anchor_mode, recent_window outside
 * [0, budget], unknown compaction), UNSUPPORTED (dtype, head_dim, a unit
 * too large for the requested path, no sm_100 device), ALLOC, CUDA.
 */
KEYDIFF_API int keydiff_create(const keydiff_config* cfg, keydiff_ctx** out);

/*
 * keydiff_evict -- one step of Eq. (block_processing) for every unit of the ctx:
 * C <- ([K || new_k], [V || new_v]); C <- pi_N(C) with pi_N = KeyDiff (Eq.
 * efficient-keydiff, anchor of normalised keys).
 *   n = len + block_B.  If n <= N the block rows are appended at rows [len, n) and
 *   nothing is scored (Sec. 2.3: eviction only when the budget is exceeded).
 *   Otherwise the n keys are scored, the N with the largest eviction score e = -s are
 *   kept (ties: lower token index wins), and K and V are compacted in place in
 *   original token order; rows in front of the first evicted row are not touched.
 *   Afterwards len = min(N, n) for every unit.
 *   With recent_window = w > 0 (Sec. 3.2, sliding window; the paper gives no formula, this is the
 *   reading taken): the last w of the n tokens are always kept, the N - w tokens with the largest e are
 *   kept among the first n - w, and the anchor is still formed from all n keys.
 *   With compaction = KEYDIFF_COMPACT_SLOT_REUSE the n candidates are numbered slots 0 .. len-1 first,
 *   block rows len .. n-1 after; scores and selection are the same (ties: lower candidate number wins);
 *   kept cache rows are not touched, and the kept block rows, in block order, are written into the freed
 *   slots (those of evicted cache rows, then slots >= len that were still empty) in ascending slot
 *   order.  The ctx keeps each slot's token position (keydiff_get_positions); the sliding window then
 *   means the tokens at the last w positions of the sequence.  An append-only step is the same as in
 *   the ordered layout.
 * k_cache, v_cache: device, in/out, caller-owned.  new_k, new_v: device, read only,
 * caller-owned; they may be reused once the work enqueued on `stream` has completed.
 * budget_N, n_kv_heads, head_dim restate the ctx's values and must equal them;
 * 1 <= block_B <= max_block.  stream: a cudaStream_t (NULL = legacy default stream).
 * Asynchronous: returns after enqueueing.  Host-detectable errors (INVALID_ARG,
 * STATE) enqueue nothing and leave len unchanged.  Device-side anomalies (a bounded
 * wait that expired) are written to the status word (keydiff_get_scratch) and the
 * kernels return normally; the call itself has returned KEYDIFF_OK long before.  A non-zero
 * status word means that the cache rows, scores and lists of that step (and of every later
 * step of the ctx: the word is never cleared) are unspecified; restore the caches from a
 * copy and use a new ctx (keydiff_set_len / keydiff_set_positions).  (With slot reuse a thread block whose own
 * wait expired places no further rows; the ordered kernel carries on to its normal end -- a check in its store
 * loops was measured at 3-5 % of the step -- so rows that never arrived on chip may be stored.)  Non-finite keys give an
 * unspecified selection, never a fault.
 */
KEYDIFF_API int keydiff_evict(keydiff_ctx* ctx, void* k_cache, void* v_cache,
                  const void* new_k, const void* new_v,
                  int32_t budget_N, int32_t block_B, int32_t n_kv_heads, int32_t head_dim,
                  void* stream);

/*
 * keydiff_evict_host -- the same step with the BLOCK in host memory (the caches stay on
 * the device): copies new_k/new_v (host, block_B rows per unit, same layout) to ctx-owned
 * device staging, runs keydiff_evict on `stream`, then copies the kept-index list
 * (U*N int32, see keydiff_get_scratch) and the status word back into kept_idx_host /
 * status_host on `stream` (host; either may be NULL to skip).  The block travels on a copy stream
 * of the ctx into one of two staging sets, and `stream` waits for it: the copy of one call
 * overlaps the kernels of the call before it.  It starts as soon as the call is made, without
 * waiting for work queued on `stream`, so the host block must hold its data when the call is made;
 * it may be reused once the work enqueued on `stream` has completed.  Pinned host memory makes the
 * copies asynchronous; the call itself does not synchronise.  While `stream` is being captured all
 * copies stay on `stream`.  When kept_idx_host is pinned (page-locked) memory and the fused path serves an
 * evicting step, the kernel writes the list into it directly while it runs (through the buffer's device
 * alias) instead of a copy afterwards; either way the list is complete once the work on `stream` is.
 * Staging buffers, copy stream and events are created on first use (that
 * first call synchronises and may return ALLOC).
 */
KEYDIFF_API int keydiff_evict_host(keydiff_ctx* ctx, void* k_cache, void* v_cache,
                       const void* new_k_host, const void* new_v_host,
                       int32_t budget_N, int32_t block_B, int32_t n_kv_heads, int32_t head_dim,
                       int32_t* kept_idx_host, int32_t* status_host, void* stream);

/* keydiff_destroy -- free the scratch and the ctx.  Synchronises the device.  NULL is OK. */
KEYDIFF_API int keydiff_destroy(keydiff_ctx* ctx);

/*
 * keydiff_set_incremental -- choose how the fused path obtains the anchor of App. B.1 (first
 * expression), mu = (1/n) sum_i k_i/||k_i||.  The cache is carried from block to block (Eq.
 * block_processing), so the sum over a step's n rows is the sum over the rows already cached plus the
 * sum over the B new rows.  With on != 0 (the default) the context keeps the cached rows' sum per unit
 * on the device: an evicting step adds the block rows' terms, subtracts the evicted rows' terms (both
 * recomputed from the same bf16 rows by the same arithmetic), and the next step needs only the block
 * normalised before it can score.  The value is the same sum in a different order of additions (fp32
 * partial sums folded in double precision); scores stay within the library's tolerance.  The running
 * sum is rebuilt from all n rows on the first evicting step, after any append-only step,
 * keydiff_set_len or keydiff_reset, and every 1024 evicting steps.  With on == 0 every step rebuilds it.
 * REQUIREMENT with on != 0: between two keydiff_evict calls nobody else may change rows [0, len) of
 * k_cache; after changing them call keydiff_set_len(ctx, len).  The staged path ignores the setting.
 * Errors: INVALID_ARG (NULL ctx).
 */
KEYDIFF_API int keydiff_set_incremental(keydiff_ctx* ctx, int32_t on);

/* Cache length bookkeeping (host side, no device work).  C_0 = empty: reset sets len = 0;
 * set_len resumes from a cache the caller restored (0 <= len <= N); both make the next evicting step
 * rebuild the running anchor sum (keydiff_set_incremental). */
KEYDIFF_API int keydiff_reset(keydiff_ctx* ctx);
KEYDIFF_API int keydiff_get_len(const keydiff_ctx* ctx, int32_t* len_out);
KEYDIFF_API int keydiff_set_len(keydiff_ctx* ctx, int32_t len);

/*
 * keydiff_get_scratch -- device pointers into ctx-owned scratch, valid until destroy;
 * contents are those of the most recent evicting step once its stream work completed.
 *   scores   : [U][N + max_block] fp32, e_i = -s_i for i < n (the eviction score, +0 for -0)
 *   kept_idx : [U][N] int32, ascending token indices (into the n concatenated rows) of
 *              the kept tokens = source row of every destination row
 *   first_evicted : [U] int32, index of the first evicted token (rows before it did not move)
 *   status   : [1] int32, 0 or a KEYDIFF_ERR_* code set by a kernel
 * Any output pointer may be NULL.
 */
KEYDIFF_API int keydiff_get_scratch(const keydiff_ctx* ctx, const float** scores, const int32_t** kept_idx,
                        const int32_t** first_evicted, const int32_t** status);

/*
 * keydiff_get_positions -- slot reuse only (else KEYDIFF_ERR_STATE): device pointer to pos[U][N] int32,
 * the token position (0-based index in the sequence) held by each of the first len slots, valid once
 * the stream work of the latest step has completed, and the position the next new token will get.
 * keydiff_set_len(len) declares slots 0 .. len-1 to hold tokens 0 .. len-1 and keydiff_reset starts a new
 * sequence; both are host-side bookkeeping, and the array itself is rewritten to that identity map only
 * by the NEXT step (until then it still shows the previous sequence).  keydiff_set_positions writes it
 * at once.  In this mode kept_idx[u][s] (keydiff_get_scratch) is the candidate number slot s now holds
 * (s itself for a cache row that stayed, len + j for block row j), and the moved-rows counter counts
 * the block rows written.  Either output pointer may be NULL.
 */
KEYDIFF_API int keydiff_get_positions(const keydiff_ctx* ctx, const int32_t** pos, long long* next_pos);

/*
 * keydiff_set_positions -- slot reuse only (else KEYDIFF_ERR_STATE): resume from a cache the caller
 * restored.  With slot reuse the cache is not in token order, so keydiff_set_len (slot s = token s) cannot
 * describe a cache that has already evicted; this call hands the saved position array back.  (The sliding
 * window of Sec. 3.2 is defined on these positions, and Eq. block_processing carries the cache, hence
 * its positions, from block to block.)
 *   pos_device : device, [U][N] int32 as keydiff_get_positions returned it (rows [0, len) of every unit
 *                are used), copied into the ctx on `stream`; NULL = the identity map (slot s = token s)
 *   len        : cached tokens per unit, 0 <= len <= N
 *   next_pos   : position the next new token gets, len <= next_pos < 2^31; every stored position must
 *                be below it (not checked)
 * The running anchor sum is rebuilt by the next evicting step.  Asynchronous on `stream`; later steps
 * must be enqueued on the same stream or ordered after it.  Errors: INVALID_ARG, STATE (not slot reuse,
 * or the ctx's device is not current), CUDA.
 */
KEYDIFF_API int keydiff_set_positions(keydiff_ctx* ctx, const int32_t* pos_device, int32_t len, long long next_pos,
                                      void* stream);

/*
 * keydiff_get_moved_rows -- device pointer to a 64-bit counter: the number of kept rows (per
 * tensor) whose position changed, summed over all units and all evicting steps since create
 * (= sum over units of N - first_evicted).  Benchmarks use it to count the bytes a step had to
 * move.  Read it after synchronising the stream.
 */
KEYDIFF_API int keydiff_get_moved_rows(const keydiff_ctx* ctx, const unsigned long long** counter);

/* Launch facts of the chosen path, for benchmarks: path actually used (KEYDIFF_PATH_*),
 * kernels launched per evicting step, cluster size (1 for the staged path).  With slot reuse on the fused
 * path a step that has to rebuild the running anchor sum (keydiff_set_incremental) launches two more. */
KEYDIFF_API int keydiff_get_launch_info(const keydiff_ctx* ctx, int32_t* path, int32_t* launches_per_step,
                            int32_t* cluster_size);

/*
 * keydiff_evict_static -- the eviction step for callers that cannot allocate device memory.
 * (The paper has no counterpart for this entry point; it exists for deployment reasons only.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside an inference server whose
 * own memory pool has already claimed the GPU, in a plugin that is only ever handed tensors, or in
 * a latency-critical loop where an allocation (which synchronises the device) is not acceptable.
 * keydiff_create must allocate its scratch, so it is unusable there.  This call allocates nothing
 * and frees nothing: its scratch is a 16 MiB array built into the library image (each GPU that
 * loads the library carries those 16 MiB until the process exits).
 *
 * It computes exactly what keydiff_evict computes (staged kernels; same scores, same selection,
 * same in-place compaction in token order), but keeps no context: the caller passes the current
 * cache length `len` (0 <= len <= budget_N) and tracks the new one itself, min(budget_N, len +
 * block_B).  k_cache/v_cache: device, in/out, [n_units][budget_N][128] bf16; new_k/new_v: device,
 * read only, [n_units][block_B][128] bf16; all 16-byte aligned.  eps: 0 selects 1e-8.
 * Asynchronous on `stream`.
 *
 * Limit: the step's scratch -- n_units * (8*(len+block_B) + 4*budget_N + 4) bytes plus the anchor
 * partials, each part rounded up to 256 bytes -- must fit in 16 MiB (about 160 units at N=8192,
 * B=128; about 2100 units at N=512, B=128) and len+block_B must not exceed 51200; otherwise the call
 * returns KEYDIFF_ERR_TOO_LARGE and enqueues nothing.
 *
 * Set-up: the first call on each device -- whatever it does, an append-only step included -- looks up
 * the array's device address (cudaGetSymbolAddress) and sets one kernel attribute before it enqueues
 * anything; the device that holds the tensors must be current (checked for k_cache: KEYDIFF_ERR_STATE).
 * Make that first call before starting any stream capture.  Later calls do no set-up.
 *
 * Sharing: every call on a device uses the same array, and the array keeps whatever the previous
 * call left in it (the call clears the one counter that has to start at zero).  Two calls whose
 * GPU work can overlap -- different streams, or different host threads without ordering -- race
 * on the scratch and corrupt each other; order them on one stream or with events.
 */
KEYDIFF_API int keydiff_evict_static(void* k_cache, void* v_cache, const void* new_k, const void* new_v,
                                     int32_t len, int32_t budget_N, int32_t block_B, int32_t n_units,
                                     int32_t head_dim, float eps, void* stream);

/*
 * keydiff_selftest_bounded_wait -- failure-detection self test (the paper has no counterpart).  Every
 * wait of the kernels on a copy in flight is bounded; when one runs out, the kernel writes
 * KEYDIFF_ERR_TIMEOUT to its status word and still returns normally.  This call shows that behaviour
 * without disturbing anything: it launches one small CTA on `stream` whose threads wait, through the same
 * wait routine and with a limit of `polls` polls (1..4096), on a barrier that nothing ever completes.
 * After the stream work has completed, *status_device (device, int32, caller-owned, zeroed by the
 * caller) holds KEYDIFF_ERR_TIMEOUT.  Errors: INVALID_ARG, CUDA.
 */
KEYDIFF_API int keydiff_selftest_bounded_wait(int32_t* status_device, int32_t polls, void* stream);

/*
 * keydiff_debug_fail_alloc -- test hook: the nth device allocation (1-based) that the next keydiff_create
 * makes on this process fails once, as if the device were out of memory; keydiff_create must then
 * release what it had allocated and return KEYDIFF_ERR_ALLOC.  0 disarms.  The hook is disarmed when
 * keydiff_create returns.  Not thread-safe.
 */
KEYDIFF_API int keydiff_debug_fail_alloc(int32_t nth);

/* Text of a status code; never NULL. */
KEYDIFF_API const char* keydiff_strerror(int code);

/* cudaError_t value of the most recent failed CUDA call made by this library on the
 * calling thread (0 if none). */
KEYDIFF_API int keydiff_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* KEYDIFF_H_ */
