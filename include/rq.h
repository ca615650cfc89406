/*
 * rq.h — C ABI of the sparse-decode library: query-aware (Quest-style) sparse
 * decode attention over exponentially decaying key/value memory, for NVIDIA
 * B200 (sm_100a).
 *
 * The method (paper sections in brackets):
 *   [Eq. 1]   k~_t = g_t*k~_{t-1} + (1-g_t)*k_t and the same for v with the
 *             same gate; zero initial state; state kept in fp32.
 *   [App. A.1, "Sparse inference settings"]  the cache of k~, v~ is split into
 *             pages (blocks) and every page keeps the per-channel minimum and
 *             maximum of its stored keys.
 *   [Eq. 3]   each decode query scores every page by the upper bound
 *             U_p = sum_i max(q_i*min_p[i], q_i*max_p[i]) and keeps the top
 *             `budget_pages` pages per head; the first page(s) and the newest
 *             page(s) are always kept and count inside the budget; equal
 *             scores go to the lower page index.
 *   [Eq. 4]   softmax attention over the valid tokens of the kept pages only,
 *             on the decayed keys and decayed values.
 *
 * Conventions
 *   - Every function returns an int status (RQ_OK = 0, otherwise RQ_ERR_*).
 *     Argument errors are found on the host before anything is enqueued; no
 *     function aborts, throws or traps the device.
 *   - Pointers are DEVICE pointers unless the name of the function ends in
 *     `_host` or the parameter is documented as host memory.
 *   - The caller owns every byte of device memory.  The library allocates no
 *     device memory and keeps no state of a cache outside the caller's buffers
 *     (it only remembers, per device, launch parameters it has looked up once);
 *     `rq_sizes` tells the caller how much to allocate and `rq_cache_init`
 *     adopts the buffers.  Buffers must be 256-byte aligned and must outlive
 *     the `rq_cache`.  (rq_attend_pages_noalloc is the one call that uses a
 *     fixed array inside the library instead of a workspace.)
 *   - `stream` is a `cudaStream_t` passed as `void*` (NULL = default stream).
 *     Work is enqueued on it and the call returns without synchronising,
 *     except where stated.  Calls on one cache must be stream-ordered; two
 *     calls on the same cache running concurrently race on its workspace.
 *   - Shapes: B = batch, H = heads (q heads = kv heads), D = head_dim,
 *     S = page_size.  All sequences of a batch have the same length.
 *   - Layouts in device memory (row-major, last index contiguous):
 *       kv        [B][H][page_capacity][2][S][D]  storage dtype; [..][0] keys, [..][1] values
 *       meta      [B][H][page_capacity][2][D]     storage dtype; [..][0] min,  [..][1] max
 *       state     [B][H][2][D]                    fp32; [..][0] k~ state, [..][1] v~ state
 *       workspace opaque
 *     page_capacity = ceil(capacity_tokens / S).
 */
#ifndef RQ_H_
#define RQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* exported-symbol marker (the library is built with hidden default visibility) */
#if defined(__GNUC__)
#define RQ_API __attribute__((visibility("default")))
#else
#define RQ_API
#endif

#define RQ_VERSION_MAJOR 0
#define RQ_VERSION_MINOR 1

/* status codes */
#define RQ_OK 0
#define RQ_ERR_INVALID_ARG 1 /* NULL / misaligned pointer, non-positive size, bad enum    */
#define RQ_ERR_UNSUPPORTED 2 /* a shape or dtype outside the compiled set (see rq_sizes) */
#define RQ_ERR_CAPACITY 3    /* the call would exceed capacity_tokens / max_budget_pages  */
#define RQ_ERR_CUDA 4        /* a CUDA runtime call or launch failed                      */
#define RQ_ERR_TIMEOUT 5     /* a bounded device-side wait ran out (device status only)   */

/* element types */
#define RQ_F32 0
#define RQ_BF16 1

/* Description of a cache.  Supported: head_dim in {64, 128}; page_size in
 * {16, 64}; dtype and gate_dtype each RQ_F32 or RQ_BF16; capacity such that
 * page_capacity <= 32768. */
typedef struct rq_config {
    int32_t batch;            /* B >= 1                                                     */
    int32_t heads;            /* H >= 1                                                     */
    int32_t head_dim;         /* D                                                          */
    int32_t page_size;        /* S, tokens per page                                         */
    int64_t capacity_tokens;  /* most tokens a sequence may ever hold                       */
    int32_t dtype;            /* type of q, k, v, o, the cache and the page bounds          */
    int32_t gate_dtype;       /* type of g                                                  */
    int32_t n_sink_pages;     /* first pages always kept (paper: "the first block"); >= 0   */
    int32_t n_local_pages;    /* newest pages always kept (paper: "local blocks"); >= 0     */
    int32_t max_budget_pages; /* largest budget_pages any later call will pass              */
    int32_t reserved;         /* must be 0                                                  */
} rq_config;

/* Host-side handle: plain data, copyable, holds no resources. */
typedef struct rq_cache {
    rq_config cfg;
    void *kv;
    void *meta;
    void *state;
    void *workspace;
    int64_t len;           /* tokens currently in every sequence                           */
    int64_t page_capacity; /* ceil(capacity_tokens / page_size)                            */
    /* reserved[0]: decode steps taken so far (kept by the library).
     * reserved[1]: testing aid: poll limit of the device-side waits for asynchronous copies;
     *              0 = the built-in limit, < 0 = no poll at all, so that the first wait of every
     *              warp gives up, the kernels let their copies land and return, and the device
     *              status reads RQ_ERR_TIMEOUT; call rq_cache_reset before the cache is used again.
     * reserved[2]: how rq_decode_step runs: 0 = the library chooses, 1 = always as separate
     *              kernels, 2 / 4 / 8 = as one launch with that many groups of heads whenever the
     *              shape allows it.  The results are the same.
     * reserved[3]: must be 0. */
    int64_t reserved[4];
} rq_cache;

/* Bytes the caller must allocate for a configuration.  Host only, no CUDA
 * call.  Any output pointer may be NULL.
 * Errors: INVALID_ARG (NULL cfg, non-positive sizes, bad enums, reserved != 0),
 * UNSUPPORTED (shape outside the supported set). */
RQ_API int rq_sizes(const rq_config *cfg, size_t *kv_bytes, size_t *meta_bytes,
             size_t *state_bytes, size_t *workspace_bytes);

/* Adopt caller-allocated device buffers of at least rq_sizes() bytes each and
 * start an empty cache: enqueues the clearing of the running state and of the
 * workspace's status word; kv and meta are not cleared (every page is
 * initialised when its first token is written).  `out` is host memory.
 * Errors: as rq_sizes; INVALID_ARG for a NULL or not 256-byte-aligned buffer. */
RQ_API int rq_cache_init(rq_cache *out, const rq_config *cfg, void *kv, void *meta,
                  void *state, void *workspace, void *stream);

/* Forget all tokens: len = 0 and zero running state (enqueued on stream). */
RQ_API int rq_cache_reset(rq_cache *cache, void *stream);

/* Prefill [Eq. 1 + App. A.1]: run the gated decay recurrence over T new tokens,
 * continuing from the cache's running state (zero for an empty cache), round
 * every state to the storage dtype, write it to the paged cache at positions
 * len .. len+T-1, bring the min/max of every touched page up to date, leave
 * the fp32 state after the last token in `state`, and set len += T.
 *   k, v : [B][T][H][D] of cfg.dtype, element (b,t,h,d) at
 *          b*stride_b + t*stride_t + h*stride_h + d  (strides in elements, all
 *          multiples of 16 bytes; d contiguous; base 16-byte aligned)
 *   g    : same indexing, of cfg.gate_dtype, values in [0, 1]; the same gate
 *          drives k and v.
 * The same call on the same inputs gives the same bits.  How a prompt is cut into calls, and how the
 * library cuts a long prompt of few heads into time chunks that run side by side, changes the order of
 * the fp32 operations: states agree within rounding (a few 1e-7 relative), not bit for bit.
 * Errors: INVALID_ARG (NULL, T < 0, misaligned), CAPACITY (len + T exceeds
 * capacity_tokens; nothing is enqueued), CUDA.  T == 0 is a no-op. */
RQ_API int rq_build_cache(rq_cache *cache, const void *k, const void *v, const void *g,
                   int64_t T, int64_t stride_b, int64_t stride_t, int64_t stride_h,
                   void *stream);

/* One decode step [Eq. 1, Eq. 3, Eq. 4], in this order: (1) one step of the
 * recurrence with (k_t, v_t, g_t), append the rounded state to the cache,
 * update the newest page's min/max, len += 1; (2) score all pages with q;
 * (3) keep min(budget_pages, #pages) pages per (b,h); (4) attend over their
 * valid tokens — the query sees its own token.  Depending on the shape the
 * step is one kernel launch or several (rq_decode_step_launches); the results
 * are the same.  On an error the cache's length is unchanged.
 *   q, k_t, v_t, o : [B][H][D] contiguous, cfg.dtype;  g_t : [B][H][D], cfg.gate_dtype
 *   budget_pages   : 1 .. cfg.max_budget_pages (>= #pages means dense attention)
 *   scale          : softmax scale; <= 0 selects 1/sqrt(D)
 *   sel_idx_out    : NULL, or int32 [B][H][budget_pages]; receives the kept
 *                    page indices in ascending order, unused tail = -1
 * Errors: INVALID_ARG, CAPACITY (len == capacity_tokens, or budget_pages >
 * max_budget_pages; nothing is enqueued), CUDA. */
RQ_API int rq_decode_step(rq_cache *cache, const void *q, const void *k_t, const void *v_t,
                   const void *g_t, int32_t budget_pages, float scale, void *o,
                   int32_t *sel_idx_out, void *stream);

/* The same step for callers whose tensors live in HOST memory: q, k_t, v_t, g_t are brought
 * to the device, the step runs, o (and sel_idx_out if not NULL) are copied back to host
 * memory, all on `stream`.  Pinned (page-locked or registered), 16-byte aligned inputs are read
 * by one small gather kernel straight from host memory; other inputs go through four
 * asynchronous copies (synchronous for pageable memory, as usual).  A pinned, 16-byte aligned o
 * is written by the attention kernel itself; any other o is filled by a copy from a staging
 * buffer.  The outputs are valid after the stream is synchronised.  Bytes moved per call: 4 inputs + 1 output of B*H*D elements
 * (+ the index list). */
RQ_API int rq_decode_step_host(rq_cache *cache, const void *q_host, const void *k_t_host,
                        const void *v_t_host, const void *g_t_host,
                        int32_t budget_pages, float scale, void *o_host,
                        int32_t *sel_idx_out_host, void *stream);

/* rq_decode_step with per-kernel device timing, for benchmarks: CUDA events are
 * recorded on `stream` between the kernels of the step, the stream is
 * SYNCHRONISED, and the elapsed microseconds of every kernel go to
 * kernel_us[0 .. RQ_PROFILE_SLOTS-1] (host memory), in launch order;
 * rq_profile_slot_name(i) names slot i.  The computation and its results are
 * those of rq_decode_step [Eq. 1, Eq. 3, Eq. 4].
 * Errors: as rq_decode_step; INVALID_ARG for NULL kernel_us. */
#define RQ_PROFILE_SLOTS 3
RQ_API int rq_decode_step_profiled(rq_cache *cache, const void *q, const void *k_t,
                                   const void *v_t, const void *g_t, int32_t budget_pages,
                                   float scale, void *o, int32_t *sel_idx_out,
                                   float *kernel_us, void *stream);

/* Name of the kernel timed in slot i ("" if out of range). */
RQ_API const char *rq_profile_slot_name(int slot);

/* Stage export [Eq. 3 only]: score and select against the current cache without
 * changing it.  scores_out: NULL or fp32 [B][H][P] with P = ceil(len / S);
 * idx_out: int32 [B][H][budget_pages] as in rq_decode_step (must not be NULL).
 * Errors: INVALID_ARG (also for an empty cache), CAPACITY, CUDA. */
RQ_API int rq_select_pages(rq_cache *cache, const void *q, int32_t budget_pages,
                    float *scores_out, int32_t *idx_out, void *stream);

/* Stage export [Eq. 4 only]: attention over caller-chosen pages.
 *   idx : int32 [B][H][n_idx], page indices in [0, P); duplicates are attended
 *         twice; an entry < 0 is skipped; an entry >= P is skipped and sets
 *         the device status to RQ_ERR_INVALID_ARG.
 * At least one valid page per (b,h) is required for a defined result.
 * Errors: INVALID_ARG, CAPACITY (n_idx > max_budget_pages), CUDA. */
RQ_API int rq_attend_pages(rq_cache *cache, const void *q, const int32_t *idx, int32_t n_idx,
                    float scale, void *o, void *stream);

/* The paper has no counterpart to this entry point; it exists for one kind of caller.
 *
 * rq_attend_pages for callers that are not allowed to allocate device memory and therefore
 * have no workspace to hand over: a plug-in inside a serving engine that owns every byte of
 * the GPU, code on a latency path where cudaMalloc is banned because it synchronises the
 * device, a process whose memory pool is already carved up.  Such a caller passes only the
 * inputs (the paged cache it already holds, the query, the page list) and the output; the
 * partial results and counters of the kernel live in a fixed 4 MiB array that is part of the
 * library's image on every GPU that loads it, until the process exits.
 *   cfg      : the configuration the cache was built with (host memory)
 *   kv       : the paged cache, layout as above (device)
 *   len      : tokens in every sequence, 1 .. cfg->capacity_tokens
 *   q, o     : [B][H][D] of cfg->dtype (device);  idx : int32 [B][H][n_idx] as in rq_attend_pages,
 *              except that an entry >= P is skipped without being reported
 *   scale    : softmax scale; <= 0 selects 1/sqrt(D)
 * Limit: 256 + B*H*256 + B*H*r*(D+4)*4 bytes must fit in the 4 MiB, where r is the number of
 * partial records per head (CTAs per head, about 2 * SMs / (B*H), when B*H is at most the
 * number of resident CTAs; otherwise up to 4 per CTA); the headline shape (B*H = 32, D = 128)
 * needs 0.16 MiB.  A shape beyond the limit is refused with RQ_ERR_CAPACITY before anything is
 * enqueued.  The call allocates nothing and calls no allocating routine; it enqueues one small
 * memset (status and counters must start at zero: the array keeps what the last call left) and
 * one kernel on `stream` and returns without synchronising.
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress) and
 * sets a kernel attribute; make that first call outside any stream capture.
 * All calls share the one array: two calls whose kernels overlap on the GPU (different streams,
 * or different host threads) race on it and give wrong results; calls on one stream are safe.
 * Errors: as rq_sizes for cfg; INVALID_ARG (NULL pointer, n_idx < 1, len out of range);
 * CAPACITY (shape beyond the limit); CUDA. */
RQ_API int rq_attend_pages_noalloc(const rq_config *cfg, const void *kv, int64_t len, const void *q,
                                   const int32_t *idx, int32_t n_idx, float scale, void *o,
                                   void *stream);

/* SnapKV-style reduction of the cache [App. A.1, "Sparse inference settings", SnapKV paragraph;
 * Sec. 2.2, Table 1]: after the prompt, the queries of its last `window` positions (the
 * observation window, at most 64; the paper uses 64) rate every position by the attention they pay
 * to it, importance[j] = sum_i softmax_j(scale * q_i . k~_j) with query i (at position len - window
 * + i) seeing the positions up to its own; the `keep` most important entries are retained: the
 * window's own positions always (they count inside keep), then the most important earlier
 * positions, equal importance to the lower position.
 *   q_window       : [B][window][H][D] of cfg.dtype (device)
 *   idx_out        : int32 [B][H][keep] (device): retained positions, ascending; -1 beyond len
 *   importance_out : NULL or fp32 [B][H][len] (device)
 *   scratch        : device memory of rq_snapkv_scratch_bytes() bytes for the cache's current
 *                    length, 256-byte aligned, free again when the call's work has run
 *   scale          : softmax scale; <= 0 selects 1/sqrt(D)
 * Errors: INVALID_ARG (NULL, window outside 1..64 or longer than the cache, keep < 1), CUDA. */
RQ_API int rq_snapkv_scratch_bytes(const rq_cache *cache, size_t *bytes);
RQ_API int rq_snapkv_select(rq_cache *cache, const void *q_window, int32_t window, int32_t keep, float scale,
                            int32_t *idx_out, float *importance_out, void *scratch, void *stream);

/* The second half of the reduction [same passage: only the selected entries stay in the cache and
 * later attention runs over them alone]: copies the `keep` positions idx[b][h][0..keep)
 * (ascending, all < len) of every head of `src` into `dst`, an initialised cache of the same shape
 * and types with capacity_tokens >= keep (plus the tokens to be decoded), as its positions
 * 0..keep-1; rebuilds the page bounds of dst from the copied keys and carries the recurrence state
 * over, so that rq_decode_step on dst continues Eq. 1 and attends over the retained entries and
 * the tokens appended since (with budget_pages >= its pages: over all of them).  Whatever dst held
 * is dropped.
 * Errors: INVALID_ARG (shapes differ, dst is src, keep outside 1..len), CAPACITY, CUDA. */
RQ_API int rq_snapkv_compact(const rq_cache *src, const int32_t *idx, int32_t keep, rq_cache *dst, void *stream);

/* MoBA-style block-sparse PREFILL attention over the cache the prompt was prefilled into [Sec. 2.2,
 * Eq. 3 and Eq. 4, Table 1 row MoBA; App. A.1, "Sparse inference settings", MoBA paragraph]: the
 * query of every prompt position t is routed to budget_blocks KV blocks of `block` positions: the
 * complete blocks before its own are scored with their mean-pooled representatives (q . mean of the
 * block's stored decayed keys) and the best are taken, equal scores to the lower block; the first
 * block and the query's own block are always taken and count inside budget_blocks; with fewer
 * blocks than that before it, a query attends everything before it.  Attention is softmax over the
 * positions <= t of the chosen blocks, on the decayed keys and values as stored.
 *   q          : [B][T][H][D] of cfg.dtype (device), T = the cache's current length
 *   block      : 64, 128, ... (a multiple of 64 and of the page size); at most 2048 blocks per prompt
 *   o          : [B][T][H][D] of cfg.dtype (device)
 *   blocks_out : NULL or int32 [B][H][T][budget_blocks] (device): chosen blocks, ascending, -1 beyond
 *   means_out  : NULL or fp32 [B][H][blocks][D] (device): the representatives
 *   scratch    : device memory of rq_moba_scratch_bytes() bytes, 256-byte aligned
 *   scale      : softmax scale; <= 0 selects 1/sqrt(D)
 * Errors: INVALID_ARG (NULL, empty cache, block or budget_blocks < 2 out of range), CUDA. */
RQ_API int rq_moba_scratch_bytes(const rq_cache *cache, int32_t block, int32_t budget_blocks, size_t *bytes);
RQ_API int rq_moba_prefill(rq_cache *cache, const void *q, int32_t block, int32_t budget_blocks, float scale, void *o,
                           int32_t *blocks_out, float *means_out, void *scratch, void *stream);

/* Tokens in the cache (host bookkeeping; no CUDA call).  -1 for NULL. */
RQ_API int64_t rq_cache_len(const rq_cache *cache);

/* Kernel launches the next rq_decode_step on this cache will enqueue for this budget when
 * sel_idx_out is NULL [no counterpart in the paper: bookkeeping for benchmarks]: ONE when the whole
 * step runs as one launch (chosen by the library for 64 to 128 (batch, head) pairs of 4096 to
 * 12284 pages each that split into 4, 8 or 2 equal groups which keep the GPU's resident CTAs
 * busy, budget below the number of pages; cache.reserved[2] asks for it on other shapes);
 * otherwise three (update + scoring, selection, attention), or two when the context is short
 * enough (at most 256 pages per head, at least 16 heads) for one CTA per head to do the first
 * two kernels' work in one launch.  A non-NULL sel_idx_out can add a launch that sorts the list.
 * The first call on a device looks up launch parameters (occupancy).  -1 for an invalid cache. */
RQ_API int rq_decode_step_launches(const rq_cache *cache, int32_t budget_pages);

/* Benchmarking aid [no counterpart in the paper]: one launch that reads `bytes` bytes (rounded
 * down to a multiple of 16) of device memory at `buf` (16-byte aligned) once, with plain 16-byte
 * loads, and folds them into the 64 words at `sink` (device memory, 256 bytes, 4-byte aligned).
 * Timed by the caller, it shows what a single launch of the decode step's size can draw from
 * HBM on the GPU at hand.  Enqueued on `stream`; returns INVALID_ARG or CUDA on failure. */
RQ_API int rq_probe_read(const void *buf, size_t bytes, void *sink, void *stream);

/* Synchronises `stream`, reads the device status word into *status_out (host
 * memory; RQ_OK if no kernel reported anything) and clears it.
 * Returns RQ_OK, INVALID_ARG or CUDA. */
RQ_API int rq_device_status(rq_cache *cache, int32_t *status_out, void *stream);

/* Static text for a status code; never NULL. */
RQ_API const char *rq_status_string(int status);

/* RQ_VERSION_MAJOR * 1000 + RQ_VERSION_MINOR of the loaded library. */
RQ_API int rq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RQ_H_ */
