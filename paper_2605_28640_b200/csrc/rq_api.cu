// Host side of the C ABI declared in rq.h: argument checks, workspace carving
// and kernel sequencing.  No device memory is allocated here.
#include <math.h>
#include <string.h>

#include "rq_internal.h"

namespace rq {

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

static int check_config(const rq_config *c)
{
    if (!c) return RQ_ERR_INVALID_ARG;
    if (c->batch < 1 || c->heads < 1 || c->head_dim < 1 || c->page_size < 1 || c->capacity_tokens < 1)
        return RQ_ERR_INVALID_ARG;
    if ((c->dtype != RQ_F32 && c->dtype != RQ_BF16) || (c->gate_dtype != RQ_F32 && c->gate_dtype != RQ_BF16))
        return RQ_ERR_INVALID_ARG;
    if (c->n_sink_pages < 0 || c->n_local_pages < 0 || c->max_budget_pages < 1 || c->reserved != 0)
        return RQ_ERR_INVALID_ARG;
    if (c->head_dim != 64 && c->head_dim != 128) return RQ_ERR_UNSUPPORTED;
    if (c->page_size != 16 && c->page_size != 64) return RQ_ERR_UNSUPPORTED;
    const int64_t pc = (c->capacity_tokens + c->page_size - 1) / c->page_size;
    if (pc > (int64_t)kTopkThreads * kTopkMaxPerThread) return RQ_ERR_UNSUPPORTED;
    if ((int64_t)c->batch * c->heads > 65535) return RQ_ERR_UNSUPPORTED;
    return RQ_OK;
}

static size_t elem_size(int dtype) { return dtype == RQ_BF16 ? 2 : 4; }

WorkspaceLayout workspace_layout(const rq_config &c)
{
    WorkspaceLayout w;
    const size_t BH = (size_t)c.batch * c.heads;
    const size_t pc = (size_t)((c.capacity_tokens + c.page_size - 1) / c.page_size);
    size_t off = 0;
    w.status = off;  off += align256(64 * sizeof(int32_t));
    w.tickets = off; off += align256(BH * (size_t)kCtrStride * sizeof(int32_t));
    const size_t SH = BH <= (size_t)kStepMaxHeads ? BH : 0;      // heads the one-launch step keeps records for
    w.absmax = off;   off += align256(2 * SH * sizeof(float));
    w.step_ctr = off; off += align256(2 * SH * (size_t)kStepCtrInts * sizeof(int32_t));
    w.list = off;     off += align256(SH * (size_t)c.max_budget_pages * sizeof(int2));
    w.hist = off;     off += align256(SH * (size_t)kStepBins * sizeof(uint32_t));
    w.range = off;    off += align256(SH * sizeof(float2));
    w.scores = off;  off += align256(BH * pc * sizeof(float));
    w.sel = off;     off += align256(BH * (size_t)c.max_budget_pages * sizeof(int32_t));
    const size_t slots = (size_t)attend_slots_per_head((int64_t)c.max_budget_pages * (c.page_size / 16));
    w.partial = off; off += align256(BH * slots * (size_t)(c.head_dim + 4) * sizeof(float));
    w.staging = off; off += align256(5 * BH * (size_t)c.head_dim * 4);
    w.scan = off;    off += align256(kScanScratchBytes);
    w.total = off;
    return w;
}

}  // namespace rq (reopened below)

int rq::stream_grid(int64_t units, int heads, int resident_ctas, int warps_per_cta, int max_ctas)
{
    int64_t g = units / (2 * warps_per_cta);
    if (g > resident_ctas) g = resident_ctas;
    if (g > max_ctas) g = max_ctas;
    // whole CTAs per head when that leaves at most 15 % of the CTAs out; otherwise all CTAs run
    // and their warps spread over the heads on their own (the kernels handle both)
    if (g >= heads && heads > 0 && (g - g % heads) * 100 >= g * 85) g -= g % heads;
    if (g < 1) g = 1;
    return (int)g;
}

namespace rq {

// SMs of the current device, looked up once per device.  (These per-device tables, like the ones
// in the launchers, are filled without a lock: two threads that make their first call on a device
// at the same time both look the value up and store the same number.)
int sm_count()
{
    static int cached[64];
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return kTargetSMs;
    if (cached[dev] == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            cached[dev] = n;
        else
            cached[dev] = kTargetSMs;
    }
    return cached[dev];
}

// rq_cache::reserved: [0] number of decode steps taken; a step works as step number reserved[0] + 1
// and commits that number when all its launches succeeded.  (Its parity picks the copy of the
// heads' largest |stored key| that the step reads, the update writing the other one, and the set of
// per-head counters the one-launch step uses, the step clearing the other one.)  [1] poll limit of
// device-side copy waits (0: the default, < 0: none at all; a testing aid), [2] choice of the decode
// path (0: automatic, 1: always the separate kernels, 2, 4, 8: the one-launch step with that many
// waves whenever the shape allows it)
static float *absmax_of(const rq_cache *c)
{
    if ((int64_t)c->cfg.batch * c->cfg.heads > kStepMaxHeads) return nullptr;
    return (float *)((char *)c->workspace + workspace_layout(c->cfg).absmax);
}

static DecodeArgs decode_args(const rq_cache *c, int64_t len)
{
    DecodeArgs a;
    a.absmax = absmax_of(c);
    a.epoch = (int32_t)((c->reserved[0] + 1) & 0x3fffffff);
    a.poll_limit = (int32_t)c->reserved[1];
    a.kv = c->kv; a.meta = c->meta; a.state = (float *)c->state;
    a.B = c->cfg.batch; a.H = c->cfg.heads; a.D = c->cfg.head_dim; a.S = c->cfg.page_size;
    a.dtype = c->cfg.dtype; a.gate_dtype = c->cfg.gate_dtype;
    a.len = len; a.page_cap = c->page_capacity;
    a.n_sink = c->cfg.n_sink_pages; a.n_local = c->cfg.n_local_pages;
    a.status = (int32_t *)((char *)c->workspace + workspace_layout(c->cfg).status);
    return a;
}

static bool aligned(const void *p, size_t a) { return ((uintptr_t)p & (a - 1)) == 0; }

static int check_cache(const rq_cache *c)
{
    if (!c || !c->kv || !c->meta || !c->state || !c->workspace) return RQ_ERR_INVALID_ARG;
    return check_config(&c->cfg);
}

// Optional per-kernel timing: when `ev` is not NULL an event is recorded after
// every kernel of a decode step (ev[0] before the first one).
static void mark(cudaEvent_t *ev, int i, cudaStream_t s)
{
    if (ev) cudaEventRecord(ev[i], s);
}

// (optionally append a token, then) score + select into `idx` (device, stride idx_stride), for a
// cache of length len after the append.  *unordered: the list came out in no particular order.
static int select_into(const rq_cache *c, int64_t len, const void *q, const void *k_t, const void *v_t,
                       const void *g_t, int do_update, int budget, float *scores, int32_t *idx, int idx_stride,
                       cudaStream_t s, cudaEvent_t *ev = nullptr, bool *unordered = nullptr)
{
    DecodeArgs a = decode_args(c, len);
    const WorkspaceLayout w = workspace_layout(c->cfg);
    int32_t *ctr = (int32_t *)((char *)c->workspace + w.tickets);
    const int64_t P = (len + c->cfg.page_size - 1) / c->cfg.page_size;
    if (unordered) *unordered = false;
    if (P <= kSmallStepPages && c->cfg.batch * c->cfg.heads >= kSmallStepMinHeads) {
        // a short context: one launch instead of two (the per-kernel marks then show the whole under "score")
        int32_t *other = a.absmax && do_update ? (int32_t *)((char *)c->workspace + w.step_ctr) +
                                                     (size_t)((a.epoch & 1) ^ 1) * a.B * a.H * kStepCtrInts
                                               : nullptr;
        if (launch_score_select(a, q, k_t, v_t, g_t, scores, do_update, budget, idx, idx_stride, ctr, do_update, other, s) !=
            cudaSuccess)
            return RQ_ERR_CUDA;
        mark(ev, 1, s);
        mark(ev, 2, s);
        return RQ_OK;
    }
    // forced pages inside the budget (sinks first, then local pages from the newest backwards): the
    // scoring kernel leaves them out of its histogram, the selection takes them outright
    const int K = (int)(budget < P ? budget : P);
    int ns = a.n_sink < K ? a.n_sink : K;
    if (ns > P) ns = (int)P;
    int nl = a.n_local < K - ns ? a.n_local : K - ns;
    if (nl > P - ns) nl = (int)(P - ns);
    a.n_sink = ns;
    a.n_local = nl;
    // the scoring kernel counts the scores into value buckets for the selection when the heads are
    // few and short enough for that path and the budget leaves something to select
    ScoreHist hs = {nullptr, nullptr, nullptr};
    if (a.absmax) {
        char *ws = (char *)c->workspace;
        if (do_update) hs.ctr_other = (int32_t *)(ws + w.step_ctr) + (size_t)((a.epoch & 1) ^ 1) * a.B * a.H * kStepCtrInts;
        if (topk_uses_hist(P) && K < P) {
            hs.hist = (uint32_t *)(ws + w.hist);
            hs.range = (float2 *)(ws + w.range);
            if (unordered) *unordered = true;
        }
    }
    if (launch_score(a, q, k_t, v_t, g_t, scores, ctr + 3, do_update, hs, sm_count(), s) != cudaSuccess) return RQ_ERR_CUDA;
    mark(ev, 1, s);
    if (launch_topk(a, scores, budget, idx, idx_stride, ctr, do_update, hs, s) != cudaSuccess) return RQ_ERR_CUDA;
    mark(ev, 2, s);
    return RQ_OK;
}

static int attend_from(const rq_cache *c, int64_t len, const void *q, const int32_t *idx, int n_idx,
                       int idx_stride, float scale, void *o, cudaStream_t s, cudaEvent_t *ev = nullptr)
{
    DecodeArgs a = decode_args(c, len);
    const WorkspaceLayout w = workspace_layout(c->cfg);
    float *partial = (float *)((char *)c->workspace + w.partial);
    if (!(scale > 0.0f)) scale = 1.0f / sqrtf((float)a.D);
    int32_t *tickets = (int32_t *)((char *)c->workspace + w.tickets);
    const AttendCounters ctr = {tickets, tickets + 1, tickets + 2};
    if (launch_attend(a, q, idx, n_idx, idx_stride, scale, partial, ctr, o, sm_count(), s) != cudaSuccess)
        return RQ_ERR_CUDA;
    mark(ev, 3, s);
    return RQ_OK;
}

static StepBuffers step_buffers(const rq_cache *c, const WorkspaceLayout &w)
{
    StepBuffers b;
    char *ws = (char *)c->workspace;
    b.scores = (float *)(ws + w.scores);
    b.list = (int2 *)(ws + w.list);
    b.list_stride = c->cfg.max_budget_pages;
    b.partial = (float *)(ws + w.partial);
    b.slots = attend_slots_per_head((int64_t)c->cfg.max_budget_pages * (c->cfg.page_size / 16));
    b.ctr = (int32_t *)(ws + w.step_ctr);
    b.hist = (uint32_t *)(ws + w.hist);
    return b;
}

// Waves of the one-launch step for the next decode step (args for the length after the append),
// 0 if the step runs as separate kernels.
static int step_waves(const rq_cache *c, const DecodeArgs &a, int budget, int *grid)
{
    const int64_t choice = c->reserved[2];
    if (choice == 1) return 0;
    const int forced = choice == 2 || choice == 4 || choice == 8 ? (int)choice : 0;
    const int waves = step_plan(a, budget, sm_count(), forced, grid);
    if (waves <= 0) return 0;
    const int team = *grid / (a.B * a.H / waves);
    const int slots = attend_slots_per_head((int64_t)c->cfg.max_budget_pages * (c->cfg.page_size / 16));
    return team <= slots ? waves : 0;
}

static int decode_step_impl(rq_cache *cache, const void *q, const void *k_t, const void *v_t,
                            const void *g_t, int32_t budget_pages, float scale, void *o,
                            int32_t *sel_idx_out, cudaStream_t s, cudaEvent_t *ev)
{
    const int rc = check_cache(cache);
    if (rc != RQ_OK) return rc;
    if (!q || !k_t || !v_t || !g_t || !o || budget_pages < 1) return RQ_ERR_INVALID_ARG;
    const rq_config &c = cache->cfg;
    if (budget_pages > c.max_budget_pages) return RQ_ERR_CAPACITY;
    if (cache->len >= c.capacity_tokens) return RQ_ERR_CAPACITY;
    const WorkspaceLayout w = workspace_layout(c);
    float *scores = (float *)((char *)cache->workspace + w.scores);
    int32_t *sel = sel_idx_out ? sel_idx_out : (int32_t *)((char *)cache->workspace + w.sel);

    mark(ev, 0, s);
    // the length and the step number are committed only when every launch of the step succeeded
    const int64_t new_len = cache->len + 1;
    const int64_t P = (new_len + c.page_size - 1) / c.page_size;
    int st;
    int grid = 0;
    DecodeArgs a = decode_args(cache, new_len);
    const int waves = step_waves(cache, a, budget_pages, &grid);
    if (waves > 0) {
        // one launch; the list lands in the workspace in no particular order and is sorted for the caller
        const StepBuffers b = step_buffers(cache, w);
        if (!(scale > 0.0f)) scale = 1.0f / sqrtf((float)a.D);
        st = launch_step(a, q, k_t, v_t, g_t, budget_pages, scale, b, o, waves, grid, s) == cudaSuccess ? RQ_OK : RQ_ERR_CUDA;
        mark(ev, 1, s);
        if (st == RQ_OK && sel_idx_out &&
            launch_sort_list(b.list, b.list_stride, budget_pages, (int)P, a.B * a.H, sel_idx_out, budget_pages, s) != cudaSuccess)
            st = RQ_ERR_CUDA;
        mark(ev, 2, s);
        mark(ev, 3, s);
        if (st == RQ_OK) cache->reserved[0] += 1;
    } else {
        bool unordered = false;
        st = select_into(cache, new_len, q, k_t, v_t, g_t, 1, budget_pages, scores, sel, budget_pages, s, ev, &unordered);
        if (st == RQ_OK) {
            const int n_idx = (int)(budget_pages < P ? budget_pages : P);
            st = attend_from(cache, new_len, q, sel, n_idx, budget_pages, scale, o, s, ev);
        }
        // the caller's copy of the list is ascending (in place, behind the attention kernel, which does not care)
        if (st == RQ_OK && unordered && sel_idx_out &&
            launch_sort_list32(sel, budget_pages, budget_pages, (int)P, c.batch * c.heads, sel, budget_pages, s) != cudaSuccess)
            st = RQ_ERR_CUDA;
        if (st == RQ_OK) cache->reserved[0] += 1;
    }
    if (st != RQ_OK) return st;
    cache->len = new_len;
    return RQ_OK;
}

// Gather of the four per-step input tensors from pinned host memory (read over the bus by the
// device) into the staging area: nv 16-byte vectors each for q, k_t, v_t and ng for g_t.
__global__ void stage_in_kernel(const uint4 *q, const uint4 *k, const uint4 *v, const uint4 *g, uint4 *dq,
                                uint4 *dk, uint4 *dv, uint4 *dg, int nv, int ng)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < nv) { dq[i] = q[i]; return; }
    i -= nv;
    if (i < nv) { dk[i] = k[i]; return; }
    i -= nv;
    if (i < nv) { dv[i] = v[i]; return; }
    i -= nv;
    if (i < ng) dg[i] = g[i];
}

// Plain streaming read of a buffer: 16-byte loads, eight in flight per thread, the words folded
// into one value per CTA so that the loads cannot be dropped.  A yardstick for what one launch of
// a given size can draw from HBM, nothing of the method.
__global__ void __launch_bounds__(256) probe_read_kernel(const uint4 *src, size_t n16, uint32_t *sink)
{
    constexpr int U = 8;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    uint32_t acc = 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += stride * U) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t j = i + (size_t)u * stride;
            v[u] = j < n16 ? __ldcs(src + j) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
    acc = __reduce_xor_sync(0xffffffffu, acc);
    if ((threadIdx.x & 31) == 0) atomicXor(sink + (blockIdx.x & 63), acc);
}

// Device address of a host buffer if it is pinned (or registered) and 16-byte aligned.
static bool device_view(const void *host, const void **dev)
{
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    if (at.type != cudaMemoryTypeHost || !at.devicePointer || ((uintptr_t)at.devicePointer & 15)) return false;
    *dev = at.devicePointer;
    return true;
}

}  // namespace rq

using namespace rq;

extern "C" {

int rq_sizes(const rq_config *cfg, size_t *kv_bytes, size_t *meta_bytes, size_t *state_bytes,
             size_t *workspace_bytes)
{
    const int rc = check_config(cfg);
    if (rc != RQ_OK) return rc;
    const size_t BH = (size_t)cfg->batch * cfg->heads;
    const size_t pc = (size_t)((cfg->capacity_tokens + cfg->page_size - 1) / cfg->page_size);
    const size_t es = elem_size(cfg->dtype);
    if (kv_bytes) *kv_bytes = BH * pc * 2 * cfg->page_size * cfg->head_dim * es;
    if (meta_bytes) *meta_bytes = BH * pc * 2 * cfg->head_dim * es;
    if (state_bytes) *state_bytes = BH * 2 * cfg->head_dim * sizeof(float);
    if (workspace_bytes) *workspace_bytes = workspace_layout(*cfg).total;
    return RQ_OK;
}

int rq_cache_init(rq_cache *out, const rq_config *cfg, void *kv, void *meta, void *state,
                  void *workspace, void *stream)
{
    if (!out) return RQ_ERR_INVALID_ARG;
    const int rc = check_config(cfg);
    if (rc != RQ_OK) return rc;
    if (!kv || !meta || !state || !workspace) return RQ_ERR_INVALID_ARG;
    if (!aligned(kv, 256) || !aligned(meta, 256) || !aligned(state, 256) || !aligned(workspace, 256))
        return RQ_ERR_INVALID_ARG;
    memset(out, 0, sizeof(*out));
    out->cfg = *cfg;
    out->kv = kv; out->meta = meta; out->state = state; out->workspace = workspace;
    out->page_capacity = (cfg->capacity_tokens + cfg->page_size - 1) / cfg->page_size;
    return rq_cache_reset(out, stream);
}

int rq_cache_reset(rq_cache *cache, void *stream)
{
    const int rc = check_cache(cache);
    if (rc != RQ_OK) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t BH = (size_t)cache->cfg.batch * cache->cfg.heads;
    const WorkspaceLayout w = workspace_layout(cache->cfg);
    if (cudaMemsetAsync(cache->state, 0, BH * 2 * cache->cfg.head_dim * sizeof(float), s) != cudaSuccess)
        return RQ_ERR_CUDA;
    // status word and the split-K arrival counters (adjacent regions)
    if (cudaMemsetAsync((char *)cache->workspace + w.status, 0, w.scores - w.status, s) != cudaSuccess)
        return RQ_ERR_CUDA;
    cache->len = 0;
    return RQ_OK;
}

int rq_build_cache(rq_cache *cache, const void *k, const void *v, const void *g, int64_t T,
                   int64_t stride_b, int64_t stride_t, int64_t stride_h, void *stream)
{
    const int rc = check_cache(cache);
    if (rc != RQ_OK) return rc;
    if (T < 0) return RQ_ERR_INVALID_ARG;
    if (T == 0) return RQ_OK;
    if (!k || !v || !g) return RQ_ERR_INVALID_ARG;
    const rq_config &c = cache->cfg;
    // 16-byte vectors of the narrower of the two element types must stay aligned
    const size_t es = elem_size(c.dtype), gs = elem_size(c.gate_dtype);
    const size_t emin = es < gs ? es : gs;
    if (!aligned(k, 16) || !aligned(v, 16) || !aligned(g, 16)) return RQ_ERR_INVALID_ARG;
    if (stride_b < 0 || stride_t < 0 || stride_h < 0) return RQ_ERR_INVALID_ARG;
    if ((stride_b * emin) % 16 || (stride_t * emin) % 16 || (stride_h * emin) % 16) return RQ_ERR_INVALID_ARG;
    if (cache->len + T > c.capacity_tokens) return RQ_ERR_CAPACITY;
    const WorkspaceLayout w = workspace_layout(c);
    ScanArgs a;
    a.k = k; a.v = v; a.g = g;
    a.sb = stride_b; a.st = stride_t; a.sh = stride_h;
    a.kv = cache->kv; a.meta = cache->meta; a.state = (float *)cache->state;
    a.B = c.batch; a.H = c.heads; a.D = c.head_dim; a.S = c.page_size;
    a.dtype = c.dtype; a.gate_dtype = c.gate_dtype;
    a.len0 = cache->len; a.T = T; a.page_cap = cache->page_capacity;
    a.absmax = absmax_of(cache);
    a.chunk_scratch = (float *)((char *)cache->workspace + w.scan);
    if (launch_scan(a, (cudaStream_t)stream) != cudaSuccess) return RQ_ERR_CUDA;
    cache->len += T;
    return RQ_OK;
}

int rq_decode_step(rq_cache *cache, const void *q, const void *k_t, const void *v_t, const void *g_t,
                   int32_t budget_pages, float scale, void *o, int32_t *sel_idx_out, void *stream)
{
    return decode_step_impl(cache, q, k_t, v_t, g_t, budget_pages, scale, o, sel_idx_out,
                            (cudaStream_t)stream, nullptr);
}

int rq_decode_step_profiled(rq_cache *cache, const void *q, const void *k_t, const void *v_t,
                            const void *g_t, int32_t budget_pages, float scale, void *o,
                            int32_t *sel_idx_out, float *kernel_us, void *stream)
{
    if (!kernel_us) return RQ_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    cudaEvent_t ev[RQ_PROFILE_SLOTS + 1];
    int made = 0;
    for (; made <= RQ_PROFILE_SLOTS; ++made)
        if (cudaEventCreate(&ev[made]) != cudaSuccess) break;
    int st = made == RQ_PROFILE_SLOTS + 1 ? RQ_OK : RQ_ERR_CUDA;
    if (st == RQ_OK)
        st = decode_step_impl(cache, q, k_t, v_t, g_t, budget_pages, scale, o, sel_idx_out, s, ev);
    if (st == RQ_OK && cudaStreamSynchronize(s) != cudaSuccess) st = RQ_ERR_CUDA;
    if (st == RQ_OK) {
        for (int i = 0; i < RQ_PROFILE_SLOTS; ++i) {
            float ms = 0.0f;
            if (cudaEventElapsedTime(&ms, ev[i], ev[i + 1]) != cudaSuccess) st = RQ_ERR_CUDA;
            kernel_us[i] = ms * 1000.0f;
        }
    }
    for (int i = 0; i < made; ++i) cudaEventDestroy(ev[i]);
    return st;
}

const char *rq_profile_slot_name(int slot)
{
    // (when the step runs as one launch, slot 0 holds the whole step and slot 1 the sorting of the list)
    static const char *names[RQ_PROFILE_SLOTS] = {"score", "topk", "attend"};
    return slot >= 0 && slot < RQ_PROFILE_SLOTS ? names[slot] : "";
}

int rq_decode_step_host(rq_cache *cache, const void *q_host, const void *k_t_host,
                        const void *v_t_host, const void *g_t_host, int32_t budget_pages, float scale,
                        void *o_host, int32_t *sel_idx_out_host, void *stream)
{
    const int rc = check_cache(cache);
    if (rc != RQ_OK) return rc;
    if (!q_host || !k_t_host || !v_t_host || !g_t_host || !o_host || budget_pages < 1)
        return RQ_ERR_INVALID_ARG;
    const rq_config &c = cache->cfg;
    if (budget_pages > c.max_budget_pages) return RQ_ERR_CAPACITY;
    if (cache->len >= c.capacity_tokens) return RQ_ERR_CAPACITY;
    cudaStream_t s = (cudaStream_t)stream;
    const WorkspaceLayout w = workspace_layout(c);
    const size_t n = (size_t)c.batch * c.heads * c.head_dim;
    const size_t slot = n * 4;
    char *stg = (char *)cache->workspace + w.staging;
    void *dq = stg, *dk = stg + slot, *dv = stg + 2 * slot, *dg = stg + 3 * slot, *dout = stg + 4 * slot;
    const size_t eb = n * elem_size(c.dtype), gb = n * elem_size(c.gate_dtype);
    // Pinned host buffers are readable from the device: one small kernel gathers all four into
    // the staging area (one launch instead of four copies).  Anything else goes through copies.
    const void *src[4] = {q_host, k_t_host, v_t_host, g_t_host};
    const void *dsrc[4];
    bool direct = true;
    for (int i = 0; i < 4 && direct; ++i) direct = device_view(src[i], &dsrc[i]);
    if (direct) {
        const int nv = (int)(eb / 16), ng = (int)(gb / 16);
        const int total = 3 * nv + ng;
        stage_in_kernel<<<(total + 255) / 256, 256, 0, s>>>((const uint4 *)dsrc[0], (const uint4 *)dsrc[1],
                                                           (const uint4 *)dsrc[2], (const uint4 *)dsrc[3],
                                                           (uint4 *)dq, (uint4 *)dk, (uint4 *)dv, (uint4 *)dg, nv, ng);
        if (cudaGetLastError() != cudaSuccess) return RQ_ERR_CUDA;
    } else if (cudaMemcpyAsync(dq, q_host, eb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
               cudaMemcpyAsync(dk, k_t_host, eb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
               cudaMemcpyAsync(dv, v_t_host, eb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
               cudaMemcpyAsync(dg, g_t_host, gb, cudaMemcpyHostToDevice, s) != cudaSuccess) {
        return RQ_ERR_CUDA;
    }
    int32_t *sel = (int32_t *)((char *)cache->workspace + w.sel);
    // A pinned output buffer is writable from the device: the kernel that produces the output
    // writes it there itself, which saves the copy operation behind it.
    const void *o_view = nullptr;
    const bool o_direct = device_view(o_host, &o_view);
    const int st = rq_decode_step(cache, dq, dk, dv, dg, budget_pages, scale, o_direct ? const_cast<void *>(o_view) : dout,
                                  sel_idx_out_host ? sel : nullptr, stream);
    if (st != RQ_OK) return st;
    if (!o_direct && cudaMemcpyAsync(o_host, dout, eb, cudaMemcpyDeviceToHost, s) != cudaSuccess) return RQ_ERR_CUDA;
    if (sel_idx_out_host) {
        const size_t ib = (size_t)c.batch * c.heads * budget_pages * sizeof(int32_t);
        if (cudaMemcpyAsync(sel_idx_out_host, sel, ib, cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return RQ_ERR_CUDA;
    }
    return RQ_OK;
}

int rq_select_pages(rq_cache *cache, const void *q, int32_t budget_pages, float *scores_out,
                    int32_t *idx_out, void *stream)
{
    const int rc = check_cache(cache);
    if (rc != RQ_OK) return rc;
    if (!q || !idx_out || budget_pages < 1 || cache->len < 1) return RQ_ERR_INVALID_ARG;
    const rq_config &c = cache->cfg;
    if (budget_pages > c.max_budget_pages) return RQ_ERR_CAPACITY;
    cudaStream_t s = (cudaStream_t)stream;
    const WorkspaceLayout w = workspace_layout(c);
    float *scores = (float *)((char *)cache->workspace + w.scores);
    bool unordered = false;
    const int st = select_into(cache, cache->len, q, nullptr, nullptr, nullptr, 0, budget_pages, scores, idx_out, budget_pages, s,
                               nullptr, &unordered);
    if (st != RQ_OK) return st;
    const int64_t Pn = (cache->len + c.page_size - 1) / c.page_size;
    if (unordered && launch_sort_list32(idx_out, budget_pages, budget_pages, (int)Pn, c.batch * c.heads, idx_out, budget_pages,
                                        s) != cudaSuccess)
        return RQ_ERR_CUDA;
    if (scores_out) {
        const int64_t P = (cache->len + c.page_size - 1) / c.page_size;
        // workspace rows are page_capacity apart; the caller's are P apart
        if (cudaMemcpy2DAsync(scores_out, (size_t)P * sizeof(float), scores,
                              (size_t)cache->page_capacity * sizeof(float), (size_t)P * sizeof(float),
                              (size_t)c.batch * c.heads, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
            return RQ_ERR_CUDA;
    }
    return RQ_OK;
}

int rq_attend_pages(rq_cache *cache, const void *q, const int32_t *idx, int32_t n_idx, float scale,
                    void *o, void *stream)
{
    const int rc = check_cache(cache);
    if (rc != RQ_OK) return rc;
    if (!q || !idx || !o || n_idx < 1 || cache->len < 1) return RQ_ERR_INVALID_ARG;
    if (n_idx > cache->cfg.max_budget_pages) return RQ_ERR_CAPACITY;
    // the flash-decode counters must be zero at launch (in a decode step the selection kernel does this)
    const WorkspaceLayout w = workspace_layout(cache->cfg);
    if (cudaMemsetAsync((char *)cache->workspace + w.tickets, 0, w.scores - w.tickets, (cudaStream_t)stream) != cudaSuccess)
        return RQ_ERR_CUDA;
    return attend_from(cache, cache->len, q, idx, n_idx, n_idx, scale, o, (cudaStream_t)stream);
}

int rq_probe_read(const void *buf, size_t bytes, void *sink, void *stream)
{
    if (!buf || !sink || bytes < 16 || !aligned(buf, 16) || !aligned(sink, 4)) return RQ_ERR_INVALID_ARG;
    const size_t n16 = bytes / 16;
    size_t ctas = (n16 + 256 * 8 - 1) / (256 * 8);
    const size_t most = (size_t)sm_count() * 8;
    if (ctas > most) ctas = most;
    probe_read_kernel<<<(unsigned)ctas, 256, 0, (cudaStream_t)stream>>>((const uint4 *)buf, n16, (uint32_t *)sink);
    return cudaGetLastError() == cudaSuccess ? RQ_OK : RQ_ERR_CUDA;
}

int rq_snapkv_scratch_bytes(const rq_cache *cache, size_t *bytes)
{
    const int rc = check_cache(cache);
    if (rc != RQ_OK) return rc;
    if (!bytes) return RQ_ERR_INVALID_ARG;
    *bytes = snap_scratch_bytes(cache->cfg.batch * cache->cfg.heads, cache->len > 0 ? cache->len : 1);
    return RQ_OK;
}

int rq_snapkv_select(rq_cache *cache, const void *q_window, int32_t window, int32_t keep, float scale,
                     int32_t *idx_out, float *importance_out, void *scratch, void *stream)
{
    const int rc = check_cache(cache);
    if (rc != RQ_OK) return rc;
    if (!q_window || !idx_out || !scratch || !aligned(scratch, 256)) return RQ_ERR_INVALID_ARG;
    if (window < 1 || window > 64 || keep < 1 || cache->len < window) return RQ_ERR_INVALID_ARG;
    const rq_config &c = cache->cfg;
    cudaStream_t s = (cudaStream_t)stream;
    SnapArgs a;
    a.kv = cache->kv; a.page_cap = cache->page_capacity; a.len = cache->len;
    a.B = c.batch; a.H = c.heads; a.D = c.head_dim; a.S = c.page_size; a.dtype = c.dtype;
    a.qw = q_window; a.W = window;
    a.scale = scale > 0.0f ? scale : 1.0f / sqrtf((float)c.head_dim);
    const int BH = c.batch * c.heads;
    snap_carve(scratch, BH, cache->len, &a.imp, &a.stats, &a.rowstat);
    a.status = (int32_t *)((char *)cache->workspace + workspace_layout(c).status);
    if (launch_snap_scores(a, s) != cudaSuccess) return RQ_ERR_CUDA;
    if (launch_snap_select(a.imp, BH, cache->len, window, keep, idx_out, s) != cudaSuccess) return RQ_ERR_CUDA;
    if (importance_out && cudaMemcpyAsync(importance_out, a.imp, (size_t)BH * cache->len * sizeof(float),
                                          cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return RQ_ERR_CUDA;
    return RQ_OK;
}

int rq_snapkv_compact(const rq_cache *src, const int32_t *idx, int32_t keep, rq_cache *dst, void *stream)
{
    int rc = check_cache(src);
    if (rc != RQ_OK) return rc;
    rc = check_cache(dst);
    if (rc != RQ_OK) return rc;
    if (!idx || keep < 1 || keep > src->len) return RQ_ERR_INVALID_ARG;
    const rq_config &a = src->cfg, &b = dst->cfg;
    if (a.batch != b.batch || a.heads != b.heads || a.head_dim != b.head_dim || a.page_size != b.page_size ||
        a.dtype != b.dtype || a.gate_dtype != b.gate_dtype || dst->kv == src->kv)
        return RQ_ERR_INVALID_ARG;
    if (keep > b.capacity_tokens) return RQ_ERR_CAPACITY;
    cudaStream_t s = (cudaStream_t)stream;
    rc = rq_cache_reset(dst, stream);                    // empties dst, clears its bookkeeping
    if (rc != RQ_OK) return rc;
    const int BH = a.batch * a.heads;
    if (launch_snap_compact(src->kv, src->page_capacity, dst->kv, dst->meta, dst->page_capacity, a.page_size, a.head_dim,
                            a.dtype, idx, keep, absmax_of(dst), BH, s) != cudaSuccess)
        return RQ_ERR_CUDA;
    // the recurrence goes on from where the prompt ended
    if (cudaMemcpyAsync(dst->state, src->state, (size_t)BH * 2 * a.head_dim * sizeof(float), cudaMemcpyDeviceToDevice, s) !=
        cudaSuccess)
        return RQ_ERR_CUDA;
    dst->len = keep;
    return RQ_OK;
}

static bool moba_shape_ok(const rq_cache *cache, int32_t block, int32_t budget_blocks)
{
    return cache->len >= 1 && block >= 64 && block % 64 == 0 && block % cache->cfg.page_size == 0 && budget_blocks >= 2 &&
           (cache->len + block - 1) / block <= 2048;
}

int rq_moba_scratch_bytes(const rq_cache *cache, int32_t block, int32_t budget_blocks, size_t *bytes)
{
    const int rc = check_cache(cache);
    if (rc != RQ_OK) return rc;
    if (!bytes || !moba_shape_ok(cache, block, budget_blocks)) return RQ_ERR_INVALID_ARG;
    *bytes = moba_scratch_bytes(cache->cfg.batch * cache->cfg.heads, cache->len, cache->cfg.head_dim, block, budget_blocks);
    return RQ_OK;
}

int rq_moba_prefill(rq_cache *cache, const void *q, int32_t block, int32_t budget_blocks, float scale, void *o,
                    int32_t *blocks_out, float *means_out, void *scratch, void *stream)
{
    const int rc = check_cache(cache);
    if (rc != RQ_OK) return rc;
    if (!q || !o || !scratch || !aligned(scratch, 256) || !aligned(q, 16) || !aligned(o, 16)) return RQ_ERR_INVALID_ARG;
    if (!moba_shape_ok(cache, block, budget_blocks)) return RQ_ERR_INVALID_ARG;
    const rq_config &c = cache->cfg;
    cudaStream_t s = (cudaStream_t)stream;
    MobaArgs a;
    a.kv = cache->kv; a.page_cap = cache->page_capacity; a.len = cache->len;
    a.B = c.batch; a.H = c.heads; a.D = c.head_dim; a.S = c.page_size; a.dtype = c.dtype;
    a.q = q; a.block = block; a.K = budget_blocks; a.o = o;
    a.scale = scale > 0.0f ? scale : 1.0f / sqrtf((float)c.head_dim);
    const int BH = c.batch * c.heads;
    moba_carve(scratch, BH, cache->len, c.head_dim, block, &a.means, &a.sel);
    a.status = (int32_t *)((char *)cache->workspace + workspace_layout(c).status);
    if (launch_moba(a, s) != cudaSuccess) return RQ_ERR_CUDA;
    const size_t nb = (size_t)((cache->len + block - 1) / block);
    if (blocks_out && cudaMemcpyAsync(blocks_out, a.sel, (size_t)BH * cache->len * budget_blocks * sizeof(int32_t),
                                      cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return RQ_ERR_CUDA;
    if (means_out && cudaMemcpyAsync(means_out, a.means, (size_t)BH * nb * c.head_dim * sizeof(float), cudaMemcpyDeviceToDevice,
                                     s) != cudaSuccess)
        return RQ_ERR_CUDA;
    return RQ_OK;
}

int64_t rq_cache_len(const rq_cache *cache) { return cache ? cache->len : -1; }

int rq_decode_step_launches(const rq_cache *cache, int32_t budget_pages)
{
    if (!cache || check_cache(cache) != RQ_OK) return -1;
    const rq_config &c = cache->cfg;
    const int64_t P = (cache->len + 1 + c.page_size - 1) / c.page_size;     // after the step's append
    int grid = 0;
    const DecodeArgs a = decode_args(cache, cache->len + 1);
    if (budget_pages >= 1 && step_waves(cache, a, budget_pages, &grid) > 0) return 1;
    return P <= kSmallStepPages && c.batch * c.heads >= kSmallStepMinHeads ? 2 : 3;
}

int rq_device_status(rq_cache *cache, int32_t *status_out, void *stream)
{
    const int rc = check_cache(cache);
    if (rc != RQ_OK) return rc;
    if (!status_out) return RQ_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    int32_t *dev = (int32_t *)((char *)cache->workspace + workspace_layout(cache->cfg).status);
    if (cudaMemcpyAsync(status_out, dev, sizeof(int32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return RQ_ERR_CUDA;
    if (cudaMemsetAsync(dev, 0, sizeof(int32_t), s) != cudaSuccess) return RQ_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return RQ_ERR_CUDA;
    return RQ_OK;
}

const char *rq_status_string(int status)
{
    switch (status) {
    case RQ_OK: return "ok";
    case RQ_ERR_INVALID_ARG: return "invalid argument";
    case RQ_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case RQ_ERR_CAPACITY: return "capacity exceeded";
    case RQ_ERR_CUDA: return "CUDA error";
    case RQ_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
    }
}

int rq_version(void) { return RQ_VERSION_MAJOR * 1000 + RQ_VERSION_MINOR; }

}  // extern "C"
