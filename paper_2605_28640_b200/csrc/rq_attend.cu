// Sparse flash-decode over the selected pages only (Eq. 4), split-K with the
// combine folded into the same launch.
//
// Work decomposition.  The unit of work is a tile: 16 consecutive token rows
// of one selected page, i.e. a 16 x D block of decayed keys and the matching
// block of decayed values (for 16-token pages a tile is the whole page and its
// keys and values are adjacent in the cache).  A head's tiles are numbered in
// the order of its index list and handed out one at a time through a per-head
// ticket counter.  The grid is sized to what the GPU holds at once.  When it is
// a whole number of CTAs per head (the usual case) head h is served by the CTAs
// h, h + BH, h + 2 BH, ...: they sit on SMs all over the chip, so every head's
// group is equally fast, and inside a group a warp that the memory system
// serves more slowly simply pulls fewer tickets; everybody finishes together.
// Otherwise (fewer CTAs than heads, or a head count that would leave many CTAs
// out) the warps are spread evenly over the heads and every warp sweeps forward
// from its starting head, helping the heads that still have tiles.  The per-head counters are zero at launch: the selection
// kernel clears them (a memset does when this kernel is launched on its own).
//
// Data movement.  Each warp runs its own pipeline: lane 0 issues one bulk
// (TMA, 1-D) copy for the key block and one for the value block of a tile into
// the warp's ring of shared-memory stages, completion is counted on the
// stage's mbarrier, and the warp consumes the stages in issue order and
// refills a stage as soon as it has been read.  The first tickets of a warp
// are its own by position, later ones come from the counter, and the ticket
// and the page index of a refill are fetched one refill ahead, so neither the
// atomic nor the index load is waited for.  No warp waits for another warp
// inside the stream.
//
// Arithmetic (plain fp32 ALU work; a decode query is a GEMV): a warp-wide
// 16-byte shared-memory read covers whole rows, lane -> (row, channel group);
// row dot products are reduced over the lanes of a row, the softmax runs
// online per warp in the exp2 domain, V is accumulated per lane for its
// channel group.  At the end the warps of a CTA are merged through shared
// memory into one partial (m, l, acc[D]) per head; the arrival that completes
// a head's count combines the head's partials into the output row.
#include <limits.h>
#include <math.h>
#include <math_constants.h>

#include <algorithm>

#include "rq_async.cuh"
#include "rq_device.cuh"
#include "rq_internal.h"
#include "rq_stream.cuh"

namespace rq {

namespace {

template <typename T, int D, int S>
__global__ void __launch_bounds__(kAttendWarps * 32) attend_kernel(DecodeArgs a, const T *q,
                                                                   const int32_t *idx, int n_idx,
                                                                   int idx_stride, float scale_log2,
                                                                   float *partial, int slots_per_head,
                                                                   AttendCounters ctr, T *o)
{
    using G = AttendGeom<T, D, S>;
    constexpr int CH = G::CH, LPR = G::LPR, TR = G::TR, TPP = G::TPP;
    constexpr int NW = G::NW, DEPTH = G::DEPTH;
    constexpr unsigned FULL = 0xffffffffu;

    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *ring = smem;
    uint64_t *bars = reinterpret_cast<uint64_t *>(ring + G::RING_BYTES);
    int2 *infos = reinterpret_cast<int2 *>(bars + NW * DEPTH);       // x: head (-1 = end), y: valid rows
    float *sm_m = reinterpret_cast<float *>(infos + NW * DEPTH);
    float *sm_l = sm_m + NW;
    int *sm_t = reinterpret_cast<int *>(sm_l + NW);
    int *sm_h = sm_t + NW;
    float *sm_acc = reinterpret_cast<float *>(sm_h + NW);            // [NW][D]

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int cgp = lane % LPR;
    const int BH = a.B * a.H;
    const int64_t P = (a.len + S - 1) / S;
    const int per_head = n_idx * TPP;                // tiles per head (host: < 2^20)
    const int NC = gridDim.x;                        // CTAs in the grid
    const int TW = NC * NW;                          // warps in the grid
    const int wg = blockIdx.x * NW + warp;

    const uint64_t stream_policy = l2_evict_first_policy();
    const int poll_limit = a.poll_limit == 0 ? kMbarPollLimit : (a.poll_limit < 0 ? 0 : a.poll_limit);
    uint64_t *mybars = bars + warp * DEPTH;
    int2 *myinfo = infos + warp * DEPTH;
    unsigned char *myring = ring + (size_t)warp * DEPTH * G::STAGE_BYTES;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < DEPTH; ++s) mbar_init(&mybars[s], 1);
        mbar_init_fence();
    }
    __syncthreads();
    grid_dependency_wait();          // the index list and the cache come from earlier kernels
    grid_launch_dependents();

    const T *kvbase = static_cast<const T *>(a.kv);

    // ------------------------------------------------------------ issue side
    // fixed: a whole number of CTAs per head; all warps of CTA c serve head c % BH and never change.
    const bool fixed = NC >= BH && NC % BH == 0;
    const int h0 = fixed ? (int)(blockIdx.x % BH) : (int)((int64_t)wg * BH / TW);
    // Warps that start on head h.  Each owns DEPTH tickets by position, so its ring fills
    // without waiting for an atomic; the counter hands out the tickets after those.
    auto first_warp = [&](int h) -> int { return (int)(((int64_t)h * TW + BH - 1) / BH); };   // sweeping mode
    auto owners = [&](int h) -> int {
        if (fixed) return ((NC - h + BH - 1) / BH) * NW;
        return first_warp(h + 1) - first_warp(h);
    };
    int k = 0;                                       // sweep position: head (h0 + k) % BH
    int ih = h0;                                     // head being pulled from
    int base = owners(h0) * DEPTH;                   // first ticket of head ih that the counter hands out
    bool drained = false;                            // no head has tiles left
    int n_own = DEPTH;                               // own tickets not yet issued
    int t_own = (fixed ? (int)(blockIdx.x / BH) * NW + warp : wg - first_warp(h0)) * DEPTH;   // next own ticket
    int pg_own = -1;                                 // lane j < DEPTH: page of own ticket j
    if (lane < DEPTH && t_own + lane < per_head)
        pg_own = __ldg(idx + (int64_t)h0 * idx_stride + (t_own + lane) / TPP);
    int tA = 0, pgA = -1, tB = 0;                    // lane 0: next ticket + its page, ticket after it

    auto prime = [&]() {                             // lane 0: first two counter tickets of head ih
        tA = base + atomicAdd(ctr.next + ih * kCtrStride, 2);
        tB = tA + 1;
        pgA = tA < per_head ? __ldg(idx + (int64_t)ih * idx_stride + tA / TPP) : -1;
    };
    // move to the next head of the sweep that still has tickets
    auto advance = [&]() {
        for (;;) {
            if (fixed || k + 1 >= BH) { drained = true; return; }
            const int j = k + 1 + lane;
            int c = INT_MAX;
            if (j < BH) {
                const int h = (h0 + j) % BH;
                c = owners(h) * DEPTH + ld_volatile(ctr.next + h * kCtrStride);
            }
            const unsigned m = __ballot_sync(FULL, c < per_head);
            if (m) {
                k += __ffs(m);
                ih = (h0 + k) % BH;
                base = owners(ih) * DEPTH;
                if (lane == 0) prime();
                return;
            }
            k = min(k + 32, BH - 1);
        }
    };
    // lane 0: start the copies of tile t of head h (page pg) into a stage
    auto start_copies = [&](int stage, int h, int t, int pg) {
        const int tile = t % TPP;
        int valid = 0;
        if (pg >= 0) {
            if (pg < P) {
                const int64_t left = a.len - ((int64_t)pg * S + tile * TR);
                valid = left >= TR ? TR : (left > 0 ? (int)left : 0);
            } else {
                atomicExch(a.status, RQ_ERR_INVALID_ARG);
            }
        }
        myinfo[stage] = make_int2(h, valid);
        if (valid > 0) {
            const T *kb = kvbase + (((int64_t)h * a.page_cap + pg) * 2) * S * D + tile * TR * D;
            unsigned char *dst = myring + (size_t)stage * G::STAGE_BYTES;
            mbar_arrive_expect_tx(&mybars[stage], G::STAGE_BYTES);
            bulk_g2s_hint(dst, kb, G::TILE_BYTES, &mybars[stage], stream_policy);
            bulk_g2s_hint(dst + G::TILE_BYTES, kb + (int64_t)S * D, G::TILE_BYTES, &mybars[stage], stream_policy);
        }
    };
    // put the next tile into a stage (or the end mark); called by the whole warp
    auto refill = [&](int stage) {
        while (n_own > 0) {                          // own tickets first
            const int t = t_own, pg = __shfl_sync(FULL, pg_own, DEPTH - n_own);
            ++t_own;
            --n_own;
            if (t < per_head) {
                if (lane == 0) start_copies(stage, h0, t, pg);
                return;
            }
        }
        for (;;) {
            if (drained) {
                if (lane == 0) myinfo[stage] = make_int2(-1, 0);
                return;
            }
            int t = 0, pg = -1;
            if (lane == 0) {
                t = tA;
                pg = pgA;
                tA = tB;
                pgA = tA < per_head ? __ldg(idx + (int64_t)ih * idx_stride + tA / TPP) : -1;
                tB = base + atomicAdd(ctr.next + ih * kCtrStride, 1);
            }
            t = __shfl_sync(FULL, t, 0);
            if (t < per_head) {
                if (lane == 0) start_copies(stage, ih, t, pg);
                return;
            }
            advance();                               // this head has no tickets left
        }
    };

    if (lane == 0) prime();
#pragma unroll
    for (int s = 0; s < DEPTH; ++s) refill(s);
    __syncwarp();

    // ------------------------------------------------------------ consume side
    int cur = -1;                                    // head of the running accumulation
    int tiles = 0;                                   // tiles of `cur` consumed by this warp
    int slot = 0;                                    // lane 0, sweeping only: this warp's partial slot in `cur`
    AttendState<T> st;
#pragma unroll
    for (int c = 0; c < CH; ++c) { st.qf[c] = 0.0f; st.acc[c] = 0.0f; }
    st.m = -CUDART_INF_F;
    st.l = 0.0f;
    int stage = 0;
    uint32_t phase = 0;                              // one parity bit per stage
    bool dead = false;                               // a wait ran out: stop streaming, finish cleanly

    // after a partial of head h has been written by this warp: count it, and combine if it was the last
    auto arrive = [&](int h, int count_word, int expect_ctas, int n_fixed) {
        // The partial was written by several lanes: the warp barrier orders those stores before
        // lane 0's release; the same atomic acquires the partials of the arrivals before it.
        __syncwarp();
        int last = 0;
        if (lane == 0) {
            int old;
            asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;"
                         : "=r"(old)
                         : "l"(ctr.done + h * kCtrStride), "r"(count_word)
                         : "memory");
            const int now = old + count_word;
            last = (now & kDoneTileMask) == per_head && (now >> kDoneTileBits) == expect_ctas;
        }
        last = __shfl_sync(FULL, last, 0);
        if (last) {
            __syncwarp();
            const int n = n_fixed >= 0 ? n_fixed : min(ld_volatile(ctr.nslot + h * kCtrStride), slots_per_head);
            combine_head<T, D>(partial + (int64_t)h * slots_per_head * (D + 4), n, o + (int64_t)h * D, lane);
        }
    };
    // sweeping mode: the warp writes its own partial for head h
    auto flush_warp = [&](int h) {
        attend_merge_rows<T, D, S>(st);
        const int s = __shfl_sync(FULL, slot, 0);
        if (s >= slots_per_head) {                   // cannot happen: a warp joins a head by holding one of its tiles
            if (lane == 0) atomicExch(a.status, RQ_ERR_CAPACITY);
            return;
        }
        float *dst = partial + ((int64_t)h * slots_per_head + s) * (D + 4);
        if (lane == 0) *reinterpret_cast<float2 *>(dst) = make_float2(st.m, st.l);
        if (lane < LPR) {
#pragma unroll
            for (int c = 0; c < CH; c += 4)
                *reinterpret_cast<float4 *>(dst + 4 + cgp * CH + c) = make_float4(st.acc[c], st.acc[c + 1], st.acc[c + 2], st.acc[c + 3]);
        }
        arrive(h, tiles, 0, -1);
    };

    for (;;) {
        const int2 inf = myinfo[stage];
        if (inf.x < 0) break;
        if (inf.x != cur) {
            if (cur >= 0) flush_warp(cur);           // only a sweeping warp changes head
            cur = inf.x;
            tiles = 0;
            if (!fixed && lane == 0) slot = atomicAdd(ctr.nslot + cur * kCtrStride, 1);
            attend_begin_head<T, D>(st, q, cur, scale_log2, lane);
        }
        const int valid = inf.y;
        if (valid > 0 && !dead) {
            if (!mbar_wait(&mybars[stage], (phase >> stage) & 1u, poll_limit)) {
                // give every copy in flight (this one too) the usual bounded chance to land, then stop
                for (int s = 0; s < DEPTH; ++s)
                    if (myinfo[s].x >= 0 && myinfo[s].y > 0) mbar_wait(&mybars[s], (phase >> s) & 1u);
                if (lane == 0) atomicExch(a.status, RQ_ERR_TIMEOUT);
                dead = true;
            }
            phase ^= 1u << stage;
        }
        if (valid > 0 && !dead) {
            const T *ks = reinterpret_cast<const T *>(myring + (size_t)stage * G::STAGE_BYTES);
            const T *vs = ks + TR * D;
            attend_tile<T, D, S>(st, ks, vs, valid, lane);
        }
        ++tiles;
        __syncwarp();                                // every lane is done with the stage
        if (dead) drained = true;
        refill(stage);
        __syncwarp();
        stage = stage + 1 == DEPTH ? 0 : stage + 1;
    }

    if (!fixed) {
        if (cur >= 0 && !dead) flush_warp(cur);
        return;
    }

    // fixed mode: merge the CTA's warps (all on head h0) into one partial in slot blockIdx / BH
    attend_merge_rows<T, D, S>(st);
    if (dead || cur < 0) { st.m = -CUDART_INF_F; st.l = 0.0f; tiles = 0; }
    if (lane == 0) { sm_m[warp] = st.m; sm_l[warp] = st.l; sm_t[warp] = tiles; sm_h[warp] = dead; }
    if (lane < LPR) {
#pragma unroll
        for (int c = 0; c < CH; ++c) sm_acc[warp * D + cgp * CH + c] = (dead || cur < 0) ? 0.0f : st.acc[c];
    }
    __syncthreads();
    if (warp != 0) return;
    constexpr int CPL = D / 32;                      // channels per lane in the merge
    float m_all = -CUDART_INF_F, l_all = 0.0f;
    int t_all = 0, any_dead = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) { m_all = fmaxf(m_all, sm_m[w]); t_all += sm_t[w]; any_dead |= sm_h[w]; }
    float out[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) out[c] = 0.0f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
        const float f = sm_m[w] == -CUDART_INF_F ? 0.0f : exp2f(sm_m[w] - m_all);
        l_all = fmaf(f, sm_l[w], l_all);
#pragma unroll
        for (int c = 0; c < CPL; ++c) out[c] = fmaf(f, sm_acc[w * D + lane * CPL + c], out[c]);
    }
    if (any_dead) return;                            // status already says why; the head stays incomplete
    const int rank = blockIdx.x / BH;
    float *dst = partial + ((int64_t)h0 * slots_per_head + rank) * (D + 4);
    if (lane == 0) *reinterpret_cast<float2 *>(dst) = make_float2(m_all, l_all);
#pragma unroll
    for (int c = 0; c < CPL; ++c) dst[4 + lane * CPL + c] = out[c];
    const int team = (NC - h0 + BH - 1) / BH;        // CTAs on this head; each arrives exactly once
    arrive(h0, t_all + (1 << kDoneTileBits), team, team);
}

}  // namespace

namespace {

// CTAs of this kernel one SM holds at once, found once per device.
template <typename T, int D, int S>
cudaError_t attend_occupancy(int *ctas_per_sm)
{
    using G = AttendGeom<T, D, S>;
    static int cached[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (cached[dev] == 0) {
        e = cudaFuncSetAttribute(attend_kernel<T, D, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        int n = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, attend_kernel<T, D, S>, G::NW * 32, G::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        cached[dev] = n > 0 ? n : 1;
    }
    *ctas_per_sm = cached[dev];
    return cudaSuccess;
}

template <typename T, int D, int S>
cudaError_t launch_attend_t(const DecodeArgs &a, const void *q, const int32_t *idx, int n_idx, int idx_stride,
                            float scale, float *partial, const AttendCounters &ctr, void *o, int sm_count,
                            cudaStream_t s)
{
    using G = AttendGeom<T, D, S>;
    const int64_t per_head = (int64_t)n_idx * G::TPP;
    const int64_t W = (int64_t)a.B * a.H * per_head;
    if (W <= 0 || per_head > kDoneTileMask) return cudaErrorInvalidValue;
    int occ = 1;
    cudaError_t e = attend_occupancy<T, D, S>(&occ);
    if (e != cudaSuccess) return e;
    const int grid = attend_grid(W, a.B * a.H, occ * sm_count);
    const int slots = attend_slots_per_head(per_head);
    const float scale_log2 = scale * 1.4426950408889634f;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(G::NW * 32);
    cfg.dynamicSmemBytes = G::SMEM_BYTES;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, attend_kernel<T, D, S>, a, (const T *)q, idx, n_idx, idx_stride, scale_log2,
                              partial, slots, ctr, (T *)o);
}

// the same launch with the number of partial records per head given by the caller
template <typename T, int D, int S>
cudaError_t launch_attend_slots_t(const DecodeArgs &a, const void *q, const int32_t *idx, int n_idx, int idx_stride,
                                  float scale, float *partial, int slots, const AttendCounters &ctr, void *o,
                                  int sm_count, cudaStream_t s)
{
    using G = AttendGeom<T, D, S>;
    const int64_t W = (int64_t)a.B * a.H * n_idx * G::TPP;
    int occ = 1;
    cudaError_t e = attend_occupancy<T, D, S>(&occ);
    if (e != cudaSuccess) return e;
    const int grid = attend_grid(W, a.B * a.H, occ * sm_count);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(G::NW * 32);
    cfg.dynamicSmemBytes = G::SMEM_BYTES;
    cfg.stream = s;
    return cudaLaunchKernelEx(&cfg, attend_kernel<T, D, S>, a, (const T *)q, idx, n_idx, idx_stride,
                              scale * 1.4426950408889634f, partial, slots, ctr, (T *)o);
}

cudaError_t launch_attend_slots(const DecodeArgs &a, const void *q, const int32_t *idx, int n_idx, int idx_stride,
                                float scale, float *partial, int slots, const AttendCounters &ctr, void *o,
                                int sm_count, cudaStream_t s)
{
#define RQ_ATT(T, D, S) return launch_attend_slots_t<T, D, S>(a, q, idx, n_idx, idx_stride, scale, partial, slots, ctr, o, sm_count, s)
    if (a.dtype == RQ_BF16) {
        if (a.D == 128 && a.S == 16) RQ_ATT(bf16, 128, 16);
        if (a.D == 128 && a.S == 64) RQ_ATT(bf16, 128, 64);
        if (a.D == 64 && a.S == 16) RQ_ATT(bf16, 64, 16);
        if (a.D == 64 && a.S == 64) RQ_ATT(bf16, 64, 64);
    } else {
        if (a.D == 128 && a.S == 16) RQ_ATT(float, 128, 16);
        if (a.D == 128 && a.S == 64) RQ_ATT(float, 128, 64);
        if (a.D == 64 && a.S == 16) RQ_ATT(float, 64, 16);
        if (a.D == 64 && a.S == 64) RQ_ATT(float, 64, 64);
    }
#undef RQ_ATT
    return cudaErrorInvalidValue;
}

}  // namespace

int attend_grid(int64_t tiles, int heads, int resident_ctas)
{
    return stream_grid(tiles, heads, resident_ctas, kAttendWarps, kAttendMaxWarps / kAttendWarps);
}

int attend_slots_per_head(int64_t tiles_per_head)
{
    // A head gets one partial per CTA that serves it (fewer than its tiles / 8, see attend_grid)
    // or, when warps sweep over heads, one per warp that held one of its tiles.
    return (int)(tiles_per_head < kAttendMaxWarps ? tiles_per_head : kAttendMaxWarps);
}

cudaError_t launch_attend(const DecodeArgs &a, const void *q, const int32_t *idx, int n_idx, int idx_stride,
                          float scale, float *partial, const AttendCounters &ctr, void *o, int sm_count,
                          cudaStream_t s)
{
#define RQ_ATT(T, D, S) return launch_attend_t<T, D, S>(a, q, idx, n_idx, idx_stride, scale, partial, ctr, o, sm_count, s)
    if (a.dtype == RQ_BF16) {
        if (a.D == 128 && a.S == 16) RQ_ATT(bf16, 128, 16);
        if (a.D == 128 && a.S == 64) RQ_ATT(bf16, 128, 64);
        if (a.D == 64 && a.S == 16) RQ_ATT(bf16, 64, 16);
        if (a.D == 64 && a.S == 64) RQ_ATT(bf16, 64, 64);
    } else {
        if (a.D == 128 && a.S == 16) RQ_ATT(float, 128, 16);
        if (a.D == 128 && a.S == 64) RQ_ATT(float, 128, 64);
        if (a.D == 64 && a.S == 16) RQ_ATT(float, 64, 16);
        if (a.D == 64 && a.S == 64) RQ_ATT(float, 64, 64);
    }
#undef RQ_ATT
    return cudaErrorInvalidValue;
}

// ---------------------------------------------------------------- attention without a workspace
// Scratch of rq_attend_pages_noalloc: lives in the library's image, so every GPU that loads the
// library holds these 4 MiB until the process exits.  Layout: status word (256 bytes), then the
// per-head counters, then the partial records.
constexpr size_t kStaticScratchBytes = (size_t)4 << 20;
static __device__ __align__(256) unsigned char g_attend_scratch[kStaticScratchBytes];

// Device address of the scratch array on the current device (the array's name is only a handle in
// host code).  Looked up once per device.
static cudaError_t static_scratch(unsigned char **out)
{
    static unsigned char *cached[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!cached[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_attend_scratch);
        if (e != cudaSuccess) return e;
        cached[dev] = static_cast<unsigned char *>(p);
    }
    *out = cached[dev];
    return cudaSuccess;
}

}  // namespace rq

extern "C" int rq_attend_pages_noalloc(const rq_config *cfg, const void *kv, int64_t len, const void *q,
                                       const int32_t *idx, int32_t n_idx, float scale, void *o, void *stream)
{
    using namespace rq;
    const int rc = rq_sizes(cfg, nullptr, nullptr, nullptr, nullptr);      // validates the configuration
    if (rc != RQ_OK) return rc;
    if (!kv || !q || !idx || !o || n_idx < 1 || len < 1 || len > cfg->capacity_tokens) return RQ_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    const int BH = cfg->batch * cfg->heads;
    const int tpp = cfg->page_size / kTileRows;
    const int64_t per_head = (int64_t)n_idx * tpp;
    if (per_head > kDoneTileMask) return RQ_ERR_CAPACITY;

    const int sms = sm_count();

    DecodeArgs a = {};
    a.kv = const_cast<void *>(kv);
    a.B = cfg->batch; a.H = cfg->heads; a.D = cfg->head_dim; a.S = cfg->page_size;
    a.dtype = cfg->dtype; a.gate_dtype = cfg->gate_dtype;
    a.len = len;
    a.page_cap = (cfg->capacity_tokens + cfg->page_size - 1) / cfg->page_size;

    // The grid and the number of partial records per head follow from the shape alone; the
    // ordinary entry point sizes its workspace for the worst case, here the exact need counts.
    int occ = 1;
    cudaError_t e = cudaErrorInvalidValue;
#define RQ_OCC(T, D, S) e = attend_occupancy<T, D, S>(&occ)
    if (a.dtype == RQ_BF16) {
        if (a.D == 128 && a.S == 16) RQ_OCC(bf16, 128, 16);
        else if (a.D == 128 && a.S == 64) RQ_OCC(bf16, 128, 64);
        else if (a.D == 64 && a.S == 16) RQ_OCC(bf16, 64, 16);
        else if (a.D == 64 && a.S == 64) RQ_OCC(bf16, 64, 64);
    } else {
        if (a.D == 128 && a.S == 16) RQ_OCC(float, 128, 16);
        else if (a.D == 128 && a.S == 64) RQ_OCC(float, 128, 64);
        else if (a.D == 64 && a.S == 16) RQ_OCC(float, 64, 16);
        else if (a.D == 64 && a.S == 64) RQ_OCC(float, 64, 64);
    }
#undef RQ_OCC
    if (e != cudaSuccess) return RQ_ERR_CUDA;
    const int grid = attend_grid((int64_t)BH * per_head, BH, occ * sms);
    const int64_t slots = (grid >= BH && grid % BH == 0) ? grid / BH : std::min<int64_t>((int64_t)grid * kAttendWarps, per_head);
    const size_t ctr_bytes = (size_t)BH * kCtrStride * sizeof(int32_t);
    const size_t need = 256 + ctr_bytes + (size_t)BH * slots * (a.D + 4) * sizeof(float);
    if (need > kStaticScratchBytes) return RQ_ERR_CAPACITY;

    unsigned char *scratch = nullptr;
    if (static_scratch(&scratch) != cudaSuccess) return RQ_ERR_CUDA;
    // the array keeps what the last call left: status and counters must start at zero
    if (cudaMemsetAsync(scratch, 0, 256 + ctr_bytes, s) != cudaSuccess) return RQ_ERR_CUDA;
    a.status = reinterpret_cast<int32_t *>(scratch);
    int32_t *ctr = reinterpret_cast<int32_t *>(scratch + 256);
    float *partial = reinterpret_cast<float *>(scratch + 256 + ctr_bytes);
    if (!(scale > 0.0f)) scale = 1.0f / sqrtf((float)a.D);
    const AttendCounters c = {ctr, ctr + 1, ctr + 2};
    if (launch_attend_slots(a, q, idx, n_idx, n_idx, scale, partial, (int)slots, c, o, sms, s) != cudaSuccess)
        return RQ_ERR_CUDA;
    return RQ_OK;
}
