// First kernel of a decode step: the single-token state update (Eq. 1) fused
// with the scoring of every page by the query's upper bound (Eq. 3 with the
// per-page min/max representatives of App. A.1).
//
// Scoring.  U_p = sum_i max(q_i min_p[i], q_i max_p[i]).  A page's bounds are
// one contiguous record [min row][max row] of 2*D elements and a head's
// records are contiguous, so scoring is one long stream per head.  Since
// min <= max, max(q*min, q*max) = q*max for q >= 0 and q*min for q < 0: a lane
// that holds part of a max row multiplies by max(q, 0), a lane that holds part
// of a min row by min(q, 0); every loaded byte is used and a record's score is
// a sum over the lanes that share it.
//
// Data movement is the flash-decode kernel's: the unit of work is 8 KiB of
// consecutive records of one head, a head's units are handed out through a
// per-head ticket counter (own tickets by position first), head h is served by
// the CTAs h, h + BH, ... (or, when the grid is not a whole number of CTAs
// per head, warps spread over the heads and sweep forward), and every warp streams its units through its own ring of
// shared-memory stages filled by bulk (TMA, 1-D) copies.  The ticket counters
// are zero at launch; the selection kernel, which always runs next, clears
// them.
//
// Update.  When a token is appended, the CTAs h, h + gridDim, ... first do head
// h's recurrence step on the fp32 state, append the rounded state to the
// cache, merge it into the newest page's bounds, and write that page's score
// from the merged bounds they hold; the stream leaves the newest page out, so
// nobody reads a record while it is being rewritten.
#include <limits.h>
#include <math_constants.h>

#include "rq_async.cuh"
#include "rq_device.cuh"
#include "rq_internal.h"
#include "rq_stream.cuh"

namespace rq {

namespace {

template <typename T, int D>
__global__ void __launch_bounds__(kScoreWarps * 32) score_kernel(DecodeArgs a, const T *q, const T *k_t,
                                                                 const T *v_t, const void *g_t, float *scores,
                                                                 int32_t *next, int do_update, ScoreHist hs)
{
    using G = ScoreGeom<T, D>;
    constexpr int CH = G::CH, RU = G::RU, VPL = G::VPL;
    constexpr int NW = G::NW, DEPTH = G::DEPTH;
    constexpr unsigned FULL = 0xffffffffu;

    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *ring = smem;
    uint64_t *bars = reinterpret_cast<uint64_t *>(ring + G::RING_BYTES);
    int4 *infos = reinterpret_cast<int4 *>(bars + NW * DEPTH);       // x: head (-1 = end), y: first record, z: records
    float *red = reinterpret_cast<float *>(infos + NW * DEPTH);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int BH = a.B * a.H;
    const int P = (int)((a.len + a.S - 1) / a.S);
    const int Ps = do_update ? P - 1 : P;            // records per head that are streamed
    const int per_head = (Ps + RU - 1) / RU;         // units per head
    const int NC = gridDim.x, TW = NC * NW;
    const int wg = blockIdx.x * NW + warp;

    const uint64_t stream_policy = l2_evict_first_policy();
    const int poll_limit = a.poll_limit == 0 ? kMbarPollLimit : (a.poll_limit < 0 ? 0 : a.poll_limit);
    uint64_t *mybars = bars + warp * DEPTH;
    int4 *myinfo = infos + warp * DEPTH;
    unsigned char *myring = ring + (size_t)warp * DEPTH * kUnitBytes;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < DEPTH; ++s) mbar_init(&mybars[s], 1);
        mbar_init_fence();
    }
    __syncthreads();
    grid_dependency_wait();          // earlier kernels may still read what the update rewrites
    grid_launch_dependents();

    const int hcur = a.epoch & 1;                    // copy of the heads' largest |stored key| that this step reads
    // forced pages inside the budget do not compete: they are not counted (the caller passes them)
    const int p_lo = hs.hist ? a.n_sink : 0, p_hi = hs.hist ? P - a.n_local : 0;
    if (do_update)
        for (int h = blockIdx.x; h < BH; h += NC) {
            const float s_new = update_head<T, D>(a, h, q, k_t, v_t, g_t, scores, red);
            if (hs.ctr_other && threadIdx.x < kStepCtrInts) hs.ctr_other[h * kStepCtrInts + threadIdx.x] = 0;
            if (hs.hist && warp == 0) {              // the newest page, scored by the update, if it competes
                const ScoreRange rg = score_range<T, D>(q, h, a.absmax[hcur * BH + h], lane);
                if (lane == 0 && P - 1 >= p_lo && P - 1 < p_hi) red_inc(hs.hist + (int64_t)h * kStepBins + rg.bucket(s_new));
            }
        }

    const T *meta = static_cast<const T *>(a.meta);

    // ------------------------------------------------------------ issue side (as in the flash-decode kernel)
    const bool fixed = NC >= BH && NC % BH == 0;
    const int h0 = fixed ? (int)(blockIdx.x % BH) : (int)((int64_t)wg * BH / TW);
    auto first_warp = [&](int h) -> int { return (int)(((int64_t)h * TW + BH - 1) / BH); };   // sweeping mode
    auto owners = [&](int h) -> int {                // warps that start on head h; each owns DEPTH tickets
        if (fixed) return ((NC - h + BH - 1) / BH) * NW;
        return first_warp(h + 1) - first_warp(h);
    };
    int k = 0;                                       // sweep position: head (h0 + k) % BH
    int ih = h0;                                     // head being pulled from
    int base = owners(h0) * DEPTH;                   // first ticket of head ih that the counter hands out
    bool drained = false;
    int n_own = DEPTH;                               // own tickets not yet issued
    int t_own = (fixed ? (int)(blockIdx.x / BH) * NW + warp : wg - first_warp(h0)) * DEPTH;
    int tA = 0;                                      // lane 0: next counter ticket

    auto advance = [&]() {                           // next head of the sweep that still has tickets
        for (;;) {
            if (fixed || k + 1 >= BH) { drained = true; return; }
            const int j = k + 1 + lane;
            int cnt = INT_MAX;
            if (j < BH) {
                const int h = (h0 + j) % BH;
                cnt = owners(h) * DEPTH + ld_volatile(next + h * kCtrStride);
            }
            const unsigned m = __ballot_sync(FULL, cnt < per_head);
            if (m) {
                k += __ffs(m);
                ih = (h0 + k) % BH;
                base = owners(ih) * DEPTH;
                if (lane == 0) tA = base + atomicAdd(next + ih * kCtrStride, 1);
                return;
            }
            k = min(k + 32, BH - 1);
        }
    };
    auto start_copy = [&](int stage, int h, int t) { // lane 0
        const int first = t * RU;
        const int n = min(RU, Ps - first);
        myinfo[stage] = make_int4(h, first, n, 0);
        const T *src = meta + ((int64_t)h * a.page_cap + first) * 2 * D;
        mbar_arrive_expect_tx(&mybars[stage], n * G::REC_BYTES);
        bulk_g2s_hint(myring + (size_t)stage * kUnitBytes, src, n * G::REC_BYTES, &mybars[stage], stream_policy);
    };
    auto refill = [&](int stage) {                   // whole warp
        while (n_own > 0) {
            const int t = t_own;
            ++t_own;
            --n_own;
            if (t < per_head) {
                if (lane == 0) start_copy(stage, h0, t);
                return;
            }
        }
        for (;;) {
            if (drained) {
                if (lane == 0) myinfo[stage] = make_int4(-1, 0, 0, 0);
                return;
            }
            int t = 0;
            if (lane == 0) {
                t = tA;
                tA = base + atomicAdd(next + ih * kCtrStride, 1);
            }
            t = __shfl_sync(FULL, t, 0);
            if (t < per_head) {
                if (lane == 0) start_copy(stage, ih, t);
                return;
            }
            advance();
        }
    };

    if (lane == 0) tA = base + atomicAdd(next + ih * kCtrStride, 1);
#pragma unroll
    for (int s = 0; s < DEPTH; ++s) refill(s);
    __syncwarp();

    // ------------------------------------------------------------ consume side
    int cur = -1;
    float qs[VPL][CH];                               // this lane's slice of q, split by sign
#pragma unroll
    for (int v = 0; v < VPL; ++v)
#pragma unroll
        for (int i = 0; i < CH; ++i) qs[v][i] = 0.0f;
    int stage = 0;
    uint32_t phase = 0;
    bool dead = false;
    ScoreRange rg = {0.0f, 0.0f};

    for (;;) {
        const int4 inf = myinfo[stage];
        if (inf.x < 0) break;
        if (inf.x != cur) {
            cur = inf.x;
            score_load_q<T, D>(q, cur, lane, qs);
            if (hs.hist) {                           // every warp computes the same bits
                rg = score_range<T, D>(q, cur, a.absmax[hcur * BH + cur], lane);
                if (lane == 0) hs.range[cur] = make_float2(rg.lo, rg.scale);
            }
        }
        if (!dead) {
            if (!mbar_wait(&mybars[stage], (phase >> stage) & 1u, poll_limit)) {
                // give every copy in flight (this one too) the usual bounded chance to land, then stop
                for (int s = 0; s < DEPTH; ++s)
                    if (myinfo[s].x >= 0) mbar_wait(&mybars[s], (phase >> s) & 1u);
                if (lane == 0) atomicExch(a.status, RQ_ERR_TIMEOUT);
                dead = true;
            }
            phase ^= 1u << stage;
        }
        if (!dead) {
            const unsigned char *ub = myring + (size_t)stage * kUnitBytes;
            if (hs.hist) {
                const int first = inf.y;
                uint32_t *hist = hs.hist + (int64_t)cur * kStepBins;
                score_unit<T, D>(ub, qs, inf.z, scores + (int64_t)cur * a.page_cap + first, lane, [&](int r, float u) {
                    const int p = first + r;
                    if (p >= p_lo && p < p_hi) red_inc(hist + rg.bucket(u));
                });
            } else {
                score_unit<T, D>(ub, qs, inf.z, scores + (int64_t)cur * a.page_cap + inf.y, lane);
            }
        }
        __syncwarp();
        if (dead) drained = true;
        refill(stage);
        __syncwarp();
        stage = stage + 1 == DEPTH ? 0 : stage + 1;
    }
}

}  // namespace

namespace {

template <typename T, int D>
cudaError_t score_occupancy(int *ctas_per_sm)
{
    using G = ScoreGeom<T, D>;
    static int cached[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (cached[dev] == 0) {
        e = cudaFuncSetAttribute(score_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        int n = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, score_kernel<T, D>, G::NW * 32, G::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        cached[dev] = n > 0 ? n : 1;
    }
    *ctas_per_sm = cached[dev];
    return cudaSuccess;
}

template <typename T, int D>
cudaError_t launch_score_t(const DecodeArgs &a, const void *q, const void *k_t, const void *v_t, const void *g_t,
                           float *scores, int32_t *next, int do_update, const ScoreHist &hs, int sm_count, cudaStream_t s)
{
    using G = ScoreGeom<T, D>;
    const int64_t P = (a.len + a.S - 1) / a.S;
    const int64_t Ps = do_update ? P - 1 : P;
    const int64_t units = (int64_t)a.B * a.H * ((Ps + G::RU - 1) / G::RU);
    int occ = 1;
    cudaError_t e = score_occupancy<T, D>(&occ);
    if (e != cudaSuccess) return e;
    const int grid = stream_grid(units, a.B * a.H, occ * sm_count, G::NW, INT_MAX);
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
    return cudaLaunchKernelEx(&cfg, score_kernel<T, D>, a, (const T *)q, (const T *)k_t, (const T *)v_t, g_t, scores,
                              next, do_update, hs);
}

}  // namespace

cudaError_t launch_score(const DecodeArgs &a, const void *q, const void *k_t, const void *v_t, const void *g_t,
                         float *scores, int32_t *next, int do_update, const ScoreHist &hs, int sm_count, cudaStream_t s)
{
    if (a.len <= 0) return cudaSuccess;
    if (a.dtype == RQ_BF16) {
        if (a.D == 128) return launch_score_t<bf16, 128>(a, q, k_t, v_t, g_t, scores, next, do_update, hs, sm_count, s);
        if (a.D == 64) return launch_score_t<bf16, 64>(a, q, k_t, v_t, g_t, scores, next, do_update, hs, sm_count, s);
    } else {
        if (a.D == 128) return launch_score_t<float, 128>(a, q, k_t, v_t, g_t, scores, next, do_update, hs, sm_count, s);
        if (a.D == 64) return launch_score_t<float, 64>(a, q, k_t, v_t, g_t, scores, next, do_update, hs, sm_count, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace rq
