// SnapKV-style reduction of the cache of decayed keys and values (App. A.1, "Sparse inference
// settings", SnapKV paragraph; Table 1, row SnapKV): the queries of the last W prompt positions
// (the observation window) rate every earlier position by the attention they pay to it, the keep
// most important entries are retained (the window itself always, inside keep) and copied into a
// new, smaller cache on which decoding then runs.
//
//   importance[j] = sum_i softmax_j(scale * q_i . k~_j),  query i at position T - W + i sees j <= T - W + i
//
// Kernels.  The importance is a dense contraction (W x D x T per head) followed by a softmax over T
// and a sum over the window.  The 64 x T scores of a head are never stored: the keys are read twice,
// once for the row statistics (maximum and sum of exponentials of every query) and once for the
// weights.
//   snap_mma_kernel<PASS 1>   bf16 caches.  Per (head, run of 128-key tiles): the scores of a tile on the
//                             tensor cores (tcgen05.mma, operands in shared memory, fp32 accumulator
//                             in tensor memory): D[query][key] with the window's queries as the M
//                             side (both halves of the 128 rows hold the same 64 queries, so that all
//                             four warps have rows to work on: the upper half takes the tile's upper 64
//                             keys), a thread per (query, half of the keys) keeps a running maximum
//                             and sum of exponentials -> partial statistics per run
//   snap_rows_kernel          per (head, query): merges the partial statistics
//   snap_mma_kernel<PASS 2>   the same products with the roles swapped, D[key][query] (keys as the M
//                             side), so that a thread owns a key and sums its weights over the
//                             queries without any exchange -> importance of the tile's keys
//   snap_tile_kernel<1 / 2>   fp32 caches: the same two passes as plain fp32 FMA code (64 x 128
//                             score tiles in registers, 8 rows x 4 keys per thread)
//   snap_select_kernel        per head: the keep - W most important positions before the window
//                             (most-significant-digit radix select on the order-preserving image of the
//                             importance, equal importance to the lower position) plus the window,
//                             written in ascending order
//   snap_compact_kernel       per (head, page of the new cache): gathers the retained rows, rebuilds
//                             the page's min/max bounds, tracks the head's largest |key|
#include <math.h>
#include <math_constants.h>

#include "rq_async.cuh"
#include "rq_device.cuh"
#include "rq_internal.h"
#include "rq_tmap.h"
#include "rq_umma.cuh"

namespace rq {

namespace {

constexpr int kSnapRows = 64;                  // queries of the window (fewer: the rest is masked)
constexpr int kSnapKeys = 128;                 // keys per tile
constexpr int kSnapThreads = 256;              // 8 row groups x 32 key groups
constexpr int kSnapBins = 2048;

template <int D>
struct SnapGeom {
    static constexpr int LD = D + 4;           // floats per row in shared memory (16-byte aligned rows, few bank conflicts)
    // queries | keys | row max | row 1/l | reduction scratch (8 x 128 floats)
    static constexpr int SMEM_BYTES = (kSnapRows + kSnapKeys) * LD * 4 + 2 * kSnapRows * 4 + 8 * kSnapKeys * 4;
};

// PASS 1: stats[bh][tile][row] = (max, sum exp) of the tile's visible scores.
// PASS 2: imp[bh][key] = sum_rows exp(s - m_row) / l_row  with rowstat[bh][row] = (m, l).
template <typename T, int D, int PASS>
__global__ void __launch_bounds__(kSnapThreads) snap_tile_kernel(const T *kv, int64_t page_cap, int S, int64_t len,
                                                                 const T *qw, int W, int H, float scale_log2,
                                                                 float2 *stats, const float2 *rowstat, float *imp,
                                                                 int ntiles)
{
    using G = SnapGeom<D>;
    constexpr int LD = G::LD;
    extern __shared__ __align__(16) float sm[];
    float *qs = sm;                              // [64][LD]
    float *ks = qs + kSnapRows * LD;             // [128][LD]
    float *rm = ks + kSnapKeys * LD;             // [64] final row maximum (pass 2)
    float *rl = rm + kSnapRows;                  // [64] 1 / final row sum  (pass 2)
    float *red = rl + kSnapRows;                 // [8][128] column sums of the row groups (pass 2)

    const int tid = threadIdx.x, tx = tid & 31, ty = tid >> 5;
    const int tile = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
    const int64_t j0 = (int64_t)tile * kSnapKeys;
    const int64_t first_q = len - W;             // position of query 0

    // the window's queries of this head, scaled: qw is [B][W][H][D]
    for (int i = tid; i < kSnapRows * (D / 4); i += kSnapThreads) {
        const int r = i / (D / 4), c4 = i % (D / 4);
        float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (r < W) {
            const T *src = qw + (((int64_t)b * W + r) * H + h) * D + c4 * 4;
            v = make_float4(load1<T>(src) * scale_log2, load1<T>(src + 1) * scale_log2, load1<T>(src + 2) * scale_log2,
                            load1<T>(src + 3) * scale_log2);
        }
        *reinterpret_cast<float4 *>(qs + r * LD + c4 * 4) = v;
    }
    // the tile's keys: position j lives in page j / S, slot j % S of the head's cache
    for (int i = tid; i < kSnapKeys * (D / 4); i += kSnapThreads) {
        const int r = i / (D / 4), c4 = i % (D / 4);
        const int64_t j = j0 + r;
        float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (j < len) {
            const T *src = kv + ((((int64_t)bh * page_cap + j / S) * 2) * S + j % S) * D + c4 * 4;
            v = make_float4(load1<T>(src), load1<T>(src + 1), load1<T>(src + 2), load1<T>(src + 3));
        }
        *reinterpret_cast<float4 *>(ks + r * LD + c4 * 4) = v;
    }
    if (PASS == 2 && tid < kSnapRows) {
        const float2 f = tid < W ? rowstat[(int64_t)bh * kSnapRows + tid] : make_float2(0.0f, 1.0f);
        rm[tid] = f.x;
        rl[tid] = 1.0f / f.y;
    }
    __syncthreads();

    // scores: rows ty * 8 .. + 7, keys tx * 4 .. + 3
    float acc[8][4];
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = 0.0f;
#pragma unroll 2
    for (int d = 0; d < D; d += 4) {
        float4 kq[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) kq[c] = *reinterpret_cast<const float4 *>(ks + (tx * 4 + c) * LD + d);
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const float4 q4 = *reinterpret_cast<const float4 *>(qs + (ty * 8 + r) * LD + d);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                acc[r][c] = fmaf(q4.x, kq[c].x, acc[r][c]);
                acc[r][c] = fmaf(q4.y, kq[c].y, acc[r][c]);
                acc[r][c] = fmaf(q4.z, kq[c].z, acc[r][c]);
                acc[r][c] = fmaf(q4.w, kq[c].w, acc[r][c]);
            }
        }
    }
    // query `row` sees key j iff row < W and j <= first_q + row (which is < len)
    auto visible = [&](int row, int c) { return row < W && j0 + tx * 4 + c <= first_q + row; };

    if (PASS == 1) {
        // per row: maximum over the tile, then sum of exponentials (exp2 domain); the lanes of a warp share the rows
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const int row = ty * 8 + r;
            float m = -CUDART_INF_F;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (visible(row, c)) m = fmaxf(m, acc[r][c]);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
            float l = 0.0f;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (visible(row, c)) l += exp2f(acc[r][c] - m);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
            if (tx == 0) stats[((int64_t)bh * ntiles + tile) * kSnapRows + row] = make_float2(m, l);
        }
    } else {
        // weights, summed over this thread's 8 rows, then over the 8 row groups through shared memory
        float col[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const int row = ty * 8 + r;
            const float m = rm[row], il = rl[row];
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (visible(row, c)) col[c] = fmaf(exp2f(acc[r][c] - m), il, col[c]);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) red[ty * kSnapKeys + tx * 4 + c] = col[c];
        __syncthreads();
        if (tid < kSnapKeys) {
            float s = 0.0f;
#pragma unroll
            for (int g = 0; g < 8; ++g) s += red[g * kSnapKeys + tid];
            if (j0 + tid < len) imp[(int64_t)bh * len + j0 + tid] = s;
        }
    }
}

// ---------------------------------------------------------------- the two passes on the tensor cores (bf16)
constexpr int kMmaKeys = 128;                  // keys per tile
constexpr int kMmaWarps = 4;                   // warps that read the accumulator: one thread per lane of it
constexpr int kMmaThreads = (kMmaWarps + 1) * 32;   // and one warp that starts the copies and the products
constexpr int kMmaStages = 2;                  // key tiles in shared memory: 97 KB with the queries, so that two CTAs share an SM
constexpr int kMmaAhead = 3;                   // tiles between an L2 prefetch and the copy of the same keys
constexpr int kMmaMaxTiles = 32;               // tiles per CTA: the search goes up to twice this

template <int D>
struct SnapMmaGeom {
    static constexpr int HALVES = D / 64;                      // 64-element (128-byte) halves of a row
    static constexpr int HALF_BYTES = 128 * 128;               // 128 rows of one half
    static constexpr int Q_BYTES = HALVES * HALF_BYTES;        // the window's queries, twice (128 rows)
    static constexpr int TILE_BYTES = HALVES * HALF_BYTES;     // 128 keys
    static constexpr int SMEM_BYTES = Q_BYTES + kMmaStages * TILE_BYTES + 1024;   // + room to align the base to 1024 bytes
};

// 2^x for x <= 0 (and -inf): the hardware approximation, relative error about 2^-22
__device__ __forceinline__ float exp2_fast(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Grid (runs of tiles, heads).  stats: [bh][runs][64]; rowstat: [bh][64]; imp: [bh][len].
// tmap: the cache as a rank-4 tensor (channel, slot, key / value, page over all heads), box = 64 channels
// x the slots of a page x keys only x the pages of 128 positions, 128-byte swizzle: one copy brings one
// 64-channel half of a tile's keys into shared memory in the layout the tensor core reads.
template <int D, int PASS>
__global__ void __launch_bounds__(kMmaThreads) snap_mma_kernel(const __grid_constant__ CUtensorMap tmap, int64_t page_cap, int S,
                                                               int64_t len, const bf16 *qw, int W, int H, float scale_log2,
                                                               float2 *stats, const float2 *rowstat, float *imp,
                                                               int ntiles, int tiles_per_cta, int32_t *status)
{
    using G = SnapMmaGeom<D>;
    constexpr int NST = kMmaStages;
    constexpr uint32_t ACC = PASS == 1 ? 128 : 64;             // columns of one accumulator
    constexpr uint32_t TCOLS = 2 * ACC;                        // two accumulators: one is filled while the other is read
    extern __shared__ __align__(1024) unsigned char dsm_raw[];
    __shared__ __align__(8) uint64_t bar[2];                   // an accumulator's product is complete
    __shared__ __align__(8) uint64_t full[NST];                // a stage's keys have landed
    __shared__ __align__(8) uint64_t acc_free[2];              // an accumulator has been read by all four warps
    __shared__ uint32_t tbase;
    __shared__ float2 qst[kSnapRows];                          // pass 1: merge of the two halves; pass 2: (max, 1 / sum) per query
    unsigned char *dsm = dsm_raw + ((1024u - (smem_addr(dsm_raw) & 1023u)) & 1023u);
    unsigned char *qs = dsm, *ks = dsm + G::Q_BYTES;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    const int t0 = blockIdx.x * tiles_per_cta, n = min(tiles_per_cta, ntiles - t0);
    const int64_t first_q = len - W;                           // position of query 0
    const int ppt = kMmaKeys / S;                              // pages per tile
    int n_issued = 0, n_landed = 0;                            // thread 0: tiles whose copies were started / seen complete

    if (tid == 0) {
        mbar_init(&bar[0], 1);
        mbar_init(&bar[1], 1);
        for (int s = 0; s < NST; ++s) mbar_init(&full[s], 1);
        mbar_init(&acc_free[0], kMmaWarps * 32);
        mbar_init(&acc_free[1], kMmaWarps * 32);
        mbar_init_fence();
    }
    if (warp == 0) tmem_alloc(&tbase, TCOLS);
    // the window's queries of this head (qw is [B][W][H][D]) in rows r and r + 64; rows beyond the window are zero
    for (int i = tid; i < 128 * (D / 8); i += kMmaThreads) {
        const int r = i / (D / 8), c = i % (D / 8), qr = r & (kSnapRows - 1);
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (qr < W) v = *reinterpret_cast<const uint4 *>(qw + (((int64_t)b * W + qr) * H + h) * D + c * 8);
        *reinterpret_cast<uint4 *>(qs + (c >> 3) * G::HALF_BYTES + umma_sw128_offset(r, c & 7)) = v;
    }
    if (PASS == 2 && tid < kSnapRows) {
        const float2 f = tid < W ? rowstat[(int64_t)bh * kSnapRows + tid] : make_float2(0.0f, 1.0f);
        qst[tid] = make_float2(f.x, 1.0f / f.y);
    }
    // the keys of tile t (relative to t0) into its stage: position j lives in page j / S, slot j % S of the
    // head's cache; pages past the head's last one hold somebody else's rows or nothing, and every key at
    // or beyond `len` is masked where the scores are used.  One thread.
    auto issue = [&](int i) {
        const int stage = i % NST;
        unsigned char *dst = ks + (size_t)stage * G::TILE_BYTES;
        const int page = (int)((int64_t)bh * page_cap + (int64_t)(t0 + i) * ppt);
        mbar_arrive_expect_tx(&full[stage], G::TILE_BYTES);
#pragma unroll
        for (int hh = 0; hh < G::HALVES; ++hh) tma_load_4d(dst + hh * G::HALF_BYTES, &tmap, hh * 64, 0, 0, page, &full[stage]);
        n_issued = i + 1;
        // two stages keep too few bytes on their way from DRAM for its latency: the keys of a later tile of this
        // CTA are asked into L2 now, so that their copy is short when its turn comes
        if (i + kMmaAhead < n) {
#pragma unroll
            for (int hh = 0; hh < G::HALVES; ++hh) tma_prefetch_4d(&tmap, hh * 64, 0, 0, page + kMmaAhead * ppt);
        }
    };
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the queries, written with ordinary stores, are read by the tensor core
    tcgen05_before_sync();
    __syncthreads();
    tcgen05_after_sync();
    const uint32_t tb = tbase;

    const int row = tid & (kSnapRows - 1), half = (tid >> 6) & 1;   // pass 1: this thread's query and half of the tile's keys
    float m = -CUDART_INF_F, l = 0.0f;                         // pass 1: running statistics
    bool ok = true;
    if (warp == kMmaWarps) {
        // ---- the producing warp: one thread starts the copies and the products; nobody else waits for it
        // except through the barriers
        if (lane == 0) {
            for (int t = NST; t < kMmaAhead && t < n; ++t) {       // the tiles between the first copies and the first prefetch
                const int page = (int)((int64_t)bh * page_cap + (int64_t)(t0 + t) * ppt);
#pragma unroll
                for (int hh = 0; hh < G::HALVES; ++hh) tma_prefetch_4d(&tmap, hh * 64, 0, 0, page);
            }
            for (int s = 0; s < NST && s < n; ++s) issue(s);
            constexpr uint32_t idesc = PASS == 1 ? umma_idesc_bf16(128, kMmaKeys) : umma_idesc_bf16(kMmaKeys, kSnapRows);
            const uint32_t qa = smem_addr(qs);
#pragma unroll 1
            for (int i = 0; i < n && ok; ++i) {
                // accumulator i & 1 has been read (tile i - 2), the tile's keys have landed
                if (i >= 2) ok = mbar_wait(&acc_free[i & 1], (uint32_t)(((i >> 1) - 1) & 1));
                ok = ok && mbar_wait(&full[i % NST], (uint32_t)((i / NST) & 1));
                if (!ok) break;
                n_landed = i + 1;
                tcgen05_after_sync();
                const uint32_t ka = smem_addr(ks + (size_t)(i % NST) * G::TILE_BYTES);
                const uint32_t acc = tb + (uint32_t)(i & 1) * ACC;
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (uint32_t)(k >> 2) * G::HALF_BYTES + (uint32_t)(k & 3) * 32u;
                    const uint64_t dq = umma_desc_sw128(qa + off), dk = umma_desc_sw128(ka + off);
                    if (PASS == 1) umma_bf16(acc, dq, dk, idesc, k > 0);
                    else umma_bf16(acc, dk, dq, idesc, k > 0);
                }
                umma_commit(&bar[i & 1]);
                // the stage of tile i - 1 is free once its product has completed; it takes tile i - 1 + NST
                if (i >= 1 && i - 1 + NST < n) {
                    ok = mbar_wait(&bar[(i - 1) & 1], (uint32_t)(((i - 1) >> 1) & 1));
                    if (ok) issue(i - 1 + NST);
                }
            }
            // after a wait that ran out: no copy may still be on its way into this CTA's shared memory when it exits
            for (int k = n_landed; k < n_issued; ++k) mbar_wait(&full[k % NST], (uint32_t)((k / NST) & 1));
        }
    } else {
#pragma unroll 1
    for (int i = 0; i < n; ++i) {
        ok = mbar_wait(&bar[i & 1], (uint32_t)((i >> 1) & 1));
        if (!__all_sync(0xffffffffu, ok)) break;               // (a warp's lanes stay together: the accumulator loads are warp-wide)
        tcgen05_after_sync();
        const int64_t j0 = (int64_t)(t0 + i) * kMmaKeys;
        const uint32_t tl = tb + (uint32_t)(i & 1) * ACC + ((uint32_t)(warp * 32) << 16);    // this warp's lanes of the accumulator
        if (PASS == 1) {
            // lane = query (both halves of the lanes hold the same 64 queries), column = key
            const int64_t pq = first_q + row;                  // query `row` sees keys up to its own position
#pragma unroll 1
            for (int cb = 0; cb < 64; cb += 32) {
                float v[32];
                tmem_ld32(tl + (uint32_t)(half * 64 + cb), v);
                const int64_t jb = j0 + half * 64 + cb;
                if (row < W && jb <= pq) {
                    const int nv = (int)min((int64_t)32, pq - jb + 1);   // visible keys among these 32
                    float tm = -CUDART_INF_F;
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        v[c] = c < nv ? v[c] * scale_log2 : -CUDART_INF_F;
                        tm = fmaxf(tm, v[c]);
                    }
                    const float mn = fmaxf(m, tm);             // finite: at least one key is visible
                    float sum = 0.0f;
#pragma unroll
                    for (int c = 0; c < 32; ++c) sum += exp2_fast(v[c] - mn);
                    l = l * exp2_fast(m - mn) + sum;           // 2^(-inf) = 0 the first time
                    m = mn;
                }
            }
        } else {
            // lane = key, column = query: the key's weights summed over the queries that see it
            const int64_t j = j0 + tid;
            const int q_lo = (int)max((int64_t)0, j - first_q);
            float acc = 0.0f;
#pragma unroll 1
            for (int cb = 0; cb < kSnapRows; cb += 32) {
                float v[32];
                tmem_ld32(tl + (uint32_t)cb, v);
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const int q = cb + c;
                    const float2 st = qst[q];
                    if (q < W && q >= q_lo) acc = fmaf(exp2_fast(fmaf(v[c], scale_log2, -st.x)), st.y, acc);
                }
            }
            if (j < len) imp[(int64_t)bh * len + j] = acc;
        }
        tcgen05_before_sync();
        mbar_arrive(&acc_free[i & 1]);                         // this thread has read the accumulator
    }
    }
    if (__any_sync(0xffffffffu, !ok) && lane == 0) atomicCAS(status, RQ_OK, RQ_ERR_TIMEOUT);
    if (PASS == 1) {
        // the two halves of a query's keys, merged through shared memory
        if (warp < kMmaWarps && half == 1) qst[row] = make_float2(m, l);
        __syncthreads();
        if (warp < kMmaWarps && half == 0) {
            const float2 o = qst[row];
            const float mn = fmaxf(m, o.x);
            float lt = 0.0f;
            if (mn > -CUDART_INF_F) lt = l * exp2f(m - mn) + o.y * exp2f(o.x - mn);
            stats[((int64_t)bh * gridDim.x + blockIdx.x) * kSnapRows + row] = make_float2(mn, lt);
        }
    }
    tcgen05_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tbase, TCOLS);
}

// Final statistics of a row: merge of its tiles' (max, sum exp).  One warp per (head, row).
__global__ void __launch_bounds__(128) snap_rows_kernel(const float2 *stats, float2 *rowstat, int ntiles, int n_rows_total)
{
    const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (w >= n_rows_total) return;
    const int bh = w / kSnapRows, row = w % kSnapRows;
    float m = -CUDART_INF_F, l = 0.0f;
    for (int t = lane; t < ntiles; t += 32) {
        const float2 f = stats[((int64_t)bh * ntiles + t) * kSnapRows + row];
        if (f.x > -CUDART_INF_F) {
            const float mn = fmaxf(m, f.x);
            l = l * exp2f(m - mn) + f.y * exp2f(f.x - mn);     // exp2f(-inf) = 0 on the first merge
            m = mn;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float mo = __shfl_xor_sync(0xffffffffu, m, off), lo = __shfl_xor_sync(0xffffffffu, l, off);
        const float mn = fmaxf(m, mo);
        const float fa = m > -CUDART_INF_F ? exp2f(m - mn) : 0.0f, fb = mo > -CUDART_INF_F ? exp2f(mo - mn) : 0.0f;
        l = l * fa + lo * fb;
        m = mn;
    }
    if (lane == 0) rowstat[w] = make_float2(m, l > 0.0f ? l : 1.0f);
}

// ---------------------------------------------------------------- token-level selection
// One CTA of 1024 threads per head.  Candidates: positions 0 .. C-1 (C = len - w, w = window
// positions kept outright); `want` of them are taken: those with the largest importance, equal
// importance to the lower position.  Radix select over the order-preserving keys, 11 bits per pass,
// reading the importances from global memory (L2) each pass; then every warp walks its own
// contiguous range twice (count, write), so the list comes out ascending.
__global__ void __launch_bounds__(1024) snap_select_kernel(const float *imp, int64_t len, int w, int keep, int32_t *idx)
{
    constexpr unsigned FULL = 0xffffffffu;
    __shared__ uint32_t hist[kSnapBins];
    __shared__ uint32_t red[32], red2[32];
    __shared__ uint32_t s_digit, s_krem, s_cnt;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bh = blockIdx.x;
    const float *x = imp + (int64_t)bh * len;
    int32_t *out = idx + (int64_t)bh * keep;
    const int C = (int)(len - w);
    const int want = keep - w;
    if (want >= C) {                                 // everything is kept
        for (int j = tid; j < keep; j += 1024) out[j] = j < len ? j : -1;
        return;
    }
    uint32_t tau = 0xffffffffu;                      // want == 0: nothing but the window
    int r_eq = 0;
    if (want > 0) {
        uint32_t prefix = 0u;
        int k = want;
        bool whole = false;
#pragma unroll 1
        for (int hi = 31; hi >= 0 && !whole; hi -= 11) {
            const int lo = hi >= 10 ? hi - 10 : 0;   // this pass decides bits hi .. lo
            const uint32_t dmask = (1u << (hi - lo + 1)) - 1u;
            const uint32_t himask = hi == 31 ? 0u : ~0u << (hi + 1);
            for (int i = tid; i < kSnapBins; i += 1024) hist[i] = 0u;
            __syncthreads();
            // eight independent loads per thread are issued before the first is used
            for (int j0 = tid; j0 < C; j0 += 8 * 1024) {
                float f[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) f[u] = j0 + u * 1024 < C ? __ldcg(x + j0 + u * 1024) : 0.0f;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const uint32_t kx = order_key(f[u]);
                    if (j0 + u * 1024 < C && (kx & himask) == (prefix & himask)) atomicAdd(&hist[(kx >> lo) & dmask], 1u);
                }
            }
            __syncthreads();
            // walk the bins from the top until k keys are covered: thread t owns bins 2t, 2t+1
            const uint32_t c0 = hist[2 * tid], c1 = hist[2 * tid + 1];
            uint32_t suf = c0 + c1;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t t = __shfl_down_sync(FULL, suf, off);
                if (lane + off < 32) suf += t;
            }
            if (lane == 0) red[warp] = suf;
            __syncthreads();
            const uint32_t wtot = red[lane];
            uint32_t wsuf = wtot;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t t = __shfl_down_sync(FULL, wsuf, off);
                if (lane + off < 32) wsuf += t;
            }
            const uint32_t above = __shfl_sync(FULL, wsuf - wtot, warp);
            const uint32_t incl1 = above + suf - c0, excl1 = incl1 - c1, incl0 = incl1 + c0, kr = (uint32_t)k;
            if (incl1 >= kr && excl1 < kr) { s_digit = 2u * tid + 1u; s_krem = kr - excl1; s_cnt = c1; }
            if (incl0 >= kr && incl1 < kr) { s_digit = 2u * tid; s_krem = kr - incl1; s_cnt = c0; }
            __syncthreads();
            prefix |= s_digit << lo;
            k = (int)s_krem;
            whole = s_cnt == s_krem;                 // the whole bin is wanted: its lowest possible key is a threshold
            __syncthreads();
        }
        tau = prefix;
        r_eq = whole ? 0x7fffffff : k;               // keys equal to tau that are taken, lowest positions first
    }
    // every warp owns a contiguous range of the candidates: count, scan over the warps, write
    const int per = (C + 31) / 32, lo_j = warp * per, hi_j = min(C, lo_j + per);
    uint32_t wgt = 0, weq = 0;
    for (int j0 = lo_j; j0 < hi_j; j0 += 8 * 32) {
        float f[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) f[u] = j0 + u * 32 + lane < hi_j ? __ldcg(x + j0 + u * 32 + lane) : 0.0f;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const bool in = j0 + u * 32 + lane < hi_j;
            const uint32_t kx = order_key(f[u]);
            wgt += __popc(__ballot_sync(FULL, in && kx > tau));
            weq += __popc(__ballot_sync(FULL, in && kx == tau));
        }
    }
    if (lane == 0) { red[warp] = wgt; red2[warp] = weq; }
    __syncthreads();
    uint32_t g_inc = red[lane], e_inc = red2[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t tg = __shfl_up_sync(FULL, g_inc, off), te = __shfl_up_sync(FULL, e_inc, off);
        if (lane >= off) { g_inc += tg; e_inc += te; }
    }
    int gt_run = (int)(__shfl_sync(FULL, g_inc, warp) - wgt), eq_run = (int)(__shfl_sync(FULL, e_inc, warp) - weq);
    const uint32_t lt = (1u << lane) - 1u;
    for (int j0 = lo_j; j0 < hi_j; j0 += 8 * 32) {
        float f[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) f[u] = j0 + u * 32 + lane < hi_j ? __ldcg(x + j0 + u * 32 + lane) : 0.0f;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int j = j0 + u * 32 + lane;
            const bool in = j < hi_j;
            const uint32_t kx = order_key(f[u]);
            const bool is_gt = in && kx > tau, is_eq = in && kx == tau;
            const uint32_t bg = __ballot_sync(FULL, is_gt), be = __ballot_sync(FULL, is_eq);
            const int gb = gt_run + __popc(bg & lt), eb = eq_run + __popc(be & lt);
            const int rank = is_gt ? gb + min(eb, r_eq) : (is_eq && eb < r_eq) ? gb + eb : -1;
            if (rank >= 0 && rank < want) out[rank] = j;
            gt_run += __popc(bg);
            eq_run += __popc(be);
        }
    }
    for (int i = tid; i < w; i += 1024) out[want + i] = C + i;       // the window, above every candidate
}

// ---------------------------------------------------------------- compaction into the new cache
// One CTA of 256 threads per (head, page of the new cache).  The page's retained rows move in 16-byte
// pieces, keys and values alike (a thread per piece, a row's pieces on neighbouring threads); the keys
// also pass through shared memory, from which a thread per channel then takes the page's bounds.
constexpr int kCompactThreads = 256;
constexpr int kCompactSmem = 64 * 128 * 4;                 // the keys of one page at most: 64 slots x 128 channels x 4 bytes

template <typename T>
__global__ void __launch_bounds__(kCompactThreads) snap_compact_kernel(const T *skv, int64_t s_page_cap, T *dkv, T *dmeta,
                                                                       int64_t d_page_cap, int S, int D, const int32_t *idx,
                                                                       int keep, float *absmax, int BH)
{
    __shared__ __align__(16) unsigned char krows[kCompactSmem];
    __shared__ int32_t src_pos[64];
    const int bh = blockIdx.y, page = blockIdx.x, tid = threadIdx.x;
    const int rb = D * (int)sizeof(T), ppr = rb / 16;        // bytes and 16-byte pieces of a row
    const int rows = min(S, keep - page * S);                // retained rows of this page (at least one)
    if (tid < S) src_pos[tid] = tid < rows ? idx[(int64_t)bh * keep + page * S + tid] : -1;
    __syncthreads();
    unsigned char *dpage = reinterpret_cast<unsigned char *>(dkv + (((int64_t)bh * d_page_cap + page) * 2) * S * D);
    const unsigned char *shead = reinterpret_cast<const unsigned char *>(skv + (int64_t)bh * s_page_cap * 2 * S * D);
    for (int i = tid; i < S * ppr; i += kCompactThreads) {
        const int r = i / ppr, c = i % ppr;
        uint4 kq = make_uint4(0u, 0u, 0u, 0u), vq = kq;      // unused slots of the last page are defined (zero)
        if (r < rows) {
            const int64_t pos = src_pos[r];
            const unsigned char *src = shead + ((pos / S) * 2 * S + pos % S) * (int64_t)rb + c * 16;
            kq = *reinterpret_cast<const uint4 *>(src);
            vq = *reinterpret_cast<const uint4 *>(src + (int64_t)S * rb);
        }
        *reinterpret_cast<uint4 *>(dpage + (int64_t)r * rb + c * 16) = kq;
        *reinterpret_cast<uint4 *>(dpage + (int64_t)(S + r) * rb + c * 16) = vq;
        *reinterpret_cast<uint4 *>(krows + r * rb + c * 16) = kq;
    }
    __syncthreads();
    float am = 0.0f;
    if (tid < D) {
        const T *kr = reinterpret_cast<const T *>(krows);
        float mn = CUDART_INF_F, mx = -CUDART_INF_F;
        for (int r = 0; r < rows; ++r) {
            const float kf = load1<T>(kr + r * D + tid);
            mn = fminf(mn, kf);
            mx = fmaxf(mx, kf);
        }
        T *mrow = dmeta + (((int64_t)bh * d_page_cap + page) * 2) * D;
        store1<T>(mrow + tid, mn);
        store1<T>(mrow + D + tid, mx);
        am = fmaxf(-mn, mx);
    }
    if (absmax && tid < D) {                                 // D is a multiple of 32: whole warps
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, off));
        if ((tid & 31) == 0) {
            atomicMax(reinterpret_cast<unsigned *>(absmax) + bh, __float_as_uint(am));
            atomicMax(reinterpret_cast<unsigned *>(absmax) + BH + bh, __float_as_uint(am));
        }
    }
}

template <typename T, int D>
cudaError_t snap_scores_t(const SnapArgs &a, cudaStream_t s)
{
    using G = SnapGeom<D>;
    static bool ready[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!ready[dev]) {
        e = cudaFuncSetAttribute(snap_tile_kernel<T, D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(snap_tile_kernel<T, D, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        ready[dev] = true;
    }
    const int BH = a.B * a.H;
    const int ntiles = (int)((a.len + kSnapKeys - 1) / kSnapKeys);
    const dim3 grid((unsigned)ntiles, (unsigned)BH);
    const float sl2 = a.scale * 1.4426950408889634f;
    snap_tile_kernel<T, D, 1><<<grid, kSnapThreads, G::SMEM_BYTES, s>>>((const T *)a.kv, a.page_cap, a.S, a.len, (const T *)a.qw,
                                                                      a.W, a.H, sl2, a.stats, nullptr, nullptr, ntiles);
    const int rows = BH * kSnapRows;
    snap_rows_kernel<<<(rows * 32 + 127) / 128, 128, 0, s>>>(a.stats, a.rowstat, ntiles, rows);
    snap_tile_kernel<T, D, 2><<<grid, kSnapThreads, G::SMEM_BYTES, s>>>((const T *)a.kv, a.page_cap, a.S, a.len, (const T *)a.qw,
                                                                      a.W, a.H, sl2, nullptr, a.rowstat, a.imp, ntiles);
    return cudaGetLastError();
}

template <int D>
cudaError_t snap_scores_mma(const SnapArgs &a, cudaStream_t s)
{
    using G = SnapMmaGeom<D>;
    static bool ready[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!ready[dev]) {
        e = cudaFuncSetAttribute(snap_mma_kernel<D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(snap_mma_kernel<D, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        ready[dev] = true;
    }
    const int BH = a.B * a.H;
    if (kMmaKeys % a.S != 0) return cudaErrorInvalidValue;
    alignas(64) CUtensorMap tmap;
    e = cache_tensor_map(&tmap, a.kv, D, a.S, (int64_t)BH * a.page_cap, kMmaKeys);
    if (e != cudaSuccess) return e;
    const int ntiles = (int)((a.len + kMmaKeys - 1) / kMmaKeys);
    // tiles per CTA: two CTAs share an SM, so the launch runs in rounds of 2 * SMs CTAs; the choice with the fewest
    // rounds * (tiles of a CTA + what a CTA costs before its first tile, about two tiles' time) ends soonest
    const int64_t slots = 2 * (int64_t)sm_count();
    int tpc = 1;
    int64_t best = INT64_MAX;
    for (int c = 1; c <= kMmaMaxTiles * 2 && c <= ntiles; ++c) {
        const int64_t ctas = (int64_t)BH * ((ntiles + c - 1) / c);
        const int64_t cost = ((ctas + slots - 1) / slots) * (c + 2);
        if (cost <= best) {                            // equal cost: the longer runs (fewer partial statistics)
            best = cost;
            tpc = c;
        }
    }
    const int runs = (ntiles + tpc - 1) / tpc;
    const dim3 grid((unsigned)runs, (unsigned)BH);
    const float sl2 = a.scale * 1.4426950408889634f;
    snap_mma_kernel<D, 1><<<grid, kMmaThreads, G::SMEM_BYTES, s>>>(tmap, a.page_cap, a.S, a.len, (const bf16 *)a.qw, a.W, a.H, sl2,
                                                                 a.stats, nullptr, nullptr, ntiles, tpc, a.status);
    const int rows = BH * kSnapRows;
    snap_rows_kernel<<<(rows * 32 + 127) / 128, 128, 0, s>>>(a.stats, a.rowstat, runs, rows);
    snap_mma_kernel<D, 2><<<grid, kMmaThreads, G::SMEM_BYTES, s>>>(tmap, a.page_cap, a.S, a.len, (const bf16 *)a.qw, a.W, a.H, sl2,
                                                                 nullptr, a.rowstat, a.imp, ntiles, tpc, a.status);
    return cudaGetLastError();
}

size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }

}  // namespace

size_t snap_scratch_bytes(int BH, int64_t len)
{
    const size_t ntiles = (size_t)((len + kSnapKeys - 1) / kSnapKeys);
    return round256((size_t)BH * len * sizeof(float))                         // importance
           + round256((size_t)BH * ntiles * kSnapRows * sizeof(float2))       // per-tile statistics
           + round256((size_t)BH * kSnapRows * sizeof(float2));               // final statistics
}

void snap_carve(void *scratch, int BH, int64_t len, float **imp, float2 **stats, float2 **rowstat)
{
    const size_t ntiles = (size_t)((len + kSnapKeys - 1) / kSnapKeys);
    char *p = (char *)scratch;
    *imp = (float *)p;
    p += round256((size_t)BH * len * sizeof(float));
    *stats = (float2 *)p;
    p += round256((size_t)BH * ntiles * kSnapRows * sizeof(float2));
    *rowstat = (float2 *)p;
}

cudaError_t launch_snap_scores(const SnapArgs &a, cudaStream_t s)
{
    if (a.W < 1 || a.W > kSnapRows || a.len < a.W) return cudaErrorInvalidValue;
    if (a.B * a.H > 65535) return cudaErrorInvalidValue;
    if (a.dtype == RQ_BF16) {
        if (a.D == 128) return snap_scores_mma<128>(a, s);
        if (a.D == 64) return snap_scores_mma<64>(a, s);
    } else {
        if (a.D == 128) return snap_scores_t<float, 128>(a, s);
        if (a.D == 64) return snap_scores_t<float, 64>(a, s);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_snap_select(const float *imp, int BH, int64_t len, int window, int keep, int32_t *idx, cudaStream_t s)
{
    int w = window < keep ? window : keep;
    if ((int64_t)w > len) w = (int)len;
    snap_select_kernel<<<(unsigned)BH, 1024, 0, s>>>(imp, len, w, keep, idx);
    return cudaGetLastError();
}

cudaError_t launch_snap_compact(const void *skv, int64_t s_page_cap, void *dkv, void *dmeta, int64_t d_page_cap, int S, int D,
                                int dtype, const int32_t *idx, int keep, float *absmax, int BH, cudaStream_t s)
{
    const dim3 grid((unsigned)((keep + S - 1) / S), (unsigned)BH);
    if (dtype == RQ_BF16)
        snap_compact_kernel<bf16><<<grid, kCompactThreads, 0, s>>>((const bf16 *)skv, s_page_cap, (bf16 *)dkv, (bf16 *)dmeta, d_page_cap, S, D, idx,
                                                     keep, absmax, BH);
    else
        snap_compact_kernel<float><<<grid, kCompactThreads, 0, s>>>((const float *)skv, s_page_cap, (float *)dkv, (float *)dmeta, d_page_cap, S, D,
                                                      idx, keep, absmax, BH);
    return cudaGetLastError();
}

}  // namespace rq
