// MoBA-style block-sparse prefill attention on the cache of decayed keys and values (Sec. 2.2, Eq. 3
// and Eq. 4, Table 1 row MoBA; App. A.1, "Sparse inference settings", MoBA paragraph): every prompt
// position routes its query to a few of the KV blocks before it, scored with mean-pooled block
// representatives, and attends over the chosen blocks only; the first block and the query's own
// block (cut at the query's position) are always among them and count inside the budget.
//
//   moba_means_kernel    per (head, block): the mean of the block's stored keys, fp32
//   moba_route_kernel    per (head, 16 consecutive queries), a warp per query: scores q . mean of the
//                        complete blocks before the query's own (a lane per block; the head's
//                        representatives staged in shared memory once per CTA when they fit), then the
//                        budget's best (equal scores to the lower block) by a bit-wise search for the
//                        threshold score, or by repeated arg-max when the budget is small or the candidates many;
//                        the list written ascending
//   moba_mma_kernel      bf16 caches.  Per (head, 128 consecutive queries): both contractions on the
//                        tensor cores (tcgen05.mma, accumulators and the weights in tensor memory),
//                        the chunks of the blocks any of the 128 queries chose walked twice (row
//                        maxima, then weights and O += P V); see the comment above the kernel
//   moba_attend_kernel   fp32 caches.  Per (head, 16 consecutive queries), a warp per query: the blocks
//                        any of the 16 queries chose pass through shared memory once, 64 positions at a
//                        time (cp.async, two buffers); a warp folds a chunk into its online softmax
//                        only if its own query chose the block (plain fp32 FMA work; the arithmetic is
//                        the decode path's tile routine)
#include <limits.h>
#include <math_constants.h>

#include "rq_async.cuh"
#include "rq_device.cuh"
#include "rq_internal.h"
#include "rq_stream.cuh"
#include "rq_tmap.h"
#include "rq_umma.cuh"

namespace rq {

namespace {

constexpr int kMobaChunk = 64;                 // positions that pass through shared memory at a time
constexpr int kMobaQueries = 16;               // queries (warps) of one attention CTA
constexpr int kMobaRouteWarps = 16;            // warps of one routing CTA
constexpr int kMobaRouteQ = 2;                 // consecutive queries of one routing warp when the representatives are staged (they share the reads)
constexpr int kMobaMaxBlocks = 2048;           // blocks of a prompt at most
constexpr unsigned FULLMASK = 0xffffffffu;

// floats of shared memory one routing warp needs: query, scores, mask words; a multiple of 4 so that
// every warp's query starts on a 16-byte boundary
__host__ __device__ inline int moba_route_floats(int D, int nb) { return (D + nb + (nb + 31) / 32 + 3) & ~3; }

__device__ __forceinline__ void cp_async16(void *dst_smem, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// ---------------------------------------------------------------- block representatives
// Grid (blocks, heads), a thread per channel; the sum runs over the block's valid positions in order.
template <typename T>
__global__ void moba_means_kernel(const T *kv, int64_t page_cap, int S, int D, int64_t len, int block, float *means, int nb)
{
    const int j = blockIdx.x, bh = blockIdx.y, c = threadIdx.x;
    const int64_t lo = (int64_t)j * block, hi = min(lo + block, len);
    float s = 0.0f;
    int64_t p = lo;
    // sixteen loads in flight at a time (a page holds a multiple of 16 positions and lo is a multiple of 64, so
    // a run of 16 stays inside one page); the additions keep the order of the positions
    for (; p + 16 <= hi; p += 16) {
        const T *src = kv + ((((int64_t)bh * page_cap + p / S) * 2) * S + p % S) * D + c;
        float x[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] = load1<T>(src + (int64_t)i * D);
#pragma unroll
        for (int i = 0; i < 16; ++i) s += x[i];
    }
    for (; p < hi; ++p) s += load1<T>(kv + ((((int64_t)bh * page_cap + p / S) * 2) * S + p % S) * D + c);
    means[((int64_t)bh * nb + j) * D + c] = s / (float)(hi - lo);
}

// The `want` best of the candidate blocks c_lo .. c_hi - 1 with scores sc[], for one warp; lane l owns the
// candidates c_lo + l + 32 r, r < R.  A candidate beats another with a higher score, or the same score and a lower
// block.  The score of the want-th best is found bit by bit on the order-preserving integer image of the scores
// (32 rounds of one comparison and one vote per owned candidate: far fewer operations than ranking every candidate
// against every other); the candidates above it are taken, and of those equal to it the lowest blocks.  Sets their
// mask bits.
template <int R>
__device__ __forceinline__ void moba_rank_take(const float *sc, uint32_t *mask, int c_lo, int c_hi, int want, int lane)
{
    uint32_t key[R];
    bool valid[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int j = c_lo + lane + 32 * r;
        valid[r] = j < c_hi;
        const uint32_t b = __float_as_uint((valid[r] ? sc[j] : 0.0f) + 0.0f);     // -0 becomes +0
        key[r] = b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
    }
    // the largest t with at least `want` keys >= t: the want-th largest key (want <= number of candidates)
    uint32_t t = 0u;
#pragma unroll 4
    for (int bit = 31; bit >= 0; --bit) {
        const uint32_t trial = t | (1u << bit);
        int cnt = 0;
#pragma unroll
        for (int r = 0; r < R; ++r) cnt += __popc(__ballot_sync(0xffffffffu, valid[r] && key[r] >= trial));
        if (cnt >= want) t = trial;
    }
    int above = 0;
#pragma unroll
    for (int r = 0; r < R; ++r) above += __popc(__ballot_sync(0xffffffffu, valid[r] && key[r] > t));
    int need = want - above;                         // of the candidates equal to the threshold, in block order
    const uint32_t lt = (1u << lane) - 1u;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const uint32_t eq = __ballot_sync(0xffffffffu, valid[r] && key[r] == t);
        const bool mine = valid[r] && (key[r] > t || (key[r] == t && __popc(eq & lt) < need));
        need = max(0, need - __popc(eq));
        const unsigned take = __ballot_sync(0xffffffffu, mine);          // blocks c_lo + 32 r + bit
        if (lane == 0 && take) {
            const int p = c_lo + 32 * r;
            mask[p >> 5] |= take << (p & 31);
            if (p & 31) mask[(p >> 5) + 1] |= take >> (32 - (p & 31));
        }
    }
}

// ---------------------------------------------------------------- routing
// Grid (ceil(T / queries of a CTA), heads); a warp per query, or per two consecutive queries when the
// representatives are staged (a lane reads a representative once for both).  Shared memory per query: the
// query (D floats), the scores of the candidate blocks (nb floats), the chosen blocks as a bit mask
// (nb / 32 words); and, when they fit (STAGED), the head's representatives for the whole CTA, rows padded
// by four floats so that the lanes of a quarter-warp, each reading its own row, hit different banks.
// q: [B][T][H][D].  sel: [BH][T][K], ascending, -1 beyond the chosen blocks.
constexpr int kMobaStagedBlocks = 128;         // representatives of up to this many blocks are staged in shared memory

// The selection of one query once the scores of its candidate blocks c_lo .. c_hi - 1 are in sc[]: the `want` best
// into the mask, the first block(s) and the own block(s) added, the chosen blocks written ascending.  One warp.
__device__ __forceinline__ void moba_route_finish(const float *sc, uint32_t *mask, int32_t *out, int words, int K, int P, int ns,
                                                  int nl, int c_lo, int c_hi, int want, int lane)
{
    if (c_hi - c_lo <= 4 * 32 && want >= 8) {
        // few candidates and more than a handful to take (a round per taken block is cheaper otherwise): the
        // threshold score by bit-wise search, a lane holding one, two or four candidates
        const int ncand = c_hi - c_lo;
        if (ncand <= 32) moba_rank_take<1>(sc, mask, c_lo, c_hi, want, lane);
        else if (ncand <= 64) moba_rank_take<2>(sc, mask, c_lo, c_hi, want, lane);
        else moba_rank_take<4>(sc, mask, c_lo, c_hi, want, lane);
        __syncwarp();
    } else {
    // the `want` best candidates, one per round: every lane's best of its blocks, then the warp's best;
    // equal scores go to the lower block
    for (int r = 0; r < want; ++r) {
        float bv = -CUDART_INF_F;
        int bj = INT_MAX;
        for (int j = c_lo + lane; j < c_hi; j += 32) {
            const float v = sc[j];
            const bool taken = (mask[j >> 5] >> (j & 31)) & 1u;
            if (!taken && (bj == INT_MAX || v > bv)) { bv = v; bj = j; }   // ascending j: '>' keeps the lower block
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(FULLMASK, bv, off);
            const int oj = __shfl_xor_sync(FULLMASK, bj, off);
            if (oj != INT_MAX && (bj == INT_MAX || ov > bv || (ov == bv && oj < bj))) { bv = ov; bj = oj; }
        }
        if (lane == 0 && bj != INT_MAX) mask[bj >> 5] |= 1u << (bj & 31);
        __syncwarp();
    }
    }
    if (lane == 0) {
        for (int j = 0; j < ns; ++j) mask[j >> 5] |= 1u << (j & 31);
        for (int j = P - nl; j < P; ++j) mask[j >> 5] |= 1u << (j & 31);
    }
    __syncwarp();
    // ascending list from the mask
    int base = 0;
    if (words <= 4) {
        // few blocks: a lane looks at its own bit of every word; a chosen block's place in the list is the
        // number of chosen blocks below it
        const uint32_t lt = (1u << lane) - 1u;
        for (int r = 0; r < words; ++r) {
            const uint32_t w = mask[r];
            if ((w >> lane) & 1u) {
                const int pos = base + __popc(w & lt);
                if (pos < K) out[pos] = r * 32 + lane;
            }
            base += __popc(w);
        }
        for (int i = base + lane; i < K; i += 32) out[i] = -1;
        return;
    }
    for (int w0 = 0; w0 < words; w0 += 32) {
        const uint32_t w = w0 + lane < words ? mask[w0 + lane] : 0u;
        const int cnt = __popc(w);
        int inc = cnt;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(FULLMASK, inc, off);
            if (lane >= off) inc += o;
        }
        int pos = base + inc - cnt;
        uint32_t bits = w;
        while (bits) {
            const int bit = __ffs(bits) - 1;
            bits &= bits - 1;
            if (pos < K) out[pos] = (w0 + lane) * 32 + bit;
            ++pos;
        }
        base += __shfl_sync(FULLMASK, inc, 31);
    }
    for (int i = base + lane; i < K; i += 32) out[i] = -1;
}

template <typename T, int D, bool STAGED>
__global__ void __launch_bounds__(kMobaRouteWarps * 32) moba_route_kernel(const T *q, const float *means, int64_t len, int H,
                                                                         int block, int nb, int K, int32_t *sel)
{
    extern __shared__ __align__(16) float rsm[];
    constexpr int LDM = STAGED ? D + 4 : D;            // floats from one representative to the next
    constexpr int QW = STAGED ? kMobaRouteQ : 1, QC = kMobaRouteWarps * QW;   // queries of a warp, of the CTA
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int words = (nb + 31) / 32;
    const int per = moba_route_floats(D, nb);
    float *wsm = rsm + (size_t)warp * QW * per;        // this warp's queries, scores and masks
    const int bh = blockIdx.y;
    const float *mh = means + (int64_t)bh * nb * D;
    if (STAGED) {
        // the representatives the CTA's queries can need: blocks before the last query's own
        float *ms = rsm + (size_t)kMobaRouteWarps * QW * per;
        const int64_t t_last = min((int64_t)blockIdx.x * QC + QC - 1, len - 1);
        const int need = (int)(t_last / block);
        for (int i = threadIdx.x; i < need * (D / 4); i += kMobaRouteWarps * 32) {
            const int j = i / (D / 4), c = i % (D / 4);
            *reinterpret_cast<float4 *>(ms + j * LDM + 4 * c) = __ldg(reinterpret_cast<const float4 *>(mh + (int64_t)j * D) + c);
        }
        __syncthreads();
        mh = ms;
    }
    const int b = bh / H, h = bh % H;
    // the first block and the own block inside the budget (K >= 2), as the first and the newest page of a decode step
    const int ns = min(1, K), nl = min(1, K - ns), want = K - ns - nl;
    const int c_lo = ns;
    int P[QW], c_hi[QW];                               // blocks a query may attend; its candidates end before c_hi
    bool active[QW];
    int c_hi_max = 0;
#pragma unroll
    for (int u = 0; u < QW; ++u) {
        const int64_t t = (int64_t)blockIdx.x * QC + warp * QW + u;
        active[u] = false;
        P[u] = c_hi[u] = 0;
        if (t >= len) continue;                        // (no CTA-wide barrier below)
        int32_t *out = sel + ((int64_t)bh * len + t) * K;
        P[u] = (int)(t / block) + 1;
        if (K >= P[u]) {                               // everything before the query
            for (int i = lane; i < K; i += 32) out[i] = i < P[u] ? i : -1;
            continue;
        }
        active[u] = true;
        c_hi[u] = P[u] - nl;                           // candidates: blocks c_lo .. c_hi - 1 (all complete)
        c_hi_max = max(c_hi_max, c_hi[u]);
        float *qs = wsm + u * per;
        uint32_t *mask = reinterpret_cast<uint32_t *>(qs + D + nb);
        for (int i = lane; i < D; i += 32) qs[i] = load1<T>(q + (((int64_t)b * len + t) * H + h) * D + i);
        for (int i = lane; i < words; i += 32) mask[i] = 0u;
    }
    if (c_hi_max == 0) return;
    __syncwarp();
    // scores: a lane per block, the block's representative read as 16-byte pieces once for the warp's queries
    for (int j0 = c_lo; j0 < c_hi_max; j0 += 32) {
        const int j = j0 + lane;
        if (j < c_hi_max) {
            const float4 *row = reinterpret_cast<const float4 *>(mh + (int64_t)j * LDM);
            // packed pairs: the even and the odd channels are summed apart and added at the end
            float2 s2[QW];
#pragma unroll
            for (int u = 0; u < QW; ++u) s2[u] = make_float2(0.0f, 0.0f);
#pragma unroll 8
            for (int i = 0; i < D / 4; ++i) {
                const float4 m4 = STAGED ? row[i] : __ldg(row + i);
#pragma unroll
                for (int u = 0; u < QW; ++u) {
                    if (!active[u]) continue;          // (the same for the whole warp)
                    const float4 q4 = *reinterpret_cast<const float4 *>(wsm + u * per + 4 * i);
                    s2[u] = fma2(make_float2(q4.x, q4.y), make_float2(m4.x, m4.y), s2[u]);
                    s2[u] = fma2(make_float2(q4.z, q4.w), make_float2(m4.z, m4.w), s2[u]);
                }
            }
#pragma unroll
            for (int u = 0; u < QW; ++u)
                if (active[u] && j < c_hi[u]) (wsm + u * per + D)[j] = s2[u].x + s2[u].y;
        }
    }
    __syncwarp();
#pragma unroll
    for (int u = 0; u < QW; ++u) {
        if (!active[u]) continue;
        const int64_t t = (int64_t)blockIdx.x * QC + warp * QW + u;
        float *sc = wsm + u * per + D;
        moba_route_finish(sc, reinterpret_cast<uint32_t *>(sc + nb), sel + ((int64_t)bh * len + t) * K, words, K, P[u], ns, nl, c_lo,
                          c_hi[u], want, lane);
    }
}

// ---------------------------------------------------------------- attention
// Grid (ceil(T / 16), heads), 16 warps, a warp per query.  Shared memory: two chunk buffers (64 key
// rows then 64 value rows each), the blocks chosen by any of the CTA's queries (bit mask) and by each
// query (16 bit masks).
template <typename T, int D>
__global__ void __launch_bounds__(kMobaQueries * 32) moba_attend_kernel(const T *kv, int64_t page_cap, int S, int64_t len,
                                                                       const T *q, int H, int block, int nb, int K,
                                                                       const int32_t *sel, float scale_log2, T *o)
{
    constexpr int CH = VecOf<T>::N, LPR = D / CH;
    constexpr int ROW_BYTES = D * (int)sizeof(T), PPR = ROW_BYTES / 16;      // 16-byte pieces of a row
    constexpr int CHUNK_BYTES = 2 * kMobaChunk * ROW_BYTES;
    constexpr int NT = kMobaQueries * 32;
    extern __shared__ __align__(16) unsigned char asmem[];
    unsigned char *buf = asmem;                                              // [2][CHUNK_BYTES]
    uint32_t *umask = reinterpret_cast<uint32_t *>(asmem + 2 * CHUNK_BYTES); // [words]
    const int words = (nb + 31) / 32;
    uint32_t *qmask = umask + words;                                         // [16][words]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    const int64_t t = (int64_t)blockIdx.x * kMobaQueries + warp;
    const bool active = t < len;

    for (int i = tid; i < words * (kMobaQueries + 1); i += NT) umask[i] = 0u;
    __syncthreads();
    if (active) {
        const int32_t *list = sel + ((int64_t)bh * len + t) * K;
        for (int i = lane; i < K; i += 32) {
            const int j = list[i];
            if (j >= 0 && j < nb) {
                atomicOr(&qmask[warp * words + (j >> 5)], 1u << (j & 31));
                atomicOr(&umask[j >> 5], 1u << (j & 31));
            }
        }
    }
    __syncthreads();

    AttendState<T> st;
    attend_begin_head<T, D>(st, q + (((int64_t)b * len + (active ? t : 0)) * H + h) * D, 0, scale_log2, lane);

    const T *head = kv + (int64_t)bh * page_cap * 2 * S * D;
    // copies of chunk `ci` of block j (positions j * block + ci * 64 ...) into buffer `bi`
    auto issue = [&](int j, int ci, int bi) {
        const int64_t p0 = (int64_t)j * block + (int64_t)ci * kMobaChunk;
        unsigned char *dst = buf + (size_t)bi * CHUNK_BYTES;
        for (int i = tid; i < kMobaChunk * PPR; i += NT) {
            const int r = i / PPR, c = i % PPR;
            const int64_t p = p0 + r;
            if (p < len) {
                const unsigned char *src =
                    reinterpret_cast<const unsigned char *>(head + (((p / S) * 2) * S + p % S) * D) + c * 16;
                cp_async16(dst + r * ROW_BYTES + c * 16, src);
                cp_async16(dst + (kMobaChunk + r) * ROW_BYTES + c * 16, src + (int64_t)S * ROW_BYTES);
            } else {                                         // rows past the prompt: defined (a masked row still multiplies its values by 0)
                *reinterpret_cast<uint4 *>(dst + r * ROW_BYTES + c * 16) = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4 *>(dst + (kMobaChunk + r) * ROW_BYTES + c * 16) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
    };
    // the chunks of the chosen blocks in ascending order: (block, chunk) -> next
    const int cpb = block / kMobaChunk;
    auto next_chunk = [&](int &j, int &ci) -> bool {     // from (j, ci) to the following chunk; false at the end
        if (j >= 0 && ci + 1 < cpb && ((int64_t)j * block + (int64_t)(ci + 1) * kMobaChunk) < len) { ++ci; return true; }
        for (int jj = j + 1; jj < nb; ++jj)
            if ((umask[jj >> 5] >> (jj & 31)) & 1u) { j = jj; ci = 0; return true; }
        return false;
    };
    int j = -1, ci = 0, bi = 0;
    bool have = next_chunk(j, ci);
    if (have) issue(j, ci, 0);
    cp_async_commit();
    while (have) {
        int jn = j, cn = ci;
        const bool have_next = next_chunk(jn, cn);
        if (have_next) issue(jn, cn, bi ^ 1);           // the other buffer was released by the barrier below
        cp_async_commit();
        cp_async_wait<1>();                              // this thread's pieces of the current chunk
        __syncthreads();                                 // everybody's
        if (active && ((qmask[warp * words + (j >> 5)] >> (j & 31)) & 1u)) {
            const T *ks = reinterpret_cast<const T *>(buf + (size_t)bi * CHUNK_BYTES);
            const T *vs = ks + kMobaChunk * D;
            const int64_t p0 = (int64_t)j * block + (int64_t)ci * kMobaChunk;
#pragma unroll 1
            for (int i = 0; i < kMobaChunk / kTileRows; ++i) {
                const int64_t pt = p0 + (int64_t)i * kTileRows;
                const int valid = (int)min((int64_t)kTileRows, t - pt + 1);   // the query sees positions up to its own
                if (valid > 0) attend_tile<T, D, kTileRows>(st, ks + i * kTileRows * D, vs + i * kTileRows * D, valid, lane);
            }
        }
        __syncthreads();                                 // the buffer may be refilled
        j = jn; ci = cn; have = have_next; bi ^= 1;
    }
    cp_async_wait<0>();
    if (active) {
        attend_merge_rows<T, D, kTileRows>(st);
        if (lane < LPR) {
            const float inv = 1.0f / st.l;               // the own block always holds the query's own position
            T *orow = o + (((int64_t)b * len + t) * H + h) * D + lane * CH;
#pragma unroll
            for (int c = 0; c < CH; ++c) store1<T>(orow + c, st.acc[c] * inv);
        }
    }
}

// ---------------------------------------------------------------- attention on the tensor cores (bf16 caches)
// Grid (ceil(T / 128), heads).  A CTA owns 128 consecutive queries of a head: they are the 128 lanes of the
// accumulators, so everything per query (mask, running maximum, sum, weights) is per thread.  The chunks
// (64 positions) of the blocks ANY of the 128 queries chose are walked twice:
//   pass 1   S = Q K^T for two chunks at a time (tcgen05.mma, 128 x 128, fp32 in tensor memory, two accumulators);
//            a thread masks its chunk for its query (block not chosen / positions after the query) and keeps the
//            running maximum
//   pass 2   S again; the thread turns its row into weights relative to the query's maximum (summed in fp32 for
//            the final division), rounds them to bf16 and writes them
//            into tensor memory (tcgen05.st) as the A operand of the second product, O += P V (128 x D, the values
//            as an MN-major operand straight from the cache's rows), accumulated in tensor memory over all chunks
// One thread of a ninth warp starts the tensor-map copies (keys and values of a chunk, two stages each) and the
// products; the eight other warps read the accumulators (two per query, half of a chunk's positions each).  They meet only through mbarriers; every wait is bounded.
constexpr int kMobaMmaQueries = 128;
constexpr int kMobaMmaWarps = 8;               // warps that read the accumulators: two per 32 lanes, half of the columns each
constexpr int kMobaMmaThreads = (kMobaMmaWarps + 1) * 32;
constexpr int kMobaMmaStages = 2;

template <int D>
struct MobaMmaGeom {
    static constexpr int HALVES = D / 64;
    static constexpr int Q_BYTES = HALVES * 128 * 128;             // 128 queries
    static constexpr int KC_BYTES = HALVES * kMobaChunk * 128;     // the keys (or the values) of a chunk
    static constexpr int OFF_K = Q_BYTES;
    static constexpr int OFF_V = OFF_K + kMobaMmaStages * KC_BYTES;
    static constexpr int OFF_MASK = OFF_V + kMobaMmaStages * KC_BYTES;
    static constexpr int FIXED_BYTES = OFF_MASK + 1024;            // + room to align the base to 1024 bytes
};

__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t saddr, uint32_t lbo_bytes)
{
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
__device__ __forceinline__ float exp2_fast(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2_bf16(float a, float b)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t *>(&h);
}

// Walk over the 64-position chunks of the chosen blocks in ascending order: (block, chunk inside the block).
// A block holds cpb chunks; the walk ends (returns n_chunks) after the last chosen block or at chunk n_chunks.
struct MobaWalk {
    int j = -1, r = 0;
};
__device__ __forceinline__ int moba_walk_next(MobaWalk &w, const uint32_t *chosen, int nb, int cpb, int n_chunks)
{
    if (w.j >= 0 && w.r + 1 < cpb && w.j * cpb + w.r + 1 < n_chunks) return w.j * cpb + ++w.r;
    int jj = w.j + 1;
    while (jj < nb) {
        const uint32_t bits = chosen[jj >> 5] >> (jj & 31);
        if (bits) {
            jj += __ffs(bits) - 1;
            break;
        }
        jj = (jj | 31) + 1;
    }
    w.j = jj;
    w.r = 0;
    return jj < nb ? min(jj * cpb, n_chunks) : n_chunks;
}

template <int D>
__global__ void __launch_bounds__(kMobaMmaThreads) moba_mma_kernel(const __grid_constant__ CUtensorMap tmap, int64_t page_cap, int S,
                                                                  int64_t len, const bf16 *q, int H, int block, int nb, int K,
                                                                  const int32_t *sel, float scale_log2, bf16 *o, int32_t *status)
{
    using G = MobaMmaGeom<D>;
    constexpr int NST = kMobaMmaStages;
    static_assert(NST == 2, "pass 1 uses the key region and the value region as its two stages of two chunks each");
    // tensor memory, 256 columns.  Pass 1: two score accumulators of 128 columns.  Pass 2: one score accumulator of 64
    // columns, the output (D columns), two weight buffers of 32 columns (64 positions as bf16 pairs).  With two key and
    // two value stages a CTA needs 97 KB of shared memory, so that TWO CTAs share an SM: each CTA's chunk is a chain of
    // dependent steps, and the two chains overlap
    constexpr uint32_t OFF_O = 64, OFF_P = 64 + D, P_COLS = 32, TCOLS = 256;
    extern __shared__ __align__(1024) unsigned char msm_raw[];
    __shared__ __align__(8) uint64_t full_k[NST], full_v[NST], s_ready[2], s_free[2], p_ready[2], pv_done[2], stat_ready;
    __shared__ __align__(8) uint64_t full1[2], s1_ready[2], s1_free[2];    // pass 1: stage landed, scores ready, scores read
    __shared__ float2 stat[2][kMobaMmaQueries];                          // pass 1: a query's statistics from its two threads
    __shared__ uint32_t tbase;
    unsigned char *msm = msm_raw + ((1024u - (smem_addr(msm_raw) & 1023u)) & 1023u);
    unsigned char *qs = msm, *kst = msm + G::OFF_K, *vst = msm + G::OFF_V;
    const int words = (nb + 31) / 32;
    uint32_t *umask = reinterpret_cast<uint32_t *>(msm + G::OFF_MASK);   // blocks chosen by any query of the CTA
    uint32_t *qmask = umask + words;                                     // [128][words] blocks chosen by each query

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // the work of a CTA grows with the position of its queries (the blocks before them): the CTAs of the last
    // queries of every head start first, so that the short ones fill the end of the launch
    const int bh = blockIdx.x, b = bh / H, h = bh % H;
    const int64_t t0 = (int64_t)(gridDim.y - 1 - blockIdx.y) * kMobaMmaQueries;
    // chunks of 64 positions up to the CTA's last query; chunk c belongs to block c * 64 / block
    const int n_chunks_all = (int)((min(t0 + kMobaMmaQueries, len) + kMobaChunk - 1) / kMobaChunk);

    if (tid == 0) {
        for (int s = 0; s < NST; ++s) { mbar_init(&full_k[s], 1); mbar_init(&full_v[s], 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&s_ready[s], 1);
            mbar_init(&pv_done[s], 1);
            mbar_init(&s_free[s], kMobaMmaWarps * 32);
            mbar_init(&p_ready[s], kMobaMmaWarps * 32);
            mbar_init(&full1[s], 1);
            mbar_init(&s1_ready[s], 1);
            mbar_init(&s1_free[s], kMobaMmaWarps * 32);
        }
        mbar_init(&stat_ready, kMobaMmaWarps * 32);
        mbar_init_fence();
    }
    if (warp == 0) tmem_alloc(&tbase, TCOLS);
    for (int i = tid; i < words * (kMobaMmaQueries + 1); i += kMobaMmaThreads) umask[i] = 0u;
    // the queries (q is [B][T][H][D]) as the K-major operand; rows past the prompt are zero
    for (int i = tid; i < 128 * (D / 8); i += kMobaMmaThreads) {
        const int r = i / (D / 8), c = i % (D / 8);
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (t0 + r < len) v = *reinterpret_cast<const uint4 *>(q + (((int64_t)b * len + t0 + r) * H + h) * D + c * 8);
        *reinterpret_cast<uint4 *>(qs + (c >> 3) * (128 * 128) + umma_sw128_offset(r, c & 7)) = v;
    }
    __syncthreads();
    if (tid < kMobaMmaQueries && t0 + tid < len) {
        const int32_t *list = sel + ((int64_t)bh * len + t0 + tid) * K;
        for (int i = 0; i < K; ++i) {
            const int j = list[i];
            if (j >= 0 && j < nb) {
                qmask[tid * words + (j >> 5)] |= 1u << (j & 31);
                atomicOr(&umask[j >> 5], 1u << (j & 31));
            }
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the queries, written with ordinary stores, are read by the tensor core
    tcgen05_before_sync();
    __syncthreads();
    tcgen05_after_sync();
    const uint32_t tb = tbase;
    // number of chunks the CTA walks in one pass: the chunks of the chosen blocks, below the CTA's last chunk
    const int cpb = block / kMobaChunk;
    const int ppc = kMobaChunk / S;                  // pages of a chunk (a page holds 16 or 64 positions)
    int n = 0;
    for (int wd = 0; wd < words; ++wd) {
        uint32_t bits = umask[wd];
        while (bits) {
            const int j = wd * 32 + __ffs(bits) - 1;
            bits &= bits - 1;
            n += max(0, min(cpb, n_chunks_all - j * cpb));
        }
    }
    // the next chunk of a walk (both roles walk the same chunks in the same order)
    auto next_chunk = [&](MobaWalk &w) { return moba_walk_next(w, umask, nb, cpb, n_chunks_all); };
    bool ok = true;

    if (warp == kMobaMmaWarps) {
        if (lane == 0) {
            // ---- copies and products; hh counts the chunks of pass 2
            MobaWalk wk, wv, w1;                     // chunk walks of pass 2's key copies and value copies, and of pass 1
            int gk_issued = 0, hv_issued = 0, gk_landed = 0, hv_landed = 0;
            auto issue_k = [&]() {                   // keys of the next chunk of the walk into stage gk_issued % NST
                const int ck_issue = next_chunk(wk);
                const int st = gk_issued % NST;
                const int page = (int)((int64_t)bh * page_cap + ck_issue * ppc);
                mbar_arrive_expect_tx(&full_k[st], G::KC_BYTES);
#pragma unroll
                for (int hf = 0; hf < G::HALVES; ++hf)
                    tma_load_4d(kst + (size_t)st * G::KC_BYTES + hf * (kMobaChunk * 128), &tmap, hf * 64, 0, 0, page, &full_k[st]);
                ++gk_issued;
            };
            auto issue_v = [&]() {
                const int cv_issue = next_chunk(wv);
                const int st = hv_issued % NST;
                const int page = (int)((int64_t)bh * page_cap + cv_issue * ppc);
                mbar_arrive_expect_tx(&full_v[st], G::KC_BYTES);
#pragma unroll
                for (int hf = 0; hf < G::HALVES; ++hf)
                    tma_load_4d(vst + (size_t)st * G::KC_BYTES + hf * (kMobaChunk * 128), &tmap, hf * 64, 0, 1, page, &full_v[st]);
                ++hv_issued;
            };
            auto product_pv = [&](int hh) -> bool {  // O += P(hh) V(hh)
                if (!mbar_wait(&p_ready[hh & 1], (uint32_t)((hh >> 1) & 1))) return false;
                if (!mbar_wait(&full_v[hh % NST], (uint32_t)((hh / NST) & 1))) return false;
                hv_landed = hh + 1;
                tcgen05_after_sync();
                constexpr uint32_t idesc = umma_idesc_bf16(128, D) | (1u << 16);       // the values are MN-major
                const uint32_t pa = tb + OFF_P + (uint32_t)(hh & 1) * P_COLS, va = smem_addr(vst + (size_t)(hh % NST) * G::KC_BYTES);
#pragma unroll
                for (int k = 0; k < kMobaChunk / 16; ++k)
                    umma_bf16_ta(tb + OFF_O, pa + k * 8, umma_desc_sw128_mn(va + k * 2048, kMobaChunk * 128), idesc,
                                 (hh > 0 || k > 0) ? 1u : 0u);
                umma_commit(&pv_done[hh & 1]);
                return true;
            };
            // ---- pass 1: the queries' maxima.  Two chunks (128 keys) per product; the key region and the value region
            // are its two stages; two accumulators of 128 columns (the columns pass 2 uses for scores, output and weights)
            const uint32_t qa = smem_addr(qs);
            const int n1 = (n + 1) / 2;
            int issued1 = 0, landed1 = 0;
            auto issue1 = [&](int it) {
                unsigned char *dst = (it & 1) ? vst : kst;
                const int cnt = min(2, n - 2 * it);
                mbar_arrive_expect_tx(&full1[it & 1], (uint32_t)cnt * G::KC_BYTES);
                for (int u = 0; u < cnt; ++u) {
                    const int c1 = next_chunk(w1);
                    const int page = (int)((int64_t)bh * page_cap + c1 * ppc);
#pragma unroll
                    for (int hf = 0; hf < G::HALVES; ++hf)
                        tma_load_4d(dst + hf * (128 * 128) + u * (kMobaChunk * 128), &tmap, hf * 64, 0, 0, page, &full1[it & 1]);
                }
                issued1 = it + 1;
            };
            issue1(0);
            if (n1 > 1) issue1(1);
            constexpr uint32_t idesc_1 = umma_idesc_bf16(128, 2 * kMobaChunk);
#pragma unroll 1
            for (int it = 0; it < n1 && ok; ++it) {
                if (it >= 2) ok = mbar_wait(&s1_free[it & 1], (uint32_t)(((it >> 1) - 1) & 1));
                ok = ok && mbar_wait(&full1[it & 1], (uint32_t)((it >> 1) & 1));
                if (!ok) break;
                landed1 = it + 1;
                tcgen05_after_sync();
                const uint32_t sa = smem_addr((it & 1) ? vst : kst);
#pragma unroll
                for (int k = 0; k < D / 16; ++k)
                    umma_bf16(tb + (uint32_t)(it & 1) * 128u, umma_desc_sw128(qa + (k >> 2) * (128 * 128) + (k & 3) * 32),
                              umma_desc_sw128(sa + (k >> 2) * (128 * 128) + (k & 3) * 32), idesc_1, k > 0);
                umma_commit(&s1_ready[it & 1]);
                if (it >= 1 && it + 1 < n1) {        // the stage of product it - 1 takes the chunks of product it + 1
                    ok = mbar_wait(&s1_ready[(it - 1) & 1], (uint32_t)(((it - 1) >> 1) & 1));
                    if (ok) issue1(it + 1);
                }
            }
            // pass 2 reuses the stages and the tensor memory: the last products are complete and their scores read
            for (int it = max(0, n1 - 2); it < n1 && ok; ++it)
                ok = mbar_wait(&s1_ready[it & 1], (uint32_t)((it >> 1) & 1)) && mbar_wait(&s1_free[it & 1], (uint32_t)((it >> 1) & 1));
            for (int k = landed1; k < issued1; ++k) mbar_wait(&full1[k & 1], (uint32_t)((k >> 1) & 1));

            // ---- pass 2: weights and output, a chunk per step
            if (ok) {
                for (int s = 0; s < NST && s < n; ++s) issue_k();
                for (int s = 0; s < NST && s < n; ++s) issue_v();
            }
            constexpr uint32_t idesc_s = umma_idesc_bf16(128, kMobaChunk);
#pragma unroll 1
            for (int hh = 0; hh < n && ok; ++hh) {
                if (hh >= 1) ok = mbar_wait(&s_free[0], (uint32_t)((hh - 1) & 1));
                ok = ok && mbar_wait(&full_k[hh % NST], (uint32_t)((hh / NST) & 1));
                if (!ok) break;
                gk_landed = hh + 1;
                tcgen05_after_sync();
                const uint32_t ka = smem_addr(kst + (size_t)(hh % NST) * G::KC_BYTES);
#pragma unroll
                for (int k = 0; k < D / 16; ++k)
                    umma_bf16(tb, umma_desc_sw128(qa + (k >> 2) * (128 * 128) + (k & 3) * 32),
                              umma_desc_sw128(ka + (k >> 2) * (kMobaChunk * 128) + (k & 3) * 32), idesc_s, k > 0);
                umma_commit(&s_ready[0]);
                if (hh >= 1) ok = product_pv(hh - 1);
                // refills: the key stage of chunk hh - 1 (its scores have been read), the value stage of chunk hh - 2 once
                // the second product of that chunk is complete
                if (ok && hh >= 1 && hh - 1 + NST < n) issue_k();
                if (ok && hh >= 2 && hh - 2 + NST < n) {
                    ok = mbar_wait(&pv_done[(hh - 2) & 1], (uint32_t)(((hh - 2) >> 1) & 1));
                    if (ok) issue_v();
                }
            }
            if (ok) ok = product_pv(n - 1);
            // after a wait that ran out: no copy may still be on its way into this CTA's shared memory when it exits
            for (int k = gk_landed; k < gk_issued; ++k) mbar_wait(&full_k[k % NST], (uint32_t)((k / NST) & 1));
            for (int k = hv_landed; k < hv_issued; ++k) mbar_wait(&full_v[k % NST], (uint32_t)((k / NST) & 1));
        }
    } else {
        // ---- the eight warps that read the accumulators: warps w and w + 4 share the 32 lanes (queries) of tensor-memory
        // subpartition w; the first takes the chunk's first 32 positions, the second the other 32
        const int lq = (warp & 3) * 32 + lane;       // this thread's query inside the CTA
        const int ch = warp >> 2;                    // which half of a chunk's positions
        const int64_t tq = t0 + lq;
        const uint32_t tl = tb + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t *mymask = qmask + lq * words;
        float m = -CUDART_INF_F, l = 0.0f, inv_l = 0.0f;
        MobaWalk wr;
        // ---- pass 1: the maximum of the scores this query attends.  A product covers two chunks; of a query's two
        // threads the first takes the first chunk, the second the other one.
        const int n1 = (n + 1) / 2;
#pragma unroll 1
        for (int it = 0; it < n1; ++it) {
            const int ca = next_chunk(wr), ja = wr.j;
            const int cb2 = 2 * it + 1 < n ? next_chunk(wr) : -1;
            const int cm = ch == 0 ? ca : cb2;       // this thread's chunk (none: -1)
            int nv = 0;
            if (cm >= 0 && tq < len) {
                const int j = ch == 0 ? ja : wr.j;
                if ((mymask[j >> 5] >> (j & 31)) & 1u) nv = (int)max((int64_t)0, min((int64_t)kMobaChunk, tq - (int64_t)cm * kMobaChunk + 1));
            }
            ok = mbar_wait(&s1_ready[it & 1], (uint32_t)((it >> 1) & 1));
            if (!__all_sync(FULLMASK, ok)) break;
            tcgen05_after_sync();
#pragma unroll 1
            for (int cb = 0; cb < kMobaChunk; cb += 32) {
                float v[32];
                tmem_ld32(tl + (uint32_t)(it & 1) * 128u + (uint32_t)(ch * kMobaChunk + cb), v);
                if (cb < nv) {
                    float tm = -CUDART_INF_F;
#pragma unroll
                    for (int i = 0; i < 32; ++i) tm = fmaxf(tm, cb + i < nv ? v[i] : -CUDART_INF_F);
                    m = fmaxf(m, tm * scale_log2);
                }
            }
            tcgen05_before_sync();
            mbar_arrive(&s1_free[it & 1]);
        }
        // the query's maximum over everything it attends: its two threads exchange theirs
        if (__all_sync(FULLMASK, ok)) {
            stat[ch][lq] = make_float2(m, 0.0f);
            mbar_arrive(&stat_ready);
            ok = mbar_wait(&stat_ready, 0u);
            if (__all_sync(FULLMASK, ok)) m = fmaxf(m, stat[ch ^ 1][lq].x);
        }
        // ---- pass 2: the same chunks one by one; of a query's two threads each takes 32 of a chunk's positions
        wr = MobaWalk();
#pragma unroll 1
        for (int hh = 0; hh < n; ++hh) {
            if (!__all_sync(FULLMASK, ok)) break;
            const int c = next_chunk(wr), j = wr.j;
            const int64_t p0 = (int64_t)c * kMobaChunk + ch * 32;    // first of this thread's 32 positions
            // positions this query attends among them: none if it did not choose the block, else those up to its own
            int nv = 0;
            if (tq < len && ((mymask[j >> 5] >> (j & 31)) & 1u)) nv = (int)max((int64_t)0, min((int64_t)32, tq - p0 + 1));
            ok = mbar_wait(&s_ready[0], (uint32_t)(hh & 1));
            if (!__all_sync(FULLMASK, ok)) break;
            tcgen05_after_sync();
            if (hh >= 2) {                           // the weights buffer hh & 1 was read by the product of chunk hh - 2
                ok = mbar_wait(&pv_done[hh & 1], (uint32_t)(((hh - 2) >> 1) & 1));
                if (!__all_sync(FULLMASK, ok)) break;
            }
            float v[32];
            tmem_ld32(tl + (uint32_t)(ch * 32), v);
            {
                // weights of 32 positions relative to the query's maximum (at most 1), rounded to bf16: 16 columns of
                // this query's lane; their sum is kept in fp32 and divides the output at the end
                uint32_t w[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float a = i < nv ? exp2_fast(fmaf(v[i], scale_log2, -m)) : 0.0f;
                    const float bq = i + 1 < nv ? exp2_fast(fmaf(v[i + 1], scale_log2, -m)) : 0.0f;
                    l += a + bq;
                    w[i >> 1] = pack2_bf16(a, bq);
                }
                tmem_st16(tl + OFF_P + (uint32_t)(hh & 1) * P_COLS + (uint32_t)(ch * 16), w);
            }
            tcgen05_before_sync();
            mbar_arrive(&s_free[0]);                 // this thread has read the scores
            if ((int64_t)c * kMobaChunk + kMobaChunk > len) {
                // the prompt ends inside this chunk: the value rows past its end hold whatever the cache's memory held;
                // a weight of zero would not stop a NaN there, so those rows are cleared once they have landed
                ok = mbar_wait(&full_v[hh % NST], (uint32_t)((hh / NST) & 1));
                if (!__all_sync(FULLMASK, ok)) break;
                const int r = tid & (kMobaChunk - 1), hf = tid >> 6;
                if (hf < G::HALVES && (int64_t)c * kMobaChunk + r >= len) {
                    uint4 *row = reinterpret_cast<uint4 *>(vst + (size_t)(hh % NST) * G::KC_BYTES + hf * (kMobaChunk * 128) + (r >> 3) * 1024 +
                                                           (r & 7) * 128);
#pragma unroll
                    for (int i = 0; i < 8; ++i) row[i] = make_uint4(0u, 0u, 0u, 0u);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // ordinary stores, read by the tensor core
            }
            tmem_st_wait();                          // the weights are in tensor memory
            tcgen05_before_sync();
            mbar_arrive(&p_ready[hh & 1]);
        }
        // the output once the last product is complete: each of a query's two threads writes half of the channels,
        // divided by the sum of the query's weights (the two threads' sums, exchanged through shared memory)
        if (__all_sync(FULLMASK, ok)) {
            stat[ch][lq] = make_float2(l, 0.0f);
            mbar_arrive(&stat_ready);
            ok = mbar_wait(&stat_ready, 1u);
        }
        if (__all_sync(FULLMASK, ok)) {
            l += stat[ch ^ 1][lq].x;
            inv_l = l > 0.0f ? 1.0f / l : 0.0f;
            ok = mbar_wait(&pv_done[(n - 1) & 1], (uint32_t)(((n - 1) >> 1) & 1));
            if (__all_sync(FULLMASK, ok)) {
                tcgen05_after_sync();
#pragma unroll 1
                for (int cb = ch * (D / 2); cb < (ch + 1) * (D / 2); cb += 32) {
                    float v[32];
                    tmem_ld32(tl + OFF_O + (uint32_t)cb, v);
                    if (tq < len) {
                        bf16 *orow = o + (((int64_t)b * len + tq) * H + h) * D + cb;
#pragma unroll
                        for (int i = 0; i < 32; i += 8)
                            *reinterpret_cast<uint4 *>(orow + i) =
                                make_uint4(pack2_bf16(v[i] * inv_l, v[i + 1] * inv_l), pack2_bf16(v[i + 2] * inv_l, v[i + 3] * inv_l),
                                           pack2_bf16(v[i + 4] * inv_l, v[i + 5] * inv_l), pack2_bf16(v[i + 6] * inv_l, v[i + 7] * inv_l));
                    }
                }
            }
        }
    }
    if (__any_sync(FULLMASK, !ok) && lane == 0) atomicCAS(status, RQ_OK, RQ_ERR_TIMEOUT);
    tcgen05_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tbase, TCOLS);
}

size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }

template <typename T, int D>
cudaError_t moba_run(const MobaArgs &a, cudaStream_t s)
{
    const int BH = a.B * a.H;
    const int nb = (int)((a.len + a.block - 1) / a.block);
    const int words = (nb + 31) / 32;
    moba_means_kernel<T><<<dim3((unsigned)nb, (unsigned)BH), D, 0, s>>>((const T *)a.kv, a.page_cap, a.S, D, a.len, a.block,
                                                                      a.means, nb);
    const bool staged = nb <= kMobaStagedBlocks;
    const int rq = staged ? kMobaRouteQ : 1;         // queries of a routing warp
    const size_t rs = (size_t)kMobaRouteWarps * rq * moba_route_floats(D, nb) * sizeof(float) + (staged ? (size_t)nb * (D + 4) * sizeof(float) : 0);
    constexpr int CHUNK_BYTES = 2 * kMobaChunk * D * (int)sizeof(T);
    const size_t as = 2 * (size_t)CHUNK_BYTES + (size_t)words * (kMobaQueries + 1) * sizeof(uint32_t);
    static bool ready[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!ready[dev]) {
        e = cudaFuncSetAttribute(moba_route_kernel<T, D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)((size_t)kMobaRouteWarps * moba_route_floats(D, kMobaMaxBlocks) * sizeof(float)));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(moba_route_kernel<T, D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)((size_t)kMobaRouteWarps * kMobaRouteQ * moba_route_floats(D, kMobaStagedBlocks) * sizeof(float) +
                                       (size_t)kMobaStagedBlocks * (D + 4) * sizeof(float)));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(moba_attend_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(2 * (size_t)CHUNK_BYTES + (size_t)(kMobaMaxBlocks / 32) * (kMobaQueries + 1) * sizeof(uint32_t)));
        if (e != cudaSuccess) return e;
        ready[dev] = true;
    }
    const dim3 rgrid((unsigned)((a.len + kMobaRouteWarps * rq - 1) / (kMobaRouteWarps * rq)), (unsigned)BH);
    if (staged)
        moba_route_kernel<T, D, true><<<rgrid, kMobaRouteWarps * 32, rs, s>>>((const T *)a.q, a.means, a.len, a.H, a.block, nb, a.K, a.sel);
    else
        moba_route_kernel<T, D, false><<<rgrid, kMobaRouteWarps * 32, rs, s>>>((const T *)a.q, a.means, a.len, a.H, a.block, nb, a.K, a.sel);
    const float sl2 = a.scale * 1.4426950408889634f;
    if constexpr (sizeof(T) == 2) {
        // bf16 caches: the attention on the tensor cores
        using G = MobaMmaGeom<D>;
        const size_t ms = (size_t)G::FIXED_BYTES + (size_t)words * (kMobaMmaQueries + 1) * sizeof(uint32_t);
        static bool mready[64];
        if (!mready[dev]) {
            e = cudaFuncSetAttribute(moba_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)((size_t)G::FIXED_BYTES + (size_t)(kMobaMaxBlocks / 32) * (kMobaMmaQueries + 1) * sizeof(uint32_t)));
            if (e != cudaSuccess) return e;
            mready[dev] = true;
        }
        alignas(64) CUtensorMap tmap;
        e = cache_tensor_map(&tmap, a.kv, D, a.S, (int64_t)BH * a.page_cap, kMobaChunk);
        if (e != cudaSuccess) return e;
        moba_mma_kernel<D><<<dim3((unsigned)BH, (unsigned)((a.len + kMobaMmaQueries - 1) / kMobaMmaQueries)), kMobaMmaThreads, ms, s>>>(
            tmap, a.page_cap, a.S, a.len, (const bf16 *)a.q, a.H, a.block, nb, a.K, a.sel, sl2, (bf16 *)a.o, a.status);
    } else {
        moba_attend_kernel<T, D><<<dim3((unsigned)((a.len + kMobaQueries - 1) / kMobaQueries), (unsigned)BH), kMobaQueries * 32, as, s>>>(
            (const T *)a.kv, a.page_cap, a.S, a.len, (const T *)a.q, a.H, a.block, nb, a.K, a.sel, sl2, (T *)a.o);
    }
    return cudaGetLastError();
}

}  // namespace

size_t moba_scratch_bytes(int BH, int64_t len, int D, int block, int K)
{
    const size_t nb = (size_t)((len + block - 1) / block);
    return round256((size_t)BH * nb * D * sizeof(float)) + round256((size_t)BH * (size_t)len * K * sizeof(int32_t));
}

void moba_carve(void *scratch, int BH, int64_t len, int D, int block, float **means, int32_t **sel)
{
    const size_t nb = (size_t)((len + block - 1) / block);
    *means = (float *)scratch;
    *sel = (int32_t *)((char *)scratch + round256((size_t)BH * nb * D * sizeof(float)));
}

cudaError_t launch_moba(const MobaArgs &a, cudaStream_t s)
{
    if (a.block < kMobaChunk || a.block % kMobaChunk != 0 || a.block % a.S != 0 || a.K < 2 || a.len < 1) return cudaErrorInvalidValue;
    if ((a.len + a.block - 1) / a.block > kMobaMaxBlocks || a.B * a.H > 65535 || (a.len + kMobaMmaQueries - 1) / kMobaMmaQueries > 65535)
        return cudaErrorInvalidValue;
    if (a.dtype == RQ_BF16) {
        if (a.D == 128) return moba_run<bf16, 128>(a, s);
        if (a.D == 64) return moba_run<bf16, 64>(a, s);
    } else {
        if (a.D == 128) return moba_run<float, 128>(a, s);
        if (a.D == 64) return moba_run<float, 64>(a, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace rq
