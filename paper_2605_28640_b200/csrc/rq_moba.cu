// MoBA-style block-sparse prefill attention on the cache of decayed keys and values (Sec. 2.2, Eq. 3
// and Eq. 4, Table 1 row MoBA; App. A.1, "Sparse inference settings", MoBA paragraph): every prompt
// position routes its query to a few of the KV blocks before it, scored with mean-pooled block
// representatives, and attends over the chosen blocks only; the first block and the query's own
// block (cut at the query's position) are always among them and count inside the budget.
//
//   moba_means_kernel    per (head, block): the mean of the block's stored keys, fp32
//   moba_route_kernel    per (head, query), one warp: scores q . mean of the complete blocks before the
//                        query's own (a lane per block), then the budget's best by repeated arg-max
//                        (equal scores to the lower block), the list written ascending
//   moba_attend_kernel   per (head, 16 consecutive queries), a warp per query: the blocks any of the 16
//                        queries chose pass through shared memory once, 64 positions at a time
//                        (cp.async, two buffers); a warp folds a chunk into its online softmax only if
//                        its own query chose the block (the arithmetic is the decode path's tile
//                        routine)
//
// This is the first correct form of the path: plain fp32 FMA work.  The attention is a dense
// contraction per (query block, KV block) and belongs on the tensor cores like the SnapKV passes; the
// routing on the query side makes that a larger kernel than this one.
#include <limits.h>
#include <math_constants.h>

#include "rq_async.cuh"
#include "rq_device.cuh"
#include "rq_internal.h"
#include "rq_stream.cuh"

namespace rq {

namespace {

constexpr int kMobaChunk = 64;                 // positions that pass through shared memory at a time
constexpr int kMobaQueries = 16;               // queries (warps) of one attention CTA
constexpr int kMobaRouteWarps = 8;             // queries (warps) of one routing CTA
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
    for (int64_t p = lo; p < hi; ++p) s += load1<T>(kv + ((((int64_t)bh * page_cap + p / S) * 2) * S + p % S) * D + c);
    means[((int64_t)bh * nb + j) * D + c] = s / (float)(hi - lo);
}

// ---------------------------------------------------------------- routing
// Grid (ceil(T / 8), heads); a warp per query.  Shared memory per warp: the query (D floats), the
// scores of the candidate blocks (nb floats), the chosen blocks as a bit mask (nb / 32 words).
// q: [B][T][H][D].  sel: [BH][T][K], ascending, -1 beyond the chosen blocks.
template <typename T, int D>
__global__ void __launch_bounds__(kMobaRouteWarps * 32) moba_route_kernel(const T *q, const float *means, int64_t len, int H,
                                                                         int block, int nb, int K, int32_t *sel)
{
    extern __shared__ __align__(16) float rsm[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int words = (nb + 31) / 32;
    float *qs = rsm + (size_t)warp * moba_route_floats(D, nb);
    float *sc = qs + D;
    uint32_t *mask = reinterpret_cast<uint32_t *>(sc + nb);
    const int64_t t = (int64_t)blockIdx.x * kMobaRouteWarps + warp;
    if (t >= len) return;                              // (no CTA-wide barrier below)
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    int32_t *out = sel + ((int64_t)bh * len + t) * K;
    const int bt = (int)(t / block), P = bt + 1;       // the query's own block; blocks it may attend
    if (K >= P) {                                      // everything before the query
        for (int i = lane; i < K; i += 32) out[i] = i < P ? i : -1;
        return;
    }
    // the first block and the own block inside the budget (K >= 2), as the first and the newest page of a decode step
    const int ns = min(1, K), nl = min(1, K - ns), want = K - ns - nl;
    const int c_lo = ns, c_hi = P - nl;                // candidates: blocks c_lo .. c_hi - 1 (all complete)
    for (int i = lane; i < D; i += 32) qs[i] = load1<T>(q + (((int64_t)b * len + t) * H + h) * D + i);
    for (int i = lane; i < words; i += 32) mask[i] = 0u;
    __syncwarp();
    // scores: a lane per block, the block's representative read as 16-byte pieces
    const float *mh = means + (int64_t)bh * nb * D;
    for (int j0 = c_lo; j0 < c_hi; j0 += 32) {
        const int j = j0 + lane;
        if (j < c_hi) {
            const float4 *row = reinterpret_cast<const float4 *>(mh + (int64_t)j * D);
            float s = 0.0f;
#pragma unroll 8
            for (int i = 0; i < D / 4; ++i) {
                const float4 m4 = __ldg(row + i);
                const float4 q4 = *reinterpret_cast<const float4 *>(qs + 4 * i);
                s = fmaf(q4.x, m4.x, s);
                s = fmaf(q4.y, m4.y, s);
                s = fmaf(q4.z, m4.z, s);
                s = fmaf(q4.w, m4.w, s);
            }
            sc[j] = s;
        }
    }
    __syncwarp();
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
    if (lane == 0) {
        for (int j = 0; j < ns; ++j) mask[j >> 5] |= 1u << (j & 31);
        for (int j = P - nl; j < P; ++j) mask[j >> 5] |= 1u << (j & 31);
    }
    __syncwarp();
    // ascending list from the mask
    int base = 0;
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

size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }

template <typename T, int D>
cudaError_t moba_run(const MobaArgs &a, cudaStream_t s)
{
    const int BH = a.B * a.H;
    const int nb = (int)((a.len + a.block - 1) / a.block);
    const int words = (nb + 31) / 32;
    moba_means_kernel<T><<<dim3((unsigned)nb, (unsigned)BH), D, 0, s>>>((const T *)a.kv, a.page_cap, a.S, D, a.len, a.block,
                                                                      a.means, nb);
    const size_t rs = (size_t)kMobaRouteWarps * moba_route_floats(D, nb) * sizeof(float);
    constexpr int CHUNK_BYTES = 2 * kMobaChunk * D * (int)sizeof(T);
    const size_t as = 2 * (size_t)CHUNK_BYTES + (size_t)words * (kMobaQueries + 1) * sizeof(uint32_t);
    static bool ready[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!ready[dev]) {
        e = cudaFuncSetAttribute(moba_route_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)((size_t)kMobaRouteWarps * moba_route_floats(D, kMobaMaxBlocks) * sizeof(float)));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(moba_attend_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(2 * (size_t)CHUNK_BYTES + (size_t)(kMobaMaxBlocks / 32) * (kMobaQueries + 1) * sizeof(uint32_t)));
        if (e != cudaSuccess) return e;
        ready[dev] = true;
    }
    moba_route_kernel<T, D><<<dim3((unsigned)((a.len + kMobaRouteWarps - 1) / kMobaRouteWarps), (unsigned)BH), kMobaRouteWarps * 32, rs,
                              s>>>((const T *)a.q, a.means, a.len, a.H, a.block, nb, a.K, a.sel);
    const float sl2 = a.scale * 1.4426950408889634f;
    moba_attend_kernel<T, D><<<dim3((unsigned)((a.len + kMobaQueries - 1) / kMobaQueries), (unsigned)BH), kMobaQueries * 32, as, s>>>(
        (const T *)a.kv, a.page_cap, a.S, a.len, (const T *)a.q, a.H, a.block, nb, a.K, a.sel, sl2, (T *)a.o);
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
    if ((a.len + a.block - 1) / a.block > kMobaMaxBlocks || a.B * a.H > 65535) return cudaErrorInvalidValue;
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
