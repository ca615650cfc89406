// Prefill: the gated decay recurrence (Eq. 1) over a whole sequence, fused with
// the paged cache write and the per-page min/max of the stored keys
// (Appendix A.1, "Sparse inference settings").  One launch, every input byte
// read once, every output byte written once, no scratch in global memory.
//
// The recurrence x~_t = g_t x~_{t-1} + (1-g_t) x_t runs along time and is
// independent per (batch, head, channel).  Work decomposition: one CTA owns
// one (batch, head) pair and 32 neighbouring channels (a lane per channel) and
// walks the whole sequence, so the state never leaves the CTA: there is no
// look-back between CTAs, no flag and no wait.  Measured on B200, 128 CTAs that
// each stream 64-byte row segments 8 KiB apart reach the same bandwidth as a
// plain copy, so nothing is lost by giving a CTA a quarter of a head's row.
//
// Inside a CTA time is cut into tiles of 128 positions that move through a
// ring of shared-memory stages filled by asynchronous copies (several tiles
// ahead of the arithmetic).  A warp owns 16 consecutive positions of the tile.
// A run of tokens acts on the incoming state as the affine map s -> A s + B
// with A = prod g and B = the run's own state from zero, and maps compose as
// (A2,B2)o(A1,B1) = (A2 A1, A2 B1 + B2).  Per tile: every thread reduces its
// run to a map (pass 1); after a barrier it composes the maps of the warps
// before it onto the state that entered the tile, and the last warp leaves the
// state for the next tile; then it applies the recurrence token by token,
// rounds to the storage type, writes the rounded rows back into the stage and
// tracks min/max of the rounded keys (pass 2); after a barrier the stage goes
// out to the cache in 16-byte pieces.  The order of all floating-point
// operations is fixed, so the result is the same bits on every run.
#include "rq_async.cuh"
#include "rq_device.cuh"
#include "rq_internal.h"

namespace rq {

namespace {

constexpr int NT = kScanThreads;
constexpr int NW = NT / 32;
constexpr int CG = kScanChannels;               // channels of one CTA: a lane per channel
constexpr int RT = kScanRunTokens;              // consecutive positions of one warp in a tile
constexpr int TT = NW * RT;                     // positions of one tile

// asynchronous copy of 16 bytes from global to shared memory
__device__ __forceinline__ void cp_async16(void *dst_smem, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ float elem_to_float(bf16 x) { return __bfloat162float(x); }
__device__ __forceinline__ float elem_to_float(float x) { return x; }
template <typename T> __device__ __forceinline__ T float_to_elem(float x);
template <> __device__ __forceinline__ bf16 float_to_elem<bf16>(float x) { return __float2bfloat16_rn(x); }
template <> __device__ __forceinline__ float float_to_elem<float>(float x) { return x; }

// bytes of one ring stage: the k, v and g segments of a tile
template <typename T, typename G> __host__ __device__ constexpr int scan_stage_bytes() { return TT * CG * (2 * (int)sizeof(T) + (int)sizeof(G)); }
// stages of the ring: as many as fit in 192 KiB, at most six
template <typename T, typename G> __host__ __device__ constexpr int scan_stages()
{
    return 192 * 1024 / scan_stage_bytes<T, G>() < 6 ? 192 * 1024 / scan_stage_bytes<T, G>() : 6;
}

template <typename T, typename G, int D, int S>
__global__ void __launch_bounds__(NT) scan_kernel(ScanArgs a, int64_t tile0, int ntiles)
{
    constexpr int NST = scan_stages<T, G>();
    constexpr int STAGE = scan_stage_bytes<T, G>();
    constexpr int EPC_T = 16 / (int)sizeof(T), EPC_G = 16 / (int)sizeof(G);   // elements per 16-byte piece
    constexpr int CPR_T = CG / EPC_T, CPR_G = CG / EPC_G;                      // pieces per row segment
    constexpr int NCH_T = TT * CPR_T, NCH_G = TT * CPR_G;                      // pieces per tile
    constexpr int WPP = S / RT;                                                // warps that share a page
    static_assert(D % CG == 0, "a head is a whole number of channel groups");
    static_assert(S % RT == 0 && TT % S == 0 && NW % WPP == 0, "a page is a whole number of warp runs inside one tile");
    static_assert(NCH_T % NT == 0 && NCH_G % NT == 0, "every thread moves the same number of pieces");
    static_assert(NST >= 2, "the ring needs two stages");

    extern __shared__ __align__(16) unsigned char dsm[];
    __shared__ float wmap[NW][3][CG];            // the warps' maps of the current tile
    __shared__ float carry[2][2][CG];            // state entering the tile (by tile parity): k, v
    __shared__ float mm[NW][2][CG];              // min / max of the warps' runs (pages wider than a run)

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int GPH = D / CG;                  // channel groups per head
    const int bh = blockIdx.x / GPH, c0 = (blockIdx.x % GPH) * CG;
    const int b = bh / a.H, h = bh % a.H;
    const int64_t end = a.len0 + a.T;
    const int64_t tail_end = (end + S - 1) / S * S;   // end of the last touched page
    const int64_t in_base = (int64_t)b * a.sb + (int64_t)h * a.sh + c0;
    const T *kp = static_cast<const T *>(a.k) + in_base;
    const T *vp = static_cast<const T *>(a.v) + in_base;
    const G *gp = static_cast<const G *>(a.g) + in_base;

    auto stage_k = [&](int st) { return reinterpret_cast<T *>(dsm + (size_t)st * STAGE); };
    auto stage_v = [&](int st) { return reinterpret_cast<T *>(dsm + (size_t)st * STAGE) + TT * CG; };
    auto stage_g = [&](int st) { return reinterpret_cast<G *>(dsm + (size_t)st * STAGE + 2 * TT * CG * sizeof(T)); };

    // start the copies of tile `rel` (positions outside the new range are left alone)
    auto issue = [&](int rel, int st) {
        const int64_t tile_start = (tile0 + rel) * TT;
        const int lo = (int)max((int64_t)0, a.len0 - tile_start), hi = (int)min((int64_t)TT, end - tile_start);
        const int64_t tok0 = tile_start - a.len0;        // input token of row 0
        T *ks = stage_k(st), *vs = stage_v(st);
        G *gs = stage_g(st);
#pragma unroll
        for (int i = 0; i < NCH_T / NT; ++i) {
            const int ch = tid + i * NT, row = ch / CPR_T, cc = ch % CPR_T;
            if (row >= lo && row < hi) {
                const int64_t src = (tok0 + row) * a.st + cc * EPC_T;
                cp_async16(ks + ch * EPC_T, kp + src);
                cp_async16(vs + ch * EPC_T, vp + src);
            }
        }
#pragma unroll
        for (int i = 0; i < NCH_G / NT; ++i) {
            const int ch = tid + i * NT, row = ch / CPR_G, cc = ch % CPR_G;
            if (row >= lo && row < hi) cp_async16(gs + ch * EPC_G, gp + (tok0 + row) * a.st + cc * EPC_G);
        }
    };

    if (tid < CG) {                              // the state the sequence starts from
        carry[0][0][tid] = a.state[(int64_t)bh * 2 * D + c0 + tid];
        carry[0][1][tid] = a.state[(int64_t)bh * 2 * D + D + c0 + tid];
    }
#pragma unroll 1
    for (int s = 0; s < NST - 1; ++s) {
        if (s < ntiles) issue(s, s);
        cp_async_commit();
    }

    T *kv = static_cast<T *>(a.kv);
    T *meta = static_cast<T *>(a.meta);

#pragma unroll 1
    for (int i = 0; i < ntiles; ++i) {
        const int st = i % NST;
        cp_async_wait<NST - 2>();                // this thread's pieces of tile i have landed ...
        __syncthreads();                         // ... and everybody else's; the stage of tile i - 1 has gone out
        if (i + NST - 1 < ntiles) issue(i + NST - 1, (i + NST - 1) % NST);
        cp_async_commit();

        T *ks = stage_k(st), *vs = stage_v(st);
        const G *gs = stage_g(st);
        const int row0 = warp * RT;
        const int64_t tile_start = (tile0 + i) * TT;
        const int64_t pos0 = tile_start + row0;
        // rows of the tile that hold new tokens: [lo, hi); rows up to fill_hi pad the last page
        const int lo = (int)max((int64_t)0, a.len0 - tile_start), hi = (int)min((int64_t)TT, end - tile_start);
        const int fill_hi = (int)min((int64_t)TT, tail_end - tile_start);

        // ---- pass 1: this thread's run as a map from a zero state (identity outside the new range)
        float gg[RT], kk[RT], vv[RT];            // g, (1-g) k, (1-g) v
        float A = 1.0f, Bk = 0.0f, Bv = 0.0f;
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            const bool valid = row0 + r >= lo && row0 + r < hi;
            const int e = (row0 + r) * CG + lane;
            const float g = valid ? elem_to_float(gs[e]) : 1.0f;
            const float om = 1.0f - g;
            gg[r] = g;
            kk[r] = valid ? om * elem_to_float(ks[e]) : 0.0f;
            vv[r] = valid ? om * elem_to_float(vs[e]) : 0.0f;
            A *= g;
            Bk = fmaf(g, Bk, kk[r]);
            Bv = fmaf(g, Bv, vv[r]);
        }
        wmap[warp][0][lane] = A;
        wmap[warp][1][lane] = Bk;
        wmap[warp][2][lane] = Bv;
        __syncthreads();

        // ---- state entering this run: the tile's incoming state through the maps of the warps before
        float sk = carry[i & 1][0][lane], sv = carry[i & 1][1][lane];
        {
            float wa[NW - 1], wk[NW - 1], wv[NW - 1];   // all loads first: only the multiply-adds form a chain
#pragma unroll
            for (int w = 0; w < NW - 1; ++w) {
                wa[w] = wmap[w][0][lane];
                wk[w] = wmap[w][1][lane];
                wv[w] = wmap[w][2][lane];
            }
#pragma unroll
            for (int w = 0; w < NW - 1; ++w) {
                if (w < warp) {
                    sk = fmaf(wa[w], sk, wk[w]);
                    sv = fmaf(wa[w], sv, wv[w]);
                }
            }
        }
        if (warp == NW - 1) {                    // state entering the next tile
            carry[(i + 1) & 1][0][lane] = fmaf(A, sk, Bk);
            carry[(i + 1) & 1][1][lane] = fmaf(A, sv, Bv);
        }

        // ---- pass 2: token by token, rounded rows back into the stage, bounds of the rounded keys
        float mn = INFINITY, mx = -INFINITY;
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            const int e = (row0 + r) * CG + lane;
            if (row0 + r >= lo && row0 + r < hi) {
                sk = fmaf(gg[r], sk, kk[r]);
                sv = fmaf(gg[r], sv, vv[r]);
                const T rk = float_to_elem<T>(sk);
                ks[e] = rk;
                vs[e] = float_to_elem<T>(sv);
                const float f = elem_to_float(rk);
                mn = fminf(mn, f);
                mx = fmaxf(mx, f);
            } else if (row0 + r >= hi && row0 + r < fill_hi) {   // unused slots of the last page
                ks[e] = float_to_elem<T>(0.0f);
                vs[e] = float_to_elem<T>(0.0f);
            }
        }
        if (WPP > 1) {
            mm[warp][0][lane] = mn;
            mm[warp][1][lane] = mx;
        }
        __syncthreads();

        // ---- page bounds: the first warp of a page writes them (merged with what the page held before)
        if (warp % WPP == 0) {
            const int64_t pstart = pos0;         // a multiple of S
            if (pstart < end && pstart + S > a.len0) {
                if (WPP > 1) {
#pragma unroll
                    for (int w = 1; w < WPP; ++w) {
                        mn = fminf(mn, mm[warp + w][0][lane]);
                        mx = fmaxf(mx, mm[warp + w][1][lane]);
                    }
                }
                T *m = meta + (((int64_t)bh * a.page_cap + pstart / S) * 2) * D + c0 + lane;
                if (pstart < a.len0) {
                    mn = fminf(mn, elem_to_float(m[0]));
                    mx = fmaxf(mx, elem_to_float(m[D]));
                }
                m[0] = float_to_elem<T>(mn);
                m[D] = float_to_elem<T>(mx);
            }
        }

        // ---- the stage's rows go out to their pages
#pragma unroll
        for (int j = 0; j < NCH_T / NT; ++j) {
            const int ch = tid + j * NT, row = ch / CPR_T, cc = ch % CPR_T;
            const int64_t pos = tile_start + row;
            if (row >= lo && row < fill_hi) {
                const int64_t page = pos / S;
                const int slot = (int)(pos % S);
                T *dst = kv + ((((int64_t)bh * a.page_cap + page) * 2) * S + slot) * D + c0 + cc * EPC_T;
                __stcs(reinterpret_cast<uint4 *>(dst), *reinterpret_cast<const uint4 *>(ks + ch * EPC_T));
                __stcs(reinterpret_cast<uint4 *>(dst + (int64_t)S * D), *reinterpret_cast<const uint4 *>(vs + ch * EPC_T));
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();
    if (tid < CG) {                              // the state after the last token
        a.state[(int64_t)bh * 2 * D + c0 + tid] = carry[ntiles & 1][0][tid];
        a.state[(int64_t)bh * 2 * D + D + c0 + tid] = carry[ntiles & 1][1][tid];
    }
}

template <typename T, typename G, int D, int S>
cudaError_t run(const ScanArgs &a, cudaStream_t s)
{
    const int64_t end = a.len0 + a.T;
    const int64_t t0 = a.len0 / TT;
    const int64_t t1 = (end + TT - 1) / TT;
    if (t1 <= t0) return cudaSuccess;
    if (t1 - t0 >= (int64_t)1 << 31) return cudaErrorInvalidValue;
    const int64_t ctas = (int64_t)a.B * a.H * (D / CG);
    if (ctas >= (int64_t)1 << 31) return cudaErrorInvalidValue;
    constexpr int DSM = scan_stages<T, G>() * scan_stage_bytes<T, G>();
    static bool ready[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!ready[dev]) {
        e = cudaFuncSetAttribute(scan_kernel<T, G, D, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, DSM);
        if (e != cudaSuccess) return e;
        ready[dev] = true;
    }
    scan_kernel<T, G, D, S><<<(unsigned)ctas, NT, DSM, s>>>(a, t0, (int)(t1 - t0));
    return cudaGetLastError();
}

template <typename T, typename G>
cudaError_t dispatch_shape(const ScanArgs &a, cudaStream_t s)
{
    if (a.D == 128 && a.S == 16) return run<T, G, 128, 16>(a, s);
    if (a.D == 128 && a.S == 64) return run<T, G, 128, 64>(a, s);
    if (a.D == 64 && a.S == 16) return run<T, G, 64, 16>(a, s);
    if (a.D == 64 && a.S == 64) return run<T, G, 64, 64>(a, s);
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_scan(const ScanArgs &a, cudaStream_t s)
{
    if (a.dtype == RQ_BF16) {
        return a.gate_dtype == RQ_BF16 ? dispatch_shape<bf16, bf16>(a, s) : dispatch_shape<bf16, float>(a, s);
    }
    return a.gate_dtype == RQ_BF16 ? dispatch_shape<float, bf16>(a, s) : dispatch_shape<float, float>(a, s);
}

}  // namespace rq
