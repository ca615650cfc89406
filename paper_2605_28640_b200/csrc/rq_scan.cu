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
// Inside a CTA time is cut into tiles of 256 positions that move through a
// ring of shared-memory stages filled by asynchronous copies (several tiles
// ahead of the arithmetic).  The kernel is bound by instruction issue, not by
// memory, so the layout is chosen for few instructions per element: a lane
// owns two neighbouring channels (one 4-byte access for a bf16 pair) and a
// half-warp owns a run of 8 consecutive positions of the tile.  A run of tokens acts on the
// incoming state as the affine map s -> A s + B with A = prod g and B = the
// run's own state from zero, and maps compose as (A2,B2)o(A1,B1) = (A2 A1,
// A2 B1 + B2).  Per tile: every thread reduces its run to a map (pass 1) and
// the two runs of a warp are composed by shuffles; after a barrier the 16
// warp maps of every channel are scanned by 16 lanes (warp w takes channels
// 2w and 2w+1), which gives the state entering every warp and the state
// entering the next tile; after a barrier every thread applies the recurrence
// token by token, rounds to the storage type, writes the rounded rows back
// into the stage and tracks min/max of the rounded keys (pass 2); then every
// warp sends its own rows out to the cache in 16-byte pieces.  Tiles that lie
// wholly inside the new tokens take a path without per-row range checks.  The
// order of all floating-point operations is fixed, so the result is the same
// bits on every run.
#include "rq_async.cuh"
#include "rq_device.cuh"
#include "rq_internal.h"

namespace rq {

namespace {


constexpr int NT = kScanThreads;
constexpr int NW = NT / 32;
constexpr int CG = kScanChannels;               // channels of one CTA: two per lane of a half-warp
constexpr int RT = kScanRunTokens;              // consecutive positions of one half-warp in a tile
constexpr int TT = 2 * NW * RT;                 // positions of one tile
constexpr int kMapStride = 3 * CG + 2;          // floats between two warps' maps: an even count, and lanes that read
                                                // the same channel of 16 consecutive maps hit 16 different banks
constexpr int kInStride = 2 * CG + 2;           // likewise for the states entering the warps
constexpr int LPC = NW;                         // lanes that scan the warp maps of one channel
static_assert(CG == 32 && (NW == 16 || NW == 32), "a half-warp holds a channel group two channels per lane; the warp maps of a channel are scanned by 16 or 32 lanes");

// asynchronous copy of 16 bytes from global to shared memory
__device__ __forceinline__ void cp_async16(void *dst_smem, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// two neighbouring elements from shared memory as floats
__device__ __forceinline__ void load2(const bf16 *p, float &x, float &y)
{
    const uint32_t w = *reinterpret_cast<const uint32_t *>(p);
    x = bf16lo(w);
    y = bf16hi(w);
}
__device__ __forceinline__ void load2(const float *p, float &x, float &y)
{
    const float2 w = *reinterpret_cast<const float2 *>(p);
    x = w.x;
    y = w.y;
}
// round two floats to the storage type, store them side by side, return the stored values
__device__ __forceinline__ void store2(bf16 *p, float &x, float &y)
{
    const uint32_t w = pack_bf16(x, y);
    *reinterpret_cast<uint32_t *>(p) = w;
    x = bf16lo(w);
    y = bf16hi(w);
}
__device__ __forceinline__ void store2(float *p, float &x, float &y) { *reinterpret_cast<float2 *>(p) = make_float2(x, y); }

// Where a row's segment sits in its tile.  With 2-byte elements a segment is 64 bytes, two rows to
// a 128-byte line, and the two half-warps of a warp read rows 8 apart, which would be the same 16
// banks: rows whose bit 3 is set swap places with their neighbour, so the two rows land in
// different halves of their lines.
template <typename X> __device__ __forceinline__ int row_slot(int row)
{
    return sizeof(X) == 2 ? row ^ ((row >> 3) & 1) : row;
}

template <bool B> struct BoolTag { static constexpr bool value = B; };

// bytes of one ring stage: the k, v and g segments of a tile
template <typename T, typename G> __host__ __device__ constexpr int scan_stage_bytes()
{
    return TT * CG * (2 * (int)sizeof(T) + (int)sizeof(G));
}
// stages of the ring: as many as fit in 192 KiB, at most four
template <typename T, typename G> __host__ __device__ constexpr int scan_stages()
{
    return 192 * 1024 / scan_stage_bytes<T, G>() < 4 ? 192 * 1024 / scan_stage_bytes<T, G>() : 4;
}

// MODE 0: the scan proper.  MODE 1: the affine map of a time chunk only (no output), for the time-chunked form.
// Time chunks (chunks > 1; few heads and a long prompt, so that one CTA per channel group would leave most of the
// chip idle): CTA x works on channel group x % units and the chunk_tiles tiles of chunk x / units.  First every
// chunk but the last is reduced to its map s -> A s + B (MODE 1), a small kernel chains the maps into the state
// that enters every chunk, then every chunk runs the scan proper from its own entry state.  The inputs of all
// chunks but the last are read twice.
//   maps   [units][chunks][3][CG]   A, B of the keys, B of the values
//   entry  [units][chunks][2][CG]   state entering a chunk (chunk 0: the cache's state)
template <typename T, typename G, int D, int S, int MODE>
__global__ void __launch_bounds__(NT) scan_kernel(ScanArgs a, int64_t tile0, int ntiles, int units, int chunks, int chunk_tiles,
                                                  float *maps, const float *entry)
{
    const int unit = blockIdx.x % units, chunk = blockIdx.x / units;
    if (MODE == 1 && chunk == chunks - 1) return;           // the last chunk's map is not needed
    tile0 += (int64_t)chunk * chunk_tiles;
    ntiles = min(chunk_tiles, ntiles - chunk * chunk_tiles);
    constexpr int NST = scan_stages<T, G>();
    constexpr int STAGE = scan_stage_bytes<T, G>();
    constexpr int EPC_T = 16 / (int)sizeof(T), EPC_G = 16 / (int)sizeof(G);   // elements per 16-byte piece
    constexpr int CPR_T = CG / EPC_T, CPR_G = CG / EPC_G;                      // pieces per row segment
    constexpr int NCH_T = TT * CPR_T, NCH_G = TT * CPR_G;                      // pieces per tile
    constexpr int WPP = S / (2 * RT);                                          // warps that share a page
    constexpr unsigned FULLMASK = 0xffffffffu;
    static_assert(D % CG == 0, "a head is a whole number of channel groups");
    static_assert(S % (2 * RT) == 0 && TT % S == 0 && NW % WPP == 0, "a page is a whole number of warps inside one tile");
    static_assert(NCH_T % NT == 0 && NCH_G % NT == 0, "every thread moves the same number of pieces");
    static_assert(NST >= 2, "the ring needs two stages");

    extern __shared__ __align__(16) unsigned char dsm[];
    __shared__ __align__(8) float wmap[NW * kMapStride];    // the warps' maps of the current tile: [warp][A, Bk, Bv][channel]
    __shared__ __align__(8) float sin_[NW * kInStride];     // state entering every warp: [warp][k, v][channel]
    __shared__ float carry[2][2][CG];                       // state entering the tile (by tile parity): k, v
    __shared__ float carry_a[2][CG];                        // MODE 1: product of the gates since the chunk began
    __shared__ float mm[NW][2][CG];                         // min / max of the warps (pages wider than a warp's 16 positions)

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int hl = lane & 15, half = lane >> 4;  // channel pair of this lane; which of the warp's two runs
    const int ch2 = 2 * hl;                      // first of this lane's two channels inside the group
    constexpr int GPH = D / CG;                  // channel groups per head
    const int bh = unit / GPH, c0 = (unit % GPH) * CG;
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
                const int dst = row_slot<T>(row) * CG + cc * EPC_T;
                cp_async16(ks + dst, kp + src);
                cp_async16(vs + dst, vp + src);
            }
        }
#pragma unroll
        for (int i = 0; i < NCH_G / NT; ++i) {
            const int ch = tid + i * NT, row = ch / CPR_G, cc = ch % CPR_G;
            if (row >= lo && row < hi)
                cp_async16(gs + row_slot<G>(row) * CG + cc * EPC_G, gp + (tok0 + row) * a.st + cc * EPC_G);
        }
    };

    if (tid < CG) {                              // the state the (chunk of the) sequence starts from
        if (MODE == 1) {
            carry[0][0][tid] = 0.0f;
            carry[0][1][tid] = 0.0f;
            carry_a[0][tid] = 1.0f;
        } else if (chunk == 0) {
            carry[0][0][tid] = a.state[(int64_t)bh * 2 * D + c0 + tid];
            carry[0][1][tid] = a.state[(int64_t)bh * 2 * D + D + c0 + tid];
        } else {
            const float *e = entry + ((int64_t)unit * chunks + chunk) * 2 * CG;
            carry[0][0][tid] = e[tid];
            carry[0][1][tid] = e[CG + tid];
        }
    }
#pragma unroll 1
    for (int s = 0; s < NST - 1; ++s) {
        if (s < ntiles) issue(s, s);
        cp_async_commit();
    }

    T *kv = static_cast<T *>(a.kv);
    T *meta = static_cast<T *>(a.meta);
    float amax = 0.0f;                           // largest |stored key| this thread has written

    // one tile; FULL: every row of the tile is a new token, so no row needs a range check
    auto tile = [&](auto full_tag, int i, int lo, int hi, int fill_hi) {
        constexpr bool FULL = decltype(full_tag)::value;
        const int st = i % NST;
        T *ks = stage_k(st), *vs = stage_v(st);
        const G *gs = stage_g(st);
        const int row0 = (2 * warp + half) * RT;
        const int64_t tile_start = (tile0 + i) * TT;

        // ---- pass 1: this thread's run as a map from a zero state (identity outside the new range)
        float2 g2[RT], k2[RT], v2[RT];                           // g, (1-g) k, (1-g) v of the two channels
        float2 A2 = make_float2(1.0f, 1.0f), Bk2 = make_float2(0.0f, 0.0f), Bv2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            const int e = row_slot<T>(row0 + r) * CG + ch2;
            float ga, gb, ka, kb, va, vb;
            load2(gs + row_slot<G>(row0 + r) * CG + ch2, ga, gb);
            load2(ks + e, ka, kb);
            load2(vs + e, va, vb);
            if (!FULL && !(row0 + r >= lo && row0 + r < hi)) {
                ga = 1.0f; gb = 1.0f;
                ka = 0.0f; kb = 0.0f;
                va = 0.0f; vb = 0.0f;
            }
            g2[r] = make_float2(ga, gb);
            const float2 o2 = fma2(g2[r], make_float2(-1.0f, -1.0f), make_float2(1.0f, 1.0f));   // 1 - g
            k2[r] = mul2(o2, make_float2(ka, kb));
            v2[r] = mul2(o2, make_float2(va, vb));
            A2 = mul2(A2, g2[r]);
            Bk2 = fma2(g2[r], Bk2, k2[r]);
            Bv2 = fma2(g2[r], Bv2, v2[r]);
        }
        const float A0 = A2.x, A1 = A2.y, Bk0 = Bk2.x, Bk1 = Bk2.y, Bv0 = Bv2.x, Bv1 = Bv2.y;
        // the map of the warp's first run, for the second run; the second run's lanes publish the warp's map
        const float LA0 = __shfl_sync(FULLMASK, A0, hl), LA1 = __shfl_sync(FULLMASK, A1, hl);
        const float LBk0 = __shfl_sync(FULLMASK, Bk0, hl), LBk1 = __shfl_sync(FULLMASK, Bk1, hl);
        const float LBv0 = __shfl_sync(FULLMASK, Bv0, hl), LBv1 = __shfl_sync(FULLMASK, Bv1, hl);
        if (half == 1) {
            float *wm = wmap + warp * kMapStride + ch2;
            *reinterpret_cast<float2 *>(wm) = make_float2(A0 * LA0, A1 * LA1);
            *reinterpret_cast<float2 *>(wm + CG) = make_float2(fmaf(A0, LBk0, Bk0), fmaf(A1, LBk1, Bk1));
            *reinterpret_cast<float2 *>(wm + 2 * CG) = make_float2(fmaf(A0, LBv0, Bv0), fmaf(A1, LBv1, Bv1));
        }
        __syncthreads();

        // ---- scan of the 16 warp maps of channels 2 warp and 2 warp + 1 (one per half-warp) by 16 lanes
        {
            const int ci = warp * (32 / LPC) + lane / LPC, m = lane % LPC;   // channel inside the group, map (= warp) index
            const float *wm = wmap + m * kMapStride + ci;
            float sa = wm[0], sbk = wm[CG], sbv = wm[2 * CG];
#pragma unroll
            for (int off = 1; off < LPC; off <<= 1) {
                const float pa = __shfl_up_sync(FULLMASK, sa, off, LPC);
                const float pbk = __shfl_up_sync(FULLMASK, sbk, off, LPC);
                const float pbv = __shfl_up_sync(FULLMASK, sbv, off, LPC);
                if (m >= off) {
                    sbk = fmaf(sa, pbk, sbk);
                    sbv = fmaf(sa, pbv, sbv);
                    sa *= pa;
                }
            }
            float ea = __shfl_up_sync(FULLMASK, sa, 1, LPC);  // maps of the warps before this one
            float ebk = __shfl_up_sync(FULLMASK, sbk, 1, LPC);
            float ebv = __shfl_up_sync(FULLMASK, sbv, 1, LPC);
            if (m == 0) { ea = 1.0f; ebk = 0.0f; ebv = 0.0f; }
            const float ck = carry[i & 1][0][ci], cv = carry[i & 1][1][ci];
            sin_[m * kInStride + ci] = fmaf(ea, ck, ebk);
            sin_[m * kInStride + CG + ci] = fmaf(ea, cv, ebv);
            if (m == LPC - 1) {                              // state entering the next tile
                carry[(i + 1) & 1][0][ci] = fmaf(sa, ck, sbk);
                carry[(i + 1) & 1][1][ci] = fmaf(sa, cv, sbv);
                if (MODE == 1) carry_a[(i + 1) & 1][ci] = sa * carry_a[i & 1][ci];
            }
        }
        if (MODE == 1) return;                               // the map needs no more of the tile (the lambda's caller goes on)
        __syncthreads();

        // ---- pass 2: token by token, rounded rows back into the stage, bounds of the rounded keys
        float sk0, sk1, sv0, sv1;
        {
            const float2 ek = *reinterpret_cast<const float2 *>(sin_ + warp * kInStride + ch2);
            const float2 ev = *reinterpret_cast<const float2 *>(sin_ + warp * kInStride + CG + ch2);
            sk0 = ek.x; sk1 = ek.y; sv0 = ev.x; sv1 = ev.y;
            if (half == 1) {                                 // through the warp's first run
                sk0 = fmaf(LA0, sk0, LBk0); sk1 = fmaf(LA1, sk1, LBk1);
                sv0 = fmaf(LA0, sv0, LBv0); sv1 = fmaf(LA1, sv1, LBv1);
            }
        }
        float2 sk2 = make_float2(sk0, sk1), sv2 = make_float2(sv0, sv1);
        float mn0 = INFINITY, mn1 = INFINITY, mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            const int e = row_slot<T>(row0 + r) * CG + ch2;
            if (FULL || (row0 + r >= lo && row0 + r < hi)) {
                sk2 = fma2(g2[r], sk2, k2[r]);
                sv2 = fma2(g2[r], sv2, v2[r]);
                float rk0 = sk2.x, rk1 = sk2.y, rv0 = sv2.x, rv1 = sv2.y;
                store2(ks + e, rk0, rk1);
                store2(vs + e, rv0, rv1);
                mn0 = fminf(mn0, rk0); mx0 = fmaxf(mx0, rk0);
                mn1 = fminf(mn1, rk1); mx1 = fmaxf(mx1, rk1);
            } else if (row0 + r >= hi && row0 + r < fill_hi) {   // unused slots of the last page
                float z0 = 0.0f, z1 = 0.0f;
                store2(ks + e, z0, z1);
                store2(vs + e, z0, z1);
            }
        }
        if (mn0 <= mx0) amax = fmaxf(amax, fmaxf(fmaxf(-mn0, mx0), fmaxf(-mn1, mx1)));   // this run held new tokens
        // the warp's two runs together (16 positions)
        mn0 = fminf(mn0, __shfl_xor_sync(FULLMASK, mn0, 16)); mn1 = fminf(mn1, __shfl_xor_sync(FULLMASK, mn1, 16));
        mx0 = fmaxf(mx0, __shfl_xor_sync(FULLMASK, mx0, 16)); mx1 = fmaxf(mx1, __shfl_xor_sync(FULLMASK, mx1, 16));
        if (WPP > 1 && half == 0) {
            *reinterpret_cast<float2 *>(&mm[warp][0][ch2]) = make_float2(mn0, mn1);
            *reinterpret_cast<float2 *>(&mm[warp][1][ch2]) = make_float2(mx0, mx1);
        }
        if (WPP > 1) __syncthreads();            // pages wider than a warp's rows: the bounds cross warps
        else __syncwarp();                       // the rows below were written by other lanes of this warp

        // ---- page bounds: the first warp of a page writes them (merged with what the page held before)
        if (warp % WPP == 0 && half == 0) {
            const int64_t pstart = tile_start + 2 * warp * RT;   // a multiple of S
            if (pstart < end && pstart + S > a.len0) {
                if (WPP > 1) {
#pragma unroll
                    for (int w = 1; w < WPP; ++w) {
                        const float2 lo2 = *reinterpret_cast<const float2 *>(&mm[warp + w][0][ch2]);
                        const float2 hi2 = *reinterpret_cast<const float2 *>(&mm[warp + w][1][ch2]);
                        mn0 = fminf(mn0, lo2.x); mn1 = fminf(mn1, lo2.y);
                        mx0 = fmaxf(mx0, hi2.x); mx1 = fmaxf(mx1, hi2.y);
                    }
                }
                T *mrow = meta + (((int64_t)bh * a.page_cap + pstart / S) * 2) * D + c0 + ch2;
                if (pstart < a.len0) {
                    float o0, o1;
                    load2(mrow, o0, o1);
                    mn0 = fminf(mn0, o0); mn1 = fminf(mn1, o1);
                    load2(mrow + D, o0, o1);
                    mx0 = fmaxf(mx0, o0); mx1 = fmaxf(mx1, o1);
                }
                store2(mrow, mn0, mn1);
                store2(mrow + D, mx0, mx1);
            }
        }

        // ---- the warp's own rows go out to their pages (no other warp touches them: no CTA barrier)
        constexpr int WROWS = 2 * RT;            // rows of a warp
        static_assert((WROWS * CPR_T) % 32 == 0, "every lane moves the same number of pieces");
#pragma unroll
        for (int j = 0; j < WROWS * CPR_T / 32; ++j) {
            const int ch = lane + j * 32, row = warp * WROWS + ch / CPR_T, cc = ch % CPR_T;
            const int64_t pos = tile_start + row;
            if (FULL || (row >= lo && row < fill_hi)) {
                const int64_t page = pos / S;
                const int slot = (int)(pos % S);
                T *dst = kv + ((((int64_t)bh * a.page_cap + page) * 2) * S + slot) * D + c0 + cc * EPC_T;
                const int src = row_slot<T>(row) * CG + cc * EPC_T;
                __stcs(reinterpret_cast<uint4 *>(dst), *reinterpret_cast<const uint4 *>(ks + src));
                __stcs(reinterpret_cast<uint4 *>(dst + (int64_t)S * D), *reinterpret_cast<const uint4 *>(vs + src));
            }
        }
    };

#pragma unroll 1
    for (int i = 0; i < ntiles; ++i) {
        cp_async_wait<NST - 2>();                // this thread's pieces of tile i have landed ...
        __syncthreads();                         // ... and everybody else's; every warp has sent its rows of tile i - 1
        if (i + NST - 1 < ntiles) issue(i + NST - 1, (i + NST - 1) % NST);
        cp_async_commit();
        // rows of the tile that hold new tokens: [lo, hi); rows up to fill_hi pad the last page
        const int64_t tile_start = (tile0 + i) * TT;
        const int lo = (int)max((int64_t)0, a.len0 - tile_start), hi = (int)min((int64_t)TT, end - tile_start);
        const int fill_hi = (int)min((int64_t)TT, tail_end - tile_start);
        if (lo == 0 && hi == TT) tile(BoolTag<true>(), i, lo, hi, fill_hi);
        else tile(BoolTag<false>(), i, lo, hi, fill_hi);
    }
    cp_async_wait<0>();
    __syncthreads();
    if (MODE == 1) {
        if (tid < CG) {                          // the chunk's map
            float *mp = maps + ((int64_t)unit * chunks + chunk) * 3 * CG;
            mp[tid] = carry_a[ntiles & 1][tid];
            mp[CG + tid] = carry[ntiles & 1][0][tid];
            mp[2 * CG + tid] = carry[ntiles & 1][1][tid];
        }
        return;
    }
    if (tid < CG && chunk == chunks - 1) {       // the state after the last token
        a.state[(int64_t)bh * 2 * D + c0 + tid] = carry[ntiles & 1][0][tid];
        a.state[(int64_t)bh * 2 * D + D + c0 + tid] = carry[ntiles & 1][1][tid];
    }
    if (a.absmax) {
        // the head's largest |stored key| (both copies): non-negative floats order like their bit patterns
        const unsigned m = __reduce_max_sync(FULLMASK, __float_as_uint(amax));
        if (lane == 0 && m != 0u) {
            atomicMax(reinterpret_cast<unsigned *>(a.absmax) + bh, m);
            atomicMax(reinterpret_cast<unsigned *>(a.absmax) + (int64_t)a.B * a.H + bh, m);
        }
    }
}

// The state entering every chunk from the chunks' maps, in order.  Grid: channel groups; a thread per (k or v, channel).
__global__ void scan_chain_kernel(const float *state, int D, int gph, int chunks, const float *maps, float *entry)
{
    const int unit = blockIdx.x, kv = threadIdx.x / CG, ch = threadIdx.x % CG;
    const int bh = unit / gph, c0 = (unit % gph) * CG;
    float s = state[(int64_t)bh * 2 * D + kv * D + c0 + ch];
    for (int c = 0; c + 1 < chunks; ++c) {
        const float *mp = maps + ((int64_t)unit * chunks + c) * 3 * CG;
        s = fmaf(mp[ch], s, mp[(1 + kv) * CG + ch]);
        entry[(((int64_t)unit * chunks + c + 1) * 2 + kv) * CG + ch] = s;
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
        e = cudaFuncSetAttribute(scan_kernel<T, G, D, S, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, DSM);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(scan_kernel<T, G, D, S, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, DSM);
        if (e != cudaSuccess) return e;
        ready[dev] = true;
    }
    // Time chunks: only where one CTA per channel group would fill less than half of the SMs and the prompt is long
    // enough for chunks of at least 16 tiles; as many chunks as give every SM a CTA, within the scratch.
    const int ntiles = (int)(t1 - t0), units = (int)ctas, sms = sm_count();
    int chunks = 1;
    if (a.chunk_scratch && 2 * units <= sms && ntiles >= 32) {
        chunks = sms / units;
        if (chunks > ntiles / 16) chunks = ntiles / 16;
        while (chunks > 1 && (size_t)units * chunks * 5 * CG * sizeof(float) > kScanScratchBytes) --chunks;
    }
    int chunk_tiles = (ntiles + chunks - 1) / chunks;
    chunks = (ntiles + chunk_tiles - 1) / chunk_tiles;
    float *maps = a.chunk_scratch, *entry = a.chunk_scratch ? a.chunk_scratch + (size_t)units * chunks * 3 * CG : nullptr;
    if (chunks > 1) {
        scan_kernel<T, G, D, S, 1><<<(unsigned)(units * chunks), NT, DSM, s>>>(a, t0, ntiles, units, chunks, chunk_tiles, maps, entry);
        scan_chain_kernel<<<(unsigned)units, 2 * CG, 0, s>>>(a.state, D, D / CG, chunks, maps, entry);
    }
    scan_kernel<T, G, D, S, 0><<<(unsigned)(units * chunks), NT, DSM, s>>>(a, t0, ntiles, units, chunks, chunk_tiles, maps, entry);
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
