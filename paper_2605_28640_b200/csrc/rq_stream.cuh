// Arithmetic of the two streaming kernels on ONE unit of data that already sits in shared
// memory, shared by the stand-alone kernels and the one-launch decode step:
//   score_unit   — Quest upper bounds of the page records of one 8 KiB unit (Eq. 3)
//   attend_tile  — one 16-row tile of a selected page folded into a warp's online softmax (Eq. 4)
//   combine_head — merge of a head's partial results
//   update_head  — one step of Eq. 1 for one head (state, cache row, newest page's bounds)
#pragma once
#include <math_constants.h>

#include "rq_async.cuh"
#include "rq_device.cuh"
#include "rq_internal.h"

namespace rq {

constexpr int kUnitBytes = 8192;                   // page records streamed per scoring unit
constexpr int kTileRows = 16;                      // token rows per attention tile
constexpr int kDoneTileBits = 20;                  // low bits of a head's done word count tiles
constexpr int kDoneTileMask = (1 << kDoneTileBits) - 1;

// ---------------------------------------------------------------- scoring
template <typename T, int D>
struct ScoreGeom {
    static constexpr int CH = VecOf<T>::N;           // elements per 16-byte vector
    static constexpr int REC_BYTES = 2 * D * (int)sizeof(T);
    static constexpr int VPR = REC_BYTES / 16;       // 16-byte vectors per record
    static constexpr int RU = kUnitBytes / REC_BYTES;   // records per unit
    static constexpr int LPP = VPR > 32 ? 32 : VPR;  // lanes that share one record in a warp-wide read
    static constexpr int VPL = VPR / LPP;            // vectors per lane and record (1 or 2)
    static constexpr int PPW = 32 / LPP;             // records per warp-wide read
    static constexpr int NR = RU / PPW;              // record groups per unit
    static constexpr int NW = kScoreWarps;
    static constexpr int DEPTH_RAW = kScoreRingBytes / (NW * kUnitBytes);
    static constexpr int DEPTH = DEPTH_RAW < 1 ? 1 : (DEPTH_RAW > 8 ? 8 : DEPTH_RAW);
    static constexpr int RING_BYTES = NW * DEPTH * kUnitBytes;
    // ring | barriers | (head, first record, records) per stage | reduction scratch of the update
    static constexpr int SMEM_BYTES = RING_BYTES + NW * DEPTH * 8 + NW * DEPTH * 16 + 64;
    static_assert(VPL == 1 || VPL == 2, "unsupported record width");
    static_assert(D <= NW * 32, "the update uses one thread per channel");
};

// This lane's slice of head `h`'s query, split by sign: a lane that reads part of a max row
// multiplies by max(q, 0), a lane that reads part of a min row by min(q, 0).
template <typename T, int D>
__device__ __forceinline__ void score_load_q(const T *q, int h, int lane, float (*qs)[VecOf<T>::N])
{
    using G = ScoreGeom<T, D>;
    const int c = lane % G::LPP;
#pragma unroll
    for (int v = 0; v < G::VPL; ++v) {
        const int vec = c + v * G::LPP;              // vector index inside the record
        const bool is_max = vec >= G::VPR / 2;
        const int ch0 = (vec % (G::VPR / 2)) * G::CH;
#pragma unroll
        for (int i = 0; i < G::CH; ++i) {
            const float x = load1<T>(q + (int64_t)h * D + ch0 + i);
            qs[v][i] = is_max ? fmaxf(x, 0.0f) : fminf(x, 0.0f);
        }
    }
}

struct NoEmit {
    __device__ __forceinline__ void operator()(int, float) const {}
};

// Scores of the first `n` records of the unit at `ub` (shared memory) -> out[0 .. n); emit(r, score)
// is called by the lane that writes record r's score.
template <typename T, int D, typename Emit = NoEmit>
__device__ __forceinline__ void score_unit(const unsigned char *ub, const float (*qs)[VecOf<T>::N], int n,
                                           float *out, int lane, Emit emit = Emit())
{
    using G = ScoreGeom<T, D>;
    constexpr int CH = G::CH, LPP = G::LPP, VPL = G::VPL, PPW = G::PPW, NR = G::NR;
    constexpr unsigned FULL = 0xffffffffu;
    const int sub = lane / LPP, c = lane % LPP;
    float val[NR];
#pragma unroll
    for (int gi = 0; gi < NR; ++gi) {
        const unsigned char *rec = ub + (size_t)(gi * PPW + sub) * G::REC_BYTES;
        float2 s2 = make_float2(0.0f, 0.0f);               // even and odd channels summed apart, then together
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            float m[CH];
            unpack16<T>(lds16(rec + (c + v * LPP) * 16), m);
#pragma unroll
            for (int i = 0; i < CH; i += 2) s2 = fma2(make_float2(qs[v][i], qs[v][i + 1]), make_float2(m[i], m[i + 1]), s2);
        }
        val[gi] = s2.x + s2.y;
    }
    // sum over the LPP lanes of a record; while more than one value is left a step also
    // halves the values a lane carries, so the whole reduction costs about NR shuffles
    int nv = NR;
#pragma unroll
    for (int off = LPP / 2; off > 0; off >>= 1) {
        if (nv > 1) {
            const int half = nv / 2;
            const bool hi = (lane & off) != 0;
#pragma unroll
            for (int i = 0; i < NR / 2; ++i) {
                if (i < half) {
                    const float send = hi ? val[i] : val[i + half];
                    const float keep = hi ? val[i + half] : val[i];
                    val[i] = keep + __shfl_xor_sync(FULL, send, off);
                }
            }
            nv = half;
        } else {
            val[0] += __shfl_xor_sync(FULL, val[0], off);
        }
    }
    // the lane now holds the sum of record group `gi` if its low lane bits are zero
    constexpr int LOG_LPP = LPP == 32 ? 5 : (LPP == 16 ? 4 : (LPP == 8 ? 3 : 2));
    constexpr int LOG_NR = NR == 32 ? 5 : (NR == 16 ? 4 : (NR == 8 ? 3 : (NR == 4 ? 2 : (NR == 2 ? 1 : 0))));
    static_assert((1 << LOG_LPP) == LPP && (1 << LOG_NR) == NR && LOG_NR <= LOG_LPP, "unsupported reduction shape");
    const int gi = (c >> (LOG_LPP - LOG_NR)) & (NR - 1);
    const bool writer = (c & ((1 << (LOG_LPP - LOG_NR)) - 1)) == 0;
    const int r = gi * PPW + sub;
    if (writer && r < n) {
        out[r] = val[0];
        emit(r, val[0]);
    }
}

// ---------------------------------------------------------------- attention
template <typename T, int D, int S>
struct AttendGeom {
    static constexpr int CH = VecOf<T>::N;         // elements per 16-byte vector
    static constexpr int LPR = D / CH;             // lanes per row
    static constexpr int RPI = 32 / LPR;           // rows per warp-wide read
    static constexpr int TR = kTileRows;           // rows per tile
    static constexpr int TPP = S / TR;             // tiles per page
    static constexpr int NI = TR / RPI;            // warp-wide reads per tile and tensor
    static constexpr int TILE_BYTES = TR * D * (int)sizeof(T);
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    static constexpr int SH = (LPR == 32 ? 5 : LPR == 16 ? 4 : LPR == 8 ? 3 : 2) - (NI == 16 ? 4 : NI == 8 ? 3 : NI == 4 ? 2 : 1);   // log2(LPR / NI)
    static_assert(SH >= 0 && (NI << SH) == LPR, "a row's score must end up in at least one lane");
    static constexpr int NW = kAttendWarps;
    static constexpr int DEPTH_RAW = kAttendRingBytes / (NW * STAGE_BYTES);
    static constexpr int DEPTH = DEPTH_RAW < 1 ? 1 : (DEPTH_RAW > 8 ? 8 : DEPTH_RAW);
    static constexpr int RING_BYTES = NW * DEPTH * STAGE_BYTES;
    // ring | barriers | (head, valid rows) per stage | per-warp m, l, tiles, head | per-warp acc
    static constexpr int SMEM_BYTES = RING_BYTES + NW * DEPTH * 8 + NW * DEPTH * 8 + 4 * NW * 4 + NW * D * 4;
    static_assert(LPR <= 32 && TR % RPI == 0 && S % TR == 0, "unsupported geometry");
    static_assert(TILE_BYTES % 16 == 0, "bulk copies move multiples of 16 bytes");
};

// Running softmax state of a warp for one head: lane -> (row group rsub = lane / LPR, channel
// group cgp = lane % LPR); acc holds the lane's CH channels summed over the rows of its group;
// l is per lane (a row's weight is added by the 2^SH lanes that hold the row's score).
template <typename T>
struct AttendState {
    float qf[VecOf<T>::N], acc[VecOf<T>::N];
    float m, l;
};

template <typename T, int D>
__device__ __forceinline__ void attend_begin_head(AttendState<T> &st, const T *q, int h, float scale_log2, int lane)
{
    constexpr int CH = VecOf<T>::N, LPR = D / CH;
    const int cgp = lane % LPR;
#pragma unroll
    for (int c = 0; c < CH; ++c) {
        st.qf[c] = load1<T>(q + (int64_t)h * D + cgp * CH + c) * scale_log2;
        st.acc[c] = 0.0f;
    }
    st.m = -CUDART_INF_F;
    st.l = 0.0f;
}

// Fold one tile (keys at ks, values at vs, both in shared memory; `valid` rows) into the state.
template <typename T, int D, int S>
__device__ __forceinline__ void attend_tile(AttendState<T> &st, const T *ks, const T *vs, int valid, int lane)
{
    using G = AttendGeom<T, D, S>;
    constexpr int CH = G::CH, LPR = G::LPR, RPI = G::RPI, NI = G::NI;
    constexpr unsigned FULL = 0xffffffffu;
    const int rsub = lane / LPR, cgp = lane % LPR;
    // K: partial dot products of NI row groups, then a reduction over the LPR lanes of a
    // row in which every step also halves the values a lane carries: afterwards a lane
    // holds the complete score of ONE row (row group cgp >> SH, shared by 2^SH lanes)
    float s[NI];
#pragma unroll
    for (int n = 0; n < NI; ++n) {
        float kf[CH];
        unpack16<T>(lds16(ks + (n * 32 + lane) * CH), kf);
        float2 d2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int c = 0; c < CH; c += 2) d2 = fma2(make_float2(st.qf[c], st.qf[c + 1]), make_float2(kf[c], kf[c + 1]), d2);
        s[n] = d2.x + d2.y;
    }
    int nv = NI;
#pragma unroll
    for (int off = LPR / 2; off > 0; off >>= 1) {
        if (nv > 1) {
            const int half = nv / 2;
            const bool hi = (lane & off) != 0;
#pragma unroll
            for (int i = 0; i < NI / 2; ++i) {
                if (i < half) {
                    const float send = hi ? s[i] : s[i + half];
                    const float keep = hi ? s[i + half] : s[i];
                    s[i] = keep + __shfl_xor_sync(FULL, send, off);
                }
            }
            nv = half;
        } else {
            s[0] += __shfl_xor_sync(FULL, s[0], off);
        }
    }
    const int row = ((cgp >> G::SH) & (NI - 1)) * RPI + rsub;
    const float sc = row < valid ? s[0] : -CUDART_INF_F;
    float m_new = fmaxf(st.m, sc);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m_new = fmaxf(m_new, __shfl_xor_sync(FULL, m_new, off));
    const float alpha = exp2f(st.m - m_new);         // 0 on the first tile (m = -inf)
    const float p_row = exp2f(sc - m_new);           // 0 for a masked row
    st.m = m_new;
    st.l = fmaf(st.l, alpha, p_row);
#pragma unroll
    for (int c = 0; c < CH; c += 2) {
        const float2 a2 = mul2(make_float2(st.acc[c], st.acc[c + 1]), make_float2(alpha, alpha));
        st.acc[c] = a2.x;
        st.acc[c + 1] = a2.y;
    }
    // V: row group n's weight comes from the lane that holds it
#pragma unroll
    for (int n = 0; n < NI; ++n) {
        const float p = __shfl_sync(FULL, p_row, rsub * LPR + (n << G::SH));
        float vf[CH];
        unpack16<T>(lds16(vs + (n * 32 + lane) * CH), vf);
#pragma unroll
        for (int c = 0; c < CH; c += 2) {
            const float2 a2 = fma2(make_float2(p, p), make_float2(vf[c], vf[c + 1]), make_float2(st.acc[c], st.acc[c + 1]));
            st.acc[c] = a2.x;
            st.acc[c + 1] = a2.y;
        }
    }
}

// Sum the warp's softmax denominators and the row groups' accumulators (all share m):
// afterwards l is the warp's total and lanes < LPR hold the channel sums.
template <typename T, int D, int S>
__device__ __forceinline__ void attend_merge_rows(AttendState<T> &st)
{
    using G = AttendGeom<T, D, S>;
    constexpr unsigned FULL = 0xffffffffu;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) st.l += __shfl_xor_sync(FULL, st.l, off);
    st.l *= 1.0f / (float)(1 << G::SH);
#pragma unroll
    for (int off = G::LPR; off < 32; off <<= 1) {
#pragma unroll
        for (int c = 0; c < G::CH; ++c) st.acc[c] += __shfl_xor_sync(FULL, st.acc[c], off);
    }
}

// Combine n partials of a head (one warp): o = sum_s 2^(m_s-M) acc_s / sum_s 2^(m_s-M) l_s.
// Lane -> (channel group g = lane % 8 of D/8 channels, subset j = lane / 8): a lane sweeps the
// partials s = j, j+4, ... with a running maximum, four records per round trip (their loads are
// all issued before the first is used); the four subsets are merged with two shuffle steps.
// A record is [m, l, -, -, acc[D]]; an empty one has m = -inf and zeros.
template <typename T, int D>
__device__ __forceinline__ void combine_head(const float *src, int n, T *o_row, int lane)
{
    constexpr int CPL = D / 8;                     // channels per lane
    constexpr int NV = CPL / 4;                    // 16-byte vectors per lane and record
    constexpr int U = 4;                           // records in flight per lane
    const int g = lane & 7, j = lane >> 3;
    float M = -CUDART_INF_F, L = 0.0f, A[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) A[c] = 0.0f;
    for (int s0 = j; s0 < n; s0 += 4 * U) {
        float2 ml[U];
        float4 v[U][NV];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int s = s0 + 4 * u;
            const float *rec = src + (int64_t)(s < n ? s : s0) * (D + 4);
            ml[u] = ld_cg_now(reinterpret_cast<const float2 *>(rec));
            if (s >= n) ml[u].x = -CUDART_INF_F;
#pragma unroll
            for (int c = 0; c < NV; ++c) v[u][c] = ld_cg_now(reinterpret_cast<const float4 *>(rec + 4 + g * CPL) + c);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            // branch-free; an empty partial or a record past the end gets weight 0
            const float Mn = fmaxf(M, ml[u].x);
            const float fo = M == -CUDART_INF_F ? 0.0f : exp2f(M - Mn);
            const float fn = ml[u].x == -CUDART_INF_F ? 0.0f : exp2f(ml[u].x - Mn);
            L = fmaf(L, fo, ml[u].y * fn);
#pragma unroll
            for (int c = 0; c < NV; ++c) {
                A[4 * c + 0] = fmaf(A[4 * c + 0], fo, v[u][c].x * fn);
                A[4 * c + 1] = fmaf(A[4 * c + 1], fo, v[u][c].y * fn);
                A[4 * c + 2] = fmaf(A[4 * c + 2], fo, v[u][c].z * fn);
                A[4 * c + 3] = fmaf(A[4 * c + 3], fo, v[u][c].w * fn);
            }
            M = Mn;
        }
    }
#pragma unroll
    for (int off = 8; off < 32; off <<= 1) {
        const float Mo = __shfl_xor_sync(0xffffffffu, M, off);
        const float Lo = __shfl_xor_sync(0xffffffffu, L, off);
        const float Mn = fmaxf(M, Mo);
        const float fa = M == -CUDART_INF_F ? 0.0f : exp2f(M - Mn), fb = Mo == -CUDART_INF_F ? 0.0f : exp2f(Mo - Mn);
        L = L * fa + Lo * fb;
#pragma unroll
        for (int c = 0; c < CPL; ++c) A[c] = A[c] * fa + __shfl_xor_sync(0xffffffffu, A[c], off) * fb;
        M = Mn;
    }
    if (j == 0) {
        const float inv = 1.0f / L;
#pragma unroll
        for (int c = 0; c < CPL; ++c) store1<T>(o_row + g * CPL + c, A[c] * inv);
    }
}

// ---------------------------------------------------------------- append
// One step of Eq. 1 for head h (thread d < D owns channel d): new state, cache row, bounds of
// the newest page, and that page's score (returned to thread 0).  `len` is the length AFTER the
// append.  red: 16 floats of shared memory.  The head's largest |stored key| is brought up to date
// in the copy that the NEXT step reads (the copy of this step is being read by the scoring warps).
template <typename T, int D>
__device__ __forceinline__ float update_head(const DecodeArgs &a, int h, const T *q, const T *k_t, const T *v_t,
                                             const void *g_t, float *scores, float *red)
{
    const int d = threadIdx.x;
    const int S = a.S;
    const int64_t pos = a.len - 1;
    const int64_t page = pos / S;
    const int slot = (int)(pos % S);
    float term = 0.0f, amax = 0.0f;
    if (d < D) {
        float *st = a.state + (int64_t)h * 2 * D;
        const float g = a.gate_dtype == RQ_BF16 ? load1<bf16>(static_cast<const bf16 *>(g_t) + (int64_t)h * D + d)
                                                : load1<float>(static_cast<const float *>(g_t) + (int64_t)h * D + d);
        const float om = 1.0f - g;
        const float sk = fmaf(g, st[d], om * load1<T>(k_t + (int64_t)h * D + d));
        const float sv = fmaf(g, st[D + d], om * load1<T>(v_t + (int64_t)h * D + d));
        st[d] = sk;
        st[D + d] = sv;
        T *pg = static_cast<T *>(a.kv) + (((int64_t)h * a.page_cap + page) * 2) * S * D;
        store1<T>(pg + (int64_t)slot * D + d, sk);
        store1<T>(pg + (int64_t)(S + slot) * D + d, sv);
        const float r = round_storage<T>(sk);
        amax = fabsf(r);
        T *m = static_cast<T *>(a.meta) + (((int64_t)h * a.page_cap + page) * 2) * D;
        float mn = r, mx = r;
        if (slot == 0) {
            // a fresh page: clear its unused slots so that later reads are defined
            for (int s2 = 1; s2 < S; ++s2) {
                store1<T>(pg + (int64_t)s2 * D + d, 0.0f);
                store1<T>(pg + (int64_t)(S + s2) * D + d, 0.0f);
            }
        } else {
            mn = fminf(load1<T>(m + d), r);
            mx = fmaxf(load1<T>(m + D + d), r);
        }
        store1<T>(m + d, mn);
        store1<T>(m + D + d, mx);
        const float qd = load1<T>(q + (int64_t)h * D + d);
        term = fmaxf(qd * mn, qd * mx);
    }
    // score of the newest page: sum of the D terms; largest |stored key| of the new row
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        term += __shfl_xor_sync(0xffffffffu, term, off);
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
    }
    if ((threadIdx.x & 31) == 0 && threadIdx.x < D) { red[threadIdx.x >> 5] = term; red[8 + (threadIdx.x >> 5)] = amax; }
    __syncthreads();
    float s = 0.0f;
    if (threadIdx.x == 0) {
        float m = 0.0f;
        for (int w = 0; w < (D + 31) / 32; ++w) { s += red[w]; m = fmaxf(m, red[8 + w]); }
        scores[(int64_t)h * a.page_cap + page] = s;
        if (a.absmax) {
            const int BH = a.B * a.H, cur = a.epoch & 1;
            const float nv = fmaxf(a.absmax[cur * BH + h], m);
            a.absmax[(cur ^ 1) * BH + h] = nv;
        }
    }
    __syncthreads();
    return s;
}

// ---------------------------------------------------------------- a-priori score range
// Every page score of head h lies in [-R, R] with R = A * sum_i |q_i|, A the largest |stored key|
// of the head (|U_p| <= sum_i |q_i| max(|min_p[i]|, |max_p[i]|)).  The one-launch step spreads
// kStepBins value buckets over that range BEFORE any score exists: bucket(u) = clamp(floor((u + R) *
// scale)), monotone in u whatever R is, so a stale or loose range costs resolution, never
// correctness.  Every warp computes the same bits (same order of operations).
struct ScoreRange {
    float lo, scale;
    __device__ __forceinline__ int bucket(float u) const
    {
        const float f = (u - lo) * scale;
        return min(max((int)f, 0), kStepBins - 1);   // a NaN product lands in bucket 0
    }
};
template <typename T, int D>
__device__ __forceinline__ ScoreRange score_range(const T *q, int h, float amax, int lane)
{
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < D / 32; ++i) s += fabsf(load1<T>(q + (int64_t)h * D + lane + 32 * i));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    const float R = amax * s;
    ScoreRange r;
    r.lo = -R;
    r.scale = (0.5f * (float)kStepBins) / R;
    // an empty or unbounded range: one bucket for everything (the selection then works on the key bits)
    if (!(R > 0.0f) || !(r.scale < CUDART_INF_F) || !(R < CUDART_INF_F)) { r.lo = 0.0f; r.scale = 0.0f; }
    return r;
}



}  // namespace rq
