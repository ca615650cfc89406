// Decode step kernels:
//   update  — one step of Eq. 1 on the fp32 state, append to the paged cache,
//             refresh the newest page's min/max
//   score   — Quest upper bound U_p = sum_i max(q_i min_p[i], q_i max_p[i]) for
//             every page (Eq. 3 with the min/max representatives of App. A.1)
//   topk    — per (b,h) selection of the budget's pages, forced first/local
//             pages inside the budget, ties to the lower page index, ascending
// All of it is bandwidth-bound GEMV-like work on plain ALUs with fp32
// accumulation; no tensor cores.
#include <math_constants.h>

#include "rq_device.cuh"
#include "rq_internal.h"

namespace rq {

namespace {

// ---------------------------------------------------------------- update
// grid: B*H CTAs of D threads; thread d owns channel d.
template <typename T, typename G, int D, int S>
__global__ void update_kernel(DecodeArgs a, const T *k_t, const T *v_t, const G *g_t)
{
    const int bh = blockIdx.x, d = threadIdx.x;
    const int64_t pos = a.len;              // position of the new token
    const int64_t page = pos / S;
    const int slot = (int)(pos % S);
    float *st = a.state + (int64_t)bh * 2 * D;
    const float g = load1<G>(g_t + (int64_t)bh * D + d);
    const float om = 1.0f - g;
    const float sk = fmaf(g, st[d], om * load1<T>(k_t + (int64_t)bh * D + d));
    const float sv = fmaf(g, st[D + d], om * load1<T>(v_t + (int64_t)bh * D + d));
    st[d] = sk;
    st[D + d] = sv;
    T *pg = static_cast<T *>(a.kv) + (((int64_t)bh * a.page_cap + page) * 2) * S * D;
    store1<T>(pg + (int64_t)slot * D + d, sk);
    store1<T>(pg + (int64_t)(S + slot) * D + d, sv);
    const float r = round_storage<T>(sk);
    T *m = static_cast<T *>(a.meta) + (((int64_t)bh * a.page_cap + page) * 2) * D;
    if (slot == 0) {
        store1<T>(m + d, r);
        store1<T>(m + D + d, r);
        // a fresh page: clear its unused slots so that later reads are defined
        for (int s2 = 1; s2 < S; ++s2) {
            store1<T>(pg + (int64_t)s2 * D + d, 0.0f);
            store1<T>(pg + (int64_t)(S + s2) * D + d, 0.0f);
        }
    } else {
        store1<T>(m + d, fminf(load1<T>(m + d), r));
        store1<T>(m + D + d, fmaxf(load1<T>(m + D + d), r));
    }
}

// ---------------------------------------------------------------- score
// A page's bounds are one contiguous record [min row][max row] of 2*D
// elements.  Since min <= max, max(q*min, q*max) = q*max for q >= 0 and q*min
// for q < 0, so a lane holding part of the max row multiplies by max(q,0) and
// a lane holding part of the min row by min(q,0); every loaded byte is used
// and the record's sum is a reduction over the lanes that share it.
constexpr int kScoreThreads = 256;
constexpr int kScoreUnroll = 8;   // records in flight per lane group

template <typename T, int D>
__global__ void __launch_bounds__(kScoreThreads) score_kernel(DecodeArgs a, const T *q, float *scores,
                                                              int64_t P, int pages_per_cta)
{
    constexpr int CH = VecOf<T>::N;
    constexpr int VPR = 2 * D / CH;                 // 16-byte vectors per record
    constexpr int LPP = VPR > 32 ? 32 : VPR;        // lanes that share one record
    constexpr int VPL = VPR / LPP;                  // vectors per lane per record (1 or 2)
    constexpr int PPW = 32 / LPP;                   // records per warp-wide load
    static_assert(VPL == 1 || VPL == 2, "unsupported record width");

    const int bh = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane / LPP, c = lane % LPP;

    // this lane's slice of q, pre-split by sign
    float qs[VPL][CH];
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        const int vec = c + v * LPP;                // vector index inside the record
        const bool is_max = vec >= VPR / 2;
        const int ch0 = (vec % (VPR / 2)) * CH;
#pragma unroll
        for (int i = 0; i < CH; ++i) {
            const float x = load1<T>(q + (int64_t)bh * D + ch0 + i);
            qs[v][i] = is_max ? fmaxf(x, 0.0f) : fminf(x, 0.0f);
        }
    }

    const T *meta = static_cast<const T *>(a.meta) + (int64_t)bh * a.page_cap * 2 * D;
    const int64_t p_begin = (int64_t)blockIdx.x * pages_per_cta;
    const int64_t p_end = min(P, p_begin + pages_per_cta);
    constexpr int WARPS = kScoreThreads / 32;
    constexpr int STEP = PPW * kScoreUnroll;        // records per warp iteration

    for (int64_t p0 = p_begin + (int64_t)warp * STEP; p0 < p_end; p0 += (int64_t)WARPS * STEP) {
        uint4 r[kScoreUnroll][VPL];
#pragma unroll
        for (int u = 0; u < kScoreUnroll; ++u) {
            const int64_t p = p0 + u * PPW + sub;
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
                if (p < p_end) r[u][v] = ldcs16(meta + p * 2 * D + (c + v * LPP) * CH);
                else r[u][v] = make_uint4(0, 0, 0, 0);
            }
        }
#pragma unroll
        for (int u = 0; u < kScoreUnroll; ++u) {
            float s = 0.0f;
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
                float m[CH];
                unpack16<T>(r[u][v], m);
#pragma unroll
                for (int i = 0; i < CH; ++i) s = fmaf(qs[v][i], m[i], s);
            }
#pragma unroll
            for (int off = LPP / 2; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
            const int64_t p = p0 + u * PPW + sub;
            if (c == 0 && p < p_end) scores[(int64_t)bh * a.page_cap + p] = s;
        }
    }
}

// ---------------------------------------------------------------- top-k
// One CTA per (b,h).  Scores become order-preserving 32-bit keys held in
// registers (consecutive pages per thread).  Forced pages (first / newest) are
// taken outright and count inside the budget.  Among the rest, the k-th
// largest key is found by a most-significant-digit radix select: the bits
// that all keys share are skipped, then each pass histograms one 8-bit digit
// of the keys that still match the prefix found so far (one private histogram
// per warp in shared memory, so equal keys only collide inside a warp) and
// walks the bins from the top until the remaining budget is used up.  Pages
// with a larger key are taken; pages with an equal key are taken in index
// order until the budget is full.  A block-wide prefix sum over the
// per-thread counts gives each taken page its slot, so the output is
// ascending and unique whatever the thread timing.
constexpr uint32_t kKeyForced = 0xffffffffu;   // above every score key
constexpr uint32_t kKeyPad = 0u;               // below every score key

template <int KPT>
__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const float *scores, int64_t score_stride,
                                                            int P, int K, int n_sink, int n_local,
                                                            int32_t *idx, int idx_stride, int budget,
                                                            int32_t *attend_ctr)
{
    constexpr int NTH = kTopkThreads, NWP = NTH / 32;
    static_assert(NWP == 32, "second-level reductions are one warp wide");
    __shared__ uint32_t hist[NWP][256];
    __shared__ uint32_t red[NWP];
    __shared__ uint32_t bins[256];
    __shared__ uint32_t s_digit, s_krem;
    const int bh = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t *out = idx + (int64_t)bh * idx_stride;
    if (tid < 3) attend_ctr[bh * kCtrStride + tid] = 0;   // the flash-decode kernel's counters of this head

    if (K >= P) {                                    // dense: every page, in order
        for (int p = tid; p < budget; p += NTH) out[p] = p < P ? p : -1;
        return;
    }
    const float *sc = scores + (int64_t)bh * score_stride;
    const int nk = (P + NTH - 1) / NTH;              // pages per thread in use (<= KPT)
    const int base = tid * nk;
    uint32_t key[KPT];
    uint32_t kmin = 0xffffffffu, kmax = 0u;
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
        const int p = base + j;
        uint32_t kx = kKeyPad;
        if (j < nk && p < P) {
            if (p < n_sink || p >= P - n_local) {
                kx = kKeyForced;
            } else {
                kx = order_key(sc[p]);
                kx = min(max(kx, 1u), 0xfffffffeu);  // stay clear of the two reserved keys
                kmin = min(kmin, kx);
                kmax = max(kmax, kx);
            }
        }
        key[j] = kx;
    }
    int k_rem = K - n_sink - n_local;                // budget left for pages that are not forced

    // range of the score keys -> bits they all share
    kmin = __reduce_min_sync(0xffffffffu, kmin);
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if (lane == 0) { red[warp] = kmin; bins[warp] = kmax; }
    __syncthreads();
    kmin = __reduce_min_sync(0xffffffffu, red[lane]);
    kmax = __reduce_max_sync(0xffffffffu, bins[lane]);
    __syncthreads();

    uint32_t tau;                                    // k-th largest key among the non-forced pages
    if (k_rem <= 0) {
        tau = 0xfffffffeu + 1u;                      // nothing but forced pages fits: take none of the rest
    } else if (kmin == kmax) {
        tau = kmin;
    } else {
        int hb = 31 - __clz(kmin ^ kmax);            // highest bit in which keys differ
        tau = hb == 31 ? 0u : (kmax >> (hb + 1)) << (hb + 1);   // shared leading bits
        while (hb >= 0) {
            const int lo = hb >= 7 ? hb - 7 : 0;     // this pass decides bits hb .. lo
            const int nb = hb - lo + 1;
            const uint32_t himask = hb == 31 ? 0u : ~0u << (hb + 1);
#pragma unroll
            for (int i = 0; i < 8; ++i) hist[warp][lane + 32 * i] = 0u;
            __syncwarp();
#pragma unroll
            for (int j = 0; j < KPT; ++j) {
                if (j >= nk) break;
                const uint32_t kx = key[j];
                if (kx != kKeyForced && kx != kKeyPad && (kx & himask) == (tau & himask))
                    atomicAdd(&hist[warp][(kx >> lo) & ((1u << nb) - 1u)], 1u);
            }
            __syncthreads();
            // bin totals, then suffix sums from the top bin down
            uint32_t c = 0;
            if (tid < 256) {
#pragma unroll 8
                for (int w = 0; w < NWP; ++w) c += hist[w][tid];
            }
            uint32_t suf = c;                        // inclusive suffix sum inside the warp
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t t = __shfl_down_sync(0xffffffffu, suf, off);
                if (lane + off < 32) suf += t;
            }
            if (tid < 256 && lane == 0) red[warp] = suf;   // warp totals (8 warps cover 256 bins)
            __syncthreads();
            if (tid < 256) {
                uint32_t above = 0;                  // keys in the warps that hold higher bins
                for (int w = warp + 1; w < 8; ++w) above += red[w];
                const uint32_t s_incl = suf + above; // keys in bins >= tid
                const uint32_t s_excl = s_incl - c;  // keys in bins >  tid
                if (s_incl >= (uint32_t)k_rem && s_excl < (uint32_t)k_rem) {
                    s_digit = (uint32_t)tid;
                    s_krem = (uint32_t)k_rem - s_excl;
                }
            }
            __syncthreads();
            tau |= s_digit << lo;
            k_rem = (int)s_krem;
            hb = lo - 1;
        }
    }

    // per-thread counts of "greater" (low half) and "equal" (high half)
    uint32_t mine = 0;
#pragma unroll
    for (int j = 0; j < KPT; ++j) mine += (key[j] > tau ? 1u : 0u) + (key[j] == tau ? 0x10000u : 0u);
    uint32_t incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += t;
    }
    if (lane == 31) red[warp] = incl;
    __syncthreads();
    const uint32_t wv = red[lane];
    uint32_t winc = wv;                              // inclusive scan of the warp totals
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, winc, off);
        if (lane >= off) winc += t;
    }
    const uint32_t total = __shfl_sync(0xffffffffu, winc, 31);
    const uint32_t before = __shfl_sync(0xffffffffu, winc - wv, warp);
    const uint32_t excl = before + incl - mine;
    const int n_gt = (int)(total & 0xffffu);
    const int r = K - n_gt;                          // how many equal keys to take
    int gt_before = (int)(excl & 0xffffu), eq_before = (int)(excl >> 16);
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
        if (key[j] > tau) {
            out[gt_before + min(eq_before, r)] = base + j;
            ++gt_before;
        } else if (key[j] == tau && key[j] != kKeyPad) {
            if (eq_before < r) out[gt_before + eq_before] = base + j;
            ++eq_before;
        }
    }
    for (int p = K + tid; p < budget; p += NTH) out[p] = -1;
}

// ---------------------------------------------------------------- dispatch helpers
#define RQ_DISPATCH_TDS(a, CALL)                                                         \
    do {                                                                                 \
        if ((a).dtype == RQ_BF16) {                                                      \
            if ((a).D == 128 && (a).S == 16) { CALL(bf16, 128, 16); }                    \
            else if ((a).D == 128 && (a).S == 64) { CALL(bf16, 128, 64); }               \
            else if ((a).D == 64 && (a).S == 16) { CALL(bf16, 64, 16); }                 \
            else if ((a).D == 64 && (a).S == 64) { CALL(bf16, 64, 64); }                 \
            else return cudaErrorInvalidValue;                                           \
        } else {                                                                         \
            if ((a).D == 128 && (a).S == 16) { CALL(float, 128, 16); }                   \
            else if ((a).D == 128 && (a).S == 64) { CALL(float, 128, 64); }              \
            else if ((a).D == 64 && (a).S == 16) { CALL(float, 64, 16); }                \
            else if ((a).D == 64 && (a).S == 64) { CALL(float, 64, 64); }                \
            else return cudaErrorInvalidValue;                                           \
        }                                                                                \
    } while (0)

}  // namespace

cudaError_t launch_update(const DecodeArgs &a, const void *k_t, const void *v_t, const void *g_t,
                          cudaStream_t s)
{
    const int BH = a.B * a.H;
#define CALL_UPD(T, D, S)                                                                              \
    if (a.gate_dtype == RQ_BF16)                                                                       \
        update_kernel<T, bf16, D, S><<<BH, D, 0, s>>>(a, (const T *)k_t, (const T *)v_t, (const bf16 *)g_t); \
    else                                                                                               \
        update_kernel<T, float, D, S><<<BH, D, 0, s>>>(a, (const T *)k_t, (const T *)v_t, (const float *)g_t)
    RQ_DISPATCH_TDS(a, CALL_UPD);
#undef CALL_UPD
    return cudaGetLastError();
}

cudaError_t launch_score(const DecodeArgs &a, const void *q, float *scores, cudaStream_t s)
{
    const int64_t P = (a.len + a.S - 1) / a.S;
    if (P <= 0) return cudaSuccess;
    const int pages_per_cta = 64;
    dim3 grid((unsigned)((P + pages_per_cta - 1) / pages_per_cta), (unsigned)(a.B * a.H));
    if (a.dtype == RQ_BF16) {
        if (a.D == 128) score_kernel<bf16, 128><<<grid, kScoreThreads, 0, s>>>(a, (const bf16 *)q, scores, P, pages_per_cta);
        else if (a.D == 64) score_kernel<bf16, 64><<<grid, kScoreThreads, 0, s>>>(a, (const bf16 *)q, scores, P, pages_per_cta);
        else return cudaErrorInvalidValue;
    } else {
        if (a.D == 128) score_kernel<float, 128><<<grid, kScoreThreads, 0, s>>>(a, (const float *)q, scores, P, pages_per_cta);
        else if (a.D == 64) score_kernel<float, 64><<<grid, kScoreThreads, 0, s>>>(a, (const float *)q, scores, P, pages_per_cta);
        else return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_topk(const DecodeArgs &a, const float *scores, int budget, int32_t *idx,
                        int idx_stride, int32_t *attend_ctr, cudaStream_t s)
{
    const int P = (int)((a.len + a.S - 1) / a.S);
    const int K = budget < P ? budget : P;
    const int BH = a.B * a.H;
    // forced pages inside the budget: sinks first, then local pages from the newest backwards
    int ns = a.n_sink < K ? a.n_sink : K;
    if (ns > P) ns = P;
    int nl = a.n_local < K - ns ? a.n_local : K - ns;
    if (nl > P - ns) nl = P - ns;
    const int per = (P + kTopkThreads - 1) / kTopkThreads;
#define CALL_TOPK(KPT) \
    topk_kernel<KPT><<<BH, kTopkThreads, 0, s>>>(scores, a.page_cap, P, K, ns, nl, idx, idx_stride, budget, attend_ctr)
    if (per <= 1) CALL_TOPK(1);
    else if (per <= 2) CALL_TOPK(2);
    else if (per <= 4) CALL_TOPK(4);
    else if (per <= 8) CALL_TOPK(8);
    else if (per <= 16) CALL_TOPK(16);
    else if (per <= 32) CALL_TOPK(32);
    else return cudaErrorInvalidValue;
#undef CALL_TOPK
    return cudaGetLastError();
}

}  // namespace rq
