// Second kernel of a decode step: per (b,h) selection of the budget's pages from
// the page scores (the TopK of Eq. 3), forced first/local pages inside the
// budget (App. A.1), ties to the lower page index, output ascending.
#include <math_constants.h>

#include "rq_device.cuh"
#include "rq_internal.h"

namespace rq {

namespace {

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
    if (tid < 4) attend_ctr[bh * kCtrStride + tid] = 0;   // this head's ticket counters of the streaming kernels

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

}  // namespace

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
