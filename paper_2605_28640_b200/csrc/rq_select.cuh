// Selection of a head's pages by one CTA of NTH threads (NTH a multiple of 32, at most 1024):
// the TopK of Eq. 3 with forced first / newest pages inside the budget (App. A.1), ties to the
// lower page index, output ascending.  The routine is written for any CTA width; the selection
// kernel runs it with 1024 threads (a narrow CTA of 128 threads takes about 2.5 times as long).
//
// Threshold search: keys (order-preserving integer image of the fp32 score) go to shared memory;
// one histogram pass over 2048 equal-width buckets of the score VALUE between the head's minimum
// and maximum (monotone, so bucket order is key order); the keys of the chosen bucket are ranked
// against each other directly; a bucket with more than kSelCandMax keys is finished by
// most-significant-digit radix passes on the key bits.  Output: one bitmap word per 32 pages for
// "above the threshold" and one for "equal to it", a prefix sum over the words' populations, then
// every thread writes the pages of its words at their ranks; equal keys are taken in index order
// until the budget is full.
#pragma once
#include <math_constants.h>

#include "rq_async.cuh"
#include "rq_device.cuh"

namespace rq {

constexpr uint32_t kSelKeyForced = 0xffffffffu;    // above every score key
constexpr int kSelDigitBits = 11;
constexpr int kSelBins = 1 << kSelDigitBits;
constexpr int kSelCandMax = 1024;

// the score a key was made from (inverse of order_key)
__device__ __forceinline__ float sel_key_value(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// bytes of shared memory select_head needs for P pages
__host__ __device__ constexpr size_t select_smem_bytes(int P)
{
    return (size_t)P * 4 + kSelBins * 4 + kSelCandMax * 4 + 2 * (size_t)((P + 31) / 32) * 4 + 128 * 4;
}

template <int NTH>
__device__ void select_head(const float *sc, int P, int K, int n_sink, int n_local, int32_t *out, int budget,
                            unsigned char *sm)
{
    constexpr int NWP = NTH / 32;
    constexpr int BPT = kSelBins / NTH;            // bins a thread owns in the suffix scan
    constexpr unsigned FULL = 0xffffffffu;
    static_assert(NTH % 32 == 0 && kSelBins % NTH == 0 && NWP <= 32, "unsupported CTA width");
    const int W = (P + 31) / 32;                     // bitmap words
    uint32_t *skey = reinterpret_cast<uint32_t *>(sm);
    uint32_t *hist = skey + P;
    uint32_t *cand = hist + kSelBins;
    uint32_t *bmg = cand + kSelCandMax;
    uint32_t *bme = bmg + W;
    uint32_t *red = bme + W;                         // [32] + [32] reduction scratch
    uint32_t *red2 = red + 32;
    uint32_t *sv = red2 + 32;                        // [0] digit, [1] k_rem, [2] cnt, [3] ncand, [4] tau
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (K >= P) {                                    // dense: every page, in order
        for (int p = tid; p < budget; p += NTH) out[p] = p < P ? p : -1;
        return;
    }
    uint32_t kmin = 0xffffffffu, kmax = 0u;
#pragma unroll 8
    for (int p = tid; p < P; p += NTH) {
        uint32_t kx = kSelKeyForced;
        if (p >= n_sink && p < P - n_local) {
            kx = order_key(__ldcg(sc + p));
            kx = min(max(kx, 1u), 0xfffffffeu);      // stay clear of the reserved key
            kmin = min(kmin, kx);
            kmax = max(kmax, kx);
        }
        skey[p] = kx;
    }
    int k_rem = K - n_sink - n_local;                // budget left for pages that are not forced

    auto block_minmax = [&](uint32_t &lo, uint32_t &hi) {
        lo = __reduce_min_sync(FULL, lo);
        hi = __reduce_max_sync(FULL, hi);
        __syncthreads();                             // earlier readers of red / red2 are done
        if (lane == 0) { red[warp] = lo; red2[warp] = hi; }
        __syncthreads();
        lo = __reduce_min_sync(FULL, lane < NWP ? red[lane] : 0xffffffffu);
        hi = __reduce_max_sync(FULL, lane < NWP ? red2[lane] : 0u);
    };
    block_minmax(kmin, kmax);

    // One histogram pass over the non-forced keys for which `in(key)` holds: bins by `bin(key)`,
    // walked from the top until k_rem keys are covered.  Leaves the chosen bin in sv[0], the
    // rank wanted inside it in sv[1] and its population in sv[2].
    auto select_bin = [&](auto in, auto bin) {
        __syncthreads();                             // earlier readers of hist / red / sv are done
        for (int i = tid; i < kSelBins; i += NTH) hist[i] = 0u;
        __syncthreads();
#pragma unroll 4
        for (int p = tid; p < P; p += NTH) {
            const uint32_t kx = skey[p];
            if (kx != kSelKeyForced && in(kx)) atomicAdd(&hist[bin(kx)], 1u);
        }
        __syncthreads();
        // thread t owns the bins [t * BPT, (t + 1) * BPT); suffix sums from the top thread down
        uint32_t tsum = 0;
#pragma unroll 8
        for (int b = 0; b < BPT; ++b) tsum += hist[tid * BPT + b];
        uint32_t suf = tsum;                         // inclusive suffix sum over the threads of the warp
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t t = __shfl_down_sync(FULL, suf, off);
            if (lane + off < 32) suf += t;
        }
        if (lane == 0) red[warp] = suf;              // warp totals
        __syncthreads();
        uint32_t above = suf - tsum;                 // keys in the bins of higher threads
        for (int w = warp + 1; w < NWP; ++w) above += red[w];
        const uint32_t kr = (uint32_t)k_rem;
        if (above < kr && above + tsum >= kr) {      // the wanted bin is one of this thread's
            uint32_t run = above;
            for (int b = BPT - 1; b >= 0; --b) {
                const uint32_t c = hist[tid * BPT + b];
                if (run < kr && run + c >= kr) { sv[0] = (uint32_t)(tid * BPT + b); sv[1] = kr - run; sv[2] = c; }
                run += c;
            }
        }
        __syncthreads();
    };
    // Most-significant-digit radix select on the key bits among the keys for which `in` holds and
    // whose extreme keys are lo_key and hi_key: returns the k_rem-th largest of them.
    auto radix_select = [&](auto in, uint32_t lo_key, uint32_t hi_key) -> uint32_t {
        if (lo_key == hi_key) return lo_key;
        int hb = 31 - __clz(lo_key ^ hi_key);        // highest bit in which the keys differ
        uint32_t t = hb == 31 ? 0u : (hi_key >> (hb + 1)) << (hb + 1);   // shared leading bits
        while (hb >= 0) {
            const int lo = hb >= kSelDigitBits - 1 ? hb - (kSelDigitBits - 1) : 0;   // this pass decides bits hb .. lo
            const uint32_t dmask = (1u << (hb - lo + 1)) - 1u;
            const uint32_t himask = hb == 31 ? 0u : ~0u << (hb + 1);
            select_bin([&](uint32_t kx) { return in(kx) && (kx & himask) == (t & himask); },
                       [&](uint32_t kx) { return (kx >> lo) & dmask; });
            t |= sv[0] << lo;
            k_rem = (int)sv[1];
            if (sv[2] == sv[1]) break;               // the whole bin is wanted: its lowest possible key is a threshold
            hb = lo - 1;
        }
        return t;
    };

    uint32_t tau;                                    // k-th largest key among the non-forced pages
    if (k_rem <= 0) {
        tau = kSelKeyForced;                         // nothing but forced pages fits: take none of the rest
    } else if (kmin == kmax) {
        tau = kmin;
    } else {
        const float v_lo = sel_key_value(kmin);
        const float scale = (float)(kSelBins - 1) / (sel_key_value(kmax) - v_lo);
        auto bucket = [&](uint32_t kx) -> uint32_t {
            const float f = (sel_key_value(kx) - v_lo) * scale;
            return (uint32_t)min(max((int)f, 0), kSelBins - 1);
        };
        if (!(scale > 0.0f) || !(scale < CUDART_INF_F)) {
            tau = radix_select([](uint32_t) { return true; }, kmin, kmax);      // range too wide for a float
        } else {
            select_bin([](uint32_t) { return true; }, bucket);
            const uint32_t b = sv[0], cnt = sv[2];
            k_rem = (int)sv[1];
            if (tid == 0) sv[3] = 0;
            __syncthreads();
            uint32_t cmin = 0xffffffffu, cmax = 0u;
#pragma unroll 4
            for (int p = tid; p < P; p += NTH) {
                const uint32_t kx = skey[p];
                if (kx != kSelKeyForced && bucket(kx) == b) {
                    cmin = min(cmin, kx);
                    cmax = max(cmax, kx);
                    if (cnt <= (uint32_t)kSelCandMax) cand[atomicAdd(&sv[3], 1u)] = kx;
                }
            }
            __syncthreads();
            if (cnt <= (uint32_t)kSelCandMax) {
                // rank every candidate against all others; the wanted one has fewer than k_rem
                // candidates above it and at least k_rem at or above it
                for (uint32_t i = tid; i < cnt; i += NTH) {
                    const uint32_t mine = cand[i];
                    uint32_t g = 0, ge = 0;
                    for (uint32_t j = 0; j < cnt; ++j) {
                        const uint32_t o = cand[j];
                        g += o > mine;
                        ge += o >= mine;
                    }
                    if (g < (uint32_t)k_rem && ge >= (uint32_t)k_rem) sv[4] = mine;
                }
                __syncthreads();
                tau = sv[4];
            } else {
                block_minmax(cmin, cmax);            // an unusually full bucket: finish on the key bits
                tau = radix_select([&](uint32_t kx) { return bucket(kx) == b; }, cmin, cmax);
            }
        }
    }

    // bitmaps: bit b of word w says whether page 32 w + b is above / equal to the threshold
    __syncthreads();
    for (int w = warp; w < W; w += NWP) {
        const int p = w * 32 + lane;
        const uint32_t kx = p < P ? skey[p] : 0u;    // 0 is below every key
        const uint32_t bg = __ballot_sync(FULL, kx > tau), be = __ballot_sync(FULL, kx == tau);
        if (lane == 0) { bmg[w] = bg; bme[w] = be; }
    }
    __syncthreads();
    // thread t owns the words [t * WPT, (t + 1) * WPT): counts of "above" (low half) and "equal"
    // (high half; both fit in 16 bits for up to 32768 pages), then an exclusive scan over threads
    const int WPT = (W + NTH - 1) / NTH;
    uint32_t mine = 0;
    for (int i = 0; i < WPT; ++i) {
        const int w = tid * WPT + i;
        if (w < W) mine += (uint32_t)__popc(bmg[w]) + ((uint32_t)__popc(bme[w]) << 16);
    }
    uint32_t incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_up_sync(FULL, incl, off);
        if (lane >= off) incl += t;
    }
    if (lane == 31) red[warp] = incl;
    __syncthreads();
    uint32_t before = 0, total = 0;
    for (int w = 0; w < NWP; ++w) {
        if (w < warp) before += red[w];
        total += red[w];
    }
    const uint32_t excl = before + incl - mine;
    const int n_gt = (int)(total & 0xffffu);
    const int r = K - n_gt;                          // how many equal keys to take
    int gb = (int)(excl & 0xffffu), eb = (int)(excl >> 16);
    for (int i = 0; i < WPT; ++i) {
        const int w = tid * WPT + i;
        if (w >= W) break;
        const uint32_t g = bmg[w];
        uint32_t bits = g | bme[w];
        while (bits) {
            const int b = __ffs(bits) - 1;
            bits &= bits - 1;
            const int page = w * 32 + b;
            if ((g >> b) & 1u) {
                out[gb + min(eb, r)] = page;
                ++gb;
            } else {
                if (eb < r) out[gb + eb] = page;
                ++eb;
            }
        }
    }
    for (int p = K + tid; p < budget; p += NTH) out[p] = -1;
}

}  // namespace rq
