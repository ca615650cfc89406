// Second kernel of a decode step: per (b,h) selection of the budget's pages from
// the page scores (the TopK of Eq. 3), forced first/local pages inside the
// budget (App. A.1), ties to the lower page index.  Two routines give the same set:
// select_rows works from the scores alone (range, value histogram, direct ranking or
// radix passes; ascending list); fast_select starts from the histogram that the scoring
// kernel filled while it scored (no pass for the range, no keys; list in no particular
// order) and hands over to select_rows whenever it cannot finish.  Also here: the
// short-context kernel that scores and selects a head in one CTA.
#include <math_constants.h>

#include "rq_async.cuh"
#include "rq_device.cuh"
#include "rq_internal.h"
#include "rq_stream.cuh"

namespace rq {

namespace {

// ---------------------------------------------------------------- top-k
// One CTA of 1024 threads per (b,h).  Scores become order-preserving 32-bit keys.  Forced pages
// (first / newest) are taken outright and count inside the budget.  Among the rest the k-th
// largest key (the threshold) is found in two steps: one histogram pass over 2048 equal-width
// buckets of the score VALUE between the head's smallest and largest score (the map score ->
// bucket is monotone, so bucket order is key order, and the bulk of the scores is resolved evenly
// whatever their sign and exponent), then the keys of the bucket that holds the threshold are
// ranked against each other directly.  A bucket with more than 1024 keys (many equal scores), or a
// score range too narrow or too wide for a float bucket width, is finished by
// most-significant-digit radix passes on the key bits instead: the bits all keys share are
// skipped, each pass histograms one 11-bit digit of the keys that still match the prefix found so
// far, and a pass whose chosen bin is wanted whole ends the search.  Pages with a key above the
// threshold are taken; pages with a key equal to it are taken in index order until the budget is
// full.  For the output, warp w owns a contiguous range of pages and walks it row by row (row j:
// pages base_w + 32 j + lane): warp ballots give every taken page its rank inside the warp and a
// scan over the warp totals its rank in the head, so the list is ascending and unique whatever
// the thread timing.
//
// A thread keeps the keys of its ROWS pages (and their bucket numbers) in registers when a head
// has at most 10240 pages: the passes over the keys then need no shared-memory traffic and no
// address arithmetic, which is what the one SM that selects a head spends its issue slots on.
// Larger heads (up to 32768 pages) keep the keys in shared memory; the code is the same.
constexpr uint32_t kKeyForced = 0xffffffffu;   // above every score key
constexpr uint32_t kKeyAbsent = 0u;            // below every score key: a row beyond the head's pages
constexpr int kDigitBits = 11;
constexpr int kBins = 1 << kDigitBits;
constexpr int kCandMax = 1024;                 // candidates ranked directly; a fuller bucket goes through the key bits

constexpr int kHistCopies = 2;                 // histogram copies; warp w adds to copy w % kHistCopies
static_assert(kTopkThreads == 1024 && kBins == 2 * kTopkThreads, "32 warps; a thread owns two bins in the suffix scan");
static_assert(kHistCopies * kBins == 4 * kTopkThreads, "a thread clears four bins");

// shared-memory scratch of a selection CTA
struct SelectScratch {
    alignas(16) uint32_t hist[kHistCopies][kBins];   // read back as 8-byte pairs
    uint32_t red[32], red2[32];                      // per-warp values of block-wide reductions
    uint32_t digit, krem, cnt, ncand, tau;           // chosen bin, rank wanted inside it, its population; candidates; threshold
    uint32_t cand[kCandMax];                         // keys of the chosen bucket
};

// After a histogram pass (all kHistCopies copies filled): walk the bins from the top until k_rem
// keys are covered.  Leaves the chosen bin in sh.digit, the rank wanted inside it in sh.krem and
// its population in sh.cnt.  Called by every thread of the CTA.
__device__ __forceinline__ void pick_bin(SelectScratch &sh, int k_rem)
{
    constexpr unsigned FULL = 0xffffffffu;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __syncthreads();                                 // the histogram is complete
    uint32_t c0 = 0, c1 = 0;                         // thread t owns bins 2t and 2t+1
#pragma unroll
    for (int w = 0; w < kHistCopies; ++w) {
        const uint2 h2 = *reinterpret_cast<const uint2 *>(&sh.hist[w][2 * tid]);
        c0 += h2.x;
        c1 += h2.y;
    }
    uint32_t suf = c0 + c1;                          // inclusive suffix sum over the threads of the warp
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_down_sync(FULL, suf, off);
        if (lane + off < 32) suf += t;
    }
    if (lane == 0) sh.red[warp] = suf;               // warp totals
    __syncthreads();
    const uint32_t wtot = sh.red[lane];
    uint32_t wsuf = wtot;                            // suffix sum over the warps, every warp on its own
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t t = __shfl_down_sync(FULL, wsuf, off);
        if (lane + off < 32) wsuf += t;
    }
    const uint32_t above = __shfl_sync(FULL, wsuf - wtot, warp);   // keys in higher warps' bins
    const uint32_t incl1 = above + suf - c0;         // keys in bins >= 2t+1
    const uint32_t excl1 = incl1 - c1;               // keys in bins >  2t+1
    const uint32_t incl0 = incl1 + c0;               // keys in bins >= 2t
    const uint32_t kr = (uint32_t)k_rem;
    if (incl1 >= kr && excl1 < kr) { sh.digit = 2u * tid + 1u; sh.krem = kr - excl1; sh.cnt = c1; }
    if (incl0 >= kr && incl1 < kr) { sh.digit = 2u * tid; sh.krem = kr - incl1; sh.cnt = c0; }
    __syncthreads();
}

// The k_rem-th largest of the cnt candidates in sh.cand (cnt <= kCandMax; they are complete): every
// candidate is ranked against all others; the wanted one has fewer than k_rem candidates above it
// and at least k_rem at or above it.  Called by every thread of the CTA.
__device__ __forceinline__ uint32_t rank_candidates(SelectScratch &sh, uint32_t cnt, int k_rem)
{
    const int tid = threadIdx.x;
    if (tid < (int)cnt) {
        const uint32_t mine = sh.cand[tid];
        uint32_t g = 0, ge = 0;
#pragma unroll 4
        for (uint32_t j = 0; j < cnt; ++j) {
            const uint32_t o = sh.cand[j];
            g += o > mine;
            ge += o >= mine;
        }
        if (g < (uint32_t)k_rem && ge >= (uint32_t)k_rem) sh.tau = mine;
    }
    __syncthreads();
    return sh.tau;
}

// From every warp's counts of keys above (wgt) and equal to (weq) the threshold: how many equal keys
// are taken in all (r) and how many pages of either kind are taken before this warp's.
__device__ __forceinline__ void scan_warp_counts(SelectScratch &sh, uint32_t wgt, uint32_t weq, int K, int &r, int &gt_run,
                                                 int &eq_run)
{
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();                                 // earlier readers of red / red2 are done
    if (lane == 0) { sh.red[warp] = wgt; sh.red2[warp] = weq; }
    __syncthreads();
    uint32_t g_inc = sh.red[lane], e_inc = sh.red2[lane];   // inclusive scans over the warps
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t tg = __shfl_up_sync(FULL, g_inc, off), te = __shfl_up_sync(FULL, e_inc, off);
        if (lane >= off) { g_inc += tg; e_inc += te; }
    }
    const int n_gt = (int)__shfl_sync(FULL, g_inc, 31);
    r = K - n_gt;                                    // how many equal keys to take
    gt_run = (int)(__shfl_sync(FULL, g_inc, warp) - wgt);   // taken before this warp
    eq_run = (int)(__shfl_sync(FULL, e_inc, warp) - weq);
}

__device__ __forceinline__ float key_value(uint32_t k) { return order_key_value(k); }

// clears what select_rows expects to find clear; a CTA barrier must lie between the two
__device__ __forceinline__ void select_prepare(SelectScratch &sh)
{
    reinterpret_cast<uint4 *>(&sh.hist[0][0])[threadIdx.x] = make_uint4(0u, 0u, 0u, 0u);
    if (threadIdx.x == 0) sh.ncand = 0;
}

// The selection proper for one head by the whole CTA (1024 threads): scores sc[0 .. P) -> out[0 .. budget).
// The histogram and the candidate counter of `sh` are clear on entry (select_prepare).  A thread's
// row j is page base_w + 32 j + lane; with SMEM_KEYS its key lives in skey[j * 1024 + tid]
// (skey: ROWS * 1024 words of shared memory), otherwise in a register.
template <int ROWS, bool SMEM_KEYS>
__device__ __forceinline__ void select_rows(SelectScratch &sh, uint32_t *skey, const float *sc, int P, int K, int n_sink,
                                            int n_local, int32_t *out, int budget, const char *kvh, int page_bytes,
                                            int n_prefetch)
{
    constexpr int NTH = kTopkThreads;
    constexpr unsigned FULL = 0xffffffffu;
    constexpr int NH = kHistCopies;
    constexpr int RR = SMEM_KEYS ? 2 : ROWS;         // register rows (the shared-memory variant keeps none)
    static_assert(ROWS % 2 == 0, "bucket numbers are kept in pairs");
    auto &hist = sh.hist;
    uint32_t *red = sh.red, *red2 = sh.red2, *cand = sh.cand;
    uint32_t &s_digit = sh.digit, &s_krem = sh.krem, &s_cnt = sh.cnt, &s_ncand = sh.ncand;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rows = (P + NTH - 1) / NTH;            // rows of 32 pages per warp (<= ROWS)
    const int base = warp * 32 * rows + lane;        // this lane's page in row 0
    auto clear_hist = [&]() { reinterpret_cast<uint4 *>(&hist[0][0])[tid] = make_uint4(0u, 0u, 0u, 0u); };
    if (K >= P) {                                    // dense: every page, in order
        for (int p = tid; p < budget; p += NTH) out[p] = p < P ? p : -1;
        return;
    }

    uint32_t key_r[RR] = {};                         // the keys of this thread's rows (register variant)
    auto key = [&](int j) -> uint32_t {
        if constexpr (SMEM_KEYS) return skey[j * NTH + tid];
        else return key_r[j];
    };
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    {
        float v[RR];
        if constexpr (!SMEM_KEYS) {                  // all loads first: one round trip
#pragma unroll
            for (int j = 0; j < ROWS; ++j) {
                const int p = base + 32 * j;
                v[j] = (j < rows && p < P) ? __ldcg(sc + p) : 0.0f;
            }
        }
#pragma unroll (SMEM_KEYS ? 4 : ROWS)
        for (int j = 0; j < ROWS; ++j) {
            const int p = base + 32 * j;
            uint32_t kx = kKeyAbsent;
            if (j < rows && p < P) {
                kx = kKeyForced;
                if (p >= n_sink && p < P - n_local) {
                    float x;
                    if constexpr (SMEM_KEYS) x = __ldcg(sc + p);
                    else x = v[j];
                    kx = min(max(order_key(x), 1u), 0xfffffffeu);   // stay clear of the reserved keys
                    kmin = min(kmin, kx);
                    kmax = max(kmax, kx);
                }
            }
            if constexpr (SMEM_KEYS) skey[j * NTH + tid] = kx;      // read back by this thread only
            else key_r[j] = kx;
        }
    }
    int k_rem = K - n_sink - n_local;                // budget left for pages that are not forced
    auto scored = [&](uint32_t kx) { return kx != kKeyAbsent && kx != kKeyForced; };

    auto block_minmax = [&](uint32_t &lo, uint32_t &hi) {
        lo = __reduce_min_sync(FULL, lo);
        hi = __reduce_max_sync(FULL, hi);
        __syncthreads();                             // earlier readers of red / red2 are done
        if (lane == 0) { red[warp] = lo; red2[warp] = hi; }
        __syncthreads();
        lo = __reduce_min_sync(FULL, red[lane]);
        hi = __reduce_max_sync(FULL, red2[lane]);
    };
    block_minmax(kmin, kmax);                        // its barriers also publish the cleared histogram

    // Most-significant-digit radix select on the key bits among the scored keys for which `in`
    // holds, whose extreme keys are lo_key and hi_key: returns a threshold t such that exactly the
    // wanted keys of that set are > t or (== t, in index order, as many as are still wanted), and
    // no key outside the set that is below lo_key is >= t.
    auto radix_select = [&](auto in, uint32_t lo_key, uint32_t hi_key) -> uint32_t {
        if (lo_key == hi_key) return lo_key;
        int hb = 31 - __clz(lo_key ^ hi_key);        // highest bit in which the keys differ
        uint32_t t = hb == 31 ? 0u : (hi_key >> (hb + 1)) << (hb + 1);   // shared leading bits
#pragma unroll 1
        while (hb >= 0) {
            const int lo = hb >= kDigitBits - 1 ? hb - (kDigitBits - 1) : 0;   // this pass decides bits hb .. lo
            const uint32_t dmask = (1u << (hb - lo + 1)) - 1u;
            const uint32_t himask = hb == 31 ? 0u : ~0u << (hb + 1);
            __syncthreads();                         // earlier readers of the histogram are done
            clear_hist();
            __syncthreads();
#pragma unroll (SMEM_KEYS ? 2 : ROWS)
            for (int j = 0; j < ROWS; ++j) {
                const uint32_t kx = key(j);
                if (scored(kx) && in(kx, j) && (kx & himask) == (t & himask))
                    atomicAdd(&hist[warp % NH][(kx >> lo) & dmask], 1u);
            }
            pick_bin(sh, k_rem);
            t |= s_digit << lo;
            k_rem = (int)s_krem;
            // The whole bin is wanted: any threshold at or below its smallest key takes it all.  The
            // bin's lowest possible key, t, may lie below lo_key, where keys outside the set may
            // sit, so the threshold is raised to lo_key (every key of the set is >= lo_key, and
            // when t < lo_key the bin holds lo_key itself, whose copies are all wanted).
            if (s_cnt == s_krem) return max(t, lo_key);
            hb = lo - 1;
        }
        return t;
    };

    uint32_t tau;                                    // k-th largest key among the non-forced pages
    if (k_rem <= 0) {
        tau = 0xfffffffeu + 1u;                      // nothing but forced pages fits: take none of the rest
    } else if (kmin == kmax) {
        tau = kmin;
    } else {
        const float v_lo = key_value(kmin);
        const float scale = (float)(kBins - 1) / (key_value(kmax) - v_lo);
        auto bucket = [&](uint32_t kx) -> uint32_t {
            const float f = (key_value(kx) - v_lo) * scale;
            return (uint32_t)min(max((int)f, 0), kBins - 1);
        };
        if (!(scale > 0.0f) || !(scale < CUDART_INF_F)) {
            // the range is too narrow or too wide for a float bucket width
            tau = radix_select([](uint32_t, int) { return true; }, kmin, kmax);
        } else {
            uint32_t bk2[RR / 2] = {};               // register variant: bucket of every key of this thread, two to a word
            auto bk = [&](uint32_t kx, int j) -> uint32_t {
                if constexpr (SMEM_KEYS) return bucket(kx);
                else return (bk2[j / 2] >> (16 * (j & 1))) & 0xffffu;
            };
#pragma unroll (SMEM_KEYS ? 2 : ROWS)
            for (int j = 0; j < ROWS; ++j) {
                const uint32_t kx = key(j);
                const uint32_t bj = scored(kx) ? bucket(kx) : 0xffffu;
                if (scored(kx)) atomicAdd(&hist[warp % NH][bj], 1u);
                if constexpr (!SMEM_KEYS) bk2[j / 2] = (j & 1) ? (bk2[j / 2] | (bj << 16)) : bj;
            }
            pick_bin(sh, k_rem);
            const uint32_t b = s_digit, cnt = s_cnt;
            k_rem = (int)s_krem;
            uint32_t cmin = 0xffffffffu, cmax = 0u;
#pragma unroll (SMEM_KEYS ? 2 : ROWS)
            for (int j = 0; j < ROWS; ++j) {
                const uint32_t kx = key(j);
                if (scored(kx) && bk(kx, j) == b) {  // a candidate: usually a handful in the whole head
                    cmin = min(cmin, kx);
                    cmax = max(cmax, kx);
                    if (cnt <= (uint32_t)kCandMax) cand[atomicAdd(&s_ncand, 1u)] = kx;
                }
            }
            __syncthreads();
            if (cnt <= (uint32_t)kCandMax) {
                tau = rank_candidates(sh, cnt, k_rem);
            } else {
                block_minmax(cmin, cmax);            // an unusually full bucket (many equal scores): finish on the key bits
                tau = radix_select([&](uint32_t kx, int j) { return bk(kx, j) == b; }, cmin, cmax);
            }
        }
    }

    // rank of every taken page: ballots inside the warp, a scan over the warp totals across warps
    uint32_t mg = 0, me = 0;                         // bit j: this lane's key of row j is greater / equal
#pragma unroll (SMEM_KEYS ? 4 : ROWS)
    for (int j = 0; j < ROWS; ++j) {
        const uint32_t kx = key(j);                  // absent rows hold key 0: neither greater nor equal
        mg |= (uint32_t)(kx > tau) << j;
        me |= (uint32_t)(kx == tau) << j;
    }
    const uint32_t wgt = __reduce_add_sync(FULL, (uint32_t)__popc(mg));   // this warp's counts
    const uint32_t weq = __reduce_add_sync(FULL, (uint32_t)__popc(me));
    int r, gt_run, eq_run;                           // equal keys to take; pages taken before this warp's
    scan_warp_counts(sh, wgt, weq, K, r, gt_run, eq_run);
    const uint32_t lt = (1u << lane) - 1u;
#pragma unroll (SMEM_KEYS ? 4 : ROWS)
    for (int j = 0; j < ROWS; ++j) {
        const bool is_gt = (mg >> j) & 1u, is_eq = (me >> j) & 1u;
        const uint32_t bg = __ballot_sync(FULL, is_gt), be = __ballot_sync(FULL, is_eq);
        const int gb = gt_run + __popc(bg & lt), eb = eq_run + __popc(be & lt);
        const int p = base + 32 * j;
        // the pages the flash-decode kernel reads first are on their way into L2 before it starts
        const int rank = is_gt ? gb + min(eb, r) : (is_eq && eb < r) ? gb + eb : -1;
        if (rank >= 0) {
            out[rank] = p;
            if (rank < n_prefetch) bulk_prefetch_l2(kvh + (int64_t)p * page_bytes, (uint32_t)page_bytes);
        }
        gt_run += __popc(bg);
        eq_run += __popc(be);
    }
    for (int p = K + tid; p < budget; p += NTH) out[p] = -1;
}

// ---------------------------------------------------------------- selection from the scoring kernel's histogram
// When the scoring kernel has already counted every competing page into 2048 value buckets of an
// a-priori range (|U_p| <= A sum_i |q_i| with A the head's largest |stored key|), the selection
// needs no pass for the range, no keys and no histogram of its own: the head's histogram and
// scores come into shared memory with two bulk copies (one round trip), the bucket b that holds
// the k_rem-th largest score and the rank k_in wanted inside it follow from suffix sums over the
// threads, pages of higher buckets go straight to the list, the pages of bucket b are ranked
// against each other by (score, lower page first) and the best k_in appended.  The list is in no
// particular order (the flash-decode kernel does not care; a caller that wants it gets it sorted by
// a kernel of its own).  Returns false, with nothing but forced pages written, when that cannot be
// done (bucket too full, counts that do not add up, copy that never came): select_rows then does
// the work.  Clears the histogram for the next step.
constexpr int kFastCandMax = 1024;

struct FastShared {                                  // dynamic shared memory of the selection kernel (register-key variants)
    alignas(16) uint32_t hist[kStepBins];
    uint32_t ckey[kFastCandMax];
    int32_t cpage[kFastCandMax];
    alignas(16) float sc[kTopkFastPages + 8];        // the head's scores from the 16-byte boundary below their start
};

__device__ __forceinline__ bool fast_select(FastShared &fs, SelectScratch &sh, uint64_t *bar, const float *sc, int P, int K,
                                            int ns, int nl, int32_t *out, int budget, uint32_t *ghist, float2 range,
                                            const char *kvh, int page_bytes, int n_prefetch)
{
    constexpr int NTH = kTopkThreads;
    constexpr unsigned FULL = 0xffffffffu;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int k_rem = K - ns - nl;
    const int p_lo = ns, p_hi = P - nl, n_forced = ns + nl;
    const int mis = (int)((reinterpret_cast<uintptr_t>(sc) >> 2) & 3);
    const float *src = sc - mis;
    const int nfl = (mis + P + 3) & ~3;
    if (tid == 0) {
        // (what the copies read was written by the kernel before this one: no fence between proxies is needed)
        mbar_arrive_expect_tx(bar, kStepBins * 4 + nfl * 4);
        bulk_g2s(fs.hist, ghist, kStepBins * 4, bar);
        bulk_g2s(fs.sc, src, nfl * 4, bar);
        sh.digit = 0xffffffffu; sh.krem = 0; sh.cnt = 0; sh.ncand = 0; sh.tau = 0;   // bucket, rank inside, its population; candidates; pages above
    }
    for (int p = tid; p < ns; p += NTH) out[p] = p;
    for (int i = tid; i < nl; i += NTH) out[ns + i] = P - nl + i;
    for (int p = K + tid; p < budget; p += NTH) out[p] = -1;
    const bool landed = mbar_wait(bar, 0);
    reinterpret_cast<uint2 *>(ghist)[tid] = make_uint2(0u, 0u);      // all zero again for the next step (the copy has read it)
    if (!__syncthreads_and(landed)) return false;
    if (k_rem <= 0) return true;

    // thread t owns bins 2t and 2t+1
    const uint2 h2 = reinterpret_cast<const uint2 *>(fs.hist)[tid];
    const int c0 = (int)h2.x, c1 = (int)h2.y;
    int suf = c0 + c1;                               // inclusive suffix sum over the lanes
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_down_sync(FULL, suf, off);
        if (lane + off < 32) suf += t;
    }
    if (lane == 0) sh.red[warp] = (uint32_t)suf;
    __syncthreads();
    const int wtot = (int)sh.red[lane];              // every warp scans the 32 warp totals on its own
    int wsuf = wtot;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_down_sync(FULL, wsuf, off);
        if (lane + off < 32) wsuf += t;
    }
    const int total = __shfl_sync(FULL, wsuf, 0);
    const int above = __shfl_sync(FULL, wsuf - wtot, warp);   // keys in higher warps' bins
    const int incl1 = above + suf - c0;              // keys in bins >= 2t+1
    const int excl1 = incl1 - c1;
    const int incl0 = incl1 + c0;
    if (total == p_hi - p_lo && k_rem <= total) {
        if (incl1 >= k_rem && excl1 < k_rem) { sh.digit = 2u * tid + 1u; sh.krem = (uint32_t)(k_rem - excl1); sh.cnt = (uint32_t)c1; }
        if (incl0 >= k_rem && incl1 < k_rem) { sh.digit = 2u * tid; sh.krem = (uint32_t)(k_rem - incl1); sh.cnt = (uint32_t)c0; }
    }
    __syncthreads();
    const int b = (int)sh.digit, k_in = (int)sh.krem, cnt_b = (int)sh.cnt;
    if (b < 0 || cnt_b > kFastCandMax) return false;

    // classify: thread t takes the 16-byte vectors t, t + 1024, ... (at most three)
    ScoreRange rg;
    rg.lo = range.x;
    rg.scale = range.y;
    constexpr int VMAX = (kTopkFastPages / 4 + 2 + NTH - 1) / NTH;
    uint32_t m_sure = 0, m_cand = 0;                 // bit 4 u + e
#pragma unroll
    for (int u = 0; u < VMAX; ++u) {
        const int fi = (u * NTH + tid) * 4;
        if (fi < nfl) {
            const float4 xv = *reinterpret_cast<const float4 *>(fs.sc + fi);
            const float xs[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int p = fi - mis + e;
                const int bk = rg.bucket(xs[e]);
                const bool in = p >= p_lo && p < p_hi;
                m_sure |= (uint32_t)(in && bk > b) << (4 * u + e);
                m_cand |= (uint32_t)(in && bk == b) << (4 * u + e);
            }
        }
    }
    // positions: scan inside the warp, then over the warp totals (32 warps on one shared-memory
    // atomic each would wait for one another)
    int ws = __popc(m_sure), wc = __popc(m_cand);
    int ps = ws, pc = wc;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t1 = __shfl_up_sync(FULL, ps, off), t2 = __shfl_up_sync(FULL, pc, off);
        if (lane >= off) { ps += t1; pc += t2; }
    }
    const int wsum = __shfl_sync(FULL, ps, 31), wcsum = __shfl_sync(FULL, pc, 31);
    ps -= ws;
    pc -= wc;
    if (lane == 0) { sh.red[warp] = (uint32_t)wsum; sh.red2[warp] = (uint32_t)wcsum; }
    __syncthreads();                                 // (the reads of red for the bucket are long done)
    {
        int a1 = (int)sh.red[lane], a2 = (int)sh.red2[lane];     // inclusive scans over the warps
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t1 = __shfl_up_sync(FULL, a1, off), t2 = __shfl_up_sync(FULL, a2, off);
            if (lane >= off) { a1 += t1; a2 += t2; }
        }
        ps += n_forced + __shfl_sync(FULL, a1, warp) - wsum;
        pc += __shfl_sync(FULL, a2, warp) - wcsum;
        const int all_s = __shfl_sync(FULL, a1, 31), all_c = __shfl_sync(FULL, a2, 31);
        if (tid == 0) { sh.tau = (uint32_t)all_s; sh.ncand = (uint32_t)all_c; }
    }
    while (m_sure) {
        const int i = __ffs(m_sure) - 1;
        m_sure &= m_sure - 1;
        const int p = ((i >> 2) * NTH + tid) * 4 - mis + (i & 3);
        if (ps < K) out[ps] = p;
        ++ps;
    }
    while (m_cand) {
        const int i = __ffs(m_cand) - 1;
        m_cand &= m_cand - 1;
        const int fi = ((i >> 2) * NTH + tid) * 4 + (i & 3);
        if (pc < kFastCandMax) { fs.ckey[pc] = order_key(fs.sc[fi]); fs.cpage[pc] = fi - mis; }
        ++pc;
    }
    __syncthreads();
    const int n_sure = (int)sh.tau, nc = (int)sh.ncand;
    if (n_sure != k_rem - k_in || nc != cnt_b) return false;         // scores and histogram disagree
    // rank of a candidate: how many candidates beat it (higher score, or equal score and lower page)
    // (a warp per candidate, the lanes share the comparisons)
    for (int j = warp; j < nc; j += NTH / 32) {
        const uint32_t kj = fs.ckey[j];
        const int pj = fs.cpage[j];
        int r = 0;
        for (int i = lane; i < nc; i += 32) {
            const uint32_t ki = fs.ckey[i];
            r += (ki > kj) || (ki == kj && fs.cpage[i] < pj);
        }
        r = __reduce_add_sync(FULL, r);
        if (lane == 0 && r < k_in) out[n_forced + n_sure + r] = pj;
    }
    // the pages the flash-decode kernel reads first are on their way into L2 before it starts: one
    // thread per page (issued by the few threads that happened to own the first ranks, the
    // prefetches held the whole CTA up for two microseconds)
    __syncthreads();
    if (tid < n_prefetch && tid < K) {
        const int p = out[tid];
        if (p >= 0 && p < P) bulk_prefetch_l2(kvh + (int64_t)p * page_bytes, (uint32_t)page_bytes);
    }
    return true;
}

// The selection kernel: one CTA per head.  SMEM_KEYS: the keys of a head (ROWS * 1024 words) live
// in dynamic shared memory.  The histogram is cleared before the wait for the scoring kernel.
template <int ROWS, bool SMEM_KEYS>
__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const float *scores, int64_t score_stride, int P, int K,
                                                            int n_sink, int n_local, int32_t *idx, int idx_stride,
                                                            int budget, int32_t *attend_ctr, const char *kv,
                                                            int64_t kv_head_bytes, int page_bytes, int n_prefetch,
                                                            uint32_t *ghist, const float2 *range)
{
    extern __shared__ __align__(16) uint32_t skey[];
    __shared__ SelectScratch sh;
    __shared__ __align__(8) uint64_t bar;
    const int bh = blockIdx.x;
    if (!SMEM_KEYS && ghist && threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_init_fence();
    }
    select_prepare(sh);
    grid_dependency_wait();          // the scores come from the kernel before; the one before that may still use the counters
    grid_launch_dependents();
    if (threadIdx.x < 4) attend_ctr[bh * kCtrStride + threadIdx.x] = 0;   // this head's ticket counters of the streaming kernels
    if constexpr (!SMEM_KEYS) {
        if (ghist && K < P) {
            __syncthreads();                         // the barrier is initialised
            FastShared &fs = *reinterpret_cast<FastShared *>(skey);
            if (fast_select(fs, sh, &bar, scores + (int64_t)bh * score_stride, P, K, n_sink, n_local,
                            idx + (int64_t)bh * idx_stride, budget, ghist + (int64_t)bh * kStepBins, range[bh],
                            kv + (int64_t)bh * kv_head_bytes, page_bytes, n_prefetch))
                return;
            __syncthreads();
            select_prepare(sh);                      // the scratch was used otherwise
            __syncthreads();
        }
    }
    select_rows<ROWS, SMEM_KEYS>(sh, skey, scores + (int64_t)bh * score_stride, P, K, n_sink, n_local,
                                 idx + (int64_t)bh * idx_stride, budget, kv + (int64_t)bh * kv_head_bytes, page_bytes,
                                 n_prefetch);
}


// ---------------------------------------------------------------- short contexts: append, score and select in one launch
// When a head has so few pages that a step is three launch latencies rather than memory traffic, one
// CTA per head does the first two kernels' work back to back: the single-token update (Eq. 1), the
// score of every page (Eq. 3; a record per group of lanes, read straight from global memory) and the
// selection, with the scores passing through the scores buffer.  The flash-decode kernel follows as usual.
template <typename T, int D, int ROWS>
__global__ void __launch_bounds__(kTopkThreads) score_select_kernel(DecodeArgs a, const T *q, const T *k_t, const T *v_t,
                                                                    const void *g_t, float *scores, int do_update, int K,
                                                                    int n_sink, int n_local, int32_t *idx, int idx_stride,
                                                                    int budget, int32_t *attend_ctr, int64_t kv_head_bytes,
                                                                    int page_bytes, int n_prefetch, int32_t *ctr_other)
{
    using G = ScoreGeom<T, D>;
    constexpr unsigned FULL = 0xffffffffu;
    __shared__ SelectScratch sh;
    __shared__ float red[32];
    const int bh = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int P = (int)((a.len + a.S - 1) / a.S);
    select_prepare(sh);
    grid_dependency_wait();          // earlier kernels may still read what the update rewrites
    grid_launch_dependents();
    if (tid < 4) attend_ctr[bh * kCtrStride + tid] = 0;   // this head's ticket counters of the flash-decode kernel
    if (do_update) {
        update_head<T, D>(a, bh, q, k_t, v_t, g_t, scores, red);   // also scores the newest page
        // the one-launch step's counters of the next step (it may be the next to run on this cache)
        if (ctr_other && tid < kStepCtrInts) ctr_other[bh * kStepCtrInts + tid] = 0;
    }

    const int Ps = do_update ? P - 1 : P;            // pages whose records are read here
    float qs[G::VPL][G::CH];
    score_load_q<T, D>(q, bh, lane, qs);
    const unsigned char *meta = static_cast<const unsigned char *>(a.meta) + (int64_t)bh * a.page_cap * G::REC_BYTES;
    float *sc = scores + (int64_t)bh * a.page_cap;
    const int sub = lane / G::LPP, c = lane % G::LPP;
    constexpr int U = 4;                             // records a lane group has in flight
    constexpr int STEP = (kTopkThreads / 32) * G::PPW;   // records the CTA covers with one warp-wide read per warp
    // (the loop bound is the same for every lane of a warp: the shuffles below need all of them)
    for (int rb = warp * G::PPW; rb < Ps; rb += U * STEP) {
        const int r0 = rb + sub;
        uint4 raw[U][G::VPL];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int rec = r0 + u * STEP;
#pragma unroll
            for (int v = 0; v < G::VPL; ++v)
                raw[u][v] = rec < Ps ? ldcs16(meta + (int64_t)rec * G::REC_BYTES + (c + v * G::LPP) * 16) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int rec = r0 + u * STEP;
            float s = 0.0f;
#pragma unroll
            for (int v = 0; v < G::VPL; ++v) {
                float m[G::CH];
                unpack16<T>(raw[u][v], m);
#pragma unroll
                for (int i = 0; i < G::CH; ++i) s = fmaf(qs[v][i], m[i], s);
            }
#pragma unroll
            for (int off = G::LPP / 2; off > 0; off >>= 1) s += __shfl_xor_sync(FULL, s, off);
            if (c == 0 && rec < Ps) sc[rec] = s;
        }
    }
    __syncthreads();                 // the head's scores are in the scores buffer
    // (a head has at most kSmallStepPages = 256 pages here, so no bucket can hold more than kCandMax keys:
    // the radix passes are reached only through a degenerate score range)
    select_rows<ROWS, false>(sh, nullptr, sc, P, K, n_sink, n_local, idx + (int64_t)bh * idx_stride, budget,
                             static_cast<const char *>(a.kv) + (int64_t)bh * kv_head_bytes, page_bytes, n_prefetch);
}

}  // namespace

bool topk_uses_hist(int64_t pages) { return pages >= kTopkHistMinPages && pages <= kTopkFastPages; }

cudaError_t launch_topk(const DecodeArgs &a, const float *scores, int budget, int32_t *idx,
                        int idx_stride, int32_t *attend_ctr, int prefetch, const ScoreHist &hs, cudaStream_t s)
{
    const int P = (int)((a.len + a.S - 1) / a.S);
    const int K = budget < P ? budget : P;
    const int BH = a.B * a.H;
    // forced pages inside the budget: sinks first, then local pages from the newest backwards
    int ns = a.n_sink < K ? a.n_sink : K;
    if (ns > P) ns = P;
    int nl = a.n_local < K - ns ? a.n_local : K - ns;
    if (nl > P - ns) nl = P - ns;
    if (P > kTopkThreads * kTopkMaxPerThread) return cudaErrorInvalidValue;
    using Kernel = void (*)(const float *, int64_t, int, int, int, int, int32_t *, int, int, int32_t *, const char *, int64_t,
                            int, int, uint32_t *, const float2 *);
    // the keys of a large head live in dynamic shared memory: allow it once per device
    constexpr int kMidRows = 16, kBigRows = kTopkMaxPerThread;
    constexpr int kMidSmem = kMidRows * kTopkThreads * (int)sizeof(uint32_t);
    constexpr int kBigSmem = kBigRows * kTopkThreads * (int)sizeof(uint32_t);
    static bool ready[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!ready[dev]) {
        const Kernel regs[5] = {topk_kernel<2, false>, topk_kernel<4, false>, topk_kernel<6, false>, topk_kernel<8, false>,
                                topk_kernel<10, false>};
        for (int i = 0; i < 5; ++i) {
            e = cudaFuncSetAttribute(regs[i], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(FastShared));
            if (e != cudaSuccess) return e;
        }
        e = cudaFuncSetAttribute(topk_kernel<kMidRows, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMidSmem);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(topk_kernel<kBigRows, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kBigSmem);
        if (e != cudaSuccess) return e;
        ready[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)BH);
    cfg.blockDim = dim3(kTopkThreads);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int64_t stride = a.page_cap;
    // pages per head whose keys and values the selection starts moving into L2 for the kernel after it
    // (the first ones of the list, which that kernel's warps read first): up to kTopkPrefetchBytes in all
    // and an eighth of a head's list
    const int es = a.dtype == RQ_BF16 ? 2 : 4;
    const int page_bytes = 2 * a.S * a.D * es;
    const int64_t kv_head_bytes = a.page_cap * (int64_t)page_bytes;
    const char *kv = static_cast<const char *>(a.kv);
    int n_prefetch = prefetch ? (int)(kTopkPrefetchBytes / BH / page_bytes) : 0;
    if (n_prefetch > K / 8) n_prefetch = K / 8;      // the head of the list only: the kernel waits for its prefetches
    const int rows = (P + kTopkThreads - 1) / kTopkThreads;
    uint32_t *ghist = hs.hist && topk_uses_hist(P) ? hs.hist : nullptr;
    Kernel kern;
    if (rows <= 10) {                                // the keys of a head fit in registers (more rows would spill)
        static const Kernel by_rows[5] = {topk_kernel<2, false>, topk_kernel<4, false>, topk_kernel<6, false>,
                                          topk_kernel<8, false>, topk_kernel<10, false>};
        kern = by_rows[(rows - 1) / 2];
        cfg.dynamicSmemBytes = ghist ? sizeof(FastShared) : 0;
    } else if (rows <= kMidRows) {
        kern = topk_kernel<kMidRows, true>;
        cfg.dynamicSmemBytes = kMidSmem;
    } else {
        kern = topk_kernel<kBigRows, true>;
        cfg.dynamicSmemBytes = kBigSmem;
    }
    return cudaLaunchKernelEx(&cfg, kern, scores, stride, P, K, ns, nl, idx, idx_stride, budget, attend_ctr, kv,
                              kv_head_bytes, page_bytes, n_prefetch, ghist, hs.range);
}

cudaError_t launch_score_select(const DecodeArgs &a, const void *q, const void *k_t, const void *v_t, const void *g_t,
                                float *scores, int do_update, int budget, int32_t *idx, int idx_stride,
                                int32_t *attend_ctr, int prefetch, int32_t *ctr_other, cudaStream_t s)
{
    const int P = (int)((a.len + a.S - 1) / a.S);
    const int K = budget < P ? budget : P;
    const int BH = a.B * a.H;
    int ns = a.n_sink < K ? a.n_sink : K;
    if (ns > P) ns = P;
    int nl = a.n_local < K - ns ? a.n_local : K - ns;
    if (nl > P - ns) nl = P - ns;
    if (P > kSmallStepPages) return cudaErrorInvalidValue;
    const int es = a.dtype == RQ_BF16 ? 2 : 4;
    const int page_bytes = 2 * a.S * a.D * es;
    const int64_t kv_head_bytes = a.page_cap * (int64_t)page_bytes;
    int n_prefetch = prefetch ? (int)(kTopkPrefetchBytes / BH / page_bytes) : 0;
    if (n_prefetch > K / 8) n_prefetch = K / 8;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)BH);
    cfg.blockDim = dim3(kTopkThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    constexpr int ROWS = 2;
    static_assert(kSmallStepPages <= ROWS * kTopkThreads, "the fused kernel keeps a head's keys in two rows");
#define RQ_LAUNCH_SMALL(T, D)                                                                                          \
    return cudaLaunchKernelEx(&cfg, score_select_kernel<T, D, ROWS>, a, (const T *)q, (const T *)k_t, (const T *)v_t,  \
                              g_t, scores, do_update, K, ns, nl, idx, idx_stride, budget, attend_ctr, kv_head_bytes,   \
                              page_bytes, n_prefetch, ctr_other)
    if (a.dtype == RQ_BF16) {
        if (a.D == 128) RQ_LAUNCH_SMALL(bf16, 128);
        if (a.D == 64) RQ_LAUNCH_SMALL(bf16, 64);
    } else {
        if (a.D == 128) RQ_LAUNCH_SMALL(float, 128);
        if (a.D == 64) RQ_LAUNCH_SMALL(float, 64);
    }
#undef RQ_LAUNCH_SMALL
    return cudaErrorInvalidValue;
}

}  // namespace rq
