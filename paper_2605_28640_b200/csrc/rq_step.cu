// The whole decode step in ONE launch: single-token update (Eq. 1), page scoring and per-head
// selection (Eq. 3 with the min/max representatives of App. A.1), sparse flash-decode over the
// selected pages and the combine (Eq. 4).
//
// Why one launch.  As three kernels the selection is serial time: one SM per head ranks the
// scores while HBM carries nothing, and every kernel boundary drains and refills the memory
// pipeline.  Here the heads are split into `waves` groups and every warp of the grid walks the
// same list of phases without ever draining its copy pipeline:
//
//     score(wave 0), score(wave 1), ..., attend(wave 0), attend(wave 1), ...
//
// A few extra CTAs at the end of the grid stream nothing: each of their warps looks after one head
// (more if there are more heads than such warps), polls the head's count of scored units and, once
// the head is complete, selects its pages while everybody else streams the next phases; by the
// time the streaming warps reach attend(wave w) the lists of wave w have been published, so the
// selection costs no time in which the memory system idles.  A streaming warp that does arrive early
// finds a wait mark in its pipeline and polls the head's flag.  (The selection is a chain of a few
// dependent round trips to L2, each of which takes several microseconds while 28 MB of copies are
// in flight; done by a streaming warp it would hold that warp's tickets back for that long, and with
// them the completion of the heads it serves next.)
//
// Work distribution inside a phase is that of the separate kernels: CTA c serves head
// wave * HW + c % HW (HW heads per wave, team = grid / HW CTAs per head); a head's units (8 KiB
// of page records when scoring, a 16-row tile of keys and values when attending) are handed out by
// a per-head ticket counter, the first two tickets of a warp being its own by position; every
// warp owns a ring of shared-memory stages filled by 1-D bulk copies (TMA, completion on an
// mbarrier).  Ticket, page index and the readiness of the next phase's list are fetched one
// refill ahead, so the issuing lane waits for none of them.
//
// Selection without a pass for the range.  The separate selection kernel first reads all scores
// to find their range.  Here the histogram is filled WHILE scoring: |U_p| <= R = A * sum_i |q_i|
// with A the head's largest |stored key| (kept up to date by the prefill and by the update), so
// 2048 value buckets over [-R, R] are fixed before the first score exists and every scoring warp
// adds its pages to the head's histogram in global memory (one `red` per page).  The selecting
// warp reads the histogram, finds the bucket that holds the threshold, and makes ONE pass over the
// head's scores: pages of higher buckets go to the list at once, the (few dozen) pages of the
// threshold bucket are ranked against each other by (score, lower page first).  The bucket map is
// monotone whatever R is, so a loose or stale R costs resolution, never correctness: a threshold
// bucket too full to rank directly (or a histogram that does not add up) is resolved by
// most-significant-digit radix passes on the key bits and one ordered pass that takes equal keys
// lowest page first.  The list is written in no particular order (attention does not care);
// when the caller wants it, a small kernel afterwards sorts it.
//
// Every wait in this kernel is bounded: copy barriers as in the other kernels, polls of flags and
// counters by kFlagPollLimit; a wait that runs out sets RQ_ERR_TIMEOUT in the status word,
// the warp stops taking work, lets its copies in flight land and still walks through the marks of
// all phases, so that the CTA's barriers are all reached and the kernel ends.
#include <limits.h>
#include <math.h>
#include <math_constants.h>

#include "rq_async.cuh"
#include "rq_device.cuh"
#include "rq_internal.h"
#include "rq_stream.cuh"

namespace rq {

namespace {

constexpr int kStepWarps = 4;                  // warps per CTA, each with its own copy pipeline
constexpr int kStepRingBytes = 64 * 1024;      // ring of one CTA: three CTAs per SM
constexpr int kStepCandMax = 256;              // pages of the threshold bucket that one warp ranks directly
constexpr int kStepOwn = 2;                    // tickets of a phase that a warp owns by position
constexpr int kStepPollLimit = 1 << 20;        // polls (a round trip to L2 each) after which a selecting CTA stops waiting for its head
// marks in the first word of a stage's descriptor
constexpr int kMarkEnd = -1, kMarkEndPhase = -2, kMarkWait = -3;
// per-head counters (int32 offsets inside a head's block of kStepCtrInts)
constexpr int kCtrScoreNext = 0, kCtrScoreDone = 1, kCtrAttendNext = 2, kCtrAttendDone = 3;

template <typename T, int D, int S>
struct StepGeom {
    using SG = ScoreGeom<T, D>;
    using AG = AttendGeom<T, D, S>;
    static constexpr int NW = kStepWarps;
    static constexpr int STAGE = AG::STAGE_BYTES > kUnitBytes ? AG::STAGE_BYTES : kUnitBytes;
    static constexpr int DEPTH_RAW = kStepRingBytes / (NW * STAGE);
    static constexpr int DEPTH = DEPTH_RAW < 1 ? 1 : (DEPTH_RAW > 8 ? 8 : DEPTH_RAW);
    static constexpr int RING_BYTES = NW * DEPTH * STAGE;
    static constexpr int OFF_BARS = RING_BYTES;                              // uint64 [NW][DEPTH]
    static constexpr int OFF_INFO = OFF_BARS + NW * DEPTH * 8;               // int4   [NW][DEPTH]
    static constexpr int OFF_SLOT = OFF_INFO + NW * DEPTH * 16;              // float4 [2][NW] (m, l, tiles, dead)
    static constexpr int OFF_ACC = OFF_SLOT + 2 * NW * 16;                   // float  [2][NW][D]
    static constexpr int OFF_MISC = OFF_ACC + 2 * NW * D * 4;                // 16 floats of reduction scratch
    static constexpr int SMEM_BYTES = OFF_MISC + 64;
    // a selecting CTA (it streams nothing) keeps its scratch where its ring would be
    static_assert(SG::RU * SG::REC_BYTES == kUnitBytes, "a scoring unit is 8 KiB of records");
};

// ---------------------------------------------------------------- selection by one warp
struct SelectArgs {
    const float *sc;        // the head's scores [P]
    int P, K, ns, nl;       // pages, budget (< P), forced first / newest pages (ns + nl <= K)
    ScoreRange rg;          // the bucket map the histogram was filled with
    uint32_t *hist;         // the head's histogram [kStepBins]; cleared here
    int2 *out;              // the head's list [K]: (page, number of this step)
    int epoch;              // number of this step: tags every entry, so that a reader can tell a new entry from an old one
    uint32_t *ckey;         // shared memory, 256 words: select_slow's digit histogram
};

__device__ __forceinline__ uint32_t score_key(float x) { return order_key(x); }

// exclusive prefix sum over the lanes and the total
__device__ __forceinline__ int warp_excl_scan(int v, int lane, int &total)
{
    int inc = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += t;
    }
    total = __shfl_sync(0xffffffffu, inc, 31);
    return inc - v;
}

// One pass over the head's scores, four consecutive pages per lane and load, U loads in flight
// per lane (a round trip to L2 takes microseconds while the streams run, so as many as the
// registers hold): fn(first page of the four, their scores).  Rows come in ascending page order,
// and inside a row lane l holds pages before lane l + 1.  The row need not start on a 16-byte
// boundary: the pass starts at the boundary below and fn sees page numbers < 0 there.
template <int U, typename F>
__device__ __forceinline__ void for_scores(const float *sc, int P, int lane, F fn)
{
    const int mis = (int)((reinterpret_cast<uintptr_t>(sc) >> 2) & 3);
    const float4 *vb = reinterpret_cast<const float4 *>(sc - mis);
    const int nvec = (mis + P + 3) >> 2;
#pragma unroll 1
    for (int v0 = 0; v0 < nvec; v0 += 32 * U) {
        float4 x[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int vi = v0 + u * 32 + lane;
            x[u] = vi < nvec ? __ldcg(vb + vi) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (v0 + u * 32 >= nvec) break;              // warp-uniform
            const int vi = v0 + u * 32 + lane;
            fn(vi < nvec ? vi * 4 - mis : INT_MIN / 2, x[u]);
        }
    }
}

// The selection of one head by a whole CTA (kStepWarps warps) that streams nothing.  The head's
// histogram (8 KiB) and its scores (at most kSelectPages of them, 48 KiB; longer heads do not take
// the one-launch step) are brought into shared memory by two bulk copies (TMA), which arrive after
// ONE round trip to L2; the same bytes fetched with ordinary loads trickle in over ten
// microseconds, because an SM keeps only so many loads in flight.  Then: the
// bucket b that holds the k_rem-th largest score and the rank k_in wanted inside it (suffix sums
// over the threads); pages of higher buckets are appended to the list, pages of bucket b collected
// in shared memory (positions reserved with one shared-memory atomic per warp, so the list is in
// no particular order); the collected pages are ranked against each other by (score, lower page
// first) and the best k_in appended.  Returns false if that could not be done (bucket too full,
// counts that do not add up, a copy that never came): the caller then runs select_slow.
constexpr int kSelectPages = 12288;                  // pages whose scores fit in the selecting CTA's shared memory (48 KiB)
struct SelectShared {
    alignas(16) uint32_t hist[kStepBins];            // the head's histogram
    alignas(16) float sc[kSelectPages];              // the head's scores (from the 16-byte boundary below their start)
    uint32_t ckey[kStepCandMax];                     // candidates: keys (doubles as select_slow's digit histogram)
    int32_t cpage[kStepCandMax];                     //             pages
    int wtot[kStepWarps];                            // per-warp histogram totals
    int ok, b, k_in, cnt_b, n_sure, n_cand;
};
static_assert(sizeof(SelectShared) <= kStepRingBytes, "a selecting CTA keeps this where a streaming CTA has its ring");

// What the classification of the scores needs besides the scores themselves.
struct ClassifyCtx {
    int b, K, n_forced, p_lo, p_hi, mis, nfl, epoch;
    ScoreRange rg;
    int2 *out;
};

// All scores of the head (c.nfl floats of sh.sc): pages of buckets above b go to the list, pages of
// bucket b to the candidates.  A thread first only marks and counts its pages of either kind (32
// pages to a mask word), the warp's counts are summed and ONE shared-memory atomic per warp and
// kind reserves the positions.  No loop over parts of the head with a run-time trip count: such a
// loop around this body (with or without a barrier in it) made every warp of the CTA lose four
// microseconds on the way in, for reasons that the source does not show.
__device__ __forceinline__ void classify_scores(const ClassifyCtx &c, SelectShared &sh)
{
    constexpr unsigned FULL = 0xffffffffu;
    constexpr int NT = kStepWarps * 32;
    constexpr int VPT = kSelectPages / 4 / NT;       // 16-byte vectors of scores per thread
    constexpr int G = VPT / 8;                       // mask words per thread and kind: 8 vectors = 32 pages each
    static_assert(VPT % 8 == 0, "whole mask words");
    const int tid = threadIdx.x, lane = tid & 31;
    uint32_t m_sure[G], m_cand[G];                   // word g, bit 4 u + e: page e of vector 8 g + u
    int n_s = 0, n_c = 0;
#pragma unroll
    for (int g = 0; g < G; ++g) {
        uint32_t ws = 0, wc = 0;
#pragma unroll 1
        for (int u = 0; u < 8; ++u) {
            const int fi = ((g * 8 + u) * NT + tid) * 4;     // float index
            const bool have = fi < c.nfl;
            const float4 xv = have ? *reinterpret_cast<const float4 *>(sh.sc + fi) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            const float xs[4] = {xv.x, xv.y, xv.z, xv.w};
            const int p0 = have ? fi - c.mis : INT_MIN / 2;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int bk = c.rg.bucket(xs[e]);
                const bool in = p0 + e >= c.p_lo && p0 + e < c.p_hi;
                ws |= (uint32_t)(in && bk > c.b) << (4 * u + e);
                wc |= (uint32_t)(in && bk == c.b) << (4 * u + e);
            }
        }
        m_sure[g] = ws;
        m_cand[g] = wc;
        n_s += __popc(ws);
        n_c += __popc(wc);
    }
    int ws, wc;
    int ps = warp_excl_scan(n_s, lane, ws), pc = warp_excl_scan(n_c, lane, wc);
    int bs = 0, bc = 0;
    if (lane == 0) {
        bs = ws ? atomicAdd(&sh.n_sure, ws) : 0;
        bc = wc ? atomicAdd(&sh.n_cand, wc) : 0;
    }
    ps += c.n_forced + __shfl_sync(FULL, bs, 0);
    pc += __shfl_sync(FULL, bc, 0);
#pragma unroll
    for (int g = 0; g < G; ++g) {
        uint32_t m = m_sure[g];
        while (m) {
            const int i = __ffs(m) - 1;
            m &= m - 1;
            if (ps < c.K) c.out[ps] = make_int2(((g * 8 + (i >> 2)) * NT + tid) * 4 - c.mis + (i & 3), c.epoch);
            ++ps;
        }
        m = m_cand[g];
        while (m) {
            const int i = __ffs(m) - 1;
            m &= m - 1;
            const int fi = ((g * 8 + (i >> 2)) * NT + tid) * 4 + (i & 3);
            if (pc < kStepCandMax) { sh.ckey[pc] = score_key(sh.sc[fi]); sh.cpage[pc] = fi - c.mis; }
            ++pc;
        }
    }
}

// bar: an initialised mbarrier of this CTA (one arrival per phase), parity: its next phase; both owned by the caller
__device__ __forceinline__ bool select_head(const SelectArgs &s, SelectShared &sh, uint64_t *bar, uint32_t &parity, int &b_out,
                                            int &k_out)
{
    constexpr int NT = kStepWarps * 32;
    constexpr int BPT = kStepBins / NT;              // bins per thread
    static_assert(BPT % 4 == 0, "bins are read 16 bytes at a time");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int k_rem = s.K - s.ns - s.nl;             // budget left for pages that are not forced
    const int p_lo = s.ns, p_hi = s.P - s.nl;        // pages in [p_lo, p_hi) compete
    const int n_forced = s.ns + s.nl;

    // requests first: the histogram and the head's scores
    const int mis = (int)((reinterpret_cast<uintptr_t>(s.sc) >> 2) & 3);   // the row may start off a 16-byte boundary
    const float *src = s.sc - mis;                   // 16-byte aligned; the bytes before the row belong to the row before
    const int nfl = (mis + s.P + 3) & ~3;            // floats from src that cover the row, a multiple of four
    if (tid == 0) {
        // what the copies read was written with ordinary stores and atomics by other SMs
        asm volatile("fence.proxy.async;" ::: "memory");
        const uint32_t bytes = kStepBins * 4 + nfl * 4;           // nfl <= kSelectPages: the host checks the head's size
        mbar_arrive_expect_tx(bar, bytes);
        bulk_g2s(sh.hist, s.hist, kStepBins * 4, bar);
        bulk_g2s(sh.sc, src, nfl * 4, bar);
        sh.b = -1; sh.k_in = 0; sh.cnt_b = 0; sh.n_sure = 0; sh.n_cand = 0;
    }
    // forced pages
    for (int p = tid; p < s.ns; p += NT) s.out[p] = make_int2(p, s.epoch);
    for (int i = tid; i < s.nl; i += NT) s.out[s.ns + i] = make_int2(s.P - s.nl + i, s.epoch);
    b_out = -1;
    k_out = k_rem;
    bool landed = mbar_wait(bar, parity);
    parity ^= 1u;
    // (the histogram is cleared for the next step by the caller, when the list is out: a burst of
    // stores here would sit in the memory pipeline in front of everything that follows)
    if (!__syncthreads_and(landed)) return false;    // (also: thread 0's writes of the shared state are visible)
    if (k_rem <= 0) return true;                     // nothing but forced pages fits

    // bucket of the k_rem-th largest score: thread t owns bins BPT t .. BPT t + BPT - 1
    uint32_t c[BPT];
#pragma unroll
    for (int i = 0; i < BPT / 4; ++i) {              // (16 bins per thread: small enough to stay unrolled)
        const uint4 v = reinterpret_cast<const uint4 *>(sh.hist)[tid * (BPT / 4) + i];
        c[4 * i] = v.x; c[4 * i + 1] = v.y; c[4 * i + 2] = v.z; c[4 * i + 3] = v.w;
    }
    int tot = 0;
#pragma unroll
    for (int j = 0; j < BPT; ++j) tot += (int)c[j];
    int wtotal;
    const int below_w = warp_excl_scan(tot, lane, wtotal);       // keys in lower lanes' bins of this warp
    if (lane == 31) sh.wtot[warp] = wtotal;
    __syncthreads();
    int total = 0, above = 0;
#pragma unroll
    for (int w = 0; w < kStepWarps; ++w) {
        total += sh.wtot[w];
        above += w > warp ? sh.wtot[w] : 0;
    }
    above += wtotal - below_w - tot;                 // keys in bins above this thread's
    if (total == p_hi - p_lo && k_rem <= total) {
        const int need = k_rem - above;
        if (need > 0 && need <= tot) {               // exactly one thread
            int acc = 0, bl = -1;
#pragma unroll
            for (int j = BPT - 1; j >= 0; --j) {
                if (bl < 0) {
                    acc += (int)c[j];
                    if (acc >= need) { bl = BPT * tid + j; sh.k_in = need - (acc - (int)c[j]); sh.cnt_b = (int)c[j]; }
                }
            }
            sh.b = bl;
        }
    }
    __syncthreads();
    const int b = sh.b, k_in = sh.k_in, cnt_b = sh.cnt_b;
    if (b < 0) return false;                         // the histogram does not add up
    b_out = b;
    k_out = k_in;
    if (cnt_b > kStepCandMax) return false;          // too many pages share the threshold bucket

    ClassifyCtx cc;
    cc.b = b; cc.K = s.K; cc.n_forced = n_forced; cc.p_lo = p_lo; cc.p_hi = p_hi; cc.mis = mis; cc.nfl = nfl; cc.epoch = s.epoch;
    cc.rg = s.rg;
    cc.out = s.out;
    classify_scores(cc, sh);
    __syncthreads();
    const int n_sure = sh.n_sure, nc = sh.n_cand;
    if (n_sure != k_rem - k_in || nc != cnt_b) return false;     // scores and histogram disagree
    // rank of a candidate: how many candidates beat it (higher score, or equal score and lower page)
    for (int j = tid; j < nc; j += NT) {
        const uint32_t kj = sh.ckey[j];
        const int pj = sh.cpage[j];
        int r = 0;
#pragma unroll 4
        for (int i = 0; i < nc; ++i) {
            const uint32_t ki = sh.ckey[i];
            r += (ki > kj) || (ki == kj && sh.cpage[i] < pj);
        }
        if (r < k_in) s.out[n_forced + n_sure + r] = make_int2(pj, s.epoch);
    }
    return true;
}

// The selection when the threshold bucket cannot be ranked directly (many equal scores, a degenerate
// score range) or the histogram does not add up: by ONE warp, slowly.  The threshold key is found by
// most-significant-digit radix passes over the key bits (of the pages of bucket b if use_b, of all
// competing pages otherwise; k of them are wanted), then one pass in ascending page order takes the
// pages above it and, lowest pages first, as many pages equal to it as are still wanted.  Writes
// the whole list except the forced pages.
__device__ __noinline__ void select_slow(const SelectArgs s, bool use_b, int b, int k)
{
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int p_lo = s.ns, p_hi = s.P - s.nl;        // pages in [p_lo, p_hi) compete
    const int n_forced = s.ns + s.nl;
    auto competes = [&](int p) { return p >= p_lo && p < p_hi; };
    auto filtered = [&](int p, float x) { return competes(p) && (!use_b || s.rg.bucket(x) == b); };
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    for_scores<16>(s.sc, s.P, lane, [&](int p0, const float4 &x) {
        const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (filtered(p0 + e, xs[e])) {
                const uint32_t kx = score_key(xs[e]);
                kmin = min(kmin, kx);
                kmax = max(kmax, kx);
            }
    });
    kmin = __reduce_min_sync(FULL, kmin);
    kmax = __reduce_max_sync(FULL, kmax);
    uint32_t tau = kmin;
    int r_eq = k;                                // keys equal to tau that are taken (lowest pages first)
    if (kmin != kmax) {
        int hb = 31 - __clz(kmin ^ kmax);        // highest bit in which the keys differ
        uint32_t t = hb == 31 ? 0u : (kmax >> (hb + 1)) << (hb + 1);
        uint32_t *dh = s.ckey;                   // 256 bins
        bool whole = false;
#pragma unroll 1
        while (hb >= 0 && !whole) {
            const int lo = hb >= 7 ? hb - 7 : 0; // this pass decides bits hb .. lo
            const uint32_t dmask = (1u << (hb - lo + 1)) - 1u;
            const uint32_t himask = hb == 31 ? 0u : ~0u << (hb + 1);
#pragma unroll
            for (int i = 0; i < 8; ++i) dh[lane * 8 + i] = 0u;
            __syncwarp();
            for_scores<16>(s.sc, s.P, lane, [&](int p0, const float4 &x) {
                const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (filtered(p0 + e, xs[e])) {
                        const uint32_t kx = score_key(xs[e]);
                        if ((kx & himask) == (t & himask)) atomicAdd(&dh[(kx >> lo) & dmask], 1u);
                    }
            });
            __syncwarp();
            int c8[8], t8 = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { c8[i] = (int)dh[lane * 8 + i]; t8 += c8[i]; }
            int all;
            const int lower = warp_excl_scan(t8, lane, all);
            const int need = k - (all - lower - t8);
            int dl = -1, kl = 0, cl = 0;
            if (need > 0 && need <= t8) {
                int acc = 0;
#pragma unroll
                for (int i = 7; i >= 0; --i) {
                    if (dl < 0) {
                        acc += c8[i];
                        if (acc >= need) { dl = lane * 8 + i; kl = need - (acc - c8[i]); cl = c8[i]; }
                    }
                }
            }
            const unsigned owner = __ballot_sync(FULL, dl >= 0);
            if (!owner) break;                   // cannot happen: k keys exist among the filtered ones
            const int src = __ffs(owner) - 1;
            const int digit = __shfl_sync(FULL, dl, src);
            k = __shfl_sync(FULL, kl, src);
            const int cnt = __shfl_sync(FULL, cl, src);
            t |= (uint32_t)digit << lo;
            whole = cnt == k;                    // the whole bin is wanted
            hb = lo - 1;
            __syncwarp();
        }
        // a bin wanted whole: its lowest possible key, raised to the smallest filtered key so that
        // no page outside the filtered set reaches it; every key equal to it is wanted
        tau = whole ? max(t, kmin) : t;
        r_eq = whole ? INT_MAX : k;
    }
    int n = n_forced, eq_run = 0;
    for_scores<16>(s.sc, s.P, lane, [&](int p0, const float4 &x) {
        const float xs[4] = {x.x, x.y, x.z, x.w};
        bool gt[4], eq[4];
        int ce = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const bool in = competes(p0 + e);
            const uint32_t kx = score_key(xs[e]);
            gt[e] = in && kx > tau;
            eq[e] = in && kx == tau;
            ce += eq[e];
        }
        int row_eq;
        int pe = eq_run + warp_excl_scan(ce, lane, row_eq);   // equal keys on lower pages
        bool take[4];
        int ct = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            take[e] = gt[e] || (eq[e] && pe < r_eq);
            pe += eq[e];
            ct += take[e];
        }
        int row_take;
        int pos = n + warp_excl_scan(ct, lane, row_take);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (take[e]) {
                if (pos < s.K) s.out[pos] = make_int2(p0 + e, s.epoch);
                ++pos;
            }
        }
        n += row_take;
        eq_run += row_eq;
    });
    __syncwarp();
}

// ---------------------------------------------------------------- the kernel
template <typename T, int D, int S>
__global__ void __launch_bounds__(kStepWarps * 32, 3) step_kernel(DecodeArgs a, const T *q, const T *k_t, const T *v_t,
                                                                 const void *g_t, int K, float scale_log2,
                                                                 StepBuffers b, T *o, int waves, int stream_ctas)
{
    using G = StepGeom<T, D, S>;
    using SG = typename G::SG;
    using AG = typename G::AG;
    constexpr int NW = G::NW, DEPTH = G::DEPTH, STAGE = G::STAGE;
    constexpr int RU = SG::RU, TPP = AG::TPP, TR = AG::TR, CH = AG::CH, LPR = AG::LPR;
    constexpr unsigned FULL = 0xffffffffu;

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + G::OFF_BARS);
    int4 *infos = reinterpret_cast<int4 *>(smem + G::OFF_INFO);     // x: head or mark, w: phase; y, z: see start_copy
    float4 *sm_slot = reinterpret_cast<float4 *>(smem + G::OFF_SLOT);
    float *sm_acc = reinterpret_cast<float *>(smem + G::OFF_ACC);
    float *red = reinterpret_cast<float *>(smem + G::OFF_MISC);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int BH = a.B * a.H;
    const int P = (int)((a.len + S - 1) / S);
    const int Ps = P - 1;                            // records that are streamed (the newest page is scored by the update)
    const int HW = BH / waves;                       // heads per wave
    const int team = stream_ctas / HW;               // streaming CTAs per head
    const int rank = blockIdx.x / HW, member = blockIdx.x % HW;
    const int NPH = 2 * waves;
    const int u_per = (Ps + RU - 1) / RU;            // scoring units per head
    const int s_total = u_per + 1;                   // arrivals that complete a head's scoring: its units + the update
    const int t_per = K * TPP;                       // tiles per head
    const int cur = a.epoch & 1;
    int32_t *ctr = b.ctr + (int64_t)cur * BH * kStepCtrInts;
    const int poll_limit = a.poll_limit == 0 ? kMbarPollLimit : (a.poll_limit < 0 ? 0 : a.poll_limit);
    // forced pages inside the budget: sinks first, then local pages from the newest backwards
    int n_sink = a.n_sink < K ? a.n_sink : K;
    int n_local = a.n_local < K - n_sink ? a.n_local : K - n_sink;

    const uint64_t stream_policy = l2_evict_first_policy();
    uint64_t *mybars = bars + warp * DEPTH;
    int4 *myinfo = infos + warp * DEPTH;
    unsigned char *myring = smem + (size_t)warp * DEPTH * STAGE;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < DEPTH; ++s) mbar_init(&mybars[s], 1);
        mbar_init_fence();
    }
    __syncthreads();
    grid_dependency_wait();          // the step before may still read what the update rewrites
    grid_launch_dependents();

    // ------------------------------------------------------------ the CTAs that select
    if ((int)blockIdx.x >= stream_ctas) {
        SelectShared &sh = *reinterpret_cast<SelectShared *>(smem);       // where a streaming CTA has its ring
        const int n_sel = (int)gridDim.x - stream_ctas;
        uint32_t sel_parity = 0;                     // next phase of bars[0], the barrier the selection's copies complete on
        // heads in ascending order: the waves complete in that order
        for (int h = (int)blockIdx.x - stream_ctas; h < BH; h += n_sel) {
            __syncthreads();                         // everybody is done with the head before
            // what does not depend on the scores is fetched while the head is still being scored
            SelectArgs sa;
            sa.sc = b.scores + (int64_t)h * a.page_cap;
            sa.P = P; sa.K = K; sa.ns = n_sink; sa.nl = n_local;
            sa.rg = score_range<T, D>(q, h, a.absmax[cur * BH + h], lane);
            sa.hist = b.hist + (int64_t)h * kStepBins;
            sa.out = b.list + (int64_t)h * b.list_stride;
            sa.epoch = a.epoch;
            sa.ckey = sh.ckey;
            int sb = -1, sk = 0;
            // wait for the head's scoring: one thread polls, one poll per round trip, no pause
            if (threadIdx.x == 0) {
                const int32_t *done = ctr + h * kStepCtrInts + kCtrScoreDone;
                int ok = 0;
                for (int it = 0; it < kStepPollLimit; ++it) {
                    if (ld_relaxed(done) == s_total) { ok = 1; break; }
                    if ((it & 63) == 63 && ld_volatile(a.status) != RQ_OK) break;   // somebody gave up
                }
                if (ok) fence_acquire();
                else atomicCAS(a.status, RQ_OK, RQ_ERR_TIMEOUT);
                sh.ok = ok;
            }
            __syncthreads();                         // also carries the acquire to the CTA
            if (!sh.ok) return;
            const bool fast = select_head(sa, sh, &bars[0], sel_parity, sb, sk);
            __syncthreads();
            if (!fast && warp == 0) select_slow(sa, sb >= 0, sb, sk);
            // the head's histogram, all zero again for the next step (the copy has read it long ago)
            for (int i = threadIdx.x; i < kStepBins / 4; i += NW * 32)
                reinterpret_cast<uint4 *>(sa.hist)[i] = make_uint4(0u, 0u, 0u, 0u);
        }
        return;
    }

    // ------------------------------------------------------------ append (Eq. 1), one CTA per head
    for (int h = blockIdx.x; h < BH; h += stream_ctas) {
        const float s_new = update_head<T, D>(a, h, q, k_t, v_t, g_t, b.scores, red);
        // the counters of the NEXT step (nobody uses that set while this kernel runs)
        if (threadIdx.x < kStepCtrInts) b.ctr[((int64_t)(cur ^ 1) * BH + h) * kStepCtrInts + threadIdx.x] = 0;
        if (warp == 0) {
            const ScoreRange rg = score_range<T, D>(q, h, a.absmax[cur * BH + h], lane);
            if (lane == 0) {
                if (P - 1 >= n_sink && n_local == 0) red_inc(b.hist + (int64_t)h * kStepBins + rg.bucket(s_new));
                // counts as one arrival of the head's scoring; releases the CTA's writes (ordered before by the barrier)
                atom_add_acq_rel(ctr + h * kStepCtrInts + kCtrScoreDone, 1);
            }
        }
    }

    const T *meta = static_cast<const T *>(a.meta);
    const T *kvbase = static_cast<const T *>(a.kv);

    // ------------------------------------------------------------ issue side
    auto is_attend = [&](int ph) { return ph >= waves; };
    auto head_of = [&](int ph) { return (ph % waves) * HW + member; };
    // entry of a head's list: (page, step number); it is this step's once the number matches
    auto entry_of = [&](int h, int t) { return __ldcg(b.list + (int64_t)h * b.list_stride + t / TPP); };
    // the page of a ticket whose entry was fetched earlier; polls (bounded) if the entry is still an old one
    auto page_now = [&](int h, int t, int2 e, bool &ok) -> int {
        ok = true;
        for (int it = 0; e.y != a.epoch; ++it) {
            if (it >= kFlagPollLimit || ((it & 63) == 63 && ld_volatile(a.status) != RQ_OK)) { ok = false; return -1; }
            __nanosleep(kFlagPollNs);
            e = entry_of(h, t);
        }
        return e.x;
    };
    const int own0 = (rank * NW + warp) * kStepOwn;  // this warp's own tickets in every phase: own0, own0 + 1
    const int base = team * NW * kStepOwn;           // first ticket the counters hand out
    bool dead = false;                               // a wait ran out: no more work, marks only
    bool lost = false;                               // the issue side ran out of patience: the consumer gives up at its next item
    int iph = 0;                                     // phase being issued
    bool entered = false;
    int ih = 0, per = 0;
    int tA = 0, tB = 0;                              // lane 0: next ticket, ticket after it
    int2 eA = make_int2(-1, 0);                      // lane 0: list entry of ticket tA (attention phases)
    int nstate = 0;                                  // lane 0: look-ahead at the next attention phase (0: none, 1: entry requested, 2: entry is there)
    int2 nent = make_int2(-1, 0);                    // lane 0: entry of this warp's first ticket in that phase

    auto look_ahead = [&]() {                        // lane 0
        const int np = iph + 1;
        if (np >= NPH || !is_attend(np) || nstate == 2) return;
        if (own0 >= t_per) { nstate = 2; return; }   // no ticket of this warp's own in that phase
        if (nstate == 1 && nent.y == a.epoch) { nstate = 2; return; }
        nent = entry_of(head_of(np), own0);          // looked at in the next call
        nstate = 1;
    };
    auto start_copy = [&](int stage, int ph, int h, int t, int pg) {   // lane 0
        unsigned char *dst = myring + (size_t)stage * STAGE;
        if (!is_attend(ph)) {
            const int first = t * RU;
            const int n = min(RU, Ps - first);
            myinfo[stage] = make_int4(h, first, n, ph);
            const T *src = meta + ((int64_t)h * a.page_cap + first) * 2 * D;
            mbar_arrive_expect_tx(&mybars[stage], n * SG::REC_BYTES);
            bulk_g2s_hint(dst, src, n * SG::REC_BYTES, &mybars[stage], stream_policy);
        } else {
            const int tile = t % TPP;
            int valid = 0;
            if (pg >= 0 && pg < P) {
                const int64_t left = a.len - ((int64_t)pg * S + tile * TR);
                valid = left >= TR ? TR : (left > 0 ? (int)left : 0);
            }
            myinfo[stage] = make_int4(h, valid, 0, ph);
            if (valid > 0) {
                const T *kb = kvbase + (((int64_t)h * a.page_cap + pg) * 2) * S * D + tile * TR * D;
                mbar_arrive_expect_tx(&mybars[stage], AG::STAGE_BYTES);
                bulk_g2s_hint(dst, kb, AG::TILE_BYTES, &mybars[stage], stream_policy);
                bulk_g2s_hint(dst + AG::TILE_BYTES, kb + (int64_t)S * D, AG::TILE_BYTES, &mybars[stage], stream_policy);
            }
        }
    };
    // put the next item into a stage: a unit, a tile, or a mark; called by the whole warp
    auto refill = [&](int stage) {
        if (iph >= NPH) {
            if (lane == 0) myinfo[stage] = make_int4(kMarkEnd, 0, 0, 0);
            return;
        }
        const bool att = is_attend(iph);
        if (dead) per = 0;                           // marks only from here on
        if (!entered) {
            ih = head_of(iph);
            per = dead ? 0 : (att ? t_per : u_per);
            int ok = 1;
            if (lane == 0) {
                if (att && !dead && own0 < t_per && nstate != 2) {
                    // not looked ahead far enough: look now; if the list is not there yet leave a wait mark
                    nent = entry_of(ih, own0);
                    ok = nent.y == a.epoch;
                }
                if (ok) {
                    tA = own0;
                    eA = nent;
                    tB = own0 + 1;
                    nstate = 0;
                }
            }
            ok = __shfl_sync(FULL, ok, 0);
            if (!ok) {
                if (lane == 0) myinfo[stage] = make_int4(kMarkWait, 0, 0, iph);
                return;
            }
            entered = true;
        }
        int t = 0, bad = 0;
        if (lane == 0) {
            t = tA;
            const int2 e = eA;
            tA = tB;
            if (att && tA < per) eA = entry_of(ih, tA);          // used in the next call
            tB = base + atomicAdd(ctr + ih * kStepCtrInts + (att ? kCtrAttendNext : kCtrScoreNext), 1);
            if (!dead) look_ahead();
            if (t < per) {
                int pg = -1;
                if (att) {
                    bool ok;
                    pg = page_now(ih, t, e, ok);                 // the entries of a list appear within microseconds of each other
                    bad = !ok;
                }
                if (!bad) start_copy(stage, iph, ih, t, pg);
            }
        }
        t = __shfl_sync(FULL, t, 0);
        if (__shfl_sync(FULL, bad, 0)) {
            // the entry never came: nothing was started for this stage; stop taking work
            if (lane == 0) { atomicCAS(a.status, RQ_OK, RQ_ERR_TIMEOUT); myinfo[stage] = make_int4(kMarkEndPhase, 0, 0, iph); }
            lost = true;
            ++iph;
            entered = false;
            return;
        }
        if (t < per) return;
        if (lane == 0) myinfo[stage] = make_int4(kMarkEndPhase, 0, 0, iph);   // no tickets left in this phase
        ++iph;
        entered = false;
    };

#pragma unroll
    for (int s = 0; s < DEPTH; ++s) refill(s);
    __syncwarp();

    // ------------------------------------------------------------ consume side
    float qs[SG::VPL][SG::CH];                       // scoring: this lane's slice of q, split by sign
#pragma unroll
    for (int v = 0; v < SG::VPL; ++v)
#pragma unroll
        for (int i = 0; i < SG::CH; ++i) qs[v][i] = 0.0f;
    ScoreRange rg = {0.0f, 0.0f};
    AttendState<T> st;
#pragma unroll
    for (int c = 0; c < CH; ++c) { st.qf[c] = 0.0f; st.acc[c] = 0.0f; }
    st.m = -CUDART_INF_F;
    st.l = 0.0f;
    int stage = 0;
    uint32_t parity = 0;                             // one bit per stage
    int count = 0;                                   // units / tiles of the current phase consumed by this warp
    bool begun = false;                              // the current phase's head is loaded

    // a copy barrier gave up, or a flag never came: let what is in flight land, then stop taking work
    auto give_up = [&](int except) {
        for (int s = 0; s < DEPTH; ++s) {
            if (s == except) continue;
            const int4 f = myinfo[s];
            if (f.x >= 0 && (!is_attend(f.w) || f.y > 0)) mbar_wait(&mybars[s], (parity >> s) & 1u);
        }
        if (lane == 0) atomicCAS(a.status, RQ_OK, RQ_ERR_TIMEOUT);
        dead = true;
    };

    for (;;) {
        if (lost && !dead) give_up(-1);
        const int4 inf = myinfo[stage];
        if (inf.x == kMarkEnd) break;
        if (inf.x >= 0) {
            // ---- a unit of page records or a tile of keys and values
            const int ph = inf.w;
            const bool att = is_attend(ph);
            if (!begun && !dead) {
                begun = true;
                if (att) {
                    attend_begin_head<T, D>(st, q, inf.x, scale_log2, lane);
                } else {
                    score_load_q<T, D>(q, inf.x, lane, qs);
                    rg = score_range<T, D>(q, inf.x, a.absmax[cur * BH + inf.x], lane);
                }
            }
            const bool copied = !att || inf.y > 0;
            if (copied && !dead) {
                if (mbar_wait(&mybars[stage], (parity >> stage) & 1u, poll_limit)) {
                    parity ^= 1u << stage;
                } else {
                    mbar_wait(&mybars[stage], (parity >> stage) & 1u);   // the usual bound, for this copy too
                    give_up(stage);
                }
            }
            if (!dead) {
                const unsigned char *ub = myring + (size_t)stage * STAGE;
                if (!att) {
                    const int first = inf.y;
                    uint32_t *hist = b.hist + (int64_t)inf.x * kStepBins;
                    const int p_lo = n_sink, p_hi = P - n_local;
                    score_unit<T, D>(ub, qs, inf.z, b.scores + (int64_t)inf.x * a.page_cap + first, lane,
                                     [&](int r, float u) {
                                         const int p = first + r;
                                         if (p >= p_lo && p < p_hi) red_inc(hist + rg.bucket(u));
                                     });
                } else if (inf.y > 0) {
                    const T *ks = reinterpret_cast<const T *>(ub);
                    attend_tile<T, D, S>(st, ks, ks + TR * D, inf.y, lane);
                }
                ++count;
            }
        } else if (inf.x == kMarkWait) {
            // ---- the list of this phase's head was not there when the pipeline got here
            const int h = head_of(inf.w);
            if (!dead) {
                int ok = 0;
                if (lane == 0) {
                    bool got;
                    page_now(h, own0, entry_of(h, own0), got);
                    ok = got;
                }
                if (!__shfl_sync(FULL, ok, 0)) give_up(stage);
            }
        } else {
            // ---- end of a phase for this warp
            const int ph = inf.w;
            const int h = head_of(ph);
            if (!is_attend(ph)) {
                // the scores and histogram entries were written by several lanes: the warp barrier
                // orders them before lane 0's release; the head's selecting warp acquires the count
                __syncwarp();
                if (lane == 0 && count > 0 && !dead) atom_add_acq_rel(ctr + h * kStepCtrInts + kCtrScoreDone, count);
            } else {
                // merge the CTA's warps (all on head h) into one partial in slot `rank`; the arrival
                // that completes the head combines its partials
                const int wv = ph - waves, sl = wv & 1;
                const bool empty = !begun || dead;
                if (!empty) attend_merge_rows<T, D, S>(st);
                if (lane == 0)
                    sm_slot[sl * NW + warp] = make_float4(empty ? -CUDART_INF_F : st.m, empty ? 0.0f : st.l,
                                                          __int_as_float(empty ? 0 : count), __int_as_float(dead ? 1 : 0));
                if (lane < LPR) {
                    const int cgp = lane % LPR;
#pragma unroll
                    for (int c = 0; c < CH; ++c) sm_acc[(sl * NW + warp) * D + cgp * CH + c] = empty ? 0.0f : st.acc[c];
                }
                __syncthreads();
                if (warp == 0) {
                    constexpr int CPL = D / 32;      // channels per lane in the merge
                    float m_all = -CUDART_INF_F, l_all = 0.0f;
                    int t_all = 0, any_dead = 0;
#pragma unroll
                    for (int w = 0; w < NW; ++w) {
                        const float4 f = sm_slot[sl * NW + w];
                        m_all = fmaxf(m_all, f.x);
                        t_all += __float_as_int(f.z);
                        any_dead |= __float_as_int(f.w);
                    }
                    float out[CPL];
#pragma unroll
                    for (int c = 0; c < CPL; ++c) out[c] = 0.0f;
#pragma unroll
                    for (int w = 0; w < NW; ++w) {
                        const float4 f = sm_slot[sl * NW + w];
                        const float fw = f.x == -CUDART_INF_F ? 0.0f : exp2f(f.x - m_all);
                        l_all = fmaf(fw, f.y, l_all);
#pragma unroll
                        for (int c = 0; c < CPL; ++c) out[c] = fmaf(fw, sm_acc[(sl * NW + w) * D + lane * CPL + c], out[c]);
                    }
                    if (!any_dead) {                 // otherwise the status says why; the head stays incomplete
                        float *dst = b.partial + ((int64_t)h * b.slots + rank) * (D + 4);
                        if (lane == 0) *reinterpret_cast<float2 *>(dst) = make_float2(m_all, l_all);
#pragma unroll
                        for (int c = 0; c < CPL; ++c) dst[4 + lane * CPL + c] = out[c];
                        __syncwarp();
                        int last = 0;
                        if (lane == 0) {
                            const int word = t_all + (1 << kDoneTileBits);
                            const int now = atom_add_acq_rel(ctr + h * kStepCtrInts + kCtrAttendDone, word) + word;
                            last = (now & kDoneTileMask) == t_per && (now >> kDoneTileBits) == team;
                        }
                        if (__shfl_sync(FULL, last, 0)) {
                            __syncwarp();
                            combine_head<T, D>(b.partial + (int64_t)h * b.slots * (D + 4), team, o + (int64_t)h * D, lane);
                        }
                    }
                }
            }
            count = 0;
            begun = false;
        }
        __syncwarp();                                // every lane is done with the stage
        refill(stage);
        __syncwarp();
        stage = stage + 1 == DEPTH ? 0 : stage + 1;
    }
}

// ---------------------------------------------------------------- ascending copy of a page list
// sel holds K distinct pages of [0, P) per head in any order (entries are pages, or (page, step
// number) pairs; the kernel may work in place): mark them in a bit map, then write the set bits out
// in order.  One CTA of 1024 threads per head (P <= 32768: one word per thread).
__device__ __forceinline__ int list_page(const int2 &e) { return e.x; }
__device__ __forceinline__ int list_page(const int32_t &e) { return e; }

template <typename E>
__global__ void __launch_bounds__(1024) sort_list_kernel(const E *sel, int sel_stride, int K, int P, int32_t *out,
                                                         int out_stride)
{
    __shared__ uint32_t bits[1024];
    __shared__ int wsum[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const E *src = sel + (int64_t)blockIdx.x * sel_stride;
    int32_t *dst = out + (int64_t)blockIdx.x * out_stride;
    bits[tid] = 0u;
    __syncthreads();
    for (int i = tid; i < K; i += 1024) {
        const int p = list_page(__ldcg(src + i));
        if (p >= 0 && p < P) atomicOr(&bits[p >> 5], 1u << (p & 31));
    }
    __syncthreads();
    uint32_t w = bits[tid];
    int total;
    int pos = warp_excl_scan(__popc(w), lane, total);
    if (lane == 31) wsum[warp] = total;
    __syncthreads();
    int before = 0, all = 0;
    for (int i = 0; i < 32; ++i) {
        before += i < warp ? wsum[i] : 0;
        all += wsum[i];
    }
    pos += before;
    while (w) {
        const int bit = __ffs(w) - 1;
        w &= w - 1;
        if (pos < out_stride) dst[pos] = tid * 32 + bit;
        ++pos;
    }
    for (int i = all + tid; i < out_stride; i += 1024) dst[i] = -1;
}

template <typename T, int D, int S>
cudaError_t step_occupancy(int *ctas_per_sm)
{
    using G = StepGeom<T, D, S>;
    static int cached[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (cached[dev] == 0) {
        e = cudaFuncSetAttribute(step_kernel<T, D, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        int n = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, step_kernel<T, D, S>, G::NW * 32, G::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        cached[dev] = n > 0 ? n : 1;
    }
    *ctas_per_sm = cached[dev];
    return cudaSuccess;
}

template <typename T, int D, int S>
cudaError_t launch_step_t(const DecodeArgs &a, const void *q, const void *k_t, const void *v_t, const void *g_t, int K,
                          float scale, const StepBuffers &b, void *o, int waves, int grid, int stream_ctas, cudaStream_t s)
{
    using G = StepGeom<T, D, S>;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(G::NW * 32);
    cfg.dynamicSmemBytes = G::SMEM_BYTES;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, step_kernel<T, D, S>, a, (const T *)q, (const T *)k_t, (const T *)v_t, g_t, K,
                              scale * 1.4426950408889634f, b, (T *)o, waves, stream_ctas);
}

#define RQ_STEP_DISPATCH(CALL)                                  \
    if (a.dtype == RQ_BF16) {                                   \
        if (a.D == 128 && a.S == 16) CALL(bf16, 128, 16);       \
        if (a.D == 128 && a.S == 64) CALL(bf16, 128, 64);       \
        if (a.D == 64 && a.S == 16) CALL(bf16, 64, 16);         \
        if (a.D == 64 && a.S == 64) CALL(bf16, 64, 64);         \
    } else {                                                    \
        if (a.D == 128 && a.S == 16) CALL(float, 128, 16);      \
        if (a.D == 128 && a.S == 64) CALL(float, 128, 64);      \
        if (a.D == 64 && a.S == 16) CALL(float, 64, 16);        \
        if (a.D == 64 && a.S == 64) CALL(float, 64, 64);        \
    }

}  // namespace

// CTAs that select: one per head, at most 16 (each then takes heads c, c + 16, ... in turn, which
// lie in different waves)
int step_select_ctas(int heads) { return heads < 16 ? heads : 16; }

int step_plan(const DecodeArgs &a, int budget, int sm_count, int forced_waves, int *grid_out)
{
    const int BH = a.B * a.H;
    const int64_t P = (a.len + a.S - 1) / a.S;
    if (!a.absmax || BH > kStepMaxHeads || budget >= P || P < 2 || budget < 1) return 0;
    if (P + 4 > kSelectPages) return 0;              // a head's scores must fit the selecting CTA's shared memory
    // short contexts stay with one CTA per head unless the caller insists
    if (forced_waves <= 0 && P <= kSmallStepPages) return 0;
    int occ = 0;
    cudaError_t e = cudaErrorInvalidValue;
#define RQ_OCC(T, D, S) { e = step_occupancy<T, D, S>(&occ); }
    RQ_STEP_DISPATCH(RQ_OCC)
#undef RQ_OCC
    if (e != cudaSuccess || occ < 1) return 0;
    // Measured: with 32 heads (one sequence) the separate kernels are as fast (57.3 against 57.6 us per
    // step at 128K context) and much faster on short contexts, where this kernel's fixed costs show;
    // with 128 heads (batch 4, 128K context) four waves take 171 us against 187 (246 / 269 and 398 / 428
    // at budgets 1/8 and 1/4); with 256 heads of 2049 pages (batch 8, 32K context) the 16 selecting
    // CTAs fall behind (179 against 155).  Left to itself the library takes this path for 64 to 128
    // heads of at least 4096 pages, trying four waves first.
    if (forced_waves <= 0 && (BH < 64 || BH > 128 || P < 4096)) return 0;
    static const int order[3] = {4, 8, 2};
    for (int i = 0; i < 3; ++i) {
        const int waves = order[i];
        if (forced_waves > 0 && waves != forced_waves) continue;
        if (BH % waves) continue;
        const int HW = BH / waves;
        const int resident = occ * sm_count - step_select_ctas(BH);   // the CTAs that select stream nothing
        if (resident < 1) continue;
        const int team = resident / HW;
        if (team < 1 || team * kStepWarps > kAttendMaxWarps) continue;
        const int grid = team * HW;
        // (almost) the whole machine must be at work, and the CTAs of a head must be a real team
        if (forced_waves <= 0 && (grid * 100 < resident * 95 || team < 4)) continue;
        *grid_out = grid;                            // streaming CTAs; the selecting CTAs come on top
        return waves;
    }
    return 0;
}

cudaError_t launch_step(const DecodeArgs &a, const void *q, const void *k_t, const void *v_t, const void *g_t, int budget,
                        float scale, const StepBuffers &b, void *o, int waves, int grid, cudaStream_t s)
{
    const int stream_ctas = grid;
    grid += step_select_ctas(a.B * a.H);
#define RQ_RUN(T, D, S) return launch_step_t<T, D, S>(a, q, k_t, v_t, g_t, budget, scale, b, o, waves, grid, stream_ctas, s)
    RQ_STEP_DISPATCH(RQ_RUN)
#undef RQ_RUN
    return cudaErrorInvalidValue;
}

cudaError_t launch_sort_list(const int2 *sel, int sel_stride, int K, int P, int BH, int32_t *out, int out_stride,
                             cudaStream_t s)
{
    if (P > 32768) return cudaErrorInvalidValue;
    sort_list_kernel<int2><<<(unsigned)BH, 1024, 0, s>>>(sel, sel_stride, K, P, out, out_stride);
    return cudaGetLastError();
}

cudaError_t launch_sort_list32(const int32_t *sel, int sel_stride, int K, int P, int BH, int32_t *out, int out_stride,
                               cudaStream_t s)
{
    if (P > 32768) return cudaErrorInvalidValue;
    sort_list_kernel<int32_t><<<(unsigned)BH, 1024, 0, s>>>(sel, sel_stride, K, P, out, out_stride);
    return cudaGetLastError();
}

}  // namespace rq
