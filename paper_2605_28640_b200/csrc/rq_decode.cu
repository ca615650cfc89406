// Decode step kernels:
//   update  — one step of Eq. 1 on the fp32 state, append to the paged cache,
//             refresh the newest page's min/max
//   score   — Quest upper bound U_p = sum_i max(q_i min_p[i], q_i max_p[i]) for
//             every page (Eq. 3 with the min/max representatives of App. A.1)
//   topk    — per (b,h) selection of the budget's pages, forced first/local
//             pages inside the budget, ties to the lower page index, ascending
//   attend  — split-K flash-decode over the selected pages only (Eq. 4) and
//             the combine of the split partials
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
// registers (KPT consecutive pages per thread); forced pages get the largest
// key.  The k-th largest key is found bit by bit (32 counting rounds, one
// barrier each); pages with a larger key are taken, pages with an equal key
// are taken in index order until the budget is full.  A block-wide prefix sum
// over the per-thread counts gives each taken page its slot, so the output is
// ascending and unique whatever the thread timing.
template <int KPT>
__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const float *scores, int64_t score_stride,
                                                            int P, int K, int n_sink, int n_local,
                                                            int32_t *idx, int idx_stride, int budget)
{
    constexpr int NTH = kTopkThreads, NWP = NTH / 32;
    __shared__ int cnt[2][NWP];
    __shared__ uint32_t wsum[NWP];
    const int bh = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t *out = idx + (int64_t)bh * idx_stride;

    if (K >= P) {                                    // dense: every page, in order
        for (int p = tid; p < budget; p += NTH) out[p] = p < P ? p : -1;
        return;
    }
    const float *sc = scores + (int64_t)bh * score_stride;
    uint32_t key[KPT];
    const int base = tid * KPT;
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
        const int p = base + j;
        uint32_t kx = 0;                             // below every real key
        if (p < P) {
            kx = order_key(sc[p]);
            if (kx == 0xffffffffu) kx = 0xfffffffeu; // keep the top key for forced pages
            if (kx == 0u) kx = 1u;
            if (p < n_sink || p >= P - n_local) kx = 0xffffffffu;
        }
        key[j] = kx;
    }

    // k-th largest key: largest tau with count(key >= tau) >= K
    uint32_t tau = 0;
    for (int bit = 31; bit >= 0; --bit) {
        const uint32_t cand = tau | (1u << bit);
        int c = 0;
#pragma unroll
        for (int j = 0; j < KPT; ++j) c += key[j] >= cand;
        c = __reduce_add_sync(0xffffffffu, c);
        if (lane == 0) cnt[bit & 1][warp] = c;
        __syncthreads();
        int tot = 0;
#pragma unroll
        for (int w = 0; w < NWP; ++w) tot += cnt[bit & 1][w];
        if (tot >= K) tau = cand;
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
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    uint32_t before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < NWP; ++w) {
        const uint32_t t = wsum[w];
        if (w < warp) before += t;
        total += t;
    }
    const uint32_t excl = before + incl - mine;
    const int n_gt = (int)(total & 0xffffu);
    const int r = K - n_gt;                          // how many equal keys to take
    int gt_before = (int)(excl & 0xffffu), eq_before = (int)(excl >> 16);
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
        if (key[j] > tau) {
            out[gt_before + min(eq_before, r)] = base + j;
            ++gt_before;
        } else if (key[j] == tau && tau != 0u) {
            if (eq_before < r) out[gt_before + eq_before] = base + j;
            ++eq_before;
        }
    }
    for (int p = K + tid; p < budget; p += NTH) out[p] = -1;
}

// ---------------------------------------------------------------- attend
// grid (nsplit, B*H), kAttendWarps warps.  Split s owns a contiguous range of
// the head's index list; its warps take the pages of that range round-robin.
// A warp reads a page's K block and V block with fully coalesced 16-byte
// loads: one load instruction covers RPI whole rows, lane -> (row, channel
// group).  Row dot products are reduced over the LPR lanes of a row; the
// softmax runs online per warp in the exp2 domain; V is accumulated per lane
// for its channel group over the rows it loaded, and the row groups are
// merged once at the end.
template <typename T, int D, int S>
__global__ void __launch_bounds__(kAttendWarps * 32) attend_kernel(DecodeArgs a, const T *q,
                                                                   const int32_t *idx, int n_idx,
                                                                   int idx_stride, float scale_log2,
                                                                   float *partial, int nsplit)
{
    constexpr int CH = VecOf<T>::N;
    constexpr int LPR = D / CH;                 // lanes per row
    constexpr int RPI = 32 / LPR;               // rows per load instruction
    constexpr int TR = 16;                      // rows handled per register tile
    constexpr int NTILE = S / TR;               // register tiles per page
    constexpr int NI = TR / RPI;                // load instructions per tile and tensor
    constexpr int NW = kAttendWarps;
    static_assert(LPR <= 32 && TR % RPI == 0 && S % TR == 0, "unsupported geometry");

    __shared__ float sm_m[NW], sm_l[NW];
    __shared__ float sm_acc[NW][D];

    const int split = blockIdx.x, bh = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rsub = lane / LPR, cgp = lane % LPR;
    const int64_t P = (a.len + S - 1) / S;

    float qf[CH];
#pragma unroll
    for (int i = 0; i < CH; ++i) qf[i] = load1<T>(q + (int64_t)bh * D + cgp * CH + i) * scale_log2;

    const int lo = (int)((int64_t)n_idx * split / nsplit);
    const int hi = (int)((int64_t)n_idx * (split + 1) / nsplit);
    const int32_t *list = idx + (int64_t)bh * idx_stride;
    const T *kvb = static_cast<const T *>(a.kv) + (int64_t)bh * a.page_cap * 2 * S * D;

    float m_run = -CUDART_INF_F, l_run = 0.0f;
    float acc[CH];
#pragma unroll
    for (int i = 0; i < CH; ++i) acc[i] = 0.0f;

    for (int it = lo + warp; it < hi; it += NW) {
        const int page = list[it];
        if (page < 0) continue;
        if (page >= P) {
            if (lane == 0) atomicExch(a.status, RQ_ERR_INVALID_ARG);
            continue;
        }
        const int valid = (int)min((int64_t)S, a.len - (int64_t)page * S);
        const T *kb = kvb + (int64_t)page * 2 * S * D;
        const T *vb = kb + S * D;
#pragma unroll 1
        for (int tile = 0; tile < NTILE; ++tile) {
            if (tile * TR >= valid) break;          // the rest of the page holds no token
            uint4 rk[NI], rv[NI];
#pragma unroll
            for (int i = 0; i < NI; ++i) rk[i] = ldcs16(kb + ((tile * NI + i) * 32 + lane) * CH);
#pragma unroll
            for (int i = 0; i < NI; ++i) rv[i] = ldcs16(vb + ((tile * NI + i) * 32 + lane) * CH);

            float s[NI];
            float m_new = m_run;
#pragma unroll
            for (int i = 0; i < NI; ++i) {
                float kf[CH];
                unpack16<T>(rk[i], kf);
                float d = 0.0f;
#pragma unroll
                for (int c = 0; c < CH; ++c) d = fmaf(qf[c], kf[c], d);
#pragma unroll
                for (int off = LPR / 2; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
                const int row = tile * TR + i * RPI + rsub;
                s[i] = row < valid ? d : -CUDART_INF_F;
                m_new = fmaxf(m_new, s[i]);
            }
#pragma unroll
            for (int off = LPR; off < 32; off <<= 1)
                m_new = fmaxf(m_new, __shfl_xor_sync(0xffffffffu, m_new, off));
            const float alpha = exp2f(m_run - m_new);    // 0 on the first tile (m_run = -inf)
            m_run = m_new;
            l_run *= alpha;
#pragma unroll
            for (int c = 0; c < CH; ++c) acc[c] *= alpha;
#pragma unroll
            for (int i = 0; i < NI; ++i) {
                const float p = exp2f(s[i] - m_new);     // 0 for masked rows
                l_run += p;
                float vf[CH];
                unpack16<T>(rv[i], vf);
#pragma unroll
                for (int c = 0; c < CH; ++c) acc[c] = fmaf(p, vf[c], acc[c]);
            }
        }
    }

    // merge the row groups of the warp (they share m_run); every lane of a row
    // added the same p, so the warp's l is the sum over one lane per row group
#pragma unroll
    for (int off = LPR; off < 32; off <<= 1) {
        l_run += __shfl_xor_sync(0xffffffffu, l_run, off);
#pragma unroll
        for (int c = 0; c < CH; ++c) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], off);
    }
    if (lane == 0) { sm_m[warp] = m_run; sm_l[warp] = l_run; }
    if (lane < LPR) {
#pragma unroll
        for (int c = 0; c < CH; ++c) sm_acc[warp][cgp * CH + c] = acc[c];
    }
    __syncthreads();

    // merge the warps and write this split's partial: [m, l, acc[D]]
    float m_all = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < NW; ++w) m_all = fmaxf(m_all, sm_m[w]);
    float *dst = partial + ((int64_t)bh * nsplit + split) * (D + 2);
    for (int d = threadIdx.x; d < D; d += NW * 32) {
        float o = 0.0f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float f = sm_m[w] == -CUDART_INF_F ? 0.0f : exp2f(sm_m[w] - m_all);
            o = fmaf(f, sm_acc[w][d], o);
        }
        dst[2 + d] = o;
    }
    if (threadIdx.x == 0) {
        float l = 0.0f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float f = sm_m[w] == -CUDART_INF_F ? 0.0f : exp2f(sm_m[w] - m_all);
            l = fmaf(f, sm_l[w], l);
        }
        dst[0] = m_all;
        dst[1] = l;
    }
}

// grid B*H, D threads: o = sum_s 2^(m_s-m) acc_s / sum_s 2^(m_s-m) l_s
template <typename T, int D>
__global__ void combine_kernel(const float *partial, int nsplit, T *o)
{
    const int bh = blockIdx.x, d = threadIdx.x;
    const float *src = partial + (int64_t)bh * nsplit * (D + 2);
    float m = -CUDART_INF_F;
    for (int s = 0; s < nsplit; ++s) m = fmaxf(m, src[(int64_t)s * (D + 2)]);
    float num = 0.0f, den = 0.0f;
    for (int s = 0; s < nsplit; ++s) {
        const float ms = src[(int64_t)s * (D + 2)];
        const float f = ms == -CUDART_INF_F ? 0.0f : exp2f(ms - m);
        num = fmaf(f, src[(int64_t)s * (D + 2) + 2 + d], num);
        den = fmaf(f, src[(int64_t)s * (D + 2) + 1], den);
    }
    store1<T>(o + (int64_t)bh * D + d, num / den);
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
                        int idx_stride, cudaStream_t s)
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
    topk_kernel<KPT><<<BH, kTopkThreads, 0, s>>>(scores, a.page_cap, P, K, ns, nl, idx, idx_stride, budget)
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

int choose_splits(int BH, int n_idx, int sm_count)
{
    // aim at four resident CTAs per SM in total
    int target = sm_count * 4;
    int ns = (target + BH - 1) / BH;
    if (ns > kMaxSplits) ns = kMaxSplits;
    if (ns > n_idx) ns = n_idx;
    if (ns < 1) ns = 1;
    return ns;
}

cudaError_t launch_attend(const DecodeArgs &a, const void *q, const int32_t *idx, int n_idx,
                          int idx_stride, float scale, float *partial, int nsplit, cudaStream_t s)
{
    const int BH = a.B * a.H;
    const float scale_log2 = scale * 1.4426950408889634f;
    dim3 grid((unsigned)nsplit, (unsigned)BH);
#define CALL_ATT(T, D, S)                                                                        \
    attend_kernel<T, D, S><<<grid, kAttendWarps * 32, 0, s>>>(a, (const T *)q, idx, n_idx,       \
                                                              idx_stride, scale_log2, partial, nsplit)
    RQ_DISPATCH_TDS(a, CALL_ATT);
#undef CALL_ATT
    return cudaGetLastError();
}

cudaError_t launch_combine(const DecodeArgs &a, const float *partial, int nsplit, void *o, cudaStream_t s)
{
    const int BH = a.B * a.H;
#define CALL_CMB(T, D, S) combine_kernel<T, D><<<BH, D, 0, s>>>(partial, nsplit, (T *)o)
    RQ_DISPATCH_TDS(a, CALL_CMB);
#undef CALL_CMB
    return cudaGetLastError();
}

}  // namespace rq
