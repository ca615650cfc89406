// Prefill: single-pass chained scan of the gated decay recurrence (Eq. 1)
// fused with the paged cache write and the per-page min/max of the stored keys
// (Appendix A.1, "Sparse inference settings").  Every input byte is read once.
//
// The recurrence x~_t = g_t x~_{t-1} + (1-g_t) x_t is a first-order linear
// recurrence, so a run of tokens acts on the incoming state as the affine map
// s -> A s + B with A = prod g and B = the run's own state from zero.  Maps
// compose as (A2,B2)o(A1,B1) = (A2 A1, A2 B1 + B2), which is associative, so
// time can be cut into pieces that are reduced independently.
//
// Work decomposition.  One CTA owns one (batch, head) pair and one chunk of
// CT consecutive cache positions.  A thread owns CH channels (one 16-byte
// vector of the storage type) and TS consecutive tokens whose k, v and g are
// fetched once, by asynchronous copies, into the thread's own slots of shared
// memory and read from there for both of its passes.  Threads with the same
// channels and consecutive token slices sit NCG lanes apart, so the carry
// between the slices of a warp moves with warp shuffles; warps exchange their
// totals through shared memory.
//
// Chaining.  A CTA takes its (chunk, head) from a ticket counter, chunk-major
// with the heads varying fastest, so every chunk before its own was taken
// earlier by a CTA that is running or done, and CTAs that run together read
// one contiguous stretch of the [B][T][H][D] inputs.  It loads its tokens,
// reduces them to the chunk's map, publishes the map (flag 1), then looks back
// over the records of the chunks before it, composing their maps until it
// meets one that already knows the state at its own end (flag 2); that gives
// the state entering the chunk.  Which chunks are composed is fixed by the
// chunk's number (back to the last multiple of eight), not by timing, so the
// result is the same bits on every run.  It publishes its own end state (flag 2)
// before the heavy part, the token-by-token application with rounding, page
// writes and page bounds, so later chunks never wait for that.  Waits on a
// flag are bounded: when the limit runs out the kernel records
// RQ_ERR_TIMEOUT in the status word and carries on with a zero carry instead
// of spinning.
#include "rq_async.cuh"
#include "rq_device.cuh"
#include "rq_internal.h"

namespace rq {

namespace {

constexpr int NT = kScanThreads;
constexpr int kLookWindow = 8;                  // chunks examined per look-back round
constexpr int kFlagPollLimit = 1 << 20;         // polls of one flag before giving up

__device__ __forceinline__ void st_release(int32_t *p, int v)
{
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// asynchronous copy of BYTES (8 or 16) from global to shared memory
template <int BYTES>
__device__ __forceinline__ void cp_async(void *dst_smem, const void *src)
{
    static_assert(BYTES == 8 || BYTES == 16, "unsupported copy size");
    if constexpr (BYTES == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst_smem)), "l"(src) : "memory");
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_addr(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// N consecutive elements of G from shared memory as floats (N * sizeof(G) in {8, 16, 32} bytes)
template <typename G, int N>
__device__ __forceinline__ void lds_n(const void *p, float *out)
{
    constexpr int BYTES = N * (int)sizeof(G);
    if constexpr (BYTES == 16) {
        unpack16<G>(lds16(p), out);
    } else if constexpr (BYTES == 32) {
        unpack16<G>(lds16(p), out);
        unpack16<G>(lds16(static_cast<const char *>(p) + 16), out + N / 2);
    } else {
        static_assert(BYTES == 8, "unsupported vector width");
        const uint2 r = *static_cast<const uint2 *>(p);
        if constexpr (sizeof(G) == 2) {
            out[0] = bf16lo(r.x); out[1] = bf16hi(r.x);
            out[2] = bf16lo(r.y); out[3] = bf16hi(r.y);
        } else {
            out[0] = __uint_as_float(r.x); out[1] = __uint_as_float(r.y);
        }
    }
}

template <typename T, typename G, int D, int S>
__global__ void __launch_bounds__(NT, 3) scan_kernel(ScanArgs a, int64_t chunk0)
{
    constexpr int CH = VecOf<T>::N;
    constexpr int NCG = D / CH;
    constexpr int NSL = NT / NCG;
    constexpr int TS = scan_ts(D, (int)sizeof(T));
    constexpr int CT = NSL * TS;
    constexpr int NW = NT / 32;
    static_assert(CT % S == 0 && S % TS == 0, "chunk must hold whole pages of whole slices");
    static_assert(NCG <= 32 && 32 % NCG == 0, "a warp must hold whole slices");

    // the warp totals are dead (several CTA barriers earlier) when the page bounds are reduced:
    // both live in the same shared memory
    constexpr int kScratchFloats = NW * 3 * D > NSL * 2 * D ? NW * 3 * D : NSL * 2 * D;
    __shared__ float scratch[kScratchFloats];
    float (*wtot)[3][D] = reinterpret_cast<float (*)[3][D]>(scratch);
    float (*mm)[2][D] = reinterpret_cast<float (*)[2][D]>(scratch);
    __shared__ float sm_agg[3][D];               // the chunk's map
    __shared__ float sm_in[2][D];                // state entering the chunk
    __shared__ int sm_ticket;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cg = tid % NCG, sl = tid / NCG;
    const int BH = a.B * a.H;
    if (tid == 0) sm_ticket = atomicAdd(a.ticket, 1);
    __syncthreads();
    const int rel = sm_ticket / BH;              // chunk number inside this call
    const int bh = sm_ticket % BH, b = bh / a.H, h = bh % a.H;
    const int64_t chunk = chunk0 + rel;
    const int64_t pos0 = chunk * CT + (int64_t)sl * TS;
    const int64_t end = a.len0 + a.T;

    const T *kp = static_cast<const T *>(a.k);
    const T *vp = static_cast<const T *>(a.v);
    const G *gp = static_cast<const G *>(a.g);

    // ---- fetch this thread's TS tokens into its own slots of shared memory with asynchronous
    // copies (identity map for positions outside the new range): the data waits there, not in
    // registers, so that three CTAs fit on an SM
    constexpr int GB = CH * (int)sizeof(G);      // bytes of this thread's gates of one token
    extern __shared__ __align__(16) unsigned char dsm[];
    uint4 *kbuf = reinterpret_cast<uint4 *>(dsm);            // [TS][NT]
    uint4 *vbuf = kbuf + TS * NT;                            // [TS][NT]
    unsigned char *gbuf = reinterpret_cast<unsigned char *>(vbuf + TS * NT);   // [TS][NT][GB]
#pragma unroll
    for (int i = 0; i < TS; ++i) {
        const int64_t pos = pos0 + i;
        const int slot = i * NT + tid;
        if (pos >= a.len0 && pos < end) {
            const int64_t src = (int64_t)b * a.sb + (pos - a.len0) * a.st + (int64_t)h * a.sh + cg * CH;
            cp_async<16>(&kbuf[slot], kp + src);
            cp_async<16>(&vbuf[slot], vp + src);
            if constexpr (GB == 32) {
                cp_async<16>(gbuf + (size_t)slot * GB, gp + src);
                cp_async<16>(gbuf + (size_t)slot * GB + 16, reinterpret_cast<const char *>(gp + src) + 16);
            } else {
                cp_async<GB>(gbuf + (size_t)slot * GB, gp + src);
            }
        } else {
            kbuf[slot] = make_uint4(0, 0, 0, 0);
            vbuf[slot] = make_uint4(0, 0, 0, 0);
            constexpr uint32_t one = sizeof(G) == 2 ? 0x3f803f80u : 0x3f800000u;   // 1.0 in G, packed
#pragma unroll
            for (int wd = 0; wd < GB / 4; ++wd) reinterpret_cast<uint32_t *>(gbuf + (size_t)slot * GB)[wd] = one;
        }
    }
    cp_async_wait_all();                         // a thread only ever reads the slots it filled itself

    // ---- the slice's own map (A, Bk, Bv) from a zero state
    float A[CH], Bk[CH], Bv[CH];
#pragma unroll
    for (int c = 0; c < CH; ++c) { A[c] = 1.0f; Bk[c] = 0.0f; Bv[c] = 0.0f; }
#pragma unroll
    for (int i = 0; i < TS; ++i) {
        float kf[CH], vf[CH];
        float gi[CH];
        unpack16<T>(kbuf[i * NT + tid], kf);
        unpack16<T>(vbuf[i * NT + tid], vf);
        lds_n<G, CH>(gbuf + (size_t)(i * NT + tid) * GB, gi);
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const float om = 1.0f - gi[c];
            Bk[c] = fmaf(gi[c], Bk[c], om * kf[c]);
            Bv[c] = fmaf(gi[c], Bv[c], om * vf[c]);
            A[c] *= gi[c];
        }
    }

    // ---- inclusive scan over the slices of this warp: carry by warp shuffle
#pragma unroll
    for (int off = NCG; off < 32; off <<= 1) {
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const float pa = __shfl_up_sync(0xffffffffu, A[c], off);
            const float pk = __shfl_up_sync(0xffffffffu, Bk[c], off);
            const float pv = __shfl_up_sync(0xffffffffu, Bv[c], off);
            if (lane >= off) {
                Bk[c] = fmaf(A[c], pk, Bk[c]);
                Bv[c] = fmaf(A[c], pv, Bv[c]);
                A[c] *= pa;
            }
        }
    }
    if (lane >= 32 - NCG) {
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            wtot[warp][0][cg * CH + c] = A[c];
            wtot[warp][1][cg * CH + c] = Bk[c];
            wtot[warp][2][cg * CH + c] = Bv[c];
        }
    }
    __syncthreads();

    // ---- map of everything in the chunk before this warp
    float Ap[CH], Pk[CH], Pv[CH];
#pragma unroll
    for (int c = 0; c < CH; ++c) { Ap[c] = 1.0f; Pk[c] = 0.0f; Pv[c] = 0.0f; }
    for (int w = 0; w < warp; ++w) {
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const float wa = wtot[w][0][cg * CH + c];
            Pk[c] = fmaf(wa, Pk[c], wtot[w][1][cg * CH + c]);
            Pv[c] = fmaf(wa, Pv[c], wtot[w][2][cg * CH + c]);
            Ap[c] *= wa;
        }
    }

    // ---- the chunk's map = (last warp's total) o (everything before the last warp)
    if (warp == NW - 1 && lane >= 32 - NCG) {
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            sm_agg[0][cg * CH + c] = A[c] * Ap[c];
            sm_agg[1][cg * CH + c] = fmaf(A[c], Pk[c], Bk[c]);
            sm_agg[2][cg * CH + c] = fmaf(A[c], Pv[c], Bv[c]);
        }
    }
    __syncthreads();

    // ---- publish the map, find the state entering the chunk, publish the state leaving it
    float *agg = a.agg + ((int64_t)bh * a.chunks_cap + rel) * 3 * D;
    float *inc = a.inc + ((int64_t)bh * a.chunks_cap + rel) * 2 * D;
    int32_t *flags = a.flags + (int64_t)bh * a.chunks_cap;
    if (tid < D) {
        const int d = tid;
        const float ca = sm_agg[0][d], cbk = sm_agg[1][d], cbv = sm_agg[2][d];
        float in_k, in_v;
        if (rel == 0) {
            in_k = a.state[(int64_t)bh * 2 * D + d];
            in_v = a.state[(int64_t)bh * 2 * D + D + d];
        } else {
            agg[d] = ca;
            agg[D + d] = cbk;
            agg[2 * D + d] = cbv;
        }
        // the D publishing threads are whole warps (D is a multiple of 32); the barrier orders their
        // stores before thread 0's release store of the flag
        asm volatile("bar.sync 1, %0;" ::"n"(D));
        if (rel != 0) {
            if (d == 0) st_release(flags + rel, 1);
            // Look back to the anchor: the last chunk before this one whose number is a multiple
            // of kLookWindow.  The state entering this chunk is the anchor's end state pushed
            // through the maps of the chunks in between, always in the same order, so the result
            // does not depend on which chunk happened to finish first.
            const int base = (rel - 1) / kLookWindow * kLookWindow;
            const int n = rel - 1 - base;          // maps to compose: chunks base+1 .. rel-1
            bool timed_out = false;
            // all flags are read together (relaxed loads, one round trip), then only the ones that
            // are not there yet are polled; the fence after the loop makes the reads acquire
            int f[kLookWindow];                    // f[u], u < n: chunk rel-1-u; f[n]: the anchor
#pragma unroll
            for (int u = 0; u < kLookWindow; ++u) f[u] = u <= n ? ld_volatile(flags + (rel - 1 - u)) : 2;
#pragma unroll
            for (int u = 0; u < kLookWindow; ++u) {
                const int need = u == n ? 2 : 1;
                int polls = 0;
                while (u <= n && f[u] < need && !timed_out) {
                    if (++polls > kFlagPollLimit) timed_out = true;
                    __nanosleep(32);
                    f[u] = ld_volatile(flags + (rel - 1 - u));
                }
            }
            __threadfence();
            const float *pa = a.agg + ((int64_t)bh * a.chunks_cap + (rel - 1)) * 3 * D + d;
            float ra[kLookWindow - 1], rbk[kLookWindow - 1], rbv[kLookWindow - 1];
#pragma unroll
            for (int u = 0; u < kLookWindow - 1; ++u) {
                if (u < n && !timed_out) {
                    ra[u] = __ldcg(pa - (int64_t)u * 3 * D);
                    rbk[u] = __ldcg(pa - (int64_t)u * 3 * D + D);
                    rbv[u] = __ldcg(pa - (int64_t)u * 3 * D + 2 * D);
                }
            }
            float acc_a = 1.0f, acc_k = 0.0f, acc_v = 0.0f;     // map of the chunks base+1 .. rel-1
#pragma unroll
            for (int u = 0; u < kLookWindow - 1; ++u) {
                if (u < n && !timed_out) {           // acc = acc o map(rel-1-u): the older map acts first
                    acc_k = fmaf(acc_a, rbk[u], acc_k);
                    acc_v = fmaf(acc_a, rbv[u], acc_v);
                    acc_a *= ra[u];
                }
            }
            in_k = 0.0f;
            in_v = 0.0f;
            if (!timed_out) {
                const float *pi = a.inc + ((int64_t)bh * a.chunks_cap + base) * 2 * D + d;
                in_k = fmaf(acc_a, __ldcg(pi), acc_k);
                in_v = fmaf(acc_a, __ldcg(pi + D), acc_v);
            }
            if (timed_out) {
                atomicExch(a.status, RQ_ERR_TIMEOUT);
                in_k = 0.0f;
                in_v = 0.0f;
            }
        }
        inc[d] = fmaf(ca, in_k, cbk);
        inc[D + d] = fmaf(ca, in_v, cbv);
        sm_in[0][d] = in_k;
        sm_in[1][d] = in_v;
        asm volatile("bar.sync 1, %0;" ::"n"(D));
        if (d == 0) st_release(flags + rel, 2);
    }
    __syncthreads();

    {
        // ---- exclusive map inside the warp = inclusive map of the previous slice
        float sk[CH], sv[CH];
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            float ea = __shfl_up_sync(0xffffffffu, A[c], NCG % 32);
            float ek = __shfl_up_sync(0xffffffffu, Bk[c], NCG % 32);
            float ev = __shfl_up_sync(0xffffffffu, Bv[c], NCG % 32);
            if (NCG == 32 || lane < NCG) { ea = 1.0f; ek = 0.0f; ev = 0.0f; }
            // state entering the chunk
            const float ck = sm_in[0][cg * CH + c];
            const float cv = sm_in[1][cg * CH + c];
            // entering this warp, then entering this slice
            const float wk = fmaf(Ap[c], ck, Pk[c]);
            const float wv = fmaf(Ap[c], cv, Pv[c]);
            sk[c] = fmaf(ea, wk, ek);
            sv[c] = fmaf(ea, wv, ev);
        }

        // ---- apply the recurrence token by token, round, store, track bounds
        T *kv = static_cast<T *>(a.kv);
        float mn[CH], mx[CH];
#pragma unroll
        for (int c = 0; c < CH; ++c) { mn[c] = INFINITY; mx[c] = -INFINITY; }
        const int64_t tail_end = (end + S - 1) / S * S;   // end of the last touched page
#pragma unroll
        for (int i = 0; i < TS; ++i) {
            const int64_t pos = pos0 + i;
            float kf[CH], vf[CH];
            float gi[CH];
            unpack16<T>(kbuf[i * NT + tid], kf);
            unpack16<T>(vbuf[i * NT + tid], vf);
            lds_n<G, CH>(gbuf + (size_t)(i * NT + tid) * GB, gi);
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const float om = 1.0f - gi[c];
                sk[c] = fmaf(gi[c], sk[c], om * kf[c]);
                sv[c] = fmaf(gi[c], sv[c], om * vf[c]);
            }
            const bool valid = pos >= a.len0 && pos < end;
            const bool fill = pos >= end && pos < tail_end;   // unused slots of the last page
            if (valid || fill) {
                const int64_t page = pos / S;
                const int slot = (int)(pos % S);
                T *dst = kv + ((((int64_t)bh * a.page_cap + page) * 2) * S + slot) * D + cg * CH;
                uint4 wk, wv;
                if (valid) {
                    wk = pack16<T>(sk);
                    wv = pack16<T>(sv);
                    float rk_[CH];
                    unpack16<T>(wk, rk_);
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        mn[c] = fminf(mn[c], rk_[c]);
                        mx[c] = fmaxf(mx[c], rk_[c]);
                    }
                } else {
                    wk = make_uint4(0, 0, 0, 0);
                    wv = wk;
                }
                *reinterpret_cast<uint4 *>(dst) = wk;
                *reinterpret_cast<uint4 *>(dst + (int64_t)S * D) = wv;
            }
        }
        // the owner of the last new token leaves the fp32 state behind
        if (end - 1 >= pos0 && end - 1 < pos0 + TS) {
            float *st = a.state + (int64_t)bh * 2 * D;
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                st[cg * CH + c] = sk[c];
                st[D + cg * CH + c] = sv[c];
            }
        }

        // ---- page bounds: reduce the slices of each page through shared memory
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            mm[sl][0][cg * CH + c] = mn[c];
            mm[sl][1][cg * CH + c] = mx[c];
        }
        __syncthreads();
        constexpr int SPP = S / TS;      // slices per page
        constexpr int PPC = CT / S;      // pages per chunk
        T *meta = static_cast<T *>(a.meta);
        for (int idx = tid; idx < PPC * D; idx += NT) {
            const int pg = idx / D, d = idx % D;
            const int64_t page = chunk * PPC + pg;
            const int64_t pstart = page * S;
            if (pstart >= end || pstart + S <= a.len0) continue;   // no new token in this page
            float lo = INFINITY, hi = -INFINITY;
#pragma unroll
            for (int s2 = 0; s2 < SPP; ++s2) {
                lo = fminf(lo, mm[pg * SPP + s2][0][d]);
                hi = fmaxf(hi, mm[pg * SPP + s2][1][d]);
            }
            T *m = meta + (((int64_t)bh * a.page_cap + page) * 2) * D + d;
            if (pstart < a.len0) {                                  // page already held tokens
                lo = fminf(lo, load1<T>(m));
                hi = fmaxf(hi, load1<T>(m + D));
            }
            store1<T>(m, lo);
            store1<T>(m + D, hi);
        }
    }
}

template <typename T, typename G, int D, int S>
cudaError_t run(const ScanArgs &a, cudaStream_t s)
{
    constexpr int CH = VecOf<T>::N;
    constexpr int CT = (NT / (D / CH)) * scan_ts(D, (int)sizeof(T));
    const int64_t end = a.len0 + a.T;
    const int64_t c0 = a.len0 / CT;
    const int64_t c1 = (end + CT - 1) / CT;
    const int64_t nchunks = c1 - c0;
    if (nchunks <= 0) return cudaSuccess;
    if (nchunks > a.chunks_cap) return cudaErrorInvalidValue;
    const int64_t ctas = nchunks * a.B * a.H;
    if (ctas >= (int64_t)1 << 31) return cudaErrorInvalidValue;
    // the ticket counter and this call's flags start at zero
    cudaError_t e = cudaMemsetAsync(a.ticket, 0, sizeof(int32_t), s);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(a.flags, 0, (size_t)a.B * a.H * a.chunks_cap * sizeof(int32_t), s);
    if (e != cudaSuccess) return e;
    constexpr int TS = scan_ts(D, (int)sizeof(T));
    constexpr int DSM = TS * NT * (32 + CH * (int)sizeof(G));    // k, v and g slots of every thread
    static bool ready[64];
    int dev = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!ready[dev]) {
        e = cudaFuncSetAttribute(scan_kernel<T, G, D, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, DSM);
        if (e != cudaSuccess) return e;
        ready[dev] = true;
    }
    scan_kernel<T, G, D, S><<<(unsigned)ctas, NT, DSM, s>>>(a, c0);
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
