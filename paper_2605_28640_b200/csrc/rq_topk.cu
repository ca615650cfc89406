// Second kernel of a decode step: per (b,h) selection of the budget's pages from
// the page scores (the TopK of Eq. 3), forced first/local pages inside the
// budget (App. A.1), ties to the lower page index, output ascending.  The
// routine itself is select_head in rq_select.cuh.
#include <math_constants.h>

#include "rq_async.cuh"
#include "rq_device.cuh"
#include "rq_internal.h"
#include "rq_select.cuh"

namespace rq {

namespace {

// One CTA per (b,h) runs the selection routine; it also clears the ticket counters of the two
// streaming kernels for its head.
template <int NTH>
__global__ void __launch_bounds__(NTH) topk_select_kernel(const float *scores, int64_t score_stride, int P, int K,
                                                         int n_sink, int n_local, int32_t *idx, int idx_stride,
                                                         int budget, int32_t *attend_ctr)
{
    extern __shared__ __align__(16) unsigned char sel_smem[];
    const int bh = blockIdx.x;
    grid_dependency_wait();
    grid_launch_dependents();
    if (threadIdx.x < 4) attend_ctr[bh * kCtrStride + threadIdx.x] = 0;
    select_head<NTH>(scores + (int64_t)bh * score_stride, P, K, n_sink, n_local, idx + (int64_t)bh * idx_stride, budget,
                     sel_smem);
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
    if (P > kTopkThreads * kTopkMaxPerThread) return cudaErrorInvalidValue;
    // the keys of a head live in dynamic shared memory: allow the largest head once per device
    static bool ready[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!ready[dev]) {
        e = cudaFuncSetAttribute(topk_select_kernel<kTopkThreads>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)select_smem_bytes(kTopkThreads * kTopkMaxPerThread));
        if (e != cudaSuccess) return e;
        ready[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)BH);
    cfg.blockDim = dim3(kTopkThreads);
    cfg.dynamicSmemBytes = select_smem_bytes(P);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int64_t stride = a.page_cap;
    return cudaLaunchKernelEx(&cfg, topk_select_kernel<kTopkThreads>, scores, stride, P, K, ns, nl, idx, idx_stride,
                              budget, attend_ctr);
}

}  // namespace rq
