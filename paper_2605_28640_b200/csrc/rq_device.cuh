// Device-side helpers: 128-bit vector access for bf16 / fp32 rows, conversion,
// order-preserving keys.  sm_100a only.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rq {

typedef __nv_bfloat16 bf16;

// Number of elements of T in one 16-byte vector.
template <typename T> struct VecOf { static constexpr int N = 16 / sizeof(T); };

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Round-to-nearest-even pack of two floats into one bf16x2 word (lo = a).
__device__ __forceinline__ uint32_t pack_bf16(float a, float b)
{
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&h);
}

// ---- raw 16-byte loads (read-only path) ----
__device__ __forceinline__ uint4 ldg16(const void *p) { return __ldg(reinterpret_cast<const uint4 *>(p)); }
// streaming variant: data that is read once
__device__ __forceinline__ uint4 ldcs16(const void *p) { return __ldcs(reinterpret_cast<const uint4 *>(p)); }

// Expand one 16-byte vector of T into floats.
// Two fp32 operations in one instruction (packed pairs); each half is rounded like the scalar operation, so the
// results are the same bits as two scalar instructions.
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c)
{
    unsigned long long ra = *reinterpret_cast<unsigned long long *>(&a), rb = *reinterpret_cast<unsigned long long *>(&b),
                       rc = *reinterpret_cast<unsigned long long *>(&c), rd;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd) : "l"(ra), "l"(rb), "l"(rc));
    return *reinterpret_cast<float2 *>(&rd);
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b)
{
    unsigned long long ra = *reinterpret_cast<unsigned long long *>(&a), rb = *reinterpret_cast<unsigned long long *>(&b), rd;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(ra), "l"(rb));
    return *reinterpret_cast<float2 *>(&rd);
}

template <typename T> __device__ __forceinline__ void unpack16(const uint4 &r, float *out);
template <> __device__ __forceinline__ void unpack16<bf16>(const uint4 &r, float *out)
{
    out[0] = bf16lo(r.x); out[1] = bf16hi(r.x);
    out[2] = bf16lo(r.y); out[3] = bf16hi(r.y);
    out[4] = bf16lo(r.z); out[5] = bf16hi(r.z);
    out[6] = bf16lo(r.w); out[7] = bf16hi(r.w);
}
template <> __device__ __forceinline__ void unpack16<float>(const uint4 &r, float *out)
{
    out[0] = __uint_as_float(r.x); out[1] = __uint_as_float(r.y);
    out[2] = __uint_as_float(r.z); out[3] = __uint_as_float(r.w);
}

// Round floats to T (RNE) and pack into one 16-byte vector.
template <typename T> __device__ __forceinline__ uint4 pack16(const float *in);
template <> __device__ __forceinline__ uint4 pack16<bf16>(const float *in)
{
    uint4 r;
    r.x = pack_bf16(in[0], in[1]); r.y = pack_bf16(in[2], in[3]);
    r.z = pack_bf16(in[4], in[5]); r.w = pack_bf16(in[6], in[7]);
    return r;
}
template <> __device__ __forceinline__ uint4 pack16<float>(const float *in)
{
    uint4 r;
    r.x = __float_as_uint(in[0]); r.y = __float_as_uint(in[1]);
    r.z = __float_as_uint(in[2]); r.w = __float_as_uint(in[3]);
    return r;
}

// Value that storage type T holds for x, widened back to float.
template <typename T> __device__ __forceinline__ float round_storage(float x);
template <> __device__ __forceinline__ float round_storage<bf16>(float x)
{
    return __bfloat162float(__float2bfloat16_rn(x));
}
template <> __device__ __forceinline__ float round_storage<float>(float x) { return x; }

// Scalar element access.
template <typename T> __device__ __forceinline__ float load1(const T *p);
template <> __device__ __forceinline__ float load1<bf16>(const bf16 *p) { return __bfloat162float(*p); }
template <> __device__ __forceinline__ float load1<float>(const float *p) { return *p; }
template <typename T> __device__ __forceinline__ void store1(T *p, float x);
template <> __device__ __forceinline__ void store1<bf16>(bf16 *p, float x) { *p = __float2bfloat16_rn(x); }
template <> __device__ __forceinline__ void store1<float>(float *p, float x) { *p = x; }

// Load N consecutive elements of G (N*sizeof(G) in {8, 16, 32} bytes, aligned
// to that size or to 16) as floats.
template <typename G, int N> __device__ __forceinline__ void load_n(const G *p, float *out)
{
    constexpr int BYTES = N * (int)sizeof(G);
    if constexpr (BYTES == 16) {
        uint4 r = ldg16(p);
        unpack16<G>(r, out);
    } else if constexpr (BYTES == 32) {
        uint4 r0 = ldg16(p);
        uint4 r1 = ldg16(reinterpret_cast<const char *>(p) + 16);
        unpack16<G>(r0, out);
        unpack16<G>(r1, out + N / 2);
    } else {
        static_assert(BYTES == 8, "unsupported vector width");
        uint2 r = __ldg(reinterpret_cast<const uint2 *>(p));
        if constexpr (sizeof(G) == 2) {
            out[0] = bf16lo(r.x); out[1] = bf16hi(r.x);
            out[2] = bf16lo(r.y); out[3] = bf16hi(r.y);
        } else {
            out[0] = __uint_as_float(r.x); out[1] = __uint_as_float(r.y);
        }
    }
}

// Monotone map float -> uint32: a < b  <=>  key(a) < key(b); -0 and +0 collapse.
__device__ __forceinline__ uint32_t order_key(float x)
{
    uint32_t b = __float_as_uint(x + 0.0f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// the float a key was made from (inverse of order_key)
__device__ __forceinline__ float order_key_value(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

}  // namespace rq
