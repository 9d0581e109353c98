// Per-lane vectors of the gather kernels (16-byte or scalar loads of fp32 / bf16 features, widened to
// fp32) and the element store shared by them.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace gnnfd {

// ---- per-lane vectors: VECN elements of T, widened to fp32

template <typename T, int VECN> struct Vec;

template <> struct Vec<float, 4> {
    float4 v;
    __device__ __forceinline__ void load(const float* p) { v = __ldg(reinterpret_cast<const float4*>(p)); }
    __device__ __forceinline__ void zero() { v = make_float4(0.f, 0.f, 0.f, 0.f); }
    __device__ __forceinline__ float get(int i) const { return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w; }
};
template <> struct Vec<float, 1> {
    float v;
    __device__ __forceinline__ void load(const float* p) { v = __ldg(p); }
    __device__ __forceinline__ void zero() { v = 0.f; }
    __device__ __forceinline__ float get(int) const { return v; }
};
template <> struct Vec<__nv_bfloat16, 8> {
    uint4 v;
    __device__ __forceinline__ void load(const __nv_bfloat16* p) { v = __ldg(reinterpret_cast<const uint4*>(p)); }
    __device__ __forceinline__ void zero() { v = make_uint4(0u, 0u, 0u, 0u); }
    __device__ __forceinline__ float get(int i) const
    {
        const uint32_t w = (i >> 1) == 0 ? v.x : (i >> 1) == 1 ? v.y : (i >> 1) == 2 ? v.z : v.w;
        return __uint_as_float((i & 1) ? (w & 0xffff0000u) : (w << 16));   // bf16 -> fp32 is exact
    }
};
template <> struct Vec<__nv_bfloat16, 1> {
    unsigned short v;
    __device__ __forceinline__ void load(const __nv_bfloat16* p) { v = __ldg(reinterpret_cast<const unsigned short*>(p)); }
    __device__ __forceinline__ void zero() { v = 0; }
    __device__ __forceinline__ float get(int) const { return __uint_as_float((uint32_t)v << 16); }
};

__device__ __forceinline__ void store_elem(void* out, int out_bf16, int64_t idx, float val)
{
    if (out_bf16) static_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16_rn(val);
    else __stcs(static_cast<float*>(out) + idx, val);
}

}  // namespace gnnfd
