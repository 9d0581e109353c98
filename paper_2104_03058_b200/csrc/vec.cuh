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

// Two adjacent 16-byte vectors with one 32-byte load (p must be 32-byte aligned): half the load
// instructions and, when a lane's two vectors sit next to each other, half the cache lines touched
// per instruction.
__device__ __forceinline__ void load_pair(Vec<float, 4>& a, Vec<float, 4>& b, const float* p)
{
    uint32_t r[8];
    asm volatile("ld.global.nc.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "l"(p));
    a.v = make_float4(__uint_as_float(r[0]), __uint_as_float(r[1]), __uint_as_float(r[2]), __uint_as_float(r[3]));
    b.v = make_float4(__uint_as_float(r[4]), __uint_as_float(r[5]), __uint_as_float(r[6]), __uint_as_float(r[7]));
}
__device__ __forceinline__ void load_pair(Vec<__nv_bfloat16, 8>& a, Vec<__nv_bfloat16, 8>& b, const __nv_bfloat16* p)
{
    asm volatile("ld.global.nc.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(a.v.x), "=r"(a.v.y), "=r"(a.v.z), "=r"(a.v.w), "=r"(b.v.x), "=r"(b.v.y), "=r"(b.v.z), "=r"(b.v.w)
                 : "l"(p));
}
// scalar vectors have no pair form; never called (the callers test the vector width first)
template <typename T>
__device__ __forceinline__ void load_pair(Vec<T, 1>& a, Vec<T, 1>& b, const T* p) { a.load(p); b.load(p + 1); }

__device__ __forceinline__ void store_elem(void* out, int out_bf16, int64_t idx, float val)
{
    if (out_bf16) static_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16_rn(val);
    else __stcs(static_cast<float*>(out) + idx, val);
}

}  // namespace gnnfd
