// Device helpers shared by the kernels: streaming 128-bit loads, storage-format
// unpacking to fp32, warp reductions.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace stmoe_dev {

constexpr int kWarp = 32;
constexpr unsigned kFull = 0xffffffffu;

// 16-byte load of weight data that is read exactly once per launch: bypass L1 so the
// activations that every row re-reads stay resident there.
__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Programmatic dependent launch.  pdl_wait: block until the kernel launched before this one
// in the stream has completed and its writes are visible (returns at once when the launch was
// an ordinary one).  pdl_launch_dependents: allow the next kernel in the stream, if it was
// launched with programmatic serialization, to start occupying SMs as this grid's CTAs retire.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

__device__ __forceinline__ float4 ld_f4(const float *p) { return *reinterpret_cast<const float4 *>(p); }

__device__ __forceinline__ float bf16_to_f32(uint16_t v) { return __uint_as_float((uint32_t)v << 16); }

// Storage formats.  kEpl = elements per 16-byte load.
template <int DT> struct Fmt;

template <> struct Fmt<0> {  // fp32
    static constexpr int kEpl = 4;
    static constexpr int kBytes = 4;
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&f)[4])
    {
        f[0] = __uint_as_float(v.x), f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z), f[3] = __uint_as_float(v.w);
    }
};

template <> struct Fmt<1> {  // bf16
    static constexpr int kEpl = 8;
    static constexpr int kBytes = 2;
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&f)[8])
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

template <> struct Fmt<2> {  // fp8 e4m3 (scale applied per row by the caller)
    static constexpr int kEpl = 16;
    static constexpr int kBytes = 1;
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&f)[16])
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t lo, hi;  // two packed f16x2
            asm("{.reg .b16 a, b;\n\t"
                "mov.b32 {a, b}, %2;\n\t"
                "cvt.rn.f16x2.e4m3x2 %0, a;\n\t"
                "cvt.rn.f16x2.e4m3x2 %1, b;}"
                : "=r"(lo), "=r"(hi)
                : "r"(w[i]));
            const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&lo));
            const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&hi));
            f[4 * i] = a.x, f[4 * i + 1] = a.y, f[4 * i + 2] = b.x, f[4 * i + 3] = b.y;
        }
    }
};

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
    return v;
}

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long t = __shfl_xor_sync(kFull, v, o);
        v = t > v ? t : v;
    }
    return v;
}

// Order-preserving map of a float onto an unsigned integer (larger float -> larger key).
__device__ __forceinline__ uint32_t float_key(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

}  // namespace stmoe_dev
