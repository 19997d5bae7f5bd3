// nfad_storage.cuh -- the three storage types (how a 16-byte packet widens to fp32 values and narrows
// back with one round-to-nearest-even) and the cache-hinted packet accesses.  Device code only, with no
// dependence on the CUDA runtime headers, so that kernels generated at run time can include it too.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#ifdef __CUDACC_RTC__
typedef unsigned int uint32_t;
typedef unsigned long long uint64_t;
typedef unsigned long long uintptr_t;
#else
#include <stdint.h>
#endif

namespace nfad {

// Resident CTAs per SM the compiler must leave room for (a register cap).  The 16-bit kernels
// are issue-bound with short dependency chains through MUFU: 5 CTAs (40 warps, <= 48 registers)
// measured 3-5 % faster than the 4 the compiler picks by itself (7 or more spill and lose 30 %); the fp32-storage kernels
// hold their chains in double precision and need 64 registers (4 CTAs; a tighter cap spills, a looser one measured slower).

// ---------------------------------------------------------------- storage types

struct StoreF32 {
    using elem = float;
    static constexpr int kVec = 4;             // elements per 16-byte packet
    static constexpr int kMinBlocks = 4;
    static __device__ __forceinline__ void unpack(const uint4& p, float (&v)[4])
    {
        v[0] = __uint_as_float(p.x); v[1] = __uint_as_float(p.y);
        v[2] = __uint_as_float(p.z); v[3] = __uint_as_float(p.w);
    }
    static __device__ __forceinline__ uint4 pack(const float (&v)[4])
    {
        return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
    }
    static __device__ __forceinline__ float load1(const elem* p) { return *p; }
    static __device__ __forceinline__ void store1(elem* p, float v) { *p = v; }
};

struct StoreBF16 {
    using elem = __nv_bfloat16;
    static constexpr int kVec = 8;
    static constexpr int kMinBlocks = 5;
    // a bf16 is the upper half of an fp32: widening is a shift or a mask
    static __device__ __forceinline__ void unpack(const uint4& p, float (&v)[8])
    {
        const uint32_t w[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ uint32_t pack2(float lo, float hi)
    {
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);   // cvt.rn.bf16x2.f32: round to nearest even
        return *reinterpret_cast<uint32_t*>(&h);
    }
    static __device__ __forceinline__ uint4 pack(const float (&v)[8])
    {
        return make_uint4(pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
    }
    static __device__ __forceinline__ float load1(const elem* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void store1(elem* p, float v) { *p = __float2bfloat16_rn(v); }
};

struct StoreF16 {
    using elem = __half;
    static constexpr int kVec = 8;
    static constexpr int kMinBlocks = 5;
    static __device__ __forceinline__ void unpack(const uint4& p, float (&v)[8])
    {
        const uint32_t w[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
            v[2 * i] = f.x;
            v[2 * i + 1] = f.y;
        }
    }
    static __device__ __forceinline__ uint32_t pack2(float lo, float hi)
    {
        __half2 h = __floats2half2_rn(lo, hi);              // cvt.rn.f16x2.f32
        return *reinterpret_cast<uint32_t*>(&h);
    }
    static __device__ __forceinline__ uint4 pack(const float (&v)[8])
    {
        return make_uint4(pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
    }
    static __device__ __forceinline__ float load1(const elem* p) { return __half2float(*p); }
    static __device__ __forceinline__ void store1(elem* p, float v) { *p = __float2half_rn(v); }
};

// ---------------------------------------------------------------- memory access with cache hints

// Inputs are read once: streaming (evict-first) loads.
__device__ __forceinline__ uint4 load_packet(const uint4* p) { return __ldcs(p); }

// Output slot `keep`: true for a tensor the next kernel reads at once (y, grad_in),
// false for one that is read much later or never by this stream (the saved f').
template <bool kKeep> __device__ __forceinline__ void store_packet(uint4* p, const uint4& v)
{
    if (kKeep) *p = v;
    else __stcs(p, v);
}

}  // namespace nfad
