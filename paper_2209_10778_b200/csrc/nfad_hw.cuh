// nfad_hw.cuh -- the few places where the activation math names a hardware
// instruction.  Everything above this header is plain IEEE fp32 arithmetic
// (+, -, *, fmaf) compiled with contraction off, so its rounding behaviour is
// fixed by the source text alone.
#pragma once

#ifndef __CUDACC_RTC__
#include <cuda_runtime.h>
#endif

#define NFAD_DEV __device__ __forceinline__

namespace nfad {
namespace hw {

// 2^a, MUFU.EX2 with the scaling that keeps subnormal results (no flush to zero).
NFAD_DEV float ex2_approx(float a)
{
    float r;
    asm("ex2.approx.f32 %0, %1;" : "=f"(r) : "f"(a));
    return r;
}

// 2^a, one MUFU.EX2; results below 2^-126 are flushed to zero.
NFAD_DEV float ex2_approx_ftz(float a)
{
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(a));
    return r;
}

// min(max(a, lo), hi) that returns NaN for a NaN (plain fminf / fmaxf drop it).
NFAD_DEV float clamp_nan(float a, float lo, float hi)
{
    float r;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(lo));
    asm("min.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(r), "f"(hi));
    return r;
}

// log2(a), MUFU.LG2 (keeps subnormal inputs).
NFAD_DEV float lg2_approx(float a)
{
    float r;
    asm("lg2.approx.f32 %0, %1;" : "=f"(r) : "f"(a));
    return r;
}

// min(a, hi) that returns NaN for a NaN.
NFAD_DEV float min_nan(float a, float hi)
{
    float r;
    asm("min.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(hi));
    return r;
}

// max(a, lo) that returns NaN for a NaN.
NFAD_DEV float max_nan(float a, float lo)
{
    float r;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(lo));
    return r;
}

// 1/a for a normal a, MUFU.RCP (about 1 ulp).
NFAD_DEV float rcp_approx(float a)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(a));
    return r;
}

// 1/a for a normal double a: MUFU.RCP64H, an estimate from the upper word good to about 20 bits.
NFAD_DEV double rcp64_approx(double a)
{
    double r;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(r) : "d"(a));
    return r;
}

// the two 32-bit words of a double, and a double from them
NFAD_DEV int double_hi(double a) { return __double2hiint(a); }
NFAD_DEV int double_lo(double a) { return __double2loint(a); }
NFAD_DEV double double_from(int hi, int lo) { return __hiloint2double(hi, lo); }
// float -> double, exact (one conversion instruction on the special-function unit; forming the same bits with
// integer operations was measured 6-15 % slower: these kernels have no issue slots to spare for it)
NFAD_DEV double to_double(float x) { return double(x); }

// double -> float, round to nearest even (subnormal results included)
NFAD_DEV float to_float(double a) { return __double2float_rn(a); }

// Packed fp32: two independent IEEE operations (round to nearest even) in one instruction.
NFAD_DEV float2 fma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
NFAD_DEV float2 mul2(float2 a, float2 b) { return __fmul2_rn(a, b); }
NFAD_DEV float2 add2(float2 a, float2 b) { return __fadd2_rn(a, b); }

NFAD_DEV int float_as_int(float a) { return __float_as_int(a); }
NFAD_DEV float int_as_float(int a) { return __int_as_float(a); }

}  // namespace hw
}  // namespace nfad
