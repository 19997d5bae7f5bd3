// nfad_hw.cuh -- the few places where the activation math names a hardware
// instruction.  Everything above this header is plain IEEE fp32 arithmetic
// (+, -, *, fmaf) compiled with contraction off, so its rounding behaviour is
// fixed by the source text alone.
#pragma once

#include <cuda_runtime.h>

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

// 1/a for a normal a, MUFU.RCP (about 1 ulp).
NFAD_DEV float rcp_approx(float a)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(a));
    return r;
}

NFAD_DEV int float_as_int(float a) { return __float_as_int(a); }
NFAD_DEV float int_as_float(int a) { return __int_as_float(a); }

}  // namespace hw
}  // namespace nfad
