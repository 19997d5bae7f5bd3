// nfad_numerics.cuh -- building blocks under the dual-number primitives.
//
// Two precision policies:
//   Fast  for bf16 / fp16 storage: plain fp32 on MUFU ex2 / rcp, results good to a few fp32 ulp,
//         i.e. to ~2^-13 of a 16-bit ulp.
//   Wide  for fp32 storage: double precision (nfad_dual_wide.cuh), results within a rounding of
//         the exact value; the one rounding is the final conversion to fp32.
//
// No exponential here is used to form 1 - sigmoid, 1 + tanh or 1 + erf by subtraction: each
// gate has a form in which both tails keep their relative accuracy.
#pragma once

#ifndef NFAD_HW_PROVIDED
#include "nfad_hw.cuh"
#endif

namespace nfad {

struct Fast {};
struct Wide {};

// ---------------------------------------------------------------- scaled complementary error function, Fast
//
// erfc(z)/2 = exp(-z^2) * W(z) for z >= 0, with W(z) = erfcx(z)/2.  W(z) (z + k) is a smooth
// function of q = (z - k)/(z + k) in [-1, 1), k = fl(3/sqrt2); it is fitted by one polynomial on
// z in [0, 10.8] (beyond that exp(-z^2) is zero in fp32).  The caller owns the exponential, so
// that the value Phi and the tangent phi share it.
//
// Every coefficient is pre-multiplied by 2^-64.  The caller's exponential carries the matching
// 2^+64 (so that it cannot underflow in MUFU's flush-to-zero range) and the product of the two is
// the first place where a result may become subnormal.  Returns 2^-64 W(z).
//   degree 6: weighted so that both W and the combination W - z/sqrt(pi) (which carries the
//             cancellation of the GELU derivative for x < 0) keep a relative error below 2^-16;
//   degree 4: W alone to 2^-12.3, enough for a 16-bit VALUE (a quarter of an fp16 ulp).
constexpr float kErfcxShift = 2.1213202476501465f;     // k
// r = 1/(z + k), formed by the caller (who may fold a scale of z into that sum)
template <int kDegree> NFAD_DEV float half_erfcx_fast_scaled(float r)
{
    const float k = kErfcxShift;
    const float s = 5.42101086e-20f;           // 2^-64
    float q = fmaf(-2.0f * k, r, 1.0f);
    float p;
    if (kDegree == 6) {
        p = 0.000961262616f * s;
        p = fmaf(p, q, 0.00436418364f * s);
        p = fmaf(p, q, -0.00761994533f * s);
        p = fmaf(p, q, -0.0332778953f * s);
        p = fmaf(p, q, 0.162689358f * s);
        p = fmaf(p, q, -0.36016348f * s);
        p = fmaf(p, q, 0.515539289f * s);
    } else {
        p = -0.00805392209f * s;
        p = fmaf(p, q, -0.0296229441f * s);
        p = fmaf(p, q, 0.162969887f * s);
        p = fmaf(p, q, -0.360796034f * s);
        p = fmaf(p, q, 0.515540838f * s);
    }
    return p * r;
}

// Fast exponential of an argument given in base 2 and raised by 64: one MUFU.EX2, so that the
// flush-to-zero unit never sees a result below 2^-126 until the true value is below 2^-190.
// Returns 2^64 2^a.
constexpr float kTwoPowMinus64 = 5.42101086e-20f;
NFAD_DEV float exp2_fast_times_2p64(float a_plus_64) { return hw::ex2_approx_ftz(a_plus_64); }

}  // namespace nfad
