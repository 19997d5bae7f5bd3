// nfad_numerics.cuh -- fp32 building blocks under the dual-number primitives.
//
// Two precision policies:
//   Full  for fp32 storage: results good to about an fp32 ulp.  Pure IEEE
//         arithmetic (add, mul, fmaf and one refined reciprocal), arguments and
//         selected intermediates carried as unevaluated sums hi + lo.  This code
//         relies on error-free transformations and must be compiled with
//         floating-point contraction OFF (-fmad=false).
//   Fast  for bf16 / fp16 storage: results good to a few fp32 ulp, i.e. ~2^-13
//         of a 16-bit ulp.  Built on MUFU ex2 / rcp; no compensation.
//
// Every exponential here has a non-positive argument: the callers evaluate
// exp(-|v|) and pick the branch by sign, which is what keeps sigmoid, tanh and
// the normal CDF free of cancellation in both tails.
#pragma once

#ifndef NFAD_HW_PROVIDED
#include "nfad_hw.cuh"
#endif

namespace nfad {

struct Full { static constexpr bool kCompensated = true; };
struct Fast { static constexpr bool kCompensated = false; };

// An unevaluated sum h + l.
struct F2 { float h, l; };

// a*b = h + l exactly.
NFAD_DEV F2 two_prod(float a, float b)
{
    float h = a * b;
    return {h, fmaf(a, b, -h)};
}

// a+b = h + l exactly, given |a| >= |b| (or a == 0).
NFAD_DEV F2 fast_two_sum(float a, float b)
{
    float h = a + b;
    return {h, b - (h - a)};
}

// a+b = h + l exactly, any magnitudes.
NFAD_DEV F2 two_sum(float a, float b)
{
    float h = a + b;
    float bb = h - a;
    return {h, (a - (h - bb)) + (b - bb)};
}

// v * 2^n with the scale applied in two steps so that a subnormal result is
// rounded once.  n in [-250, 250].
NFAD_DEV float scale_pow2(float v, int n)
{
    int n1 = n < -100 ? -100 : (n > 100 ? 100 : n);
    int n2 = n - n1;
    n2 = n2 < -126 ? -126 : n2;
    float s1 = hw::int_as_float((n1 + 127) << 23);
    float s2 = hw::int_as_float((n2 + 127) << 23);
    return (v * s1) * s2;
}

// ---------------------------------------------------------------- exp, Full

// e^(ah+al) = h + l for any finite ah (|al| tiny against ah).  Cody-Waite
// reduction a = n ln2 + r with the reduced argument kept as a pair, a degree-5
// minimax for (e^r - 1 - r)/r^2, and the final 1 + r + r^2 q(r) summed without
// rounding loss.  |error| of h + l is ~2^-28 relative; h alone is the rounded
// value (<= 0.5 ulp + 2^-28).  Results below 2^-126 lose l.
NFAD_DEV F2 exp_full(float ah, float al)
{
    const float kLog2e = 1.44269502f;
    const float kMagic = 12582912.0f;          // 1.5 * 2^23: adding it rounds to an integer
    const float kLn2Hi = 0.693147182f;         // 0x3f317218
    const float kLn2Lo = -1.90465421e-09f;     // ln2 - kLn2Hi
    ah = ah < -170.0f ? -170.0f : (ah > 100.0f ? 100.0f : ah);
    float t = fmaf(ah, kLog2e, kMagic);
    float n = t - kMagic;
    int ni = hw::float_as_int(t) - 0x4B400000;
    float rh = fmaf(n, -kLn2Hi, ah);           // exact
    float rl = fmaf(n, -kLn2Lo, al);
    float r = rh + rl;
    float dl = (rh - r) + rl;                  // what the rounding of r dropped
    float q = 0.000199696486f;
    q = fmaf(q, r, 0.00139308674f);
    q = fmaf(q, r, 0.0083331801f);
    q = fmaf(q, r, 0.0416665077f);
    q = fmaf(q, r, 0.166666672f);
    q = fmaf(q, r, 0.5f);
    float w = fmaf(r * r, q, dl);              // e^(r+dl) - 1 - r, to first order in dl
    F2 g = fast_two_sum(r, w);
    float ph = 1.0f + g.h;
    float pl = (g.h - (ph - 1.0f)) + g.l;      // 1 + g = ph + pl exactly (|g.h| < 1)
    return {scale_pow2(ph, ni), scale_pow2(pl, ni)};
}

// ---------------------------------------------------------------- exp, Fast

// 2^a for a <= 0 (a already multiplied by log2 e by the caller).
NFAD_DEV float exp2_fast(float a) { return hw::ex2_approx(a); }

// ---------------------------------------------------------------- logistic pair

// For e = exp(-|v|) in (0, 1]:  big = 1/(1+e),  small = e/(1+e) = 1 - big.
// sigmoid(v) is `big` for v >= 0 and `small` for v < 0; its complement is the other.
struct LogisticPair { float big, small_; };

NFAD_DEV LogisticPair logistic_pair_full(F2 e)
{
    float dh = 1.0f + e.h;
    float dl = (e.h - (dh - 1.0f)) + e.l;      // 1 + e = dh + dl
    float r0 = hw::rcp_approx(dh);
    float rho = fmaf(-dh, r0, 1.0f);
    rho = fmaf(-dl, r0, rho);                  // 1 - (dh+dl) r0
    float rh = fmaf(r0, rho, r0);              // 1/(1+e), ~0.5 ulp
    float rl = fmaf(r0, rho, r0 - rh);         // and what that rounding dropped
    float sm = fmaf(e.h, rh, fmaf(e.h, rl, e.l * rh));
    return {rh, sm};
}

NFAD_DEV LogisticPair logistic_pair_fast(float e)
{
    float r = hw::rcp_approx(1.0f + e);
    return {r, e * r};
}

// ---------------------------------------------------------------- scaled complementary error function

// erfc(z)/2 = exp(-z^2) * W(z) for z >= 0, with W(z) = erfcx(z)/2.
// W(z) (z + k) is a smooth function of q = (z - k)/(z + k) in [-1, 1); it is
// fitted by one polynomial on z in [0, 10.8] (beyond that exp(-z^2) is zero in
// fp32).  k = fl(3/sqrt2).  Returns W(z); the caller owns the exponential, so
// that the value Phi and the tangent phi share it.
NFAD_DEV float half_erfcx_full(float z)
{
    const float k = 2.1213202476501465f;
    F2 d = two_sum(z, k);                      // z + k exactly
    float r0 = hw::rcp_approx(d.h);
    float rho = fmaf(-d.h, r0, 1.0f);
    rho = fmaf(-d.l, r0, rho);
    float r = fmaf(r0, rho, r0);               // 1/(z+k)
    float q = fmaf(-2.0f * k, r, 1.0f);        // (z-k)/(z+k)
    float p = 4.23795245e-05f;
    p = fmaf(p, q, 9.49347959e-05f);
    p = fmaf(p, q, -0.0001815203f);
    p = fmaf(p, q, -0.000733935158f);
    p = fmaf(p, q, 0.000731255859f);
    p = fmaf(p, q, 0.00493023125f);
    p = fmaf(p, q, -0.00740043446f);
    p = fmaf(p, q, -0.0334202126f);
    p = fmaf(p, q, 0.162647396f);
    p = fmaf(p, q, -0.360152066f);
    p = fmaf(p, q, 0.515540004f);
    return p * r;
}

NFAD_DEV float half_erfcx_fast(float z)
{
    const float k = 2.1213202476501465f;
    float r = hw::rcp_approx(z + k);
    float q = fmaf(-2.0f * k, r, 1.0f);
    float p = -0.00018698952f;
    p = fmaf(p, q, -0.000633997901f);
    p = fmaf(p, q, 0.000762930082f);
    p = fmaf(p, q, 0.00489306729f);
    p = fmaf(p, q, -0.00741203828f);
    p = fmaf(p, q, -0.0334145501f);
    p = fmaf(p, q, 0.162648439f);
    p = fmaf(p, q, -0.360152334f);
    p = fmaf(p, q, 0.515540004f);
    return p * r;
}

}  // namespace nfad
