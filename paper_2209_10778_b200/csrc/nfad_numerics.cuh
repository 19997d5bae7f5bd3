// nfad_numerics.cuh -- fp32 building blocks under the dual-number primitives.
//
// Two precision policies:
//   Full  for fp32 storage: results good to about an fp32 ulp.  Pure IEEE
//         arithmetic (add, mul, fmaf) plus one reciprocal seed that is refined
//         at once, with values carried as unevaluated sums hi + lo ("two-float")
//         wherever a rounding would otherwise be amplified or accumulated.
//         This code relies on error-free transformations and must be compiled
//         with floating-point contraction OFF (-fmad=false).
//   Fast  for bf16 / fp16 storage: results good to a few fp32 ulp, i.e. to
//         ~2^-13 of a 16-bit ulp.  Built on MUFU ex2 / rcp; no compensation.
//
// Every exponential here has a non-positive argument: the callers evaluate
// exp(-|v|) and pick the branch by sign, which is what keeps sigmoid, tanh and
// the normal CDF free of cancellation in both tails.
#pragma once

#ifndef NFAD_HW_PROVIDED
#include "nfad_hw.cuh"
#endif

namespace nfad {

struct Full {};
struct Fast {};

// ---------------------------------------------------------------- two-float arithmetic

// An unevaluated sum h + l, |l| << |h| (not necessarily normalised).
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

NFAD_DEV float f2_value(F2 a) { return a.h + a.l; }

// products and sums good to ~2^-44 relative
NFAD_DEV F2 f2_mul(F2 a, float b)
{
    F2 p = two_prod(a.h, b);
    p.l = fmaf(a.l, b, p.l);
    return p;
}
NFAD_DEV F2 f2_mul(F2 a, F2 b)
{
    F2 p = two_prod(a.h, b.h);
    p.l = fmaf(a.h, b.l, fmaf(a.l, b.h, p.l));
    return p;
}
NFAD_DEV F2 f2_add(F2 a, F2 b)
{
    F2 s = two_sum(a.h, b.h);
    s.l += a.l + b.l;
    return s;
}
// c + a for |c| >= |a.h|
NFAD_DEV F2 f2_add_big(float c, F2 a)
{
    F2 s = fast_two_sum(c, a.h);
    s.l += a.l;
    return s;
}

// 1/(d.h + d.l) as a two-float: MUFU seed, one Newton step carried in the low part.
NFAD_DEV F2 f2_rcp(F2 d)
{
    float r0 = hw::rcp_approx(d.h);
    float rho = fmaf(-d.h, r0, 1.0f);
    rho = fmaf(-d.l, r0, rho);                 // 1 - d r0, exact to ~2^-48
    float rh = fmaf(r0, rho, r0);
    float rl = fmaf(r0, rho, r0 - rh);         // what the rounding of rh dropped
    return {rh, rl};
}

// ---------------------------------------------------------------- powers of two

// 2^n as a float, n clamped to the normal range below (n <= 0 in every use).
NFAD_DEV float pow2_clamped(int n)
{
    n = n < -126 ? -126 : n;
    return hw::int_as_float((n + 127) << 23);
}

// v * 2^n with the scale applied in two steps, so that a result in the
// subnormal range is rounded exactly once.  n in [-250, 0].
NFAD_DEV float scale_pow2(float v, int n)
{
    int n1 = n < -100 ? -100 : n;
    int n2 = n - n1;
    n2 = n2 < -126 ? -126 : n2;
    float s1 = hw::int_as_float((n1 + 127) << 23);
    float s2 = hw::int_as_float((n2 + 127) << 23);
    return (v * s1) * s2;
}

// ---------------------------------------------------------------- exp, Full

// e^(ah+al) = 2^n (p.h + p.l), p in [0.70, 1.42], for -300 < ah <= 0 (|al| tiny
// against ah).  The power of two is NOT applied: callers multiply by it last,
// where it is exact, so that a result near or below 2^-126 is rounded once.
// Cody-Waite reduction a = n ln2 + r with the reduced argument kept as a pair, a
// degree-5 minimax for (e^r - 1 - r)/r^2, and the final 1 + r + r^2 q(r) summed
// without rounding loss.  p.h + p.l is good to ~2^-28 relative.
struct ExpParts { F2 p; int n; };

NFAD_DEV ExpParts exp_parts_full(float ah, float al)
{
    const float kLog2e = 1.44269502f;
    const float kMagic = 12582912.0f;          // 1.5 * 2^23: adding it rounds to an integer
    const float kLn2Hi = 0.693147182f;         // 0x3f317218
    const float kLn2Lo = -1.90465421e-09f;     // ln2 - kLn2Hi
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
    float w = fmaf(r * r, q, dl);              // e^(r+dl) - 1 - r, to first order in dl (|dl| < 2^-25)
    F2 g = fast_two_sum(r, w);
    float ph = 1.0f + g.h;
    float pl = (g.h - (ph - 1.0f)) + g.l;      // 1 + g = ph + pl exactly (|g.h| < 1)
    return {{ph, pl}, ni};
}

// Leaner variant: e^(ah+al) = 2^n (1 + g) with g one float (|g| < 0.42), good to ~0.4 units of
// 2^-24 relative to the result.  Callers multiply by (1 + g) with one fused multiply-add,
// m (1 + g) = fmaf(m, g, m), so that 1 + g itself is never rounded.
struct ExpG { float g; int n; };

NFAD_DEV ExpG exp_g_full(float ah, float al)
{
    const float kLog2e = 1.44269502f;
    const float kMagic = 12582912.0f;
    const float kLn2Hi = 0.693147182f;
    const float kLn2Lo = -1.90465421e-09f;
    float t = fmaf(ah, kLog2e, kMagic);
    float n = t - kMagic;
    int ni = hw::float_as_int(t) - 0x4B400000;
    float rh = fmaf(n, -kLn2Hi, ah);           // exact
    float r = rh + fmaf(n, -kLn2Lo, al);
    float q = 0.000199696486f;
    q = fmaf(q, r, 0.00139308674f);
    q = fmaf(q, r, 0.0083331801f);
    q = fmaf(q, r, 0.0416665077f);
    q = fmaf(q, r, 0.166666672f);
    q = fmaf(q, r, 0.5f);
    return {fmaf(r * r, q, r), ni};
}

// ---------------------------------------------------------------- exp, Fast


// ---------------------------------------------------------------- scaled complementary error function

// erfc(z)/2 = exp(-z^2) * W(z) for z >= 0, with W(z) = erfcx(z)/2.
// W(z) (z + k) is a smooth function of q = (z - k)/(z + k) in [-1, 1); it is
// fitted by one polynomial on z in [0, 10.8] (beyond that exp(-z^2) is zero in
// fp32), k = fl(3/sqrt2).  Returns W(z); the caller owns the exponential, so
// that the value Phi and the tangent phi share it.
NFAD_DEV F2 half_erfcx_full(float z)
{
    const float k = 2.1213202476501465f;
    F2 r = f2_rcp(two_sum(z, k));              // 1/(z+k)
    float q = fmaf(-2.0f * k, r.h, 1.0f);      // (z-k)/(z+k)
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
    // last Horner step c0 + q p without losing its rounding: the sum stays in [0.28, 1.07], so c0 - s.h is
    // exact and a second fused multiply-add returns what the first one rounded away
    const float c0 = 0.515540004f;
    F2 s;
    s.h = fmaf(p, q, c0);
    s.l = fmaf(p, q, c0 - s.h);
    return f2_mul(s, r);
}

// Fast policy: a degree-6 fit of the same function, weighted so that both W and the
// combination W - z/sqrt(pi) (which carries the cancellation of the GELU derivative for
// x < 0) keep a relative error below 2^-16, with every coefficient pre-multiplied by 2^-64.
// The caller's exponential carries the matching 2^+64 (so that it cannot underflow in
// MUFU's flush-to-zero range) and the product of the two is the first place where a result
// may become subnormal.  Returns 2^-64 W(z).
NFAD_DEV float half_erfcx_fast_scaled(float z)
{
    const float k = 2.1213202476501465f;
    const float s = 5.42101086e-20f;           // 2^-64
    float r = hw::rcp_approx(z + k);
    float q = fmaf(-2.0f * k, r, 1.0f);
    float p = 0.000961262616f * s;
    p = fmaf(p, q, 0.00436418364f * s);
    p = fmaf(p, q, -0.00761994533f * s);
    p = fmaf(p, q, -0.0332778953f * s);
    p = fmaf(p, q, 0.162689358f * s);
    p = fmaf(p, q, -0.36016348f * s);
    p = fmaf(p, q, 0.515539289f * s);
    return p * r;
}

// Fast exponential of a non-positive argument given in base 2: one MUFU.EX2 on the
// argument raised by 64, so that the flush-to-zero unit never sees a result below 2^-126
// until the true value is below 2^-190.  Returns 2^64 2^a.
constexpr float kTwoPowMinus64 = 5.42101086e-20f;
NFAD_DEV float exp2_fast_times_2p64(float a_plus_64) { return hw::ex2_approx_ftz(a_plus_64); }

}  // namespace nfad
