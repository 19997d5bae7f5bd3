// nfad_dual_fast.cuh -- the chains of the four activations under the Fast policy (16-bit storage), written ONCE for
// one element per call (policy `Fast`, lanes = float) and for two (policy `Fast2`, lanes = float2).
//
// Why two widths.  The 16-bit kernels are bound by instruction issue, not by memory: 15 to 25 instructions per
// element, more than half of them fp32 multiplies, adds and fused multiply-adds.  sm_100 has packed forms of those
// three (fma.rn.f32x2 and friends: two independent IEEE operations, one issue slot), so the same chain on a pair of
// elements needs half the issue slots for that part.  What has no packed form (the exponential and reciprocal units,
// min / max, selects, |x|) is issued once per lane, and a pair of registers per operand costs registers: pairs pay
// where a chain is long enough to be short of issue slots and a tile shape holds them without spilling (the GELU-erf
// kernels, the value-only GELU-tanh), and cost a few per cent elsewhere, so each kernel picks its width (nfad_ops.cuh).
//
// Every function below is a template over the policy and calls only the `ln::` operations, each of which is the same
// IEEE operation per lane in both widths (explicit fma / mul / add: nothing is left to contraction).  A lane of a pair
// therefore sees exactly the scalar operation sequence, and the two widths agree bit for bit.
//
// The algebra is the one of nfad_dual.cuh (Section II-C approach 3, Eq. 3; Section III-A): a dual number is
// (value, tangent) per lane, a primitive returns both from one exponential.  Only what the four activation chains
// need is here; sequences composed at run time use the general-purpose primitives of nfad_dual.cuh.
#pragma once

#include "nfad_numerics.cuh"

namespace nfad {

struct Fast2 {};

template <class P> struct Lanes {};                    // no lanes: the policy is not a Fast one
template <> struct Lanes<Fast> { using type = float; };
template <> struct Lanes<Fast2> { using type = float2; };

namespace ln {
// one element
NFAD_DEV float fma(float a, float b, float c) { return __fmaf_rn(a, b, c); }
NFAD_DEV float mul(float a, float b) { return __fmul_rn(a, b); }
NFAD_DEV float add(float a, float b) { return __fadd_rn(a, b); }
NFAD_DEV float ex2_ftz(float a) { return hw::ex2_approx_ftz(a); }
NFAD_DEV float rcp(float a) { return hw::rcp_approx(a); }
NFAD_DEV float abs(float a) { return fabsf(a); }
NFAD_DEV float clamp_nan(float a, float lo, float hi) { return hw::clamp_nan(a, lo, hi); }
NFAD_DEV float min_nan(float a, float hi) { return hw::min_nan(a, hi); }
NFAD_DEV float max_nan(float a, float lo) { return hw::max_nan(a, lo); }
NFAD_DEV float if_negative(float x, float a, float b) { return x < 0.0f ? a : b; }          // x < 0 ? a : b
// two elements
NFAD_DEV float2 bc(float c) { return make_float2(c, c); }
NFAD_DEV float2 fma(float2 a, float2 b, float2 c) { return hw::fma2(a, b, c); }
NFAD_DEV float2 fma(float2 a, float b, float c) { return hw::fma2(a, bc(b), bc(c)); }
NFAD_DEV float2 fma(float2 a, float b, float2 c) { return hw::fma2(a, bc(b), c); }
NFAD_DEV float2 fma(float2 a, float2 b, float c) { return hw::fma2(a, b, bc(c)); }
NFAD_DEV float2 mul(float2 a, float2 b) { return hw::mul2(a, b); }
NFAD_DEV float2 mul(float2 a, float b) { return hw::mul2(a, bc(b)); }
NFAD_DEV float2 add(float2 a, float2 b) { return hw::add2(a, b); }
NFAD_DEV float2 add(float2 a, float b) { return hw::add2(a, bc(b)); }
NFAD_DEV float2 ex2_ftz(float2 a) { return make_float2(hw::ex2_approx_ftz(a.x), hw::ex2_approx_ftz(a.y)); }
NFAD_DEV float2 rcp(float2 a) { return make_float2(hw::rcp_approx(a.x), hw::rcp_approx(a.y)); }
NFAD_DEV float2 abs(float2 a) { return make_float2(fabsf(a.x), fabsf(a.y)); }
NFAD_DEV float2 clamp_nan(float2 a, float lo, float hi) { return make_float2(hw::clamp_nan(a.x, lo, hi), hw::clamp_nan(a.y, lo, hi)); }
NFAD_DEV float2 min_nan(float2 a, float hi) { return make_float2(hw::min_nan(a.x, hi), hw::min_nan(a.y, hi)); }
NFAD_DEV float2 max_nan(float2 a, float lo) { return make_float2(hw::max_nan(a.x, lo), hw::max_nan(a.y, lo)); }
NFAD_DEV float2 if_negative(float2 x, float2 a, float2 b) { return make_float2(x.x < 0.0f ? a.x : b.x, x.y < 0.0f ? a.y : b.y); }
}  // namespace ln

// independent variables (one per lane), each with tangent exactly 1
template <class P> struct SeedOf { typename Lanes<P>::type x; };
template <> struct Dual<Fast2> { float2 v, t; };
template <> struct Gate<Fast2> { float2 v, t; };

// x * b:  value x b.v,  tangent b.v + x b.t   (Eq. 3); xv is the factor of the value's product, xt of the tangent's
// (they differ only in how far each is clamped: see evaluate)
template <class P> NFAD_DEV Gate<P> dual_mul(const SeedOf<P>& xv, const SeedOf<P>& xt, const Gate<P>& b)
{
    return {ln::mul(xv.x, b.v), ln::fma(xt.x, b.t, b.v)};
}

// c1 x + c3 x^3, tangent c1 + k3 x^2 (k3 = 3 c3, rounded once by the caller)
template <class P> NFAD_DEV Dual<P> dual_odd_cubic(P, float c1, float c3, float k3, const SeedOf<P>& a)
{
    auto s = ln::mul(a.x, a.x);
    return {ln::mul(a.x, ln::fma(s, c3, c1)), ln::fma(s, k3, c1)};
}

// L(w) = 1/(1+exp(-w)), L' = L (1 - L), one form for both signs.  E = 2^-64 exp(-w) comes from one exponential on the
// argument lowered by 64 (flushed to zero only where exp(-w) < 2^-62, far below what a 16-bit result keeps; the caller
// keeps scale * w >= -133, beyond which the slope's E r would be inf * 0); r = 1/(E + 2^-64); L = 2^-64 r and
// 1 - L = E r, with no subtraction anywhere, so both tails keep their relative accuracy.
// sigmoid of the seed: the slope is L (E r)
template <class P> NFAD_DEV Gate<P> dual_sigmoid(P, InRange, const SeedOf<P>& a)
{
    auto E = ln::ex2_ftz(ln::fma(a.x, -1.44269502f, -64.0f));
    auto r = ln::rcp(ln::add(E, kTwoPowMinus64));
    auto L = ln::mul(r, kTwoPowMinus64);
    return {L, ln::mul(L, ln::mul(E, r))};
}
// sigmoid of a dual w (the caller keeps w.v >= -133): the slope is L (E r) w'.  (1 + tanh u)/2 is this with w = 2u.
template <class P> NFAD_DEV Gate<P> dual_sigmoid(InRange, const Dual<P>& w)
{
    auto E = ln::ex2_ftz(ln::fma(w.v, -1.44269502f, -64.0f));
    auto r = ln::rcp(ln::add(E, kTwoPowMinus64));
    auto L = ln::mul(r, kTwoPowMinus64);
    return {L, ln::mul(ln::mul(L, ln::mul(E, r)), w.t)};
}

// 2^-64 W(z) from r = 1/(z + k): the fit described at half_erfcx_fast_scaled (nfad_numerics.cuh), per lane
template <int kDegree, class T> NFAD_DEV T half_erfcx_lanes_scaled(T r)
{
    const float k = kErfcxShift;
    const float s = 5.42101086e-20f;           // 2^-64
    T q = ln::fma(r, -2.0f * k, 1.0f);
    T p;
    if (kDegree == 6) {
        p = ln::fma(q, 0.000961262616f * s, 0.00436418364f * s);
        p = ln::fma(p, q, -0.00761994533f * s);
        p = ln::fma(p, q, -0.0332778953f * s);
        p = ln::fma(p, q, 0.162689358f * s);
        p = ln::fma(p, q, -0.36016348f * s);
        p = ln::fma(p, q, 0.515539289f * s);
    } else {
        p = ln::fma(q, -0.00805392209f * s, -0.0296229441f * s);
        p = ln::fma(p, q, 0.162969887f * s);
        p = ln::fma(p, q, -0.360796034f * s);
        p = ln::fma(p, q, 0.515540838f * s);
    }
    return ln::mul(p, r);
}

// H = (1 + erf(c x))/2 of the seed,  H' = c exp(-(c x)^2)/sqrt(pi).  With z = c |x|, E = exp(-z^2) and
// W = erfcx(z)/2:  erfc(z)/2 = E W, so  x < 0: H = E W,  x >= 0: H = 1 - E W, and the same E serves the tangent.
// E is formed as 2^64 E and W as 2^-64 W, so that neither underflows before their product does.
template <int kDegree, class P> NFAD_DEV Gate<P> dual_half_one_plus_erf_scaled(P, float c, const SeedOf<P>& x)
{
    const float kInvSqrtPiScaled = 0.564189612865448f * 5.42101086e-20f;
    auto xa = ln::abs(x.x);
    auto e64 = ln::ex2_ftz(ln::fma(ln::mul(xa, xa), (c * c) * -1.44269502f, 64.0f));
    auto a = ln::mul(e64, half_erfcx_lanes_scaled<kDegree>(ln::rcp(ln::fma(xa, c, kErfcxShift))));
    return {ln::if_negative(x.x, a, ln::fma(a, -1.0f, 1.0f)), ln::mul(e64, kInvSqrtPiScaled * c)};
}

// softplus hands w = exp(x) to tanh (x <= 20 by the caller's clamp): every later use of softplus in the Mish chain is
// an algebraic function of w, so the logarithm itself is never needed.  w is formed as 2^-64 (2^64 w) so that a result
// below 2^-126 is rounded by the multiplier and not flushed by the exponential unit.
template <> struct SoftplusDual<Fast> { float w; };
template <> struct SoftplusDual<Fast2> { float2 w; };
template <class P> NFAD_DEV SoftplusDual<P> dual_softplus(P, const SeedOf<P>& a)
{
    return {ln::mul(ln::ex2_ftz(ln::fma(a.x, 1.44269502f, 64.0f)), kTwoPowMinus64)};
}
// tanh(log1p(w)) = ((1+w)^2 - 1)/((1+w)^2 + 1) = n/(n + 2), n = w (w + 2): one form for both signs, every term
// positive.  T' = (dn/dx) 2/(n + 2)^2 = 4 w (w + 1)/(n + 2)^2.  Formed with the halves h = (w + 2)/2, m = n/2 = w h and
// r = 2/(n + 2) = 1/(w h + 1), so that no factor 2 or 4 costs an operation:  T = m r,  T' = (w r) (w r + r).
// Needs w <= 2^29 (x <= 20), so that the factors stay inside fp32's range.
template <class P> NFAD_DEV Gate<P> dual_tanh_of_softplus(const SoftplusDual<P>& p)
{
    auto w = p.w;
    auto h = ln::fma(w, 0.5f, 1.0f);
    auto r = ln::rcp(ln::fma(w, h, 1.0f));
    return {ln::mul(ln::mul(w, h), r), ln::mul(ln::mul(w, r), ln::fma(w, r, r))};
}
NFAD_DEV Gate<Fast> dual_tanh(const SoftplusDual<Fast>& p) { return dual_tanh_of_softplus<Fast>(p); }
NFAD_DEV Gate<Fast2> dual_tanh(const SoftplusDual<Fast2>& p) { return dual_tanh_of_softplus<Fast2>(p); }

}  // namespace nfad
