// nfad_dual_wide.cuh -- the dual-number algebra in double precision (policy `Wide`), used for fp32 storage.
//
// Why doubles for fp32 tensors.  The tolerance of the pass is a few fp32 ulp of an fp64 oracle, for the value
// f(x) and for f'(x) = h + x h', whose two terms cancel on the negative axis.  Holding that with fp32 arithmetic
// alone takes error-free transformations around every sensitive step (the exponential's argument, the
// reciprocal, the products that feed the cancellation): 60 to 120 instructions per element, which made these
// kernels issue-bound far below the memory roofline.  This part executes fp64 fused multiply-adds at half the
// fp32 rate, and in double precision every step is a single instruction with 29 spare bits: a chain is 25 to 35
// fp64 operations, results are within a rounding of the oracle (the one rounding is the final conversion to
// fp32, which also rounds a subnormal result exactly once), and nothing needs compensation.
//
// The algebra is the same as under the Fast policy (Section II-C approach 3, Eq. 3; Section III-A for the
// primitive set): a primitive returns its value and its derivative together, sharing the one exponential that
// both need, in forms where 1 - sigmoid, 1 + tanh and 1 + erf are never formed by subtraction.
#pragma once

#include "nfad_numerics.cuh"

namespace nfad {

namespace wide {

// 1/d for a normal d > 0: the hardware's estimate from the upper word (about 20 bits) refined by Newton steps;
// one step leaves a relative error near 2^-40 (what the four activations need), two go below 2^-52.
template <int kSteps = 2> NFAD_DEV double rcp(double d)
{
    double r = hw::rcp64_approx(d);
#pragma unroll
    for (int i = 0; i < kSteps; ++i) {
        double e = fma(-d, r, 1.0);
        r = fma(r, e, r);
    }
    return r;
}

// e^a for |a| <= 700: a = n ln2 + r with |r| <= ln2/2 (n taken from the low word of a sum with 1.5 * 2^52), a minimax
// polynomial for e^r, and 2^n added into the exponent field (the result stays normal for |a| <= 700; every caller keeps
// its argument inside that).  Degree 6 leaves a relative error of 2^-29 (a thirtieth of an fp32 ulp: what the four
// activations need), degree 11 of 2^-55 (the general-purpose primitives, whose results other operations may cancel).
template <int kDegree> NFAD_DEV double exp_bounded(double a)
{
    const double kMagic = 6755399441055744.0;
    double t = fma(a, 1.4426950408889634, kMagic);
    double n = t - kMagic;
    int ni = hw::double_lo(t);
    double r = fma(n, -0.6931471805599453, a);
    if (kDegree != 6) r = fma(n, -2.3190468138462996e-17, r);      // the rest of ln2: |n| reaches 1000
    double p;
    if (kDegree == 6) {
        p = 0.0013836846134577057;
        p = fma(p, r, 0.008374815798301793);
        p = fma(p, r, 0.04166822556692284);
        p = fma(p, r, 0.16666420169946367);
        p = fma(p, r, 0.4999999207982802);
        p = fma(p, r, 1.0000000363231765);
        p = fma(p, r, 1.0000000005541663);
    } else {
        p = 2.5110095611886237e-08;
        p = fma(p, r, 2.7632715071632255e-07);
        p = fma(p, r, 2.7557240761739257e-06);
        p = fma(p, r, 2.4801485278370062e-05);
        p = fma(p, r, 0.00019841269890193705);
        p = fma(p, r, 0.0013888888952505406);
        p = fma(p, r, 0.008333333333319546);
        p = fma(p, r, 0.04166666666648738);
        p = fma(p, r, 0.1666666666666668);
        p = fma(p, r, 0.5000000000000019);
        p = fma(p, r, 1.0);
        p = fma(p, r, 1.0);
    }
    return hw::double_from(hw::double_hi(p) + (ni << 20), hw::double_lo(p));
}
NFAD_DEV double exp_neg(double a) { return exp_bounded<11>(a); }

// kappa e^(-g s) for s >= 0 with g s <= 700, to 2^-29: the degree-6 form of exp_bounded with both constants folded in,
// so that neither costs an operation.  -g s = n ln2 + r with r = -g r', r' = s + n ln2/g: the polynomial runs in r'
// with its coefficients multiplied by kappa (-g)^i (g and kappa are compile-time constants at every call).
NFAD_DEV double exp_neg_scaled(double s, double g, double kappa)
{
    const double kMagic = 6755399441055744.0;
    double t = fma(s, -g * 1.4426950408889634, kMagic);
    double n = t - kMagic;
    int ni = hw::double_lo(t);
    double rp = fma(n, 0.6931471805599453 / g, s);
    const double m = -g;
    double p = kappa * 0.0013836846134577057 * (m * m * m * m * m * m);
    p = fma(p, rp, kappa * 0.008374815798301793 * (m * m * m * m * m));
    p = fma(p, rp, kappa * 0.04166822556692284 * (m * m * m * m));
    p = fma(p, rp, kappa * 0.16666420169946367 * (m * m * m));
    p = fma(p, rp, kappa * 0.4999999207982802 * (m * m));
    p = fma(p, rp, kappa * 1.0000000363231765 * m);
    p = fma(p, rp, kappa * 1.0000000005541663);
    return hw::double_from(hw::double_hi(p) + (ni << 20), hw::double_lo(p));
}

// erfc(z)/2 = exp(-z^2) W(z) for z >= 0.  W(z) (z + k) is a smooth function of q = (z - k)/(z + k) in [-1, 1), fitted
// by one polynomial on z in [0, 15], k = 3/sqrt(2).  Returns W(z); the caller owns the exponential, so that value and
// slope share it.
//   half_erfcx:     everything in double, degree 22 (relative error 2^-52, the arithmetic's), for the general-purpose erf;
//   half_erfcx_mix: r = 1/(z + k) and the final product in double, the polynomial itself in fp32 on the otherwise idle
//                   fp32 pipe (q in (-1, 1) and a result in [0.28, 1.07] make that a well-conditioned Horner chain: the
//                   result is good to about 0.8 fp32 ulp, which the activations' tolerance has room for).
NFAD_DEV double half_erfcx(double z)
{
    const double k = 2.1213202476501465;
    const double c[23] = {0.5155400178331069, -0.3601520858466969, 0.16264707189352245, -0.03341999312315092, -0.007398367634744453,
                          0.004930386718851745, 0.0007266182227491928, -0.0007395124001504905, -0.0001814263229256693,
                          0.00010917379216550876, 5.572919709637488e-05, -9.368798767498136e-06, -1.4631205627619127e-05,
                          -2.479590212362355e-06, 2.582014193120429e-06, 1.580743084650836e-06, -1.5835451846490903e-08,
                          -4.0458837978587706e-07, -1.5996308446846036e-07, 2.7211538400833845e-08, 3.937772165516381e-08,
                          1.0068658595420031e-08, 4.3545861799549443e-10};
    double r = rcp<2>(z + k);
    double q = fma(-2.0 * k, r, 1.0);
    double p = c[22];
#pragma unroll
    for (int i = 21; i >= 0; --i) p = fma(p, q, c[i]);
    return p * r;
}
// The argument is kappa (z + k) and the result W(z)/kappa, for any constant kappa > 0 the caller wants folded in.
NFAD_DEV double half_erfcx_mix(double z_plus_k_scaled, double kappa)
{
    double r = rcp<1>(z_plus_k_scaled);                                          // 1/(kappa (z + k))
    float q = hw::to_float(fma(-2.0 * 2.1213202476501465 * kappa, r, 1.0));      // (z - k)/(z + k)
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
    return double(p) * r;
}

// log(u) for a normal u > 0, relative error about 2^-45 away from u = 1 (absolute 2^-45 near it): u = 2^k m with m in
// [sqrt(1/2), sqrt(2)), log m = 2 atanh(s), s = (m - 1)/(m + 1).
NFAD_DEV double log_pos(double u)
{
    int hi = hw::double_hi(u);
    int k = (hi >> 20) - 1023;
    int mh = (hi & 0x000fffff) | 0x3ff00000;
    if (mh >= 0x3ff6a09e) { mh -= 0x00100000; k += 1; }     // m >= sqrt(2): halve it
    double m = hw::double_from(mh, hw::double_lo(u));
    double s = (m - 1.0) * rcp<2>(m + 1.0);
    double s2 = s * s;
    double p = 0.13333333333333333;                           // 2/15
    p = fma(p, s2, 0.15384615384615385);
    p = fma(p, s2, 0.18181818181818182);
    p = fma(p, s2, 0.22222222222222222);
    p = fma(p, s2, 0.2857142857142857);
    p = fma(p, s2, 0.4);
    p = fma(p, s2, 0.66666666666666663);
    p = fma(p, s2, 2.0);
    return fma(double(k), 0.6931471805599453, s * p);
}

}  // namespace wide

template <> struct Dual<Wide> { double v, t; };
template <> struct Gate<Wide> { double v, t; };

// the one rounding of each result: the conversion to fp32 (round to nearest even, subnormal results included)
NFAD_DEV float dual_value(const Dual<Wide>& a) { return hw::to_float(a.v); }
NFAD_DEV float dual_tangent(const Dual<Wide>& a) { return hw::to_float(a.t); }
NFAD_DEV float dual_value(const Gate<Wide>& a) { return hw::to_float(a.v); }
NFAD_DEV float dual_tangent(const Gate<Wide>& a) { return hw::to_float(a.t); }
NFAD_DEV Dual<Wide> as_dual(const Gate<Wide>& a) { return {a.v, a.t}; }

// ----------------------------------------------------------------- add, scale, mul (Eq. 3)

NFAD_DEV Dual<Wide> dual_add(const Dual<Wide>& a, const Dual<Wide>& b) { return {a.v + b.v, a.t + b.t}; }
NFAD_DEV Dual<Wide> dual_add_const(double c, const Dual<Wide>& a) { return {c + a.v, a.t}; }
NFAD_DEV Dual<Wide> dual_scale(double c, const Dual<Wide>& a) { return {c * a.v, c * a.t}; }
NFAD_DEV Dual<Wide> dual_scale(Wide, double c, const Seed& a) { return {c * hw::to_double(a.x), c}; }
NFAD_DEV Dual<Wide> dual_mul(Wide, const Seed& a, const Seed& b) { return {hw::to_double(a.x) * hw::to_double(b.x), hw::to_double(a.x) + hw::to_double(b.x)}; }
NFAD_DEV Dual<Wide> dual_mul(const Seed& a, const Dual<Wide>& b) { return {hw::to_double(a.x) * b.v, fma(hw::to_double(a.x), b.t, b.v)}; }
NFAD_DEV Gate<Wide> dual_mul(const Seed& a, const Gate<Wide>& b) { return {hw::to_double(a.x) * b.v, fma(hw::to_double(a.x), b.t, b.v)}; }
NFAD_DEV Dual<Wide> dual_mul(const Dual<Wide>& a, const Dual<Wide>& b) { return {a.v * b.v, fma(a.v, b.t, a.t * b.v)}; }

// c1 x + c3 x^3 with tangent c1 + k3 x^2 (k3 = 3 c3)
NFAD_DEV Dual<Wide> dual_odd_cubic(Wide, double c1, double c3, double k3, const Seed& a)
{
    double x = hw::to_double(a.x);
    double s = x * x;
    return {x * fma(c3, s, c1), fma(k3, s, c1)};
}

NFAD_DEV Dual<Wide> as_wide(const Seed& a) { return {hw::to_double(a.x), 1.0}; }
NFAD_DEV Dual<Wide> as_wide(const Dual<Wide>& a) { return a; }

// ----------------------------------------------------------------- the logistic gates

// L(w) = 1/(1 + exp(-w)) and dL/dw = L (1 - L), one form for both signs: E = exp(-w), L = 1/(1 + E), 1 - L = E L
// (no subtraction anywhere; doubles have the range for E on either side).  The slope is returned times `slope_in`
// (the chain rule's next factor).  |w| <= 700.  kPrecise: the exponential and the reciprocal to 2^-52 instead of 2^-29.
template <bool kPrecise> NFAD_DEV Gate<Wide> logistic_wide(double w, double slope_in)
{
    double E = wide::exp_bounded<kPrecise ? 11 : 6>(-w);
    double L = wide::rcp<kPrecise ? 2 : 1>(1.0 + E);
    return {L, (L * (E * L)) * slope_in};
}
NFAD_DEV double clamp700(double v) { return v != v ? v : fmin(fmax(v, -700.0), 700.0); }

// of the seed (an activation's own gate: |x| is bounded by its caller) and of any dual (clamped here)
NFAD_DEV Gate<Wide> dual_sigmoid(Wide, const Seed& a) { return logistic_wide<false>(hw::to_double(a.x), 1.0); }
NFAD_DEV Gate<Wide> dual_sigmoid(const Dual<Wide>& a) { return logistic_wide<true>(clamp700(a.v), a.t); }

NFAD_DEV Gate<Wide> dual_sigmoid(InRange, const Dual<Wide>& a) { return logistic_wide<false>(a.v, a.t); }

// (1 + tanh u)/2 = L(2u), slope 2 L'(2u)
NFAD_DEV Gate<Wide> dual_half_one_plus_tanh(const Dual<Wide>& u) { return logistic_wide<true>(clamp700(u.v + u.v), u.t + u.t); }

// (1 + erf z)/2 = erfc(-z)/2: with E = exp(-z^2) and W = erfcx(|z|)/2 it is E W for z < 0 and 1 - E W for z >= 0;
// slope E / sqrt(pi).  Beyond |z| = 15 the gate is 0 or 1 and its slope 0 in double precision.
NFAD_DEV Gate<Wide> dual_half_one_plus_erf(const Dual<Wide>& z)
{
    double za = z.v != z.v ? z.v : fmin(fabs(z.v), 15.0);
    double E = wide::exp_bounded<11>(-(za * za));
    double a = E * wide::half_erfcx(za);
    return {z.v < 0.0 ? a : 1.0 - a, (E * 0.5641895835477563) * z.t};
}
// (1 + erf(c x))/2 of the seed, c a constant: the scale folded in (a binary operation with one constant input is unary,
// Section III-A), so that -c^2 x^2 and c |x| + k each are one operation.  |c x| <= 15.
NFAD_DEV Gate<Wide> dual_half_one_plus_erf_scaled(Wide, double c, const Seed& a)
{
    const double kappa = 0.5641895835477563 * c;             // the slope is kappa E: E is formed times kappa, W over kappa
    double x = hw::to_double(a.x);
    double Ek = wide::exp_neg_scaled(x * x, c * c, kappa);
    double v = Ek * wide::half_erfcx_mix(fma(fabs(x), c * kappa, 2.1213202476501465 * kappa), kappa);
    return {a.x < 0.0f ? v : 1.0 - v, Ek};
}

// ----------------------------------------------------------------- softplus, and tanh of a softplus

// softplus remembers w = exp(v) itself: its slope sigmoid(v) and tanh(softplus) are algebraic in w
// (tag Precise: the exponential and the reciprocal to 2^-52 instead of 2^-29, as in the general-purpose primitives)
struct Precise {};
template <> struct SoftplusDual<Wide> { double w; };
NFAD_DEV SoftplusDual<Wide> dual_softplus(Wide, const Seed& a) { return {wide::exp_bounded<6>(hw::to_double(a.x))}; }
NFAD_DEV SoftplusDual<Wide> dual_softplus(Wide, Precise, const Seed& a) { return {wide::exp_bounded<11>(hw::to_double(a.x))}; }

// one form for both signs, every term positive:  T = n/(n + 2),  n = w (w + 2),  w = e^v;
// T' = (dn/dv) 2/(n + 2)^2 = 4 w (w + 1)/(n + 2)^2.  Formed with the halves h = (w + 2)/2, m = n/2 = w h and
// r = 2/(n + 2) = 1/(w h + 1), so that no factor 2 or 4 costs an operation:  T = m r,  T' = (w r) (w r + r).
// |v| <= 150 keeps w h inside the range of a double.
template <int kRcpSteps> NFAD_DEV Gate<Wide> tanh_of_softplus_wide(double w)
{
    double h = fma(w, 0.5, 1.0);
    double r = wide::rcp<kRcpSteps>(fma(w, h, 1.0));
    return {(w * h) * r, (w * r) * fma(w, r, r)};
}
NFAD_DEV Gate<Wide> dual_tanh(const SoftplusDual<Wide>& p) { return tanh_of_softplus_wide<1>(p.w); }
NFAD_DEV Gate<Wide> dual_tanh(Precise, const SoftplusDual<Wide>& p) { return tanh_of_softplus_wide<2>(p.w); }

// ----------------------------------------------------------------- general-purpose primitives
//
// exp, log1p, tanh, erf and softplus with its value, for sequences composed at run time; good to about 2^-38
// of the value where the function is well conditioned.  A user who writes 1 + tanh(u) gets the cancellation
// that expression has (in double precision it costs digits only beyond |u| ~ 9).

// exp:  v = e^a, v' = v.  The argument is clamped to [-700, 700]; the positive side is formed as 1/e^-a.
NFAD_DEV Dual<Wide> dual_exp(const Dual<Wide>& a)
{
    double m = wide::exp_neg(-fmin(fabs(a.v), 700.0));
    double v = a.v > 0.0 ? wide::rcp<2>(m) : m;
    v = a.v != a.v ? a.v : v;
    return {v, v * a.t};
}

// log1p:  v = log(1 + a), v' = 1/(1 + a), a > -1.  log(u) a/(u - 1) with u = fl(1 + a) removes the rounding of u.
NFAD_DEV Dual<Wide> dual_log1p(const Dual<Wide>& a)
{
    double u = 1.0 + a.v;
    double um1 = u - 1.0;
    double v = um1 == 0.0 ? a.v : wide::log_pos(u) * (a.v * wide::rcp<2>(um1));
    return {v, a.t * wide::rcp<2>(u)};
}

// tanh:  (1 - e)/(1 + e) with e = exp(-2|a|), an odd series below 2^-4 where that cancels; v' = 4e/(1+e)^2.
NFAD_DEV Dual<Wide> dual_tanh(const Dual<Wide>& a)
{
    double aa = fmin(fabs(a.v), 350.0);
    double e = wide::exp_neg(-2.0 * aa);
    double r = wide::rcp<2>(1.0 + e);
    double big = (1.0 - e) * r;
    double a2 = aa * aa;
    double ser = fma(a2, fma(a2, fma(a2, fma(a2, 0.021869488536155203, -0.053968253968253971), 0.13333333333333333), -0.33333333333333331), 1.0);
    double v = copysign(aa < 0.0625 ? aa * ser : big, a.v);
    v = a.v != a.v ? a.v : v;
    return {v, ((4.0 * e) * (r * r)) * a.t};
}

// erf:  1 - erfc for |a| >= 0.5, the Maclaurin series below; v' = 2/sqrt(pi) exp(-a^2).
NFAD_DEV Dual<Wide> dual_erf(const Dual<Wide>& a)
{
    double aa = fmin(fabs(a.v), 15.0);
    double a2 = aa * aa;
    double E = wide::exp_neg(-a2);
    double big = fma(-2.0, E * wide::half_erfcx(aa), 1.0);
    double s = -1.6365844691234924e-07;                     // 2/sqrt(pi) (-1)^j / (j! (2j+1)), j = 9 ... 0
    s = fma(s, a2, 1.6462114365889248e-06);
    s = fma(s, a2, -1.492565035840625e-05);
    s = fma(s, a2, 0.00012055332981789664);
    s = fma(s, a2, -0.0008548327023450853);
    s = fma(s, a2, 0.005223977625442188);
    s = fma(s, a2, -0.026866170645131252);
    s = fma(s, a2, 0.11283791670955126);
    s = fma(s, a2, -0.37612638903183754);
    s = fma(s, a2, 1.1283791670955126);
    double v = copysign(aa < 0.5 ? aa * s : big, a.v);
    v = a.v != a.v ? a.v : v;
    return {v, (E * 1.1283791670955126) * a.t};
}

// softplus with its value:  v = max(a, 0) + log1p(exp(-|a|)),  v' = sigmoid(a)
NFAD_DEV Dual<Wide> dual_softplus(const Dual<Wide>& a)
{
    double e = wide::exp_neg(-fmin(fabs(a.v), 700.0));
    Dual<Wide> l = dual_log1p(Dual<Wide>{e, 0.0});
    double r = wide::rcp<2>(1.0 + e);
    double v = fmax(a.v, 0.0) + l.v;
    v = a.v != a.v ? a.v : v;
    return {v, (a.v < 0.0 ? e * r : r) * a.t};
}

}  // namespace nfad
