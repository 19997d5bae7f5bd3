// nfad_dual.cuh -- the device-side dual-number algebra of nested Forward-AD.
//
// A dual number carries a value v and a tangent t = dv/dx.  Every primitive
// computes its value and its derivative TOGETHER (Section II-C, approach 3: the
// derivative of a node is calculated when the node is executed), sharing the one
// exponential that both need; a unary primitive applies the chain rule
// t_out = prim'(v) * t_in, and the product of two duals of the same source
// applies the product rule of Eq. 3.  The seed is x' = 1 (Section II-D), held
// as a type (`Seed`) rather than a register, so that no multiply by 1 is ever
// emitted (the single-operator shortcut of Section IV, "Efficiency").
//
// Primitive set (Section III-A: unary operations, binary operations whose two
// inputs come from the same source, binary operations with one constant, and
// the closed symbolic forms tanh / sigmoid / softplus that frameworks ship as
// single operators):
//     dual_add  dual_mul  dual_scale  dual_add_const
//     dual_exp  dual_log1p  dual_tanh  dual_erf  dual_softplus  dual_sigmoid
// and two "binary with a constant, hence unary" fusions that keep the tails
// free of cancellation:
//     dual_half_one_plus_tanh(u) = (1 + tanh u)/2 = sigmoid(2u)
//     dual_half_one_plus_erf(z)  = (1 + erf z)/2  = erfc(-z)/2
// and one fusion of mul / scale / add_const over the seed alone, with its derivative
// in closed form like any other primitive:
//     dual_odd_cubic(c1, c3, x)  = c1 x + c3 x^3,  tangent c1 + 3 c3 x^2
//
// Policies.  Fast (16-bit storage): a value and a tangent are one float each.
// Full (fp32 storage): values and the tangents of the polynomial part of a
// chain are unevaluated sums hi + lo; a gate's tangent is one float.  The pairs
// keep (a) the bits of an exponential's argument that |arg| would amplify and
// (b) a result of the form 1 - small as (1, -small); values are rounded once, at
// the store.
//
// Gates.  sigmoid, (1+tanh)/2, (1+erf)/2 and tanh(softplus) all behave like
// exp(-|v|) on their small side.  Under Full they return a `Gate`: a dual whose
// value and tangent share a power-of-two factor that is applied last (it is
// exact), so that nothing on the way is rounded in the subnormal range.
#pragma once

#include "nfad_numerics.cuh"

namespace nfad {

// The independent variable: value x, tangent exactly 1.
struct Seed { float x; };

template <class P> struct Dual;
template <> struct Dual<Fast> { float v, t; };
template <> struct Dual<Full> { F2 v, t; };

template <class P> struct Gate;
template <> struct Gate<Fast> { float v, t; };
template <> struct Gate<Full> { F2 v; float t; float sc; int n; };   // (v, t) times sc = 2^max(n,-126), times 2^(n+126) if n < -126

// A constant known to more than fp32 precision.
struct Const2 { float h, l; };
// The same, split so that the high part is a positive multiple of 2^-20 (and the low part
// correspondingly larger).  For e >= 0 and s = fl(h + e) < 16 the difference s - h is then
// exact (a multiple of s's last place that fits 24 bits), which makes the rounding error of
// a fused multiply-add onto h recoverable with one more fused multiply-add.
struct SplitConst { float h, l; };

NFAD_DEV float dual_value(const Dual<Fast>& a) { return a.v; }
NFAD_DEV float dual_tangent(const Dual<Fast>& a) { return a.t; }
NFAD_DEV float dual_value(const Gate<Fast>& a) { return a.v; }
NFAD_DEV float dual_tangent(const Gate<Fast>& a) { return a.t; }
NFAD_DEV float dual_value(const Dual<Full>& a) { return f2_value(a.v); }       // the one rounding
NFAD_DEV float dual_tangent(const Dual<Full>& a) { return f2_value(a.t); }
// The scale is a power of two: exact, unless the result is subnormal, where it is the one
// rounding.  The second factor exists only below 2^-126 (rare, so a branch).
NFAD_DEV float gate_rest(const Gate<Full>& a) { return pow2_clamped(a.n + 126); }
NFAD_DEV float dual_value(const Gate<Full>& a)
{
    float y = f2_value(a.v) * a.sc;
    if (a.n < -126) y *= gate_rest(a);
    return y;
}
NFAD_DEV float dual_tangent(const Gate<Full>& a)
{
    float t = a.t * a.sc;
    if (a.n < -126) t *= gate_rest(a);
    return t;
}

// A gate as an ordinary dual (for further generic composition).
NFAD_DEV Dual<Fast> as_dual(const Gate<Fast>& a) { return {a.v, a.t}; }
NFAD_DEV Dual<Full> as_dual(const Gate<Full>& a) { return {{a.v.h * a.sc, a.v.l * a.sc}, {a.t * a.sc, 0.0f}}; }

// ----------------------------------------------------------------- add, scale (linear)

NFAD_DEV Dual<Fast> dual_add(const Dual<Fast>& a, const Dual<Fast>& b) { return {a.v + b.v, a.t + b.t}; }
NFAD_DEV Dual<Full> dual_add(const Dual<Full>& a, const Dual<Full>& b) { return {f2_add(a.v, b.v), f2_add(a.t, b.t)}; }

// c + a (binary with one constant input: unary, tangent unchanged)
NFAD_DEV Dual<Fast> dual_add_const(float c, const Dual<Fast>& a) { return {c + a.v, a.t}; }
NFAD_DEV Dual<Full> dual_add_const(float c, const Dual<Full>& a)
{
    F2 s = two_sum(c, a.v.h);
    s.l += a.v.l;
    return {s, a.t};
}

// c * a
NFAD_DEV Dual<Fast> dual_scale(Const2 c, const Dual<Fast>& a) { return {c.h * a.v, c.h * a.t}; }
NFAD_DEV Dual<Full> dual_scale(Const2 c, const Dual<Full>& a)
{
    return {f2_mul(a.v, F2{c.h, c.l}), f2_mul(a.t, F2{c.h, c.l})};
}
// (a seed does not say which policy its result takes: the caller passes it as a tag)
NFAD_DEV Dual<Fast> dual_scale(Fast, Const2 c, const Seed& a) { return {c.h * a.x, c.h}; }
NFAD_DEV Dual<Full> dual_scale(Full, Const2 c, const Seed& a) { return {f2_mul(F2{c.h, c.l}, a.x), {c.h, c.l}}; }

// ----------------------------------------------------------------- mul (product rule, Eq. 3)

NFAD_DEV Dual<Fast> dual_mul(Fast, const Seed& a, const Seed& b) { return {a.x * b.x, a.x + b.x}; }
NFAD_DEV Dual<Full> dual_mul(Full, const Seed& a, const Seed& b) { return {two_prod(a.x, b.x), {a.x + b.x, 0.0f}}; }

// x * b:  value x b.v,  tangent 1 * b.v + x * b.t
NFAD_DEV Dual<Fast> dual_mul(const Seed& a, const Dual<Fast>& b) { return {a.x * b.v, fmaf(a.x, b.t, b.v)}; }
NFAD_DEV Gate<Fast> dual_mul(const Seed& a, const Gate<Fast>& b) { return {a.x * b.v, fmaf(a.x, b.t, b.v)}; }
NFAD_DEV Dual<Full> dual_mul(const Seed& a, const Dual<Full>& b)
{
    return {f2_mul(b.v, a.x), f2_add(f2_mul(b.t, a.x), b.v)};
}
NFAD_DEV Gate<Full> dual_mul(const Seed& a, const Gate<Full>& b)
{
    return {f2_mul(b.v, a.x), fmaf(a.x, b.t, b.v.h) + b.v.l, b.sc, b.n};
}

NFAD_DEV Dual<Fast> dual_mul(const Dual<Fast>& a, const Dual<Fast>& b)
{
    return {a.v * b.v, fmaf(a.v, b.t, a.t * b.v)};
}
NFAD_DEV Dual<Full> dual_mul(const Dual<Full>& a, const Dual<Full>& b)
{
    return {f2_mul(a.v, b.v), f2_add(f2_mul(a.v, b.t), f2_mul(a.t, b.v))};
}

// ----------------------------------------------------------------- odd cubic of the seed
//
// p(x) = c1 x + c3 x^3 = x (c1 + c3 x^2),  p'(x) = c1 + 3 c3 x^2   (k3 = 3 c3 is passed in).
// Full: both brackets are formed as two-floats from the exact square x^2 = s.h + s.l; the
// high part is one fused multiply-add onto c1.h and the low part recovers its rounding error
// (see SplitConst) plus the terms of the constants' and the square's low parts.  Needs
// c1 + k x^2 < 15.
NFAD_DEV F2 cubic_bracket(SplitConst c1, Const2 k, F2 s)
{
    float h = fmaf(k.h, s.h, c1.h);
    float l = fmaf(k.h, s.h, c1.h - h);
    l += fmaf(k.h, s.l, fmaf(k.l, s.h, c1.l));
    return {h, l};
}
NFAD_DEV Dual<Full> dual_odd_cubic(Full, SplitConst c1, Const2 c3, Const2 k3, const Seed& a)
{
    F2 s = two_prod(a.x, a.x);
    return {f2_mul(cubic_bracket(c1, c3, s), a.x), cubic_bracket(c1, k3, s)};
}
NFAD_DEV Dual<Fast> dual_odd_cubic(Fast, SplitConst c1, Const2 c3, Const2 k3, const Seed& a)
{
    float s = a.x * a.x;
    float c = c1.h + c1.l;
    return {a.x * fmaf(c3.h, s, c), fmaf(k3.h, s, c)};
}

// ----------------------------------------------------------------- chain rule's last factor

// d * (tangent of the input); free for the seed
NFAD_DEV float chain(float d, const Seed&) { return d; }
NFAD_DEV float chain(float d, const Dual<Fast>& a) { return d * a.t; }
NFAD_DEV float chain(float d, const Dual<Full>& a) { return fmaf(d, a.t.l, d * a.t.h); }

NFAD_DEV float in_v(const Seed& a) { return a.x; }
NFAD_DEV float in_v(const Dual<Fast>& a) { return a.v; }
NFAD_DEV F2 in_v2(const Seed& a) { return {a.x, 0.0f}; }
NFAD_DEV F2 in_v2(const Dual<Full>& a) { return a.v; }

// ----------------------------------------------------------------- the logistic function and its slope

// L(w) = 1/(1+exp(-w)), L' = L (1 - L), from one e = exp(-|w|):
//   big = 1/(1+e), small = e big = 1 - big;  L = small for w < 0, big for w >= 0.
// Fast: (value, slope).
// The slope is returned times slope_in * slope_const (the chain rule's next factor and a
// compile-time constant, folded in here so that the 2^-64 costs no instruction).
NFAD_DEV Gate<Fast> logistic_fast(float w, float minus_log2e_scale, float slope_in, float slope_const)
{
    float e64 = exp2_fast_times_2p64(fmaf(fabsf(w), minus_log2e_scale, 64.0f));   // 2^64 e
    float big = hw::rcp_approx(fmaf(e64, kTwoPowMinus64, 1.0f));
    float small64 = e64 * big;                                                    // 2^64 small
    return {w < 0.0f ? small64 * kTwoPowMinus64 : big, (small64 * big) * (slope_in * (slope_const * kTwoPowMinus64))};
}

// Full: |w| = -(ah + al).  For w < 0 the common factor 2^n of e is left out of
// value and slope (they carry it as `sc`); for w >= 0 the value is the pair (1, -small).
// The exponential comes as 2^n (1 + g) and is applied as m (1 + g) = fmaf(m, g, m), so 1 + g is
// never rounded; 1/(1+e) is a Newton-refined reciprocal of the exactly known 1 + e.  Every fp32
// input was run against the fp64 oracle with this arithmetic (see tests/certify_fp32_exhaustive.py).
// kFineSlope spends six more instructions on the slope (two-float 1/(1+e), its square formed
// exactly): needed where the slope is multiplied by a large chain-rule factor, as in GELU-tanh.
template <bool kFineSlope>
NFAD_DEV Gate<Full> logistic_full(float ah, float al, bool neg)
{
    ExpG E = exp_g_full(ah, al);
    float sc = pow2_clamped(E.n);
    float e = fmaf(sc, E.g, sc);
    float dh = 1.0f + e;
    float dl = e - (dh - 1.0f);                // 1 + e = dh + dl
    F2 big2 = f2_rcp(F2{dh, dl});              // 1/(1+e); the low part is dead code unless kFineSlope
    float big = big2.h;
    float pr = fmaf(big, E.g, big);            // small / 2^n
    float dd;                                  // big small / 2^n
    if (kFineSlope) {
        F2 bb = two_prod(big, big);
        bb.l = fmaf(big + big, big2.l, bb.l);  // 1/(1+e)^2
        dd = fmaf(bb.h, E.g, bb.h) + bb.l;
    } else {
        dd = pr * big;
    }
    F2 v = neg ? F2{pr, 0.0f} : F2{1.0f, -(pr * sc)};
    float d = neg ? dd : dd * sc;
    return {v, d, neg ? sc : 1.0f, neg ? E.n : 0};
}

// ----------------------------------------------------------------- sigmoid

template <class In> NFAD_DEV Gate<Fast> dual_sigmoid_fast(const In& a)
{
    return logistic_fast(in_v(a), -1.44269502f, chain(1.0f, a), 1.0f);
}
template <class In> NFAD_DEV Gate<Full> dual_sigmoid_full(const In& a)
{
    F2 v = in_v2(a);
    bool neg = v.h < 0.0f;
    Gate<Full> g = logistic_full<false>(-fabsf(v.h), neg ? v.l : -v.l, neg);
    return {g.v, chain(g.t, a), g.sc, g.n};
}
NFAD_DEV Gate<Fast> dual_sigmoid(Fast, const Seed& a) { return dual_sigmoid_fast(a); }
NFAD_DEV Gate<Full> dual_sigmoid(Full, const Seed& a) { return dual_sigmoid_full(a); }
NFAD_DEV Gate<Fast> dual_sigmoid(const Dual<Fast>& a) { return dual_sigmoid_fast(a); }
NFAD_DEV Gate<Full> dual_sigmoid(const Dual<Full>& a) { return dual_sigmoid_full(a); }

// ----------------------------------------------------------------- (1 + tanh u)/2

// H = (1 + tanh u)/2 = L(2u),  dH/du = 2 L'(2u)   [= (1 - tanh^2 u)/2]
NFAD_DEV Gate<Fast> dual_half_one_plus_tanh(const Dual<Fast>& u)
{
    return logistic_fast(u.v, -2.88539004f, u.t, 2.0f);
}
NFAD_DEV Gate<Full> dual_half_one_plus_tanh(const Dual<Full>& u)
{
    bool neg = u.v.h < 0.0f;
    float two_ul = u.v.l + u.v.l;
    Gate<Full> g = logistic_full<true>(-2.0f * fabsf(u.v.h), neg ? two_ul : -two_ul, neg);
    return {g.v, chain(g.t + g.t, u), g.sc, g.n};
}

// ----------------------------------------------------------------- (1 + erf z)/2

// H = (1 + erf z)/2 = erfc(-z)/2,  H' = exp(-z^2)/sqrt(pi).
// With E = exp(-z^2) and W = erfcx(|z|)/2:  erfc(|z|)/2 = E W, so
//   z < 0:  H = E W           z >= 0:  H = 1 - E W
// and the same E serves the tangent.
NFAD_DEV Gate<Fast> dual_half_one_plus_erf(const Dual<Fast>& z)
{
    // E is formed as 2^64 exp(-z^2) and W as 2^-64 W: see half_erfcx_fast_scaled
    const float kInvSqrtPiScaled = 0.564189612865448f * 5.42101086e-20f;
    float za = fabsf(z.v);
    float e64 = exp2_fast_times_2p64(fmaf(za * za, -1.44269502f, 64.0f));
    float a = e64 * half_erfcx_fast_scaled(za);
    return {z.v < 0.0f ? a : 1.0f - a, e64 * (kInvSqrtPiScaled * z.t)};
}

NFAD_DEV Gate<Full> dual_half_one_plus_erf(const Dual<Full>& z)
{
    const F2 kInvSqrtPi = {0.564189612865448f, -2.9317691e-08f};
    bool neg = z.v.h < 0.0f;
    float za = fabsf(z.v.h);
    float zla = neg ? -z.v.l : z.v.l;          // |z| = za + zla
    F2 sq = two_prod(za, za);
    ExpParts E = exp_parts_full(-sq.h, -sq.l); // exp(-za^2): the square is exact
    F2 a = f2_mul(half_erfcx_full(za), E.p);   // erfc(za)/2, without 2^n
    // its slope's magnitude at za, without 2^n: one rounding, of the leading product
    float t0 = fmaf(E.p.h, kInvSqrtPi.h, fmaf(E.p.h, kInvSqrtPi.l, E.p.l * kInvSqrtPi.h));
    // first order in the low part of the argument: the value moves by -t0 zla,
    // the exponential by the factor (1 - 2 za zla)
    a.l = fmaf(-t0, zla, a.l);
    t0 = fmaf(t0, -2.0f * (za * zla), t0);
    float sc = pow2_clamped(E.n);
    F2 v = neg ? a : F2{1.0f, -(f2_value(a) * sc)};
    float d = neg ? t0 : t0 * sc;
    return {v, chain(d, z), neg ? sc : 1.0f, neg ? E.n : 0};
}

// ----------------------------------------------------------------- softplus, and tanh of a softplus

// p = softplus(v) = log1p(exp v),  p' = sigmoid(v).
// The result remembers exp(-|v|): every later use of p (its tangent, tanh p) is
// an algebraic function of it, so the logarithm itself is never needed here.
template <class P> struct SoftplusDual;
template <> struct SoftplusDual<Fast> { float e; bool neg; };
template <> struct SoftplusDual<Full> { ExpParts E; bool neg; };

NFAD_DEV SoftplusDual<Fast> dual_softplus(Fast, const Seed& a)
{
    return {exp2_fast_times_2p64(fmaf(fabsf(a.x), -1.44269502f, 64.0f)) * kTwoPowMinus64, a.x < 0.0f};
}
NFAD_DEV SoftplusDual<Full> dual_softplus(Full, const Seed& a)
{
    return {exp_parts_full(-fabsf(a.x), 0.0f), a.x < 0.0f};
}

// tanh(log1p(w)) = ((1+w)^2 - 1)/((1+w)^2 + 1) = n/(n+2), n = w^2 + 2w, w = e^v.
// In terms of e = exp(-|v|), all terms positive:
//   v <  0 (w = e):    T = e (e + 2) / (e^2 + 2e + 2)
//   v >= 0 (w = 1/e):  T = 1 - e (2e) / (2e^2 + 2e + 1)
// and T' = sech^2(p) sigmoid(v) = 4 e (1+e) / den^2, times e again for v >= 0.
NFAD_DEV Gate<Fast> dual_tanh(const SoftplusDual<Fast>& p)
{
    float e = p.e;
    float g = p.neg ? e + 2.0f : e + e;
    float num = e * g;
    float den = num + (p.neg ? 2.0f : fmaf(2.0f, e, 1.0f));
    float rd = hw::rcp_approx(den);
    float sm = num * rd;
    float k = (4.0f * e) * (1.0f + e) * (rd * rd);
    return {p.neg ? sm : 1.0f - sm, p.neg ? k : k * e};
}

NFAD_DEV Gate<Full> dual_tanh(const SoftplusDual<Full>& p)
{
    const bool neg = p.neg;
    float sc = pow2_clamped(p.E.n);
    F2 e = {p.E.p.h * sc, p.E.p.l * sc};
    F2 e2 = {e.h + e.h, e.l + e.l};
    F2 g = neg ? f2_add_big(2.0f, e) : e2;
    F2 num = f2_mul(e, g);
    F2 base = neg ? F2{2.0f, 0.0f} : f2_add_big(1.0f, e2);
    F2 den = f2_add(base, num);
    F2 rd = f2_rcp(den);                       // 1/den
    F2 f0 = neg ? p.E.p : e;                   // the front factor e, without 2^n on the small side
    F2 sm = f2_mul(f2_mul(f0, g), rd);
    F2 ope = f2_add_big(1.0f, e);
    F2 a1 = f2_mul(f0, ope);                                // e (1 + e)
    F2 rd2 = two_prod(rd.h, rd.h);
    rd2.l = fmaf(rd.h + rd.h, rd.l, rd2.l);                 // 1/den^2
    float tt = f2_value(f2_mul(a1, rd2)) * (neg ? 4.0f : 4.0f * e.h);
    F2 v = neg ? sm : F2{1.0f, -f2_value(sm)};
    return {v, tt, neg ? sc : 1.0f, neg ? p.E.n : 0};
}

// ----------------------------------------------------------------- general-purpose primitives (Fast policy)
//
// exp, log1p, tanh, erf and the value of softplus are not needed by the four
// activation chains above (which use the cancellation-free fusions); they are the
// remaining members of the primitive set, for sequences composed at run time.
// Plain fp32 on MUFU ex2 / lg2 / rcp: good to a few fp32 ulp of the value where the
// function itself is well conditioned; a user who writes 1 + tanh(u) gets the
// cancellation that expression has.

// exp:  v = e^a,  v' = v
NFAD_DEV Dual<Fast> dual_exp(const Dual<Fast>& a)
{
    float v = hw::ex2_approx(1.44269502f * a.v);
    return {v, v * a.t};
}

// log1p:  v = log(1 + a),  v' = 1/(1 + a).  log(u) a/(u - 1) with u = fl(1 + a) cancels
// the rounding of u to first order; a itself when u rounds to 1.
NFAD_DEV Dual<Fast> dual_log1p(const Dual<Fast>& a)
{
    float u = 1.0f + a.v;
    float lg = 0.693147182f * hw::lg2_approx(u);
    float um1 = u - 1.0f;
    float v = um1 == 0.0f ? a.v : lg * (a.v * hw::rcp_approx(um1));
    return {v, a.t * hw::rcp_approx(u)};
}

// tanh:  v' = 1 - v^2, formed as 4e/(1+e)^2 from e = exp(-2|a|) so that it stays
// accurate where v -> 1; an odd polynomial takes over for small |a|, where (1-e)/(1+e) cancels.
NFAD_DEV Dual<Fast> dual_tanh(const Dual<Fast>& a)
{
    float aa = fabsf(a.v);
    float e = hw::ex2_approx(-2.88539004f * aa);
    float r = hw::rcp_approx(1.0f + e);
    float big = (1.0f - e) * r;
    float a2 = a.v * a.v;
    float small_ = aa * fmaf(a2, fmaf(a2, fmaf(a2, -0.0539682545f, 0.133333340f), -0.333333343f), 1.0f);
    float v = copysignf(aa < 0.25f ? small_ : big, a.v);
    float slope = aa < 0.25f ? fmaf(-v, v, 1.0f) : (4.0f * e) * (r * r);
    return {v, slope * a.t};
}

// erf:  v' = 2/sqrt(pi) exp(-a^2).  1 - erfc for |a| >= 0.5, the Maclaurin series below.
NFAD_DEV Dual<Fast> dual_erf(const Dual<Fast>& a)
{
    float aa = fabsf(a.v);
    float a2 = aa * aa;
    float e64 = exp2_fast_times_2p64(fmaf(a2, -1.44269502f, 64.0f));
    float big = fmaf(-2.0f, e64 * half_erfcx_fast_scaled(aa), 1.0f);
    float ser = fmaf(a2, fmaf(a2, fmaf(a2, fmaf(a2, 0.00522397785f, -0.0268661696f), 0.112837918f), -0.376126379f), 1.12837923f);
    float v = copysignf(aa < 0.5f ? aa * ser : big, a.v);
    return {v, (e64 * (1.12837923f * kTwoPowMinus64)) * a.t};
}

// softplus with its value:  v = max(a, 0) + log1p(exp(-|a|)),  v' = sigmoid(a)
NFAD_DEV Dual<Fast> dual_softplus(const Dual<Fast>& a)
{
    float e = exp2_fast_times_2p64(fmaf(fabsf(a.v), -1.44269502f, 64.0f)) * kTwoPowMinus64;
    Dual<Fast> l = dual_log1p(Dual<Fast>{e, 0.0f});
    float r = hw::rcp_approx(1.0f + e);
    return {fmaxf(a.v, 0.0f) + l.v, (a.v < 0.0f ? e * r : r) * a.t};
}

// ----------------------------------------------------------------- the four activations (Table I)

struct GeluErf {};
struct GeluTanh {};
struct Swish {};
struct Mish {};

// The gate h(x) of each activation f(x) = x h(x), as a dual number.

// GELU, erf form: h = Phi(x) = (1 + erf(x/sqrt2))/2
template <class P> NFAD_DEV Gate<P> gate(GeluErf, Seed X)
{
    const Const2 kInvSqrt2 = {0.7071067690849304f, 1.2101617e-08f};
    Dual<P> Z = dual_scale(P{}, kInvSqrt2, X);
    return dual_half_one_plus_erf(Z);
}

// GELU, tanh form (Table I): h = (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))/2
template <class P> NFAD_DEV Gate<P> gate(GeluTanh, Seed X)
{
    // u = c x + (c a) x^3 with c = sqrt(2/pi), a = 0.044715 (the double nearest to it)
    const SplitConst kC = {0.7978849411010742f, -3.8029822e-07f};
    const Const2 kCA = {0.035677406936883926f, 1.1994162e-09f};
    const Const2 k3CA = {0.10703222453594208f, -1.2704171e-10f};
    return dual_half_one_plus_tanh(dual_odd_cubic(P{}, kC, kCA, k3CA, X));
}

// Swish (Table I, Table II): h = sigmoid(x)
template <class P> NFAD_DEV Gate<P> gate(Swish, Seed X) { return dual_sigmoid(P{}, X); }

// Mish (Table I): h = tanh(softplus(x))
template <class P> NFAD_DEV Gate<P> gate(Mish, Seed X) { return dual_tanh(dual_softplus(P{}, X)); }

struct ActOut { float y, dydx; };

// Saturation.  Beyond |x| = kFull the gate is 0 or 1 to every fp32 bit and its
// slope is exactly 0 (the exponential has underflowed to zero), so evaluating
// the gate at the clamped argument changes nothing; it is what keeps x^2, x^3
// and the error-free transformations finite for inputs up to the largest float.
// The Fast policy needs that only where an intermediate can overflow (the cubic
// of the tanh form).
template <class K> struct Saturation;
template <> struct Saturation<GeluErf> { static constexpr float kFull = 20.0f; static constexpr bool kFastClamp = false; };
template <> struct Saturation<GeluTanh> { static constexpr float kFull = 11.5f; static constexpr bool kFastClamp = true; };
template <> struct Saturation<Swish> { static constexpr float kFull = 120.0f; static constexpr bool kFastClamp = false; };
template <> struct Saturation<Mish> { static constexpr float kFull = 120.0f; static constexpr bool kFastClamp = false; };

// x -> (f(x), f'(x)) in fp32, for any finite or non-finite x.  f = x h(x): the
// last node of every chain is the product of the seed with the gate (v3 = v1 v2
// with v2 = x in the Swish example), where Eq. 3 merges the tangents.
template <class K> NFAD_DEV ActOut evaluate(K, Full, float x)
{
    constexpr float kSat = Saturation<K>::kFull;
    float xc = hw::clamp_nan(x, -kSat, kSat);
    Seed X{xc};
    Gate<Full> Y = dual_mul(X, gate<Full>(K{}, X));
    float y = dual_value(Y);
    return {x > kSat ? x : y, dual_tangent(Y)};
}

template <class K> NFAD_DEV ActOut evaluate(K, Fast, float x)
{
    const float kMax = 3.40282347e+38f;
    if (Saturation<K>::kFastClamp) {
        // the gate and the tangent's product see the clamped argument (the slope is exactly 0
        // beyond it); the value's product sees x itself, kept finite on the side where the
        // gate is 0 so that -inf gives -0
        float xg = hw::clamp_nan(x, -12.0f, 12.0f);
        Gate<Fast> H = gate<Fast>(K{}, Seed{xg});
        return {hw::max_nan(x, -kMax) * H.v, fmaf(xg, H.t, H.v)};
    }
    // +-inf become the largest float, which rounds back to inf in either 16-bit type
    float xf = hw::clamp_nan(x, -kMax, kMax);
    Gate<Fast> Y = dual_mul(Seed{xf}, gate<Fast>(K{}, Seed{xf}));
    return {dual_value(Y), dual_tangent(Y)};
}

template <class K, class P> NFAD_DEV ActOut evaluate(float x) { return evaluate(K{}, P{}, x); }

// x -> f(x) alone (a pass that will not be differentiated).  Same chain, same bits as evaluate().y; under the
// Fast policy only the side that needs it is clamped: +inf goes through as it is (every gate is exactly 1
// there, so f = x), -inf becomes the most negative float so that 0 * x gives -0.
template <class K> NFAD_DEV float evaluate_value(K, Full, float x) { return evaluate(K{}, Full{}, x).y; }
template <class K> NFAD_DEV float evaluate_value(K, Fast, float x)
{
    if (Saturation<K>::kFastClamp) return evaluate(K{}, Fast{}, x).y;
    const float xf = hw::max_nan(x, -3.40282347e+38f);
    return dual_value(dual_mul(Seed{xf}, gate<Fast>(K{}, Seed{xf})));
}

// x -> h(x) alone (what a recomputation pass re-materialises).
template <class K, class P> NFAD_DEV float evaluate_gate(float x)
{
    constexpr float kSat = Saturation<K>::kFull;
    float xc = hw::clamp_nan(x, -kSat, kSat);
    return dual_value(gate<P>(K{}, Seed{xc}));
}

}  // namespace nfad
