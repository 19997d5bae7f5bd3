// nfad_dual.cuh -- the device-side dual-number algebra of nested Forward-AD.
//
// A dual number carries a value v and a tangent t = dv/dx.  Every primitive
// computes its value and its derivative TOGETHER (Section II-C, approach 3:
// "v1' = v1(1-v1) is calculated when v1 is executed"), sharing the one
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
//
// Under the Full policy (fp32 storage) a value is an unevaluated sum v + vl so
// that (a) arguments of exponentials keep the bits that |arg| would otherwise
// amplify and (b) a result of the form 1 - small is held as (1, -small) and
// rounded once, at the store.  Under the Fast policy (16-bit storage) a value is
// one float.
#pragma once

#include "nfad_numerics.cuh"

namespace nfad {

// The independent variable: value x, tangent exactly 1.
struct Seed { float x; };

template <class P> struct Dual;
template <> struct Dual<Fast> { float v, t; };
template <> struct Dual<Full> { float v, vl, t; };

// A constant known to more than fp32 precision.
struct Const2 { float h, l; };

NFAD_DEV float dual_value(const Dual<Fast>& a) { return a.v; }
NFAD_DEV float dual_value(const Dual<Full>& a) { return a.v + a.vl; }   // the one rounding

// ----------------------------------------------------------------- add, scale (linear)

NFAD_DEV Dual<Fast> dual_add(const Dual<Fast>& a, const Dual<Fast>& b) { return {a.v + b.v, a.t + b.t}; }
NFAD_DEV Dual<Full> dual_add(const Dual<Full>& a, const Dual<Full>& b)
{
    F2 s = two_sum(a.v, b.v);
    return {s.h, s.l + (a.vl + b.vl), a.t + b.t};
}

// c + a (binary with one constant input: unary, tangent unchanged)
NFAD_DEV Dual<Fast> dual_add_const(float c, const Dual<Fast>& a) { return {c + a.v, a.t}; }
NFAD_DEV Dual<Full> dual_add_const(float c, const Dual<Full>& a)
{
    F2 s = two_sum(c, a.v);
    return {s.h, s.l + a.vl, a.t};
}

// c * a
NFAD_DEV Dual<Fast> dual_scale(Const2 c, const Dual<Fast>& a) { return {c.h * a.v, c.h * a.t}; }
NFAD_DEV Dual<Full> dual_scale(Const2 c, const Dual<Full>& a)
{
    F2 p = two_prod(c.h, a.v);
    return {p.h, fmaf(c.h, a.vl, fmaf(c.l, a.v, p.l)), c.h * a.t};
}
// (a seed does not say which policy its result takes: the caller passes it as a tag)
NFAD_DEV Dual<Fast> dual_scale(Fast, Const2 c, const Seed& a) { return {c.h * a.x, c.h}; }
NFAD_DEV Dual<Full> dual_scale(Full, Const2 c, const Seed& a)
{
    F2 p = two_prod(c.h, a.x);
    return {p.h, fmaf(c.l, a.x, p.l), c.h};
}

// ----------------------------------------------------------------- mul (product rule, Eq. 3)

NFAD_DEV Dual<Fast> dual_mul(Fast, const Seed& a, const Seed& b) { return {a.x * b.x, a.x + b.x}; }
NFAD_DEV Dual<Full> dual_mul(Full, const Seed& a, const Seed& b)
{
    F2 p = two_prod(a.x, b.x);
    return {p.h, p.l, a.x + b.x};
}

// x * b:  value x b.v,  tangent 1 * b.v + x * b.t
NFAD_DEV Dual<Fast> dual_mul(const Seed& a, const Dual<Fast>& b) { return {a.x * b.v, fmaf(a.x, b.t, b.v)}; }
NFAD_DEV Dual<Full> dual_mul(const Seed& a, const Dual<Full>& b)
{
    F2 p = two_prod(a.x, b.v);
    return {p.h, fmaf(a.x, b.vl, p.l), fmaf(a.x, b.t, b.v + b.vl)};
}

NFAD_DEV Dual<Fast> dual_mul(const Dual<Fast>& a, const Dual<Fast>& b)
{
    return {a.v * b.v, fmaf(a.v, b.t, a.t * b.v)};
}
NFAD_DEV Dual<Full> dual_mul(const Dual<Full>& a, const Dual<Full>& b)
{
    F2 p = two_prod(a.v, b.v);
    return {p.h, fmaf(a.v, b.vl, fmaf(a.vl, b.v, p.l)), fmaf(a.v, b.t, a.t * b.v)};
}

// ----------------------------------------------------------------- access helpers for unary primitives

NFAD_DEV float in_v(const Seed& a) { return a.x; }
NFAD_DEV float in_vl(const Seed&) { return 0.0f; }
NFAD_DEV float in_v(const Dual<Fast>& a) { return a.v; }
NFAD_DEV float in_vl(const Dual<Fast>&) { return 0.0f; }
NFAD_DEV float in_v(const Dual<Full>& a) { return a.v; }
NFAD_DEV float in_vl(const Dual<Full>& a) { return a.vl; }
// d * (tangent of the input): the chain rule's last factor; free for the seed
NFAD_DEV float chain(float d, const Seed&) { return d; }
NFAD_DEV float chain(float d, const Dual<Fast>& a) { return d * a.t; }
NFAD_DEV float chain(float d, const Dual<Full>& a) { return d * a.t; }

// ----------------------------------------------------------------- sigmoid

// s = sigmoid(v), s' = s (1 - s).  One exp(-|v|) gives s and 1 - s without
// subtraction; for v >= 0 the value is held as 1 - small.
template <class In> NFAD_DEV Dual<Fast> dual_sigmoid_fast(const In& a)
{
    float v = in_v(a);
    float e = exp2_fast(-1.44269502f * fabsf(v));
    LogisticPair lp = logistic_pair_fast(e);
    bool neg = v < 0.0f;
    float s = neg ? lp.small_ : lp.big;
    return {s, chain(lp.big * lp.small_, a)};
}

template <class In> NFAD_DEV Dual<Full> dual_sigmoid_full(const In& a)
{
    float v = in_v(a), vl = in_vl(a);
    bool neg = v < 0.0f;
    F2 e = exp_full(-fabsf(v), neg ? vl : -vl);
    LogisticPair lp = logistic_pair_full(e);
    float d = lp.big * lp.small_;
    return {neg ? lp.small_ : 1.0f, neg ? 0.0f : -lp.small_, chain(d, a)};
}

NFAD_DEV Dual<Fast> dual_sigmoid(Fast, const Seed& a) { return dual_sigmoid_fast(a); }
NFAD_DEV Dual<Full> dual_sigmoid(Full, const Seed& a) { return dual_sigmoid_full(a); }
NFAD_DEV Dual<Fast> dual_sigmoid(const Dual<Fast>& a) { return dual_sigmoid_fast(a); }
NFAD_DEV Dual<Full> dual_sigmoid(const Dual<Full>& a) { return dual_sigmoid_full(a); }

// ----------------------------------------------------------------- (1 + tanh u)/2

// H = (1 + tanh u)/2 = sigmoid(2u),  H' = 2 H (1 - H)   [= (1 - tanh^2 u)/2]
NFAD_DEV Dual<Fast> dual_half_one_plus_tanh(const Dual<Fast>& u)
{
    float e = exp2_fast(-2.88539004f * fabsf(u.v));
    LogisticPair lp = logistic_pair_fast(e);
    float s = u.v < 0.0f ? lp.small_ : lp.big;
    return {s, (u.t + u.t) * (lp.big * lp.small_)};
}

NFAD_DEV Dual<Full> dual_half_one_plus_tanh(const Dual<Full>& u)
{
    bool neg = u.v < 0.0f;
    float two_ul = u.vl + u.vl;
    F2 e = exp_full(-2.0f * fabsf(u.v), neg ? two_ul : -two_ul);
    LogisticPair lp = logistic_pair_full(e);
    float d = lp.big * lp.small_;
    return {neg ? lp.small_ : 1.0f, neg ? 0.0f : -lp.small_, (u.t + u.t) * d};
}

// ----------------------------------------------------------------- (1 + erf z)/2

// H = (1 + erf z)/2 = erfc(-z)/2,  H' = exp(-z^2)/sqrt(pi).
// With E = exp(-z^2) and W = erfcx(|z|)/2:  erfc(|z|)/2 = E W, so
//   z < 0:  H = E W           z >= 0:  H = 1 - E W
// and the same E serves the tangent.
NFAD_DEV Dual<Fast> dual_half_one_plus_erf(const Dual<Fast>& z)
{
    const float kInvSqrtPi = 0.564189612865448f;
    float za = fabsf(z.v);
    float e = exp2_fast(-1.44269502f * (za * za));
    float a = e * half_erfcx_fast(za);
    float h = z.v < 0.0f ? a : 1.0f - a;
    return {h, (e * kInvSqrtPi) * z.t};
}

NFAD_DEV Dual<Full> dual_half_one_plus_erf(const Dual<Full>& z)
{
    const float kInvSqrtPi = 0.564189612865448f;
    bool neg = z.v < 0.0f;
    float za = fabsf(z.v);
    float zla = neg ? -z.vl : z.vl;            // |z| = za + zla
    F2 sq = two_prod(za, za);
    F2 e = exp_full(-sq.h, -sq.l);             // exp(-za^2): the square is exact
    float w = half_erfcx_full(za);
    float t0 = e.h * kInvSqrtPi;               // |d/dz| of erfc(z)/2 at za
    float a0 = fmaf(e.h, w, e.l * w);          // erfc(za)/2
    // first order in the low part of the argument: the value moves by -t0 zla,
    // the exponential by the factor (1 - 2 za zla)
    float a = fmaf(-t0, zla, a0);
    float t = fmaf(t0, -2.0f * (za * zla), t0);
    return {neg ? a : 1.0f, neg ? 0.0f : -a, t * z.t};
}

// ----------------------------------------------------------------- softplus, and tanh of a softplus

// p = softplus(v) = log1p(exp v),  p' = sigmoid(v).
// The result remembers e = exp(-|v|): every later use of p (its own value, its
// tangent, tanh p) is an algebraic function of e.
template <class P> struct SoftplusDual;
template <> struct SoftplusDual<Fast> { float e; bool neg; float tin; float x; };
template <> struct SoftplusDual<Full> { F2 e; bool neg; float tin; float x; };

NFAD_DEV SoftplusDual<Fast> dual_softplus(Fast, const Seed& a)
{
    return {exp2_fast(-1.44269502f * fabsf(a.x)), a.x < 0.0f, 1.0f, a.x};
}
NFAD_DEV SoftplusDual<Full> dual_softplus(Full, const Seed& a)
{
    return {exp_full(-fabsf(a.x), 0.0f), a.x < 0.0f, 1.0f, a.x};
}

// tanh(log1p(w)) = ((1+w)^2 - 1)/((1+w)^2 + 1) = n/(n+2), n = w^2 + 2w, w = e^v.
// In terms of e = exp(-|v|), all terms positive:
//   v <  0 (w = e):    T = (e^2 + 2e)/(e^2 + 2e + 2)
//   v >= 0 (w = 1/e):  T = 1 - 2e^2/(1 + 2e + 2e^2)
// and T' = sech^2(p) sigmoid(v) = 4 e (1+e) / den^2, times e again for v >= 0.
NFAD_DEV Dual<Fast> dual_tanh(const SoftplusDual<Fast>& p)
{
    float e = p.e;
    float e2 = e * e;
    float num_n = fmaf(e, e, e + e);
    float den = p.neg ? num_n + 2.0f : fmaf(2.0f, e2, fmaf(2.0f, e, 1.0f));
    float rd = hw::rcp_approx(den);
    float sm = (p.neg ? num_n : e2 + e2) * rd;
    float k = (4.0f * e) * (1.0f + e) * (rd * rd);
    return {p.neg ? sm : 1.0f - sm, (p.neg ? k : k * e) * p.tin};
}

NFAD_DEV Dual<Full> dual_tanh(const SoftplusDual<Full>& p)
{
    float e = p.e.h;
    float e2 = e * e;
    float num_n = fmaf(e, e, e + e);
    float den = p.neg ? num_n + 2.0f : fmaf(2.0f, e2, fmaf(2.0f, e, 1.0f));
    float r0 = hw::rcp_approx(den);
    float rd = fmaf(r0, fmaf(-den, r0, 1.0f), r0);
    float sm = (p.neg ? num_n : e2 + e2) * rd;
    float k = (4.0f * e) * (1.0f + e) * (rd * rd);
    return {p.neg ? sm : 1.0f, p.neg ? 0.0f : -sm, (p.neg ? k : k * e) * p.tin};
}

// ----------------------------------------------------------------- the four activations (Table I)

struct GeluErf {};
struct GeluTanh {};
struct Swish {};
struct Mish {};

struct ActOut { float y, dydx; };

// Beyond |x| = kSat the gate h(x) of f = x h(x) is 0 or 1 to every fp32 bit and
// h'(x) is 0, so the chain runs on the clamped argument (which also keeps x^2,
// x^3 finite for any input) and f(x) = x is restored for x > kSat.
template <class K> struct Saturation;
template <> struct Saturation<GeluErf> { static constexpr float kSat = 20.0f; };
template <> struct Saturation<GeluTanh> { static constexpr float kSat = 20.0f; };
template <> struct Saturation<Swish> { static constexpr float kSat = 120.0f; };
template <> struct Saturation<Mish> { static constexpr float kSat = 120.0f; };

// The gate h(x) of each activation f(x) = x h(x), as a dual number.

// GELU, erf form: h = Phi(x) = (1 + erf(x/sqrt2))/2
template <class P> NFAD_DEV Dual<P> gate(GeluErf, Seed X)
{
    const Const2 kInvSqrt2 = {0.7071067690849304f, 1.2101617e-08f};
    Dual<P> Z = dual_scale(P{}, kInvSqrt2, X);
    return dual_half_one_plus_erf(Z);
}

// GELU, tanh form (Table I): h = (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))/2
template <class P> NFAD_DEV Dual<P> gate(GeluTanh, Seed X)
{
    const Const2 kA = {0.044714998453855515f, 1.5461444e-09f};   // 0.044715
    const Const2 kC = {0.7978845834732056f, -2.2670340e-08f};    // sqrt(2/pi)
    Dual<P> X2 = dual_mul(P{}, X, X);
    Dual<P> B = dual_add_const(1.0f, dual_scale(kA, X2));   // 1 + a x^2
    Dual<P> Q = dual_mul(X, B);                             // x + a x^3
    Dual<P> U = dual_scale(kC, Q);
    return dual_half_one_plus_tanh(U);
}

// Swish (Table I, Table II): h = sigmoid(x)
template <class P> NFAD_DEV Dual<P> gate(Swish, Seed X) { return dual_sigmoid(P{}, X); }

// Mish (Table I): h = tanh(softplus(x))
template <class P> NFAD_DEV Dual<P> gate(Mish, Seed X) { return dual_tanh(dual_softplus(P{}, X)); }

// f = x h(x): the last node of every chain is the product of the seed with the
// gate (v3 = v1 v2 with v2 = x in the Swish example), where Eq. 3 merges the tangents.
template <class K, class P> NFAD_DEV Dual<P> activation(K, Seed X) { return dual_mul(X, gate<P>(K{}, X)); }

// x -> (f(x), f'(x)) in fp32, for any finite or non-finite x.
template <class K, class P> NFAD_DEV ActOut evaluate(float x)
{
    constexpr float kSat = Saturation<K>::kSat;
    float xc = x < -kSat ? -kSat : (x > kSat ? kSat : x);    // NaN stays NaN
    Dual<P> Y = activation<K, P>(K{}, Seed{xc});
    float y = dual_value(Y);
    return {x > kSat ? x : y, Y.t};
}

// x -> h(x) alone (what a recomputation pass re-materialises).
template <class K, class P> NFAD_DEV float evaluate_gate(float x)
{
    constexpr float kSat = Saturation<K>::kSat;
    float xc = x < -kSat ? -kSat : (x > kSat ? kSat : x);
    return dual_value(gate<P>(K{}, Seed{xc}));
}

}  // namespace nfad
