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
// and the "binary with a constant, hence unary" fusions that keep the tails free of
// cancellation or save an operation:
//     dual_half_one_plus_tanh(u)        = (1 + tanh u)/2 = sigmoid(2u)
//     dual_half_one_plus_erf(z)         = (1 + erf z)/2  = erfc(-z)/2
//     dual_half_one_plus_erf_scaled(c, x) = (1 + erf(c x))/2 of the seed
//     dual_odd_cubic(c1, c3, x)         = c1 x + c3 x^3,  tangent c1 + 3 c3 x^2
//
// Policies.  Fast (16-bit storage): a value and a tangent are one float each, on the hardware's
// approximate exponential and reciprocal; this file holds its general-purpose primitives (for
// sequences composed at run time), nfad_dual_fast.cuh the chains of the four activations, written
// once for one element per call (Fast) and for two on packed fp32 arithmetic (Fast2).  Wide (fp32
// storage, nfad_dual_wide.cuh): the same algebra in double precision.
//
// Gates.  sigmoid, (1+tanh)/2, (1+erf)/2 and tanh(softplus) are the factors h(x) of the four
// activations f(x) = x h(x); a `Gate` is the dual number (h, h').
#pragma once

#include "nfad_numerics.cuh"

namespace nfad {

// The independent variable: value x, tangent exactly 1.
struct Seed { float x; };

template <class P> struct Dual;
template <> struct Dual<Fast> { float v, t; };

template <class P> struct Gate;
template <> struct Gate<Fast> { float v, t; };

NFAD_DEV float dual_value(const Dual<Fast>& a) { return a.v; }
NFAD_DEV float dual_tangent(const Dual<Fast>& a) { return a.t; }
NFAD_DEV float dual_value(const Gate<Fast>& a) { return a.v; }
NFAD_DEV float dual_tangent(const Gate<Fast>& a) { return a.t; }

// A gate as an ordinary dual (for further generic composition).
NFAD_DEV Dual<Fast> as_dual(const Gate<Fast>& a) { return {a.v, a.t}; }

// tag: the caller keeps the argument where a primitive needs no clamp of its own
struct InRange {};

// ----------------------------------------------------------------- add, scale (linear)

NFAD_DEV Dual<Fast> dual_add(const Dual<Fast>& a, const Dual<Fast>& b) { return {a.v + b.v, a.t + b.t}; }

// c + a (binary with one constant input: unary, tangent unchanged)
NFAD_DEV Dual<Fast> dual_add_const(float c, const Dual<Fast>& a) { return {c + a.v, a.t}; }

// c * a
NFAD_DEV Dual<Fast> dual_scale(float c, const Dual<Fast>& a) { return {c * a.v, c * a.t}; }

// ----------------------------------------------------------------- mul (product rule, Eq. 3)

NFAD_DEV Dual<Fast> dual_mul(const Dual<Fast>& a, const Dual<Fast>& b)
{
    return {a.v * b.v, fmaf(a.v, b.t, a.t * b.v)};
}

// ----------------------------------------------------------------- the logistic function and its slope

// L(w) = 1/(1+exp(-w)), L' = L (1 - L), one form for both signs.  E = 2^-64 exp(-w) comes from one exponential on
// the argument lowered by 64 (flushed to zero only where exp(-w) < 2^-62, far below what a 16-bit result keeps, and
// clamped where it would overflow: beyond w = -133 the slope's E r would be inf * 0); r = 1/(E + 2^-64);
// L = 2^-64 r  and  1 - L = E r, with no subtraction anywhere, so both tails keep their relative accuracy.
// The slope is returned times slope_in * slope_const (the chain rule's next factor and a compile-time constant).
NFAD_DEV Gate<Fast> logistic_fast(float w, float minus_log2e_scale, float slope_in, float slope_const)
{
    float E = hw::ex2_approx_ftz(hw::min_nan(fmaf(w, minus_log2e_scale, -64.0f), 126.0f));
    float r = hw::rcp_approx(E + kTwoPowMinus64);
    float L = r * kTwoPowMinus64;
    return {L, (L * (E * r)) * (slope_in * slope_const)};
}

NFAD_DEV Gate<Fast> dual_sigmoid(const Dual<Fast>& a) { return logistic_fast(a.v, -1.44269502f, a.t, 1.0f); }

// H = (1 + tanh u)/2 = L(2u),  dH/du = 2 L'(2u)   [= (1 - tanh^2 u)/2]
NFAD_DEV Gate<Fast> dual_half_one_plus_tanh(const Dual<Fast>& u) { return logistic_fast(u.v, -2.88539004f, u.t, 2.0f); }

// ----------------------------------------------------------------- (1 + erf z)/2

// H = (1 + erf z)/2 = erfc(-z)/2,  H' = exp(-z^2)/sqrt(pi).
// With E = exp(-z^2) and W = erfcx(|z|)/2:  erfc(|z|)/2 = E W, so
//   z < 0:  H = E W           z >= 0:  H = 1 - E W
// and the same E serves the tangent.  E is formed as 2^64 exp(-z^2) and W as 2^-64 W: see half_erfcx_fast_scaled.
NFAD_DEV Gate<Fast> dual_half_one_plus_erf(const Dual<Fast>& z)
{
    const float kInvSqrtPiScaled = 0.564189612865448f * 5.42101086e-20f;
    float za = fabsf(z.v);
    float e64 = exp2_fast_times_2p64(fmaf(za * za, -1.44269502f, 64.0f));
    float a = e64 * half_erfcx_fast_scaled<6>(hw::rcp_approx(za + kErfcxShift));
    return {z.v < 0.0f ? a : 1.0f - a, e64 * (kInvSqrtPiScaled * z.t)};
}
// ----------------------------------------------------------------- softplus

template <class P> struct SoftplusDual;        // what softplus hands to tanh in the Mish chain (nfad_dual_fast.cuh, nfad_dual_wide.cuh)

// ----------------------------------------------------------------- general-purpose primitives
//
// exp, log1p, tanh, erf and the value of softplus are not needed by the four activation chains (which use the
// cancellation-free fusions above); they are the remaining members of the primitive set, for sequences composed at
// run time.  Plain fp32 on MUFU ex2 / lg2 / rcp: good to a few fp32 ulp of the value where the function itself is
// well conditioned; a user who writes 1 + tanh(u) gets the cancellation that expression has.

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
    float big = fmaf(-2.0f, e64 * half_erfcx_fast_scaled<6>(hw::rcp_approx(aa + kErfcxShift)), 1.0f);
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

}  // namespace nfad

#include "nfad_dual_fast.cuh"
#include "nfad_dual_wide.cuh"

namespace nfad {

// ----------------------------------------------------------------- the four activations (Table I)

struct GeluErf {};
struct GeluTanh {};
struct Swish {};
struct Mish {};

// Where each gate is 0 or 1, and its slope 0, to every bit the storage type keeps.
//   kWide: fp32 storage.  Beyond |x| = kWide the chain runs on the clamped argument (which keeps every intermediate
//          inside the range its primitive states) and f = x is restored on the positive side.
//   kFastGateLo / kFastGateHi: 16-bit storage.  The range of x inside which no Fast intermediate overflows; an
//          infinite end means the chain needs no clamp on that side.
template <class K> struct Saturation;
template <> struct Saturation<GeluErf> {
    static constexpr float kWide = 20.0f;
    static constexpr float kFastGateLo = -3.40282347e+38f, kFastGateHi = 3.40282347e+38f;
};
template <> struct Saturation<GeluTanh> {                // the cubic overflows without a clamp; 2u(11) = 112.5 < 133
    static constexpr float kWide = 11.5f;
    static constexpr float kFastGateLo = -11.0f, kFastGateHi = 11.0f;
};
template <> struct Saturation<Swish> {                   // the logistic's slope needs w >= -133
    static constexpr float kWide = 120.0f;
    static constexpr float kFastGateLo = -130.0f, kFastGateHi = 3.40282347e+38f;
};
template <> struct Saturation<Mish> {                    // tanh(softplus) is formed from exp(x) itself: x <= 20
    static constexpr float kWide = 120.0f;
    static constexpr float kFastGateLo = -3.40282347e+38f, kFastGateHi = 20.0f;
};

// The gate h(x) of each activation f(x) = x h(x), as a dual number (per lane under Fast / Fast2).  The argument is
// inside the range that Saturation states, so the primitives run without clamps of their own.

// GELU, erf form: h = Phi(x) = (1 + erf(x/sqrt2))/2
template <class P> NFAD_DEV Gate<P> gate(P, GeluErf, SeedOf<P> X) { return dual_half_one_plus_erf_scaled<6>(P{}, 0.707106769f, X); }
NFAD_DEV Gate<Wide> gate(Wide, GeluErf, Seed X) { return dual_half_one_plus_erf_scaled(Wide{}, 0.7071067811865476, X); }

// GELU, tanh form (Table I): h = (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))/2
//   u = c x + (c a) x^3 with c = sqrt(2/pi), a = 0.044715 (the double nearest to it); the last constant is 3 c a
//   (1 + tanh u)/2 = sigmoid(2u), and the 2 goes into the cubic's constants (a scale by a constant is unary, Section
//   III-A; doubling is exact, so the value is bit for bit that of (1 + tanh u)/2 formed from u)
template <class P> NFAD_DEV Gate<P> gate(P, GeluTanh, SeedOf<P> X)
{
    return dual_sigmoid(InRange{}, dual_odd_cubic(P{}, 2.0f * 0.797884583f, 2.0f * 0.0356774069f, 2.0f * 0.107032225f, X));
}
NFAD_DEV Gate<Wide> gate(Wide, GeluTanh, Seed X)
{
    return dual_sigmoid(InRange{}, dual_odd_cubic(Wide{}, 2.0 * 0.7978845608028654, 2.0 * 0.035677408136300125, 2.0 * 0.10703222440890037, X));
}

// Swish (Table I, Table II): h = sigmoid(x)
template <class P> NFAD_DEV Gate<P> gate(P, Swish, SeedOf<P> X) { return dual_sigmoid(P{}, InRange{}, X); }
NFAD_DEV Gate<Wide> gate(Wide, Swish, Seed X) { return dual_sigmoid(Wide{}, X); }

// Mish (Table I): h = tanh(softplus(x))
template <class P> NFAD_DEV Gate<P> gate(P, Mish, SeedOf<P> X) { return dual_tanh(dual_softplus(P{}, X)); }
NFAD_DEV Gate<Wide> gate(Wide, Mish, Seed X) { return dual_tanh(dual_softplus(Wide{}, X)); }

template <class T> struct ActOutOf { T y, dydx; };
using ActOut = ActOutOf<float>;
using ActOut2 = ActOutOf<float2>;

// x -> (f(x), f'(x)) in fp32, for any finite or non-finite x.  f = x h(x): the
// last node of every chain is the product of the seed with the gate (v3 = v1 v2
// with v2 = x in the Swish example), where Eq. 3 merges the tangents.

// Wide: the chain in double precision on the clamped argument; the conversions to fp32 are the only roundings.
template <class K> NFAD_DEV ActOut evaluate(K, Wide, float x)
{
    constexpr float kSat = Saturation<K>::kWide;
    float xc = hw::clamp_nan(x, -kSat, kSat);
    Seed X{xc};
    Gate<Wide> Y = dual_mul(X, gate(Wide{}, K{}, X));
    float y = dual_value(Y);
    return {x > kSat ? x : y, dual_tangent(Y)};
}

// Fast (one element) and Fast2 (two).  The gate and the tangent's product see the argument clamped to [kFastGateLo,
// kFastGateHi], beyond which the gate is 0 or 1 and its slope 0 to every bit that a 16-bit result keeps.  The value's
// product sees x itself, kept finite so that -inf gives -0; where the gate's range has no upper end, +inf becomes the
// largest float, which rounds back to inf in either 16-bit type.
template <class K, class P> NFAD_DEV ActOutOf<typename Lanes<P>::type> evaluate(K, P, typename Lanes<P>::type x)
{
    using S = Saturation<K>;
    const float kMax = 3.40282347e+38f;
    SeedOf<P> xl, xg;
    if (S::kFastGateHi >= kMax) {
        xl.x = xg.x = ln::clamp_nan(x, S::kFastGateLo, kMax);
    } else {
        xl.x = ln::max_nan(x, -kMax);
        xg.x = S::kFastGateLo > -kMax ? ln::clamp_nan(x, S::kFastGateLo, S::kFastGateHi) : ln::min_nan(xl.x, S::kFastGateHi);
    }
    Gate<P> Y = dual_mul(xl, xg, gate(P{}, K{}, xg));
    return {Y.v, Y.t};
}

template <class K, class P> NFAD_DEV ActOut evaluate(float x) { return evaluate(K{}, P{}, x); }

// x -> f(x) alone (a pass that will not be differentiated).  Same chain without the tangent parts; under the Fast
// policies the gate's value may come from a cheaper form of the same accuracy class (value_gate), and only what the
// value needs is clamped: -inf becomes the most negative float so that 0 * x gives -0, +inf goes through as it is
// (every gate is exactly 1 there) unless the gate's own range has an upper end.
template <class K, class P> NFAD_DEV typename Lanes<P>::type value_gate(K, P, SeedOf<P> X) { return gate(P{}, K{}, X).v; }
template <class P> NFAD_DEV typename Lanes<P>::type value_gate(GeluErf, P, SeedOf<P> X)
{
    return dual_half_one_plus_erf_scaled<4>(P{}, 0.707106769f, X).v;
}
template <class K> NFAD_DEV float evaluate_value(K, Wide, float x) { return evaluate(K{}, Wide{}, x).y; }
template <class K, class P> NFAD_DEV typename Lanes<P>::type evaluate_value(K, P, typename Lanes<P>::type x)
{
    using S = Saturation<K>;
    const auto xl = ln::max_nan(x, -3.40282347e+38f);
    const auto xg = S::kFastGateHi < 3.40282347e+38f ? ln::min_nan(xl, S::kFastGateHi) : xl;
    return ln::mul(xl, value_gate(K{}, P{}, SeedOf<P>{xg}));
}

// x -> h(x) alone (what a recomputation pass re-materialises).
template <class K> NFAD_DEV float evaluate_gate(K, Wide, float x)
{
    constexpr float kSat = Saturation<K>::kWide;
    return dual_value(gate(Wide{}, K{}, Seed{hw::clamp_nan(x, -kSat, kSat)}));
}
template <class K, class P> NFAD_DEV typename Lanes<P>::type evaluate_gate(K, P, typename Lanes<P>::type x)
{
    using S = Saturation<K>;
    return gate(P{}, K{}, SeedOf<P>{ln::clamp_nan(x, S::kFastGateLo, S::kFastGateHi)}).v;
}
template <class K, class P> NFAD_DEV float evaluate_gate(float x) { return evaluate_gate(K{}, P{}, x); }

}  // namespace nfad
