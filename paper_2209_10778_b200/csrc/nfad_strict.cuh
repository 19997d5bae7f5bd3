// nfad_strict.cuh -- f'(x) for x < 0 to a fraction of an fp32 ulp of f'(x) ITSELF.
//
// For x < 0 the derivative f' = h + x h' is the difference of two positive quantities A = h and
// B = -x h' of similar size, and it changes sign (near -0.75 for the GELUs, -1.28 for Swish, -1.19
// for Mish).  Arithmetic that is good to an fp32 ulp of A and B -- all that fp32 internals can give,
// and what the regular forward pass guarantees -- is therefore not good to an fp32 ulp of A - B.
// The strict forward pass evaluates A and B for x < 0 in fp64 (cancellation-free forms: every
// exponential has a non-positive argument, 1 - sigmoid is formed as 1/(1+e), Phi as erfc/2) and
// rounds the difference once: the result is within 0.5 ulp + 2^-52 (A + B)/|A - B| ulp... i.e. within
// one fp32 ulp unless |f'| < 2^-27 (A + B), which no fp32 x reaches by more than a factor of two.
// Results below 2^-126 are rounded once to the subnormal grid by the conversion itself.
#pragma once

#include "nfad_dual.cuh"

namespace nfad {

// The argument is already clamped to [-kWide, 0): all exponentials stay finite and non-zero where it matters.
__device__ __forceinline__ double fprime_negative_f64(GeluErf, double x)
{
    const double kInvSqrt2 = 0.70710678118654752440, kInvSqrt2Pi = 0.39894228040143267794;
    double a = 0.5 * erfc(-x * kInvSqrt2);                    // Phi(x)
    double b = -x * (exp(-0.5 * x * x) * kInvSqrt2Pi);        // -x phi(x)
    return a - b;
}

__device__ __forceinline__ double fprime_negative_f64(GeluTanh, double x)
{
    const double c = 0.79788456080286535588, a = 0.044715;
    double x2 = x * x;
    double u = c * (x + a * (x2 * x));                        // < 0
    double e = exp(2.0 * u);
    double big = 1.0 / (1.0 + e);                             // 1 - S
    double s = e * big;                                       // S = (1 + tanh u)/2
    double du2 = 2.0 * c * (1.0 + 3.0 * a * x2);              // 2 u'
    return s - (-x * du2) * (s * big);
}

__device__ __forceinline__ double fprime_negative_f64(Swish, double x)
{
    double e = exp(x);
    double big = 1.0 / (1.0 + e);
    double s = e * big;
    return s - (-x) * (s * big);
}

__device__ __forceinline__ double fprime_negative_f64(Mish, double x)
{
    double w = exp(x);
    double n = w * (w + 2.0);
    double den = n + 2.0;
    double t = n / den;                                       // tanh(softplus x)
    double sech2 = 4.0 * (n + 1.0) / (den * den);
    double sig = w / (1.0 + w);
    return t - (-x) * (sech2 * sig);
}

// x -> (f(x), f'(x)): the value and, for x >= 0, the derivative from the regular fp32-storage chain
// (within a rounding of themselves there); the derivative for x < 0 from the forms above.
template <class K> __device__ __forceinline__ ActOut evaluate_strict(float x)
{
    ActOut o = evaluate(K{}, Wide{}, x);
    if (x < 0.0f) {
        constexpr float kSat = Saturation<K>::kWide;
        o.dydx = __double2float_rn(fprime_negative_f64(K{}, (double)fmaxf(x, -kSat)));
    }
    return o;
}

template <class K> struct ForwardStrictOp {
    static constexpr int kMinBlocks = 3;
    static constexpr int kUnroll = 2;
    static constexpr int kIn = 1, kOut = 2;
    static __device__ __forceinline__ constexpr bool keep(int k) { return k == 0; }
    static __device__ __forceinline__ void apply(const float (&in)[1], float (&out)[2])
    {
        ActOut o = evaluate_strict<K>(in[0]);
        out[0] = o.y;
        out[1] = o.dydx;
    }
};

}  // namespace nfad
