// nfad_ops.cuh -- the per-element bodies that the streaming engine maps over
// tensors: the nested Forward-AD forward and backward, and the two comparator
// layouts that save x instead of f'(x).
#pragma once

#include "nfad_dual.cuh"

namespace nfad {

// Forward, training: x -> (y = f(x), f'(x)).  One pass over dual numbers; f'(x)
// is the only tensor kept for back-propagation (Section II-C, approach 3).
template <class P> struct IsFast { static constexpr bool value = false; };
template <> struct IsFast<Fast> { static constexpr bool value = true; };
// the chains that evaluate a polynomial (the cubic of GELU-tanh, the scaled erfc fit of GELU-erf): mostly fused
// multiply-adds, which is what packed fp32 arithmetic halves
template <class K> struct HasPolynomial { static constexpr bool value = false; };
template <> struct HasPolynomial<GeluErf> { static constexpr bool value = true; };
template <> struct HasPolynomial<GeluTanh> { static constexpr bool value = true; };

template <class K> struct IsErf { static constexpr bool value = false; };
template <> struct IsErf<GeluErf> { static constexpr bool value = true; };

template <class K, class P> struct ForwardTrainOp {
    static constexpr int kMinBlocks = 0;
    // 16-bit storage, GELU-erf (the longest chain: 25 instructions per element, 16 of them multiply-adds): two elements
    // per call on packed fp32 arithmetic (18 instructions per element).  With four packets per thread the pairs fit the
    // 48-register cap without spills (five packets spill 48-56 bytes), and under a sustained load, where the clock sags
    // and this kernel is short of issue slots, that is worth 2 points for bf16 (0.925 -> 0.945 of the copy peak in the
    // benchmark's own timing) and 4 for fp16.  The other three chains are not short of issue slots: pairs measured
    // equal or 1-5 % slower for them (spills, or one resident CTA less), so they stay at one element per call.
    static constexpr bool kPairs = IsFast<P>::value && IsErf<K>::value;
    // packets per thread and tile, measured at 100.7M elements: 16-bit storage 5 (1-4 % faster than 4; 3 and 6 are slower
    // under the 48-register cap), 4 with pairs; fp32 storage 7 (0.76 / 0.82 / 0.95 / 0.87 of the copy peak against 0.72 /
    // 0.82 / 0.88 / 0.84 with 4; 8 and 10 fall off again)
    static constexpr int kUnroll = IsFast<P>::value ? (kPairs ? 4 : 5) : 7;
    static constexpr int kIn = 1, kOut = 2;
    static __device__ __forceinline__ constexpr bool keep(int k) { return k == 0; }   // y is consumed next; f' much later
    static __device__ __forceinline__ void apply(const float (&in)[1], float (&out)[2])
    {
        ActOut o = evaluate<K, P>(in[0]);
        out[0] = o.y;
        out[1] = o.dydx;
    }
    // the same bits as apply on each element (the chain is one template for both widths)
    static __device__ __forceinline__ void apply2(const float2 (&in)[1], float2 (&out)[2])
    {
        ActOut2 o = evaluate(K{}, Fast2{}, in[0]);
        out[0] = o.y;
        out[1] = o.dydx;
    }
};

// Forward, inference: x -> y.  Same chain; the tangent parts are dead code.
template <class K, class P> struct ForwardInferOp {
    // one input stream and one output.  16-bit storage, the two GELUs: two elements per call on packed fp32 arithmetic,
    // eight packets per thread at four resident CTAs (64 registers: a pair of registers per operand needs the room);
    // measured 0.90 / 0.94 of the copy peak (bf16; 0.86 / 0.92 fp16) against 0.85 / 0.89 (0.82 / 0.91) for one element
    // per call in its best shape.  Swish and Mish (15 and 20 instructions per element, few of them multiply-adds) stay
    // at one element per call, six packets and five CTAs: pairs measured within +-2 % there.  fp32 storage: eight
    // packets, 5-10 % faster than four.
    static constexpr bool kPairs = IsFast<P>::value && HasPolynomial<K>::value;
    static constexpr int kMinBlocks = (IsFast<P>::value && !kPairs) ? 5 : 4;
    static constexpr int kUnroll = (IsFast<P>::value && !kPairs) ? 6 : 8;
    static constexpr int kIn = 1, kOut = 1;
    static __device__ __forceinline__ constexpr bool keep(int) { return true; }
    static __device__ __forceinline__ void apply(const float (&in)[1], float (&out)[1])
    {
        out[0] = evaluate_value(K{}, P{}, in[0]);
    }
    // the same bits as apply on each element (the chain is one template for both widths)
    static __device__ __forceinline__ void apply2(const float2 (&in)[1], float2 (&out)[1])
    {
        out[0] = evaluate_value(K{}, Fast2{}, in[0]);
    }
};

// Backward of the nested layout (Eq. 4): grad_in = grad_out * f'(x), one multiply.
// One fp32 multiply followed by the store's rounding IS the single rounding of the exact
// product, for every storage type:
//   fp32: the multiply is that rounding.
//   fp16: two 11-bit significands give a product of at most 22 bits inside fp32's normal
//         range: exact, so the store's conversion is the only rounding.
//   bf16: two 8-bit significands give M 2^e with M < 2^16.  At or above 2^-126 that is exact
//         in fp32.  Below, fp32's grid is the multiples of 2^-149: a product whose leading bit
//         is at 2^-134 or higher has its last bit at 2^-149 or higher and is exact again; one
//         whose leading bit is lower is below 2^-134, half of bf16's smallest subnormal, and
//         must become a zero of its sign: fp32 rounds it to at most 2^-134 (keeping the
//         sign), which the store's round-to-nearest-even takes to that zero (2^-134 itself is
//         the tie between 0 and 2^-133, and 0 is the even one).
// So there is no double rounding to repair and no data-dependent path in this kernel.
struct BackwardOp {
    static constexpr int kIn = 2, kOut = 1;
    static constexpr int kMinBlocks = 4;   // measured: 4 is 7 % faster than 5 for this load-and-multiply kernel
    static constexpr int kUnroll = 0;
    static __device__ __forceinline__ constexpr bool keep(int) { return true; }
    static __device__ __forceinline__ void apply(const float (&in)[2], float (&out)[1]) { out[0] = __fmul_rn(in[0], in[1]); }
    static constexpr bool kPairs = false;
};

// Conventional layout: x is saved, and backward re-derives f'(x) with the full
// transcendental chain before the multiply.
template <class K, class P> struct ConvBackwardOp {
    // two input streams: their packets alone are 24-40 registers, so room for 64 (four resident CTAs) or the chain's
    // temporaries spill.  Packets per thread, measured at 100.7M elements: 16-bit storage 5 (0.90-1.02 of the copy peak
    // against 0.80-0.89 with 4), fp32 storage 3 (0.72-0.91 against 0.70-0.87).  GELU-erf, 16-bit storage: two elements
    // per call as in the training forward, three packets per thread (more spill): 0.87 -> 0.88 bf16, 0.86 -> 0.88 fp16.
    static constexpr bool kPairs = IsFast<P>::value && IsErf<K>::value;
    static constexpr int kMinBlocks = 4;
    static constexpr int kUnroll = IsFast<P>::value ? (kPairs ? 3 : 5) : 3;
    static constexpr int kIn = 2, kOut = 1;
    static __device__ __forceinline__ constexpr bool keep(int) { return true; }
    static __device__ __forceinline__ void apply(const float (&in)[2], float (&out)[1])
    {
        out[0] = __fmul_rn(in[0], evaluate<K, P>(in[1]).dydx);
    }
    static __device__ __forceinline__ void apply2(const float2 (&in)[2], float2 (&out)[1])
    {
        out[0] = hw::mul2(in[0], evaluate(K{}, Fast2{}, in[1]).dydx);
    }
};

// Recomputation layout (Section II-C, approach 2): x is saved; backward first
// re-runs the forward operators to re-materialise the intermediate the
// per-operator backward rules need (the gate h = v1 of the Swish example), then
// walks those rules: x' = g v1 + g v2 v1' with v2 = x (Eq. 2).
template <class K, class P> struct RecomputePhase1Op {
    // the same widths and tile shapes as the value-only forward
    static constexpr bool kPairs = ForwardInferOp<K, P>::kPairs;
    static constexpr int kMinBlocks = ForwardInferOp<K, P>::kMinBlocks;
    static constexpr int kUnroll = ForwardInferOp<K, P>::kUnroll;
    static constexpr int kIn = 1, kOut = 1;
    static __device__ __forceinline__ constexpr bool keep(int) { return true; }
    static __device__ __forceinline__ void apply(const float (&in)[1], float (&out)[1])
    {
        out[0] = evaluate_gate<K, P>(in[0]);
    }
    static __device__ __forceinline__ void apply2(const float2 (&in)[1], float2 (&out)[1])
    {
        out[0] = evaluate_gate(K{}, Fast2{}, in[0]);
    }
};

// h'(x) from x and the re-materialised h, by each operator's usual backward rule
// (sigmoid: h(1-h); tanh: 1-t^2; erf: exp(-z^2) 2/sqrt(pi); softplus: sigmoid(x)).
template <class K> struct GateSlope;
template <> struct GateSlope<Swish> {
    static __device__ __forceinline__ float of(float, float h) { return h * (1.0f - h); }
};
template <> struct GateSlope<GeluTanh> {
    static __device__ __forceinline__ float of(float x, float h)
    {
        float du2 = fmaf(0.2140644488f, x * x, 1.5957691216f);     // 2 sqrt(2/pi) (1 + 3 * 0.044715 x^2)
        return du2 * (h * (1.0f - h));
    }
};
template <> struct GateSlope<GeluErf> {
    static __device__ __forceinline__ float of(float x, float)
    {
        float xc = fminf(fabsf(x), 20.0f);
        return 0.3989422804f * hw::ex2_approx(-0.72134752f * (xc * xc));   // phi(x)
    }
};
template <> struct GateSlope<Mish> {
    static __device__ __forceinline__ float of(float x, float t)
    {
        float xc = fminf(fabsf(x), 120.0f);
        float e = hw::ex2_approx(-1.44269502f * xc);
        float r = hw::rcp_approx(1.0f + e);
        float sig = x < 0.0f ? e * r : r;
        return fmaf(-t, t, 1.0f) * sig;
    }
};

template <class K, class P> struct RecomputePhase2Op {
    // three input streams: three packets each and 64 registers (see ConvBackwardOp)
    static constexpr int kMinBlocks = 4;
    static constexpr int kUnroll = 3;
    static constexpr int kIn = 3, kOut = 1;            // grad_out, x, h
    static __device__ __forceinline__ constexpr bool keep(int) { return true; }
    static __device__ __forceinline__ void apply(const float (&in)[3], float (&out)[1])
    {
        float g = in[0], x = in[1], h = in[2];
        float hs = GateSlope<K>::of(x, h);
        out[0] = fmaf(g * x, hs, g * h);
    }
    static constexpr bool kPairs = false;
};

// Traffic probe: moves bytes through the same streaming engine with no arithmetic to speak
// of, to measure what a given read/write mix can reach on the device.
template <int NIN, int NOUT> struct ProbeOp {
    static constexpr int kMinBlocks = 4;
    static constexpr int kUnroll = 0;
    static constexpr int kIn = NIN, kOut = NOUT;
    static __device__ __forceinline__ constexpr bool keep(int k) { return k == 0; }
    static __device__ __forceinline__ void apply(const float (&in)[NIN], float (&out)[NOUT])
    {
        float v = in[0];
        if (NIN > 1) v = __uint_as_float(__float_as_uint(v) ^ __float_as_uint(in[1]));
        out[0] = v;
        if (NOUT > 1) out[1] = __uint_as_float(~__float_as_uint(v));
    }
    static constexpr bool kPairs = false;
};

}  // namespace nfad
