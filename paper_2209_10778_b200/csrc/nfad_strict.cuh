// nfad_strict.cuh -- f'(x) to a fraction of an fp32 ulp of f'(x) ITSELF, for every x.
//
// For x < 0 the derivative f' = h + x h' is the difference of two positive quantities A = h and
// B = -x h' of similar size, and it changes sign (near -0.75 for the GELUs, -1.28 for Swish, -1.19
// for Mish).  The regular forward pass evaluates A and B to 2^-29 of themselves -- a thirtieth of an
// fp32 ulp of the TERMS, which is what its tolerance asks for -- and that is not an fp32 ulp of
// A - B within about 2^-8 (A + B) of the sign change.  The strict pass runs the same dual-number
// chain (Section II-C approach 3, Eq. 3) on the general-purpose double-precision primitives, whose
// exponential, reciprocal and erfc are good to the last bits of a double: the error of f' is then
// 0.5 ulp + about 2^-27 (A + B)/|A - B| fp32 ulp, i.e. within one ulp even for the fp32 inputs
// nearest to the sign change (no fp32 x brings |f'| below 2^-28 (A + B)).  Results below 2^-126
// are rounded once to the subnormal grid by the conversion itself.
#pragma once

#include "nfad_dual.cuh"

namespace nfad {

// The gate h(x) of each activation on the precise primitives (the argument is already clamped to the
// activation's saturation range).
NFAD_DEV Gate<Wide> gate_precise(GeluErf, Seed X) { return dual_half_one_plus_erf(dual_scale(Wide{}, 0.7071067811865476, X)); }
NFAD_DEV Gate<Wide> gate_precise(GeluTanh, Seed X)
{
    return dual_half_one_plus_tanh(dual_odd_cubic(Wide{}, 0.7978845608028654, 0.035677408136300125, 0.10703222440890037, X));
}
NFAD_DEV Gate<Wide> gate_precise(Swish, Seed X) { return dual_sigmoid(as_wide(X)); }
NFAD_DEV Gate<Wide> gate_precise(Mish, Seed X) { return dual_tanh(Precise{}, dual_softplus(Wide{}, Precise{}, X)); }

// x -> (f(x), f'(x))
template <class K> NFAD_DEV ActOut evaluate_strict(float x)
{
    constexpr float kSat = Saturation<K>::kWide;
    float xc = hw::clamp_nan(x, -kSat, kSat);
    Seed X{xc};
    Gate<Wide> Y = dual_mul(X, gate_precise(K{}, X));
    float y = dual_value(Y);
    return {x > kSat ? x : y, dual_tangent(Y)};
}

template <class K> struct ForwardStrictOp {
    static constexpr int kMinBlocks = 0;
    static constexpr int kUnroll = 4;
    static constexpr int kIn = 1, kOut = 2;
    static constexpr bool kPairs = false;
    static __device__ __forceinline__ constexpr bool keep(int k) { return k == 0; }
    static __device__ __forceinline__ void apply(const float (&in)[1], float (&out)[2])
    {
        ActOut o = evaluate_strict<K>(in[0]);
        out[0] = o.y;
        out[1] = o.dydx;
    }
};

}  // namespace nfad
