// Test infrastructure: the library's dual-number algebra (paper_2209_10778_b200/csrc/nfad_dual*.cuh) compiled for the
// HOST, so that the chains of the four activations can be checked against the oracle without a GPU.  The hardware layer
// (nfad_hw.cuh) is replaced by plain C stand-ins: the approximate exponential and reciprocal units become exp2f and a
// division (more exact than the hardware, same formulas around them), the packed fp32 instructions become two scalar
// operations.  What this checks is the ALGEBRA -- constants, signs, clamps, the order of operations -- not the
// hardware's rounding; the GPU parity tests check the real thing.
#include <cmath>
#include <cstddef>
#include <cstring>

#define NFAD_HW_PROVIDED
#define NFAD_DEV inline
#define __fmaf_rn(a, b, c) fmaf(a, b, c)
static inline float __fmul_rn(float a, float b) { volatile float r = a * b; return r; }
static inline float __fadd_rn(float a, float b) { volatile float r = a + b; return r; }
struct float2 { float x, y; };
static inline float2 make_float2(float a, float b) { return float2{a, b}; }

namespace nfad { namespace hw {
static inline float ex2_approx(float a) { return exp2f(a); }
static inline float ex2_approx_ftz(float a) { float r = exp2f(a); return r < 1.17549435e-38f ? 0.0f : r; }
static inline float rcp_approx(float a) { return 1.0f / a; }
static inline float lg2_approx(float a) { return log2f(a); }
static inline float min_nan(float a, float hi) { return a != a ? a : (a > hi ? hi : a); }
static inline float max_nan(float a, float lo) { return a != a ? a : (a < lo ? lo : a); }
static inline float clamp_nan(float a, float lo, float hi) { return a != a ? a : (a < lo ? lo : (a > hi ? hi : a)); }
// about 20 good bits, like the hardware's estimate from the upper word
static inline double rcp64_approx(double a)
{
    double r = 1.0 / a;
    long long u;
    memcpy(&u, &r, 8);
    u &= ~0xffffffffLL;
    memcpy(&r, &u, 8);
    return r;
}
static inline int double_hi(double a) { long long u; memcpy(&u, &a, 8); return (int)(u >> 32); }
static inline int double_lo(double a) { long long u; memcpy(&u, &a, 8); return (int)(u & 0xffffffff); }
static inline double double_from(int hi, int lo)
{
    long long u = ((long long)hi << 32) | (unsigned int)lo;
    double r;
    memcpy(&r, &u, 8);
    return r;
}
static inline float to_float(double a) { return (float)a; }
static inline double to_double(float a) { return (double)a; }
static inline float2 fma2(float2 a, float2 b, float2 c) { return {fmaf(a.x, b.x, c.x), fmaf(a.y, b.y, c.y)}; }
static inline float2 mul2(float2 a, float2 b) { return {__fmul_rn(a.x, b.x), __fmul_rn(a.y, b.y)}; }
static inline float2 add2(float2 a, float2 b) { return {__fadd_rn(a.x, b.x), __fadd_rn(a.y, b.y)}; }
static inline int float_as_int(float a) { int i; memcpy(&i, &a, 4); return i; }
static inline float int_as_float(int a) { float f; memcpy(&f, &a, 4); return f; }
}}  // namespace nfad::hw

#include "nfad_dual.cuh"

using namespace nfad;

// width: 0 = one element per call (Fast), 1 = two per call (Fast2; n even), 2 = double precision (Wide)
template <class K> static void run(int width, const float* x, float* y, float* d, float* v, float* h, size_t n)
{
    if (width == 1) {
        for (size_t i = 0; i + 1 < n; i += 2) {
            float2 in = make_float2(x[i], x[i + 1]);
            ActOut2 o = evaluate(K{}, Fast2{}, in);
            float2 vv = evaluate_value(K{}, Fast2{}, in);
            float2 hh = evaluate_gate(K{}, Fast2{}, in);
            y[i] = o.y.x; y[i + 1] = o.y.y;
            d[i] = o.dydx.x; d[i + 1] = o.dydx.y;
            v[i] = vv.x; v[i + 1] = vv.y;
            h[i] = hh.x; h[i + 1] = hh.y;
        }
        return;
    }
    for (size_t i = 0; i < n; ++i) {
        if (width == 0) {
            ActOut o = evaluate(K{}, Fast{}, x[i]);
            y[i] = o.y; d[i] = o.dydx;
            v[i] = evaluate_value(K{}, Fast{}, x[i]);
            h[i] = evaluate_gate(K{}, Fast{}, x[i]);
        } else {
            ActOut o = evaluate(K{}, Wide{}, x[i]);
            y[i] = o.y; d[i] = o.dydx;
            v[i] = evaluate_value(K{}, Wide{}, x[i]);
            h[i] = evaluate_gate(K{}, Wide{}, x[i]);
        }
    }
}

// y = f(x), d = f'(x), v = f(x) from the value-only form, h = the gate alone
extern "C" void host_algebra(int kind, int width, const float* x, float* y, float* d, float* v, float* h, size_t n)
{
    switch (kind) {
    case 0: run<GeluErf>(width, x, y, d, v, h, n); break;
    case 1: run<GeluTanh>(width, x, y, d, v, h, n); break;
    case 2: run<Swish>(width, x, y, d, v, h, n); break;
    case 3: run<Mish>(width, x, y, d, v, h, n); break;
    }
}

// one general-purpose primitive applied to the dual (x, 1): value and tangent.  op: 0 exp, 1 log1p, 2 tanh, 3 erf,
// 4 softplus, 5 sigmoid, 6 (1 + tanh)/2, 7 (1 + erf)/2.  wide: 0 fp32 arithmetic, 1 double.
template <class D, class T> static void prim(int op, T x, T* v, T* t)
{
    D a{x, T(1)}, r{T(0), T(0)};
    switch (op) {
    case 0: r = dual_exp(a); break;
    case 1: r = dual_log1p(a); break;
    case 2: r = dual_tanh(a); break;
    case 3: r = dual_erf(a); break;
    case 4: r = dual_softplus(a); break;
    case 5: r = as_dual(dual_sigmoid(a)); break;
    case 6: r = as_dual(dual_half_one_plus_tanh(a)); break;
    case 7: r = as_dual(dual_half_one_plus_erf(a)); break;
    }
    *v = r.v;
    *t = r.t;
}
extern "C" void host_primitive(int op, int wide, const double* x, double* v, double* t, size_t n)
{
    for (size_t i = 0; i < n; ++i) {
        if (wide) {
            prim<Dual<Wide>, double>(op, x[i], &v[i], &t[i]);
        } else {
            float fv, ft;
            prim<Dual<Fast>, float>(op, (float)x[i], &fv, &ft);
            v[i] = fv;
            t[i] = ft;
        }
    }
}
