/*
 * nfad_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, double-precision CPU evaluation of what the nested
 * Forward-AD activation pass computes: y = f(x), the saved tensor f'(x), and
 * the backward product grad_in = grad_out * f'(x).  Forward-AD is exact
 * differentiation (Section II-C, approach 3; Section II-E), so the result it
 * reaches has a plain definition: the activation of Table I and its textbook
 * derivative.  This file writes those definitions out, one expression per
 * quantity, with no dual numbers, no blocking, no vectorisation and no code
 * shared with the CUDA path.  Only tests, the smoke check and the benchmark's
 * cpu_baseline / reference arm may call it.
 *
 * Activations (Table I, plus the erf-exact GELU the paper only cites):
 *   GELU-erf  f = x * Phi(x),                Phi = standard normal CDF
 *   GELU-tanh f = 0.5 x (1 + tanh(u)),       u = sqrt(2/pi) (x + 0.044715 x^3)
 *   Swish     f = x * sigmoid(x)                          (Table I, Table II)
 *   Mish      f = x * tanh(softplus(x))                   (Table I)
 *
 * Derivatives (product rule of Eq. 3 applied to f = x * h(x): f' = h + x h'):
 *   GELU-erf  f' = Phi(x) + x phi(x)
 *   GELU-tanh f' = S + x * 2 u'(x) * S (1 - S),  S = sigmoid(2u) = (1+tanh u)/2
 *   Swish     f' = s + x s (1 - s)                        (Table II)
 *   Mish      f' = t + x * sech^2(softplus x) * sigmoid(x)
 *
 * Rewritings used, each an exact identity chosen so that no quantity is formed
 * by subtracting nearly equal numbers (a literal "1 + tanh(u)" or "1 + erf(z)"
 * has no correct digit in double once x < -8, while the true result, about
 * 1e-21, is an ordinary fp32 number):
 *   (1 + tanh u)/2 = sigmoid(2u),   1 - tanh^2 u = 4 sigmoid(2u) sigmoid(-2u)
 *   (1 + erf(z))/2 = erfc(-z)/2
 *   1 - sigmoid(z) = sigmoid(-z)
 *   sigmoid(z) = 1/(1+exp(-z)) for z >= 0, exp(z)/(1+exp(z)) for z < 0
 *   softplus(x) = log1p(exp(x)) for x <= 0, x + log1p(exp(-x)) for x > 0
 *   1 - tanh^2 p = 1/cosh^2 p
 * The only remaining cancellation is the one inherent in f' itself, whose two
 * addends have opposite signs for x < 0.
 *
 * Backward (Eq. 4, Section II-E): grad_in = grad_out * f'.  Both factors are
 * stored values of at most 24 significant bits, so their product is exact in
 * double and is rounded once to the storage type.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_pins.py
 * (fixed points, symmetries, limits, central differences, 50-digit mpmath,
 * torch/scipy double-precision library routines, brute-force rounding).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { KIND_GELU_ERF = 0, KIND_GELU_TANH = 1, KIND_SWISH = 2, KIND_MISH = 3 };
enum { DT_F32 = 0, DT_BF16 = 1, DT_F16 = 2 };

typedef struct {
    double f;        /* f(x)                                         */
    double fprime;   /* f'(x) = term_h + term_xh                     */
    double term_h;   /* h(x),  the first addend of the product rule  */
    double term_xh;  /* x h'(x), the second addend                   */
} nfad_oracle_point;

static int g_threads = 1;

/* ---- elementary pieces -------------------------------------------------- */

static double sigmoid_d(double z)
{
    if (z >= 0.0) return 1.0 / (1.0 + exp(-z));
    double e = exp(z);
    return e / (1.0 + e);
}

static double softplus_d(double x)
{
    if (x <= 0.0) return log1p(exp(x));
    return x + log1p(exp(-x));
}

/* ---- the four activations ----------------------------------------------- */

static void gelu_erf_d(double x, nfad_oracle_point* o)
{
    const double inv_sqrt2 = 0.70710678118654752440;   /* 1/sqrt(2)    */
    const double inv_sqrt_2pi = 0.39894228040143267794; /* 1/sqrt(2 pi) */
    double Phi = 0.5 * erfc(-x * inv_sqrt2);
    double phi = exp(-0.5 * x * x) * inv_sqrt_2pi;
    o->f = x * Phi;
    o->term_h = Phi;
    o->term_xh = x * phi;
    o->fprime = o->term_h + o->term_xh;
}

static void gelu_tanh_d(double x, nfad_oracle_point* o)
{
    const double c = 0.79788456080286535588;  /* sqrt(2/pi) */
    const double a = 0.044715;                /* Table I    */
    double u = c * (x + a * x * x * x);
    double du = c * (1.0 + 3.0 * a * x * x);
    double S = sigmoid_d(2.0 * u);            /* (1 + tanh u)/2 */
    double Sc = sigmoid_d(-2.0 * u);          /* 1 - S          */
    o->f = x * S;
    o->term_h = S;
    o->term_xh = x * (2.0 * du) * S * Sc;
    o->fprime = o->term_h + o->term_xh;
}

static void swish_d(double x, nfad_oracle_point* o)
{
    double s = sigmoid_d(x);
    double sc = sigmoid_d(-x);                /* 1 - s */
    o->f = x * s;
    o->term_h = s;
    o->term_xh = x * s * sc;
    o->fprime = o->term_h + o->term_xh;
}

static void mish_d(double x, nfad_oracle_point* o)
{
    double p = softplus_d(x);
    double t = tanh(p);
    double ch = cosh(p);                      /* p <= ~710 keeps cosh finite for |x| of interest */
    double sech2 = isinf(ch) ? 0.0 : 1.0 / (ch * ch);
    o->f = x * t;
    o->term_h = t;
    o->term_xh = x * sech2 * sigmoid_d(x);
    o->fprime = o->term_h + o->term_xh;
}

int nfad_oracle_eval_point(int kind, double x, nfad_oracle_point* out)
{
    if (!out) return 3;
    switch (kind) {
    case KIND_GELU_ERF:  gelu_erf_d(x, out);  return 0;
    case KIND_GELU_TANH: gelu_tanh_d(x, out); return 0;
    case KIND_SWISH:     swish_d(x, out);     return 0;
    case KIND_MISH:      mish_d(x, out);      return 0;
    default: return 1;
    }
}

/* ---- storage formats ----------------------------------------------------- */

static double widen_f32(const void* p, size_t i)
{
    float v;
    memcpy(&v, (const char*)p + 4 * i, 4);
    return (double)v;
}

static double widen_bf16(const void* p, size_t i)
{
    uint16_t h;
    memcpy(&h, (const char*)p + 2 * i, 2);
    uint32_t w = (uint32_t)h << 16;           /* bf16 is the top half of an fp32 */
    float v;
    memcpy(&v, &w, 4);
    return (double)v;
}

static double widen_f16(const void* p, size_t i)
{
    uint16_t h;
    memcpy(&h, (const char*)p + 2 * i, 2);
    int sign = (h >> 15) & 1;
    int ex = (h >> 10) & 0x1f;
    int man = h & 0x3ff;
    double v;
    if (ex == 0)        v = ldexp((double)man, -24);               /* subnormal or zero */
    else if (ex == 31)  v = man ? NAN : INFINITY;
    else                v = ldexp((double)(man + 1024), ex - 25);
    return sign ? -v : v;
}

static double widen(int dtype, const void* p, size_t i)
{
    if (dtype == DT_F32) return widen_f32(p, i);
    if (dtype == DT_BF16) return widen_bf16(p, i);
    return widen_f16(p, i);
}

/*
 * Round a double to a binary format with `pbits` significand bits (hidden bit
 * included), minimum normal exponent `emin` and maximum exponent `emax`, with
 * round-to-nearest-even, in ONE rounding (never through fp32).  Returns the
 * rounded value as a double plus its pieces for packing.
 */
static double round_to_format(double v, int pbits, int emin, int emax, int* is_inf)
{
    *is_inf = 0;
    if (v == 0.0 || isnan(v)) return v;
    if (isinf(v)) { *is_inf = 1; return v; }
    int e;
    double m = frexp(fabs(v), &e);            /* |v| = m 2^e, m in [0.5, 1) */
    int exp_unb = e - 1;                      /* |v| = (2m) 2^(e-1)         */
    int q;                                    /* quantum exponent: result is a multiple of 2^q */
    if (exp_unb < emin) q = emin - (pbits - 1);
    else                q = exp_unb - (pbits - 1);
    double scaled = ldexp(fabs(v), -q);       /* exact: power-of-two scaling */
    double r = nearbyint(scaled);             /* default mode: ties to even  */
    double out = ldexp(r, q);
    if (out >= ldexp(1.0, emax + 1)) { *is_inf = 1; out = INFINITY; }
    (void)m;
    return v < 0 ? -out : out;
}

static void narrow_store(int dtype, double v, void* p, size_t i)
{
    int inf;
    if (dtype == DT_F32) {
        float f = (float)v;                   /* C conversion: correctly rounded, RNE */
        memcpy((char*)p + 4 * i, &f, 4);
        return;
    }
    uint16_t h;
    if (dtype == DT_BF16) {
        if (isnan(v)) h = 0x7fc0;
        else {
            double r = round_to_format(v, 8, -126, 127, &inf);
            float f = (float)r;               /* exact: r is a bf16 value */
            uint32_t w;
            memcpy(&w, &f, 4);
            h = (uint16_t)(w >> 16);
        }
    } else {
        if (isnan(v)) h = 0x7e00;
        else {
            double r = round_to_format(v, 11, -14, 15, &inf);
            uint16_t sign = signbit(r) ? 0x8000 : 0;
            double a = fabs(r);
            if (inf) h = sign | 0x7c00;
            else if (a == 0.0) h = sign;
            else if (a < ldexp(1.0, -14)) h = sign | (uint16_t)ldexp(a, 24);
            else {
                int e;
                double m = frexp(a, &e);      /* a = m 2^e, m in [0.5,1) */
                int biased = (e - 1) + 15;
                int man = (int)ldexp(m, 11) - 1024;
                h = sign | (uint16_t)(biased << 10) | (uint16_t)man;
            }
        }
    }
    memcpy((char*)p + 2 * i, &h, 2);
}

/* ---- array entry points --------------------------------------------------- */

void nfad_oracle_set_threads(int t) { g_threads = t < 1 ? 1 : t; }

int nfad_oracle_get_threads(void) { return g_threads; }

int nfad_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_num_procs();
#else
    return 1;
#endif
}

/*
 * x: n stored elements of `dtype`.  f, fprime: n doubles each (unrounded
 * results).  cond: optional n doubles, |term_h| + |term_xh|, the scale the
 * cancellation in f' is measured against; may be NULL.
 */
int nfad_oracle_forward(int kind, int dtype, const void* x, size_t n,
                        double* f, double* fprime, double* cond)
{
    if (kind < 0 || kind > 3) return 1;
    if (dtype < 0 || dtype > 2) return 2;
    if (n && (!x || !f || !fprime)) return 3;
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(static)
#endif
    for (long long i = 0; i < (long long)n; ++i) {
        nfad_oracle_point o;
        nfad_oracle_eval_point(kind, widen(dtype, x, (size_t)i), &o);
        f[i] = o.f;
        fprime[i] = o.fprime;
        if (cond) cond[i] = fabs(o.term_h) + fabs(o.term_xh);
    }
    return 0;
}

/* One correct rounding of each double to the storage type. */
int nfad_oracle_round(int dtype, const double* v, size_t n, void* out)
{
    if (dtype < 0 || dtype > 2) return 2;
    if (n && (!v || !out)) return 3;
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(static)
#endif
    for (long long i = 0; i < (long long)n; ++i) narrow_store(dtype, v[i], out, (size_t)i);
    return 0;
}

/* Stored elements to doubles (exact). */
int nfad_oracle_widen(int dtype, const void* in, size_t n, double* out)
{
    if (dtype < 0 || dtype > 2) return 2;
    if (n && (!in || !out)) return 3;
    for (size_t i = 0; i < n; ++i) out[i] = widen(dtype, in, i);
    return 0;
}

/* grad_in = RN_dtype( grad_out * fprime_saved ), product exact in double. */
int nfad_oracle_backward(int dtype, const void* grad_out, const void* fprime_saved,
                         size_t n, void* grad_in)
{
    if (dtype < 0 || dtype > 2) return 2;
    if (n && (!grad_out || !fprime_saved || !grad_in)) return 3;
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(static)
#endif
    for (long long i = 0; i < (long long)n; ++i) {
        double g = widen(dtype, grad_out, (size_t)i);
        double d = widen(dtype, fprime_saved, (size_t)i);
        narrow_store(dtype, g * d, grad_in, (size_t)i);
    }
    return 0;
}

/*
 * The whole hot path as the oracle sees it, for timing: forward in double,
 * round y and f' to the storage type, then the backward product from the
 * rounded f'.  y, fprime_saved, grad_in: n stored elements each.
 */
int nfad_oracle_forward_backward(int kind, int dtype, const void* x, const void* grad_out,
                                 size_t n, void* y, void* fprime_saved, void* grad_in)
{
    if (kind < 0 || kind > 3) return 1;
    if (dtype < 0 || dtype > 2) return 2;
    if (n && (!x || !grad_out || !y || !fprime_saved || !grad_in)) return 3;
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(static)
#endif
    for (long long i = 0; i < (long long)n; ++i) {
        nfad_oracle_point o;
        nfad_oracle_eval_point(kind, widen(dtype, x, (size_t)i), &o);
        narrow_store(dtype, o.f, y, (size_t)i);
        narrow_store(dtype, o.fprime, fprime_saved, (size_t)i);
        double g = widen(dtype, grad_out, (size_t)i);
        double d = widen(dtype, fprime_saved, (size_t)i);
        narrow_store(dtype, g * d, grad_in, (size_t)i);
    }
    return 0;
}
