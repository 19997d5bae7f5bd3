/*
 * nfad_seq_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * Double-precision evaluation of a FAD sequence: a straight-line program of
 * primitive operations (Section III-A) applied to one source x, with M results
 * (R^1 -> R^M).  The derivative of every result with respect to x is what the
 * chain rule and the product / sum rules give (Section II-D: the Jacobian of the
 * composition is the product of the primitives' Jacobians, applied to x' = 1), so
 * each register carries the value and that derivative, both in fp64, each
 * primitive written as its textbook definition and textbook derivative with libm:
 *
 *   add   v = a + b        v' = a' + b'         mul   v = a b         v' = a' b + a b'
 *   scale v = c a          v' = c a'            addc  v = c + a       v' = a'
 *   exp   v = e^a          v' = v a'            log1p v = log(1+a)    v' = a'/(1+a)
 *   tanh  v = tanh a       v' = a'/cosh^2 a     erf   v = erf a       v' = 2/sqrt(pi) e^(-a^2) a'
 *   softplus v = log(1+e^a) (two-branch form)   v' = sigmoid(a) a'
 *   sigmoid  v = 1/(1+e^-a) (two-branch form)   v' = sigmoid(a) sigmoid(-a) a'
 *   (1+tanh a)/2 = sigmoid(2a)                  v' = 2 sigmoid(2a) sigmoid(-2a) a'
 *   (1+erf a)/2 = erfc(-a)/2                    v' = e^(-a^2)/sqrt(pi) a'
 *
 * The backward of a sequence (Section II-E) is sum_k g_k * dy_k/dx, formed in fp64
 * from the stored operands and rounded once to the storage type.
 *
 * Pins: tests/test_seq_oracle_pins.py (the four activations written as programs
 * against the closed-form oracle, central differences per primitive, hand values).
 * Shares no code with the CUDA path; the program crosses the boundary as plain arrays.
 */
#include <math.h>
#include <stddef.h>

enum { OP_ADD = 0, OP_MUL, OP_SCALE, OP_ADDC, OP_EXP, OP_LOG1P, OP_TANH, OP_ERF, OP_SOFTPLUS, OP_SIGMOID, OP_H1PT, OP_H1PE, OP_OUT };
#define MAX_REGS 12
#define MAX_OUT 4

static double sig(double z)
{
    if (z >= 0.0) return 1.0 / (1.0 + exp(-z));
    double e = exp(z);
    return e / (1.0 + e);
}

/* Returns 0, or 10 for a malformed program. */
int nfad_seq_oracle_point(int n_ops, const int* op, const int* a, const int* b, const int* dst, const double* c,
                          double x, int m, double* y, double* dydx)
{
    double v[MAX_REGS], t[MAX_REGS];
    int have[MAX_REGS] = {1};
    v[0] = x;
    t[0] = 1.0;                                     /* the seed x' = 1 */
    if (m < 1 || m > MAX_OUT) return 10;
    for (int i = 0; i < n_ops; ++i) {
        int ra = a[i], rb = b[i], rd = dst[i];
        if (ra < 0 || ra >= MAX_REGS || !have[ra]) return 10;
        double av = v[ra], at = t[ra], rv, rt;
        switch (op[i]) {
        case OP_ADD:
            if (rb < 0 || rb >= MAX_REGS || !have[rb]) return 10;
            rv = av + v[rb]; rt = at + t[rb]; break;
        case OP_MUL:
            if (rb < 0 || rb >= MAX_REGS || !have[rb]) return 10;
            rv = av * v[rb]; rt = at * v[rb] + av * t[rb]; break;
        case OP_SCALE: rv = c[i] * av; rt = c[i] * at; break;
        case OP_ADDC: rv = c[i] + av; rt = at; break;
        case OP_EXP: rv = exp(av); rt = rv * at; break;
        case OP_LOG1P: rv = log1p(av); rt = at / (1.0 + av); break;
        case OP_TANH: { double ch = cosh(av); rv = tanh(av); rt = isinf(ch) ? 0.0 : at / (ch * ch); } break;
        case OP_ERF: rv = erf(av); rt = 1.1283791670955126 * exp(-av * av) * at; break;
        case OP_SOFTPLUS: rv = av <= 0.0 ? log1p(exp(av)) : av + log1p(exp(-av)); rt = sig(av) * at; break;
        case OP_SIGMOID: rv = sig(av); rt = sig(av) * sig(-av) * at; break;
        case OP_H1PT: rv = sig(2.0 * av); rt = 2.0 * sig(2.0 * av) * sig(-2.0 * av) * at; break;
        case OP_H1PE: rv = 0.5 * erfc(-av); rt = 0.5641895835477563 * exp(-av * av) * at; break;
        case OP_OUT:
            if (rd < 0 || rd >= m) return 10;
            y[rd] = av; dydx[rd] = at; continue;
        default: return 10;
        }
        if (rd < 1 || rd >= MAX_REGS) return 10;
        v[rd] = rv; t[rd] = rt; have[rd] = 1;
    }
    return 0;
}

/* x: n doubles (already widened); y, dydx: m blocks of n doubles each. */
int nfad_seq_oracle_forward(int n_ops, const int* op, const int* a, const int* b, const int* dst, const double* c,
                            const double* x, size_t n, int m, double* y, double* dydx)
{
    for (size_t i = 0; i < n; ++i) {
        double yy[MAX_OUT], dd[MAX_OUT];
        int rc = nfad_seq_oracle_point(n_ops, op, a, b, dst, c, x[i], m, yy, dd);
        if (rc) return rc;
        for (int k = 0; k < m; ++k) { y[(size_t)k * n + i] = yy[k]; dydx[(size_t)k * n + i] = dd[k]; }
    }
    return 0;
}

/* sum_k g_k d_k in fp64 (operands: m blocks of n doubles); also sum_k |g_k d_k| for tolerances. */
int nfad_seq_oracle_backward(const double* g, const double* d, size_t n, int m, double* out, double* out_abs)
{
    for (size_t i = 0; i < n; ++i) {
        double s = 0.0, sa = 0.0;
        for (int k = 0; k < m; ++k) { double p = g[(size_t)k * n + i] * d[(size_t)k * n + i]; s += p; sa += fabs(p); }
        out[i] = s;
        if (out_abs) out_abs[i] = sa;
    }
    return 0;
}
