/*
 * nfad_bias_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * Plain double-precision CPU definition of the activation pass with its
 * producer's bias folded in: the pre-activation is z = x + b with b one value
 * per column of a row-major [rows, cols] tensor, the activation and its
 * derivative are those of Table I evaluated at z, and back-propagation (Eq. 4)
 * gives grad_in = grad_out * f'(z) for x and, because dz/db = 1 for every row,
 * grad_bias[c] = sum over rows of grad_in[r, c].
 *
 * The paper treats a binary operation with one constant input as unary
 * (Section III-A) and notes that frameworks fuse such chains by hand; the
 * bias-add is that case seen from x.  Nothing here is blocked, fused or
 * reordered: one loop nest per quantity, rows outside, columns inside.
 *
 * Precision decisions, stated because the paper is silent:
 *   - z is the sum rounded ONCE to fp32 (for every storage type): it is the
 *     pre-activation an fp32-accumulating producer hands over, and the CUDA
 *     path forms it with the same single fp32 addition, so both sides evaluate
 *     the activation at the same point.
 *   - grad_in is rounded once to the storage type (as in the plain backward);
 *     grad_bias sums those ROUNDED values (what a separate reduction over the
 *     stored grad_in tensor would see), here in double, row 0 first.
 *
 * Pinned by tests/test_bias_oracle_pins.py (library erf / logistic in double at
 * the fp32-rounded sum on a non-square grid, a tie case of the fp32 addition,
 * exact rational column sums on tiny inputs, closed-form sums).
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>

typedef struct {
    double f, fprime, term_h, term_xh;
} nfad_oracle_point;

/* defined in nfad_oracle.c */
int nfad_oracle_eval_point(int kind, double x, nfad_oracle_point* out);
int nfad_oracle_widen(int dtype, const void* in, size_t n, double* out);
int nfad_oracle_round(int dtype, const double* v, size_t n, void* out);

/* the one fp32 addition: both operands are exact in fp32 */
static double add_in_fp32(double a, double b)
{
    volatile float af = (float)a;
    volatile float bf = (float)b;
    volatile float s = af + bf;
    return (double)s;
}

/*
 * x: rows*cols stored elements, row-major; bias: cols stored elements.
 * f, fprime: rows*cols doubles (unrounded results at z = fl32(x + b)).
 * cond: optional, |h| + |z h'| (the scale f' is compared against); zsum:
 * optional, the pre-activation z itself.
 */
int nfad_bias_oracle_forward(int kind, int dtype, const void* x, const void* bias, size_t rows, size_t cols,
                             double* f, double* fprime, double* cond, double* zsum)
{
    if (kind < 0 || kind > 3) return 1;
    if (dtype < 0 || dtype > 2) return 2;
    if (rows && cols && (!x || !bias || !f || !fprime)) return 3;
    double* xd = (double*)malloc((rows * cols + cols + 1) * sizeof(double));
    if (!xd) return 4;
    double* bd = xd + rows * cols;
    nfad_oracle_widen(dtype, x, rows * cols, xd);
    nfad_oracle_widen(dtype, bias, cols, bd);
    for (size_t r = 0; r < rows; ++r) {
        for (size_t c = 0; c < cols; ++c) {
            size_t i = r * cols + c;
            double z = add_in_fp32(xd[i], bd[c]);
            nfad_oracle_point o;
            nfad_oracle_eval_point(kind, z, &o);
            f[i] = o.f;
            fprime[i] = o.fprime;
            if (cond) cond[i] = fabs(o.term_h) + fabs(o.term_xh);
            if (zsum) zsum[i] = z;
        }
    }
    free(xd);
    return 0;
}

/*
 * grad_out, fprime_saved: rows*cols stored elements.  grad_in: rows*cols stored
 * elements, RN(grad_out * fprime_saved).  grad_bias: cols doubles, the column
 * sums of the rounded grad_in; grad_bias_abs: optional, the column sums of
 * their absolute values (the scale a floating-point summation is judged by).
 */
int nfad_bias_oracle_backward(int dtype, const void* grad_out, const void* fprime_saved, size_t rows, size_t cols,
                              void* grad_in, double* grad_bias, double* grad_bias_abs)
{
    if (dtype < 0 || dtype > 2) return 2;
    if (rows && cols && (!grad_out || !fprime_saved || !grad_in)) return 3;
    if (cols && !grad_bias) return 3;
    size_t n = rows * cols;
    double* gd = (double*)malloc((2 * n + 1) * sizeof(double));
    if (!gd) return 4;
    double* dd = gd + n;
    nfad_oracle_widen(dtype, grad_out, n, gd);
    nfad_oracle_widen(dtype, fprime_saved, n, dd);
    for (size_t i = 0; i < n; ++i) gd[i] = gd[i] * dd[i];          /* exact in double */
    nfad_oracle_round(dtype, gd, n, grad_in);                      /* one rounding to the storage type */
    nfad_oracle_widen(dtype, grad_in, n, gd);                      /* the stored values */
    for (size_t c = 0; c < cols; ++c) {
        grad_bias[c] = 0.0;
        if (grad_bias_abs) grad_bias_abs[c] = 0.0;
    }
    for (size_t r = 0; r < rows; ++r) {
        for (size_t c = 0; c < cols; ++c) {
            double stored = gd[r * cols + c];
            grad_bias[c] += stored;
            if (grad_bias_abs) grad_bias_abs[c] += fabs(stored);
        }
    }
    free(gd);
    return 0;
}
