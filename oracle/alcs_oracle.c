/*
 * CPU oracle for the SIMD-structured sparse convolution (pointwise first, general k x k at
 * the end of the file).
 *
 * TEST INFRASTRUCTURE ONLY: the library under test never calls this file; only the tests,
 * the smoke check and the benchmark's CPU-baseline leg may.  It shares no code with the
 * CUDA path and never sees the packed weight format.
 *
 * What it computes is the paper's convolution definition (Section 3.2.2, the unnumbered
 * equation  O(n,h,w) = sum_c sum_r sum_s W(n,c,r,s) I(c,h+r,w+s) ) for k_h = k_w = 1, with the
 * pruned weights written as explicit zeros (Section 3.2.1: all g filters of a group share
 * their zero locations).  Because pruning only replaces weights by zero, the sparse result
 * has a plain definition, and the oracle is that definition: a dense triple loop over the
 * mask-applied weights with NO zero skipping, accumulated in double precision in ascending
 * input-channel order.  Bias and ReLU are the epilogue the workload adds on top of the
 * paper's formula: y = max(acc + bias, 0).
 *
 * Block membership: block row r holds output channels r*g .. r*g+g-1 ("each 4 adjacent
 * channels", Section 3.2.1); mask[r][c] != 0 keeps the block (r, c).
 *
 * Also produced on request: the condition scale  A = |bias| + sum_c |Wm||X|,  the standard
 * forward-error scale of a dot product, against which the tests state their tolerance.
 *
 * fp16 inputs arrive as IEEE binary16 bit patterns and are decoded here, by this file's own
 * decoder, before the double-precision arithmetic.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ORACLE_MUTANT plants one deliberate mistake; used only by the tests that check that the
 * pins can tell a wrong oracle from a right one.  0 (default) is the real oracle. */
#ifndef ORACLE_MUTANT
#define ORACLE_MUTANT 0
#endif

static double half_to_double(uint16_t h)
{
    const int sign = (h >> 15) & 1;
    const int ex = (h >> 10) & 0x1f;
    const int man = h & 0x3ff;
    double v;
    if (ex == 0)
        v = ldexp((double)man, -24);                 /* zero and subnormals */
    else if (ex == 31)
        v = man ? NAN : INFINITY;
    else
        v = ldexp((double)(man | 0x400), ex - 25);   /* 1.m * 2^(ex-15) */
    return sign ? -v : v;
}

static inline double ld_f32(const void *p, size_t i) { return (double)((const float *)p)[i]; }
static inline double ld_f16(const void *p, size_t i) { return half_to_double(((const uint16_t *)p)[i]); }

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int oracle_mutant(void) { return ORACLE_MUTANT; }

static inline double masked_weight(const void *W, int is_f16, const uint8_t *mask, int g,
                                   int cin, int cout, int co, int ci)
{
#if ORACLE_MUTANT == 1            /* wrong block membership: interleaved instead of adjacent */
    const int r = co % ((cout + g - 1) / g);
#else
    const int r = co / g;
    (void)cout;
#endif
    size_t wi = (size_t)co * cin + ci;
#if ORACLE_MUTANT == 2            /* transposed weight operand (planted only for square W) */
    if (cin == cout) wi = (size_t)ci * cin + co;
#endif
    const double w = is_f16 ? ld_f16(W, wi) : ld_f32(W, wi);
    return mask[(size_t)r * cin + ci] ? w : 0.0;
}

/*
 * Full output.  W [cout][cin], mask [ceil(cout/g)][cin], X [n][cin][hw], bias [cout] or NULL.
 * Y (double, [n][cout][hw]) and A (same shape) may each be NULL.  Returns 0, or -1 on bad
 * arguments, -2 if out of memory.
 */
int oracle_conv1x1(const void *W, const uint8_t *mask, int g, const void *X, const float *bias,
                   int relu, int is_f16, int n, int cin, int cout, long hw, double *Y, double *A)
{
    if (!W || !mask || !X || g < 1 || n < 0 || cin < 0 || cout < 0 || hw < 0) return -1;
    int fail = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int in = 0; in < n; ++in) {
        for (int co = 0; co < cout; ++co) {
            double *acc = (double *)calloc((size_t)(hw > 0 ? hw : 1), sizeof(double));
            double *mag = A ? (double *)calloc((size_t)(hw > 0 ? hw : 1), sizeof(double)) : NULL;
            if (!acc || (A && !mag)) { fail = 1; free(acc); free(mag); continue; }
            for (int ci = 0; ci < cin; ++ci) {
                const double wm = masked_weight(W, is_f16, mask, g, cin, cout, co, ci);
                const size_t xoff = ((size_t)in * cin + ci) * (size_t)hw;
#if ORACLE_MUTANT == 3            /* dropped term: the last input channel is never added */
                if (ci == cin - 1 && cin > 1) continue;
#endif
                if (is_f16) {
                    for (long p = 0; p < hw; ++p) {
                        const double x = ld_f16(X, xoff + p);
                        acc[p] += wm * x;
                        if (mag) mag[p] += fabs(wm) * fabs(x);
                    }
                } else {
                    const float *xr = (const float *)X + xoff;
                    for (long p = 0; p < hw; ++p) {
                        acc[p] += wm * (double)xr[p];
                        if (mag) mag[p] += fabs(wm) * fabs((double)xr[p]);
                    }
                }
            }
            const double b = bias ? (double)bias[co] : 0.0;
            const size_t yoff = ((size_t)in * cout + co) * (size_t)hw;
            for (long p = 0; p < hw; ++p) {
#if ORACLE_MUTANT == 4            /* wrong sign on the bias */
                double s = acc[p] - b;
#elif ORACLE_MUTANT == 5          /* ReLU applied before the bias instead of after */
                double s = (relu && acc[p] < 0.0 ? 0.0 : acc[p]) + b;
#else
                double s = acc[p] + b;
#endif
#if ORACLE_MUTANT != 5
                if (relu && s < 0.0) s = 0.0;
#endif
                if (Y) Y[yoff + p] = s;
                if (A) A[yoff + p] = mag[p] + fabs(b);
            }
            free(acc);
            free(mag);
        }
    }
    return fail ? -2 : 0;
}

/*
 * Pointwise convolution with stride and a residual operand (the shape of a ResNet bottleneck's last
 * 1x1 convolution and of its projection shortcut): the paper's formula at k_h = k_w = 1 sampled at
 * stride s,
 *     O(co, oh, ow) = sum_c Wm(co, c) * I(c, oh*s, ow*s),   oh < ceil(h/s), ow < ceil(wd/s),
 * then  y = O + bias + R  and, if relu, y = max(y, 0): the residual is added BEFORE the activation.
 * X [n][cin][h][wd]; R (may be NULL) [n][cout][oh*ow] of fp32, or of binary16 if res_is_f16;
 * Y, A (double, [n][cout][oh*ow]) may each be NULL; A = |bias| + |R| + sum |Wm||I|.
 * Dense triple loop, no zero skipping.  Returns 0, -1 on bad arguments.
 */
int oracle_conv1x1_ex(const void *W, const uint8_t *mask, int g, const void *X, const float *bias,
                      const void *R, int res_is_f16, int relu, int is_f16, int n, int cin, int cout,
                      int h, int wd, int stride, double *Y, double *A)
{
    if (!W || !mask || !X || g < 1 || n < 0 || cin < 0 || cout < 0 || h < 0 || wd < 0 || stride < 1) return -1;
    const int oh = (h + stride - 1) / stride, ow = (wd + stride - 1) / stride;
    const size_t ohw = (size_t)oh * ow, hw = (size_t)h * wd;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int in = 0; in < n; ++in) {
        for (int co = 0; co < cout; ++co) {
            for (int y = 0; y < oh; ++y) {
                for (int x = 0; x < ow; ++x) {
                    double acc = 0.0, mag = 0.0;
#if ORACLE_MUTANT == 11           /* sampling grid shifted by one pixel */
                    const size_t pin = (size_t)(y * stride + (stride > 1 && y * stride + 1 < h ? 1 : 0)) * wd + (size_t)x * stride;
#else
                    const size_t pin = (size_t)(y * stride) * wd + (size_t)x * stride;
#endif
                    for (int ci = 0; ci < cin; ++ci) {
                        const double wm = masked_weight(W, is_f16, mask, g, cin, cout, co, ci);
                        const size_t xi = ((size_t)in * cin + ci) * hw + pin;
                        const double xv = is_f16 ? ld_f16(X, xi) : ld_f32(X, xi);
                        acc += wm * xv;
                        mag += fabs(wm) * fabs(xv);
                    }
                    const double b = bias ? (double)bias[co] : 0.0;
                    const size_t yo = ((size_t)in * cout + co) * ohw + (size_t)y * ow + x;
                    const double r = R ? (res_is_f16 ? ld_f16(R, yo) : ld_f32(R, yo)) : 0.0;
#if ORACLE_MUTANT == 10           /* residual added after the activation */
                    double s = acc + b;
                    if (relu && s < 0.0) s = 0.0;
                    s += r;
#else
                    double s = acc + b + r;
                    if (relu && s < 0.0) s = 0.0;
#endif
                    if (Y) Y[yo] = s;
                    if (A) A[yo] = mag + fabs(b) + fabs(r);
                }
            }
        }
    }
    return 0;
}

/*
 * Selected outputs only: idx[k] is a flat index into Y[n][cout][hw]; out[k] (and mag[k] if
 * mag != NULL) receive the same quantities as oracle_conv1x1.  For full-size workloads where
 * the whole output would take too long.
 */
int oracle_conv1x1_points(const void *W, const uint8_t *mask, int g, const void *X,
                          const float *bias, int relu, int is_f16, int n, int cin, int cout,
                          long hw, const int64_t *idx, long n_idx, double *out, double *mag)
{
    if (!W || !mask || !X || !idx || !out || g < 1) return -1;
    int bad = 0;
#pragma omp parallel for schedule(static)
    for (long k = 0; k < n_idx; ++k) {
        const int64_t f = idx[k];
        if (f < 0 || f >= (int64_t)n * cout * hw) { bad = 1; continue; }
        const long p = (long)(f % hw);
        const int co = (int)((f / hw) % cout);
        const int in = (int)(f / hw / cout);
        double s = 0.0, m = 0.0;
        for (int ci = 0; ci < cin; ++ci) {
            const double wm = masked_weight(W, is_f16, mask, g, cin, cout, co, ci);
            const size_t xi = ((size_t)in * cin + ci) * (size_t)hw + (size_t)p;
            const double x = is_f16 ? ld_f16(X, xi) : ld_f32(X, xi);
            s += wm * x;
            m += fabs(wm) * fabs(x);
        }
        const double b = bias ? (double)bias[co] : 0.0;
        s += b;
        if (relu && s < 0.0) s = 0.0;
        out[k] = s;
        if (mag) mag[k] = m + fabs(b);
    }
    return bad ? -1 : 0;
}

/* ------------------------------------------------------------------------------------------
 * General k_h x k_w convolution: the same Section 3.2.2 formula with all three sums,
 *
 *     O(co, oh, ow) = sum_c sum_r sum_s Wm(co, c, r, s) * I(c, oh*stride - pad + r, ow*stride - pad + s),
 *
 * where I is read as zero outside the image.  The paper writes the stride-1, unpadded case
 * (I(c, h+r, w+s)); stride and zero padding are what the ResNet / MobileNet layers add and
 * reduce to the paper's formula at stride = 1, pad = 0.  The pruning pattern is the one of
 * Section 3.2.1 for a general kernel: the parameters at the same location (c, r, s) of g
 * adjacent filters form one group, so the block mask is [ceil(cout/g)][cin*kh*kw] over the
 * columns of the flattened-filter matrix W*, column = (c*kh + r)*kw + s.
 *
 * As above: dense loops over the mask-applied weights, no zero skipping, double accumulation
 * in ascending (c, r, s) order, then bias and ReLU.  W is [cout][cin][kh][kw], X is
 * [n][cin][h][wd], Y and A are [n][cout][oh][ow] with oh = (h + 2*pad - kh)/stride + 1.
 */
static inline double conv2d_point(const void *W, const uint8_t *mask, int g, const void *X,
                                  int is_f16, int cin, int cout, int h, int wd, int kh, int kw,
                                  int stride, int pad, int in, int co, int oh, int ow, double *mag)
{
    const int K = cin * kh * kw;
    double s = 0.0, m = 0.0;
    for (int c = 0; c < cin; ++c)
        for (int r = 0; r < kh; ++r)
            for (int q = 0; q < kw; ++q) {
#if ORACLE_MUTANT == 6            /* flipped kernel: true convolution instead of the paper's h+r, w+s */
                const int ih = oh * stride - pad + (kh - 1 - r), iw = ow * stride - pad + (kw - 1 - q);
#elif ORACLE_MUTANT == 7          /* taps transposed: r walks the width, s the height */
                const int ih = oh * stride - pad + q, iw = ow * stride - pad + r;
#elif ORACLE_MUTANT == 8          /* stride applied to the taps as well */
                const int ih = (oh + r) * stride - pad, iw = (ow + q) * stride - pad;
#elif ORACLE_MUTANT == 9          /* padding added instead of subtracted */
                const int ih = oh * stride + pad + r, iw = ow * stride + pad + q;
#else
                const int ih = oh * stride - pad + r, iw = ow * stride - pad + q;
#endif
                if (ih < 0 || ih >= h || iw < 0 || iw >= wd) continue;   /* zero padding */
                const int col = (c * kh + r) * kw + q;
                const double wm = masked_weight(W, is_f16, mask, g, K, cout, co, col);
                const size_t xi = (((size_t)in * cin + c) * (size_t)h + (size_t)ih) * (size_t)wd + (size_t)iw;
                const double x = is_f16 ? ld_f16(X, xi) : ld_f32(X, xi);
                s += wm * x;
                m += fabs(wm) * fabs(x);
            }
    *mag = m;
    return s;
}

int oracle_conv2d_out_size(int in, int k, int stride, int pad)
{
    if (stride < 1 || k < 1 || pad < 0 || in + 2 * pad < k) return -1;
    return (in + 2 * pad - k) / stride + 1;
}

int oracle_conv2d(const void *W, const uint8_t *mask, int g, const void *X, const float *bias,
                  int relu, int is_f16, int n, int cin, int cout, int h, int wd, int kh, int kw,
                  int stride, int pad, double *Y, double *A)
{
    if (!W || !mask || !X || g < 1 || n < 0 || cin < 0 || cout < 0) return -1;
    const int oh = oracle_conv2d_out_size(h, kh, stride, pad);
    const int ow = oracle_conv2d_out_size(wd, kw, stride, pad);
    if (oh < 0 || ow < 0) return -1;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int in = 0; in < n; ++in)
        for (int co = 0; co < cout; ++co) {
            const double b = bias ? (double)bias[co] : 0.0;
            for (int y = 0; y < oh; ++y)
                for (int x = 0; x < ow; ++x) {
                    double m;
                    double s = conv2d_point(W, mask, g, X, is_f16, cin, cout, h, wd, kh, kw, stride,
                                            pad, in, co, y, x, &m) + b;
                    if (relu && s < 0.0) s = 0.0;
                    const size_t yi = (((size_t)in * cout + co) * (size_t)oh + (size_t)y) * (size_t)ow + (size_t)x;
                    if (Y) Y[yi] = s;
                    if (A) A[yi] = m + fabs(b);
                }
        }
    return 0;
}

/* Selected outputs of the general convolution: idx[k] is a flat index into Y[n][cout][oh][ow]. */
int oracle_conv2d_points(const void *W, const uint8_t *mask, int g, const void *X, const float *bias,
                         int relu, int is_f16, int n, int cin, int cout, int h, int wd, int kh,
                         int kw, int stride, int pad, const int64_t *idx, long n_idx, double *out,
                         double *mag)
{
    if (!W || !mask || !X || !idx || !out || g < 1) return -1;
    const int oh = oracle_conv2d_out_size(h, kh, stride, pad);
    const int ow = oracle_conv2d_out_size(wd, kw, stride, pad);
    if (oh < 0 || ow < 0) return -1;
    int bad = 0;
#pragma omp parallel for schedule(static)
    for (long k = 0; k < n_idx; ++k) {
        const int64_t f = idx[k];
        if (f < 0 || f >= (int64_t)n * cout * oh * ow) { bad = 1; continue; }
        const int x = (int)(f % ow);
        const int y = (int)((f / ow) % oh);
        const int co = (int)((f / ow / oh) % cout);
        const int in = (int)(f / ow / oh / cout);
        double m;
        const double b = bias ? (double)bias[co] : 0.0;
        double s = conv2d_point(W, mask, g, X, is_f16, cin, cout, h, wd, kh, kw, stride, pad, in,
                                co, y, x, &m) + b;
        if (relu && s < 0.0) s = 0.0;
        out[k] = s;
        if (mag) mag[k] = m + fabs(b);
    }
    return bad ? -1 : 0;
}
