/*
 * CPU float64 oracle for the discrete Fourier transform. TEST INFRASTRUCTURE:
 * it exists so that the CUDA library can be checked against the plain
 * definition. It shares no code with the CUDA path and must never be called
 * from it.
 *
 * What it computes (paper, Section "The M6 Memory Hierarchy": a transform of N
 * complex points, 5 N log2 N nominal operations; sign and scaling as the
 * workload statement fixes them):
 *
 *   forward  X[k] =       sum_{n=0}^{N-1} x[n] exp(-2 pi i n k / N)
 *   inverse  x[n] = (1/N) sum_{k=0}^{N-1} X[k] exp(+2 pi i n k / N)
 *
 * N <= 1024: the sum above, term by term (O(N^2)).
 * N  > 1024: textbook recursive radix-2 decimation in time, down to length 1.
 * Both are exact methods, so the oracle is the definition written out.
 *
 * Complex numbers are interleaved (re, im) doubles. Element j of transform b
 * lives at complex index b*dist + j*stride, for input and output alike.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_DIRECT_MAX 1024

/* exp(sign * 2 pi i j / n) for 0 <= j < n, argument reduced to the first
 * octant on the integer index so that no large angle ever reaches sin/cos. */
static void unit_root(int64_t j, int64_t n, int sign, double *re, double *im)
{
    /* angle = 2 pi j / n ; work in eighths of a turn: j/n = (q + f)/8 */
    int64_t j8 = 8 * j;
    int64_t q = j8 / n;           /* octant 0..7 */
    int64_t r = j8 - q * n;       /* remainder, 0 <= r < n */
    double c, s;
    if (q & 1) {                  /* odd octant: measure back from its far edge */
        double a = (M_PI / 4.0) * ((double)(n - r) / (double)n);
        c = sin(a);
        s = cos(a);
    } else {
        double a = (M_PI / 4.0) * ((double)r / (double)n);
        c = cos(a);
        s = sin(a);
    }
    /* (c, s) is the point at angle within [0, pi/4] (even octant) or the
     * mirrored one (odd octant, already swapped); rotate by (q/2) quarter turns */
    double x, y;
    switch ((q >> 1) & 3) {
    case 0:  x = c;  y = s;  break;
    case 1:  x = -s; y = c;  break;
    case 2:  x = -c; y = -s; break;
    default: x = s;  y = -c; break;
    }
    /* odd octant q = 2h+1: the angle is (h+1) quarter turns minus a, i.e. h
     * quarter turns plus (pi/2 - a), whose point (sin a, cos a) is the swapped
     * pair taken above; so the same rotation by h serves both cases. */
    *re = x;
    *im = (sign < 0) ? -y : y;
}

int oracle_unit_root(int64_t j, int64_t n, int sign, double *out2)
{
    if (n <= 0 || j < 0 || j >= n) return 1;
    unit_root(j, n, sign, &out2[0], &out2[1]);
    return 0;
}

/* The definition, term by term. sign = -1 forward, +1 inverse (no scaling here). */
void oracle_dft_direct(int64_t n, int sign, const double *in, int64_t istride,
                       double *out, int64_t ostride)
{
    double *w = (double *)malloc(sizeof(double) * 2 * (size_t)n);
    for (int64_t j = 0; j < n; ++j) unit_root(j, n, sign, &w[2 * j], &w[2 * j + 1]);
    for (int64_t k = 0; k < n; ++k) {
        double sr = 0.0, si = 0.0;
        for (int64_t m = 0; m < n; ++m) {
            int64_t idx = (m * k) % n;
            double xr = in[2 * m * istride], xi = in[2 * m * istride + 1];
            double wr = w[2 * idx], wi = w[2 * idx + 1];
            sr += xr * wr - xi * wi;
            si += xr * wi + xi * wr;
        }
        out[2 * k * ostride] = sr;
        out[2 * k * ostride + 1] = si;
    }
    free(w);
}

/* Recursive radix-2 decimation in time on a contiguous work array:
 * X[k] = E[k] + w^k O[k],  X[k + n/2] = E[k] - w^k O[k],
 * E, O the transforms of the even- and odd-indexed halves. */
static void fft_rec(int64_t n, int sign, const double *in, int64_t istride,
                    double *out, double *scratch)
{
    if (n == 1) {
        out[0] = in[0];
        out[1] = in[1];
        return;
    }
    int64_t h = n / 2;
    double *even = scratch, *odd = scratch + 2 * h;
    fft_rec(h, sign, in, 2 * istride, even, scratch + 2 * n);
    fft_rec(h, sign, in + 2 * istride, 2 * istride, odd, scratch + 2 * n);
    for (int64_t k = 0; k < h; ++k) {
        double wr, wi;
        unit_root(k, n, sign, &wr, &wi);
        double orr = odd[2 * k] * wr - odd[2 * k + 1] * wi;
        double oi = odd[2 * k] * wi + odd[2 * k + 1] * wr;
        out[2 * k] = even[2 * k] + orr;
        out[2 * k + 1] = even[2 * k + 1] + oi;
        out[2 * (k + h)] = even[2 * k] - orr;
        out[2 * (k + h) + 1] = even[2 * k + 1] - oi;
    }
}

int oracle_fft_radix2(int64_t n, int sign, const double *in, int64_t istride,
                      double *out, int64_t ostride)
{
    if (n <= 0 || (n & (n - 1))) return 1;
    /* scratch: n + n/2 + ... < 2n complex per level chain; 2n complex is enough */
    double *scratch = (double *)malloc(sizeof(double) * 2 * (size_t)(2 * n + 2));
    double *tmp = (double *)malloc(sizeof(double) * 2 * (size_t)n);
    if (!scratch || !tmp) { free(scratch); free(tmp); return 2; }
    fft_rec(n, sign, in, istride, tmp, scratch);
    for (int64_t k = 0; k < n; ++k) {
        out[2 * k * ostride] = tmp[2 * k];
        out[2 * k * ostride + 1] = tmp[2 * k + 1];
    }
    free(scratch);
    free(tmp);
    return 0;
}

/* One transform with the size rule stated at the top. method: 0 = by size,
 * 1 = force the direct sum, 2 = force the recursion. direction: -1 / +1. */
static int one_transform(int64_t n, int direction, int method,
                         const double *in, int64_t istride, double *out, int64_t ostride)
{
    int use_direct = (method == 1) || (method == 0 && n <= ORACLE_DIRECT_MAX);
    if (use_direct) {
        oracle_dft_direct(n, direction, in, istride, out, ostride);
    } else {
        int rc = oracle_fft_radix2(n, direction, in, istride, out, ostride);
        if (rc) return rc;
    }
    if (direction > 0) {
        double s = 1.0 / (double)n;
        for (int64_t k = 0; k < n; ++k) {
            out[2 * k * ostride] *= s;
            out[2 * k * ostride + 1] *= s;
        }
    }
    return 0;
}

/* Batched, strided transform. in and out must not overlap. */
int oracle_fft_c2c(int64_t n, int64_t batch, int64_t stride, int64_t dist,
                   int direction, int method, const double *in, double *out)
{
    if (n <= 0 || batch <= 0 || stride <= 0 || dist <= 0) return 1;
    if (direction != -1 && direction != 1) return 1;
    if (method != 1 && n > ORACLE_DIRECT_MAX && (n & (n - 1))) return 1;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t b = 0; b < batch; ++b) {
        int rc = one_transform(n, direction, method, in + 2 * b * dist, stride,
                               out + 2 * b * dist, stride);
        if (rc) {
#pragma omp atomic write
            fail = rc;
        }
    }
    return fail;
}

/* 2-D transform of a rows x cols row-major matrix: every row, then every column. */
int oracle_fft2d(int64_t rows, int64_t cols, int direction, const double *in, double *out)
{
    double *tmp = (double *)malloc(sizeof(double) * 2 * (size_t)rows * (size_t)cols);
    if (!tmp) return 2;
    int rc = oracle_fft_c2c(cols, rows, 1, cols, direction, 0, in, tmp);
    if (!rc) rc = oracle_fft_c2c(rows, cols, cols, 1, direction, 0, tmp, out);
    free(tmp);
    return rc;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
