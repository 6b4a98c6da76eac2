/*
 * CPU float64 oracle for range-Doppler SAR image formation. TEST
 * INFRASTRUCTURE: a straight-line restatement of the processing chain the
 * paper lists (Section "End to End: Range-Doppler SAR", "Processing and
 * validation"): range compression (FFT, matched filter, inverse FFT along
 * each pulse); azimuth FFT along each range bin; range cell migration
 * correction with an 8-tap interpolator; the azimuth filter
 * exp(+j 4 pi R0 (D - 1) / lambda), D = sqrt(1 - (lambda f_a / 2 v)^2);
 * azimuth inverse FFT. It shares no code with the CUDA path and must never be
 * called from it. All transforms go through oracle_fft_c2c (oracle_fft.c).
 *
 * Readings where the paper prints no formula (each is the standard
 * range-Doppler expression consistent with the paper's D):
 *  - replica h[n] = exp(j pi K (n/fs)^2), n = -P/2 .. P/2-1 (P pulse samples),
 *    placed circularly; matched filter H = conj(FFT(h)); the inverse FFT
 *    carries its 1/N_range.
 *  - Doppler of azimuth bin k: f = k PRF/N_a for k < N_a/2, (k - N_a) PRF/N_a above.
 *  - migration in range bins: dn(k, n) = R0(n) (1/D(f_k) - 1) / dr,
 *    R0(n) = R_c + (n - N_r/2) dr, dr = c / (2 fs);
 *    i0 = floor(dn), mu = dn - i0 (the fraction comes from dn alone: the
 *    paper's fourth fix);
 *    S'[k, n] = sum_{j=-3}^{4} w_j(mu) S[k, n + i0 + j], zero outside the row,
 *    w_j(mu) = sinc(mu - j) / sum_j' sinc(mu - j'),  sinc(x) = sin(pi x)/(pi x).
 *  - D - 1 and 1/D - 1 are evaluated without cancellation from u = (lambda f/2v)^2.
 *
 * Images are row-major [azimuth][range], interleaved (re, im) doubles.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

int oracle_fft_c2c(int64_t n, int64_t batch, int64_t stride, int64_t dist,
                   int direction, int method, const double *in, double *out);

#define ORACLE_C_LIGHT 299792458.0

typedef struct {
    int64_t n_azimuth;
    int64_t n_range;
    int64_t pulse_samples;
    double wavelength_m;
    double chirp_rate;      /* K = bandwidth / pulse length, Hz/s */
    double fs_hz;
    double prf_hz;
    double velocity_mps;
    double r_center_m;      /* slant range of range bin n_range/2 */
    int32_t rcmc_enabled;   /* 0 switches migration correction off (ablation) */
    int32_t baseband_filter;/* 1: (D-1) as the paper prescribes; 0: textbook D (ablation) */
} oracle_sar_params;

static double sinc_pi(double x)
{
    if (x == 0.0) return 1.0;
    double a = M_PI * x;
    return sin(a) / a;
}

static double doppler_hz(const oracle_sar_params *p, int64_t k)
{
    int64_t kk = (k < p->n_azimuth / 2) ? k : k - p->n_azimuth;
    return (double)kk * p->prf_hz / (double)p->n_azimuth;
}

/* H[n] = conj(FFT(h))[n], n_range complex values. */
int oracle_sar_matched_filter(const oracle_sar_params *p, double *H)
{
    int64_t nr = p->n_range, P = p->pulse_samples;
    double *h = (double *)calloc((size_t)(2 * nr), sizeof(double));
    if (!h) return 2;
    for (int64_t i = -P / 2; i < P - P / 2; ++i) {
        double t = (double)i / p->fs_hz;
        double ph = M_PI * p->chirp_rate * t * t;
        int64_t pos = (i < 0) ? nr + i : i;
        h[2 * pos] = cos(ph);
        h[2 * pos + 1] = sin(ph);
    }
    int rc = oracle_fft_c2c(nr, 1, 1, nr, -1, 0, h, H);
    for (int64_t n = 0; n < nr; ++n) H[2 * n + 1] = -H[2 * n + 1];
    free(h);
    return rc;
}

/* y[m, :] = IFFT(FFT(raw[m, :]) * H) */
int oracle_sar_range_compress(const oracle_sar_params *p, const double *raw, double *y)
{
    int64_t na = p->n_azimuth, nr = p->n_range;
    double *H = (double *)malloc(sizeof(double) * 2 * (size_t)nr);
    double *F = (double *)malloc(sizeof(double) * 2 * (size_t)na * (size_t)nr);
    if (!H || !F) { free(H); free(F); return 2; }
    int rc = oracle_sar_matched_filter(p, H);
    if (!rc) rc = oracle_fft_c2c(nr, na, 1, nr, -1, 0, raw, F);
    if (!rc) {
        for (int64_t m = 0; m < na; ++m)
            for (int64_t n = 0; n < nr; ++n) {
                double *f = F + 2 * (m * nr + n);
                double ar = f[0], ai = f[1];
                f[0] = ar * H[2 * n] - ai * H[2 * n + 1];
                f[1] = ar * H[2 * n + 1] + ai * H[2 * n];
            }
        rc = oracle_fft_c2c(nr, na, 1, nr, +1, 0, F, y);
    }
    free(H);
    free(F);
    return rc;
}

/* S[:, n] = FFT over azimuth of y[:, n] */
int oracle_sar_azimuth_fft(const oracle_sar_params *p, const double *y, double *S)
{
    return oracle_fft_c2c(p->n_azimuth, p->n_range, p->n_range, 1, -1, 0, y, S);
}

/* Migration in range bins for azimuth bin k, range bin n. */
double oracle_sar_migration_bins(const oracle_sar_params *p, int64_t k, int64_t n)
{
    double dr = ORACLE_C_LIGHT / (2.0 * p->fs_hz);
    double f = doppler_hz(p, k);
    double a = p->wavelength_m * f / (2.0 * p->velocity_mps);
    double u = a * a;
    double sq = sqrt(1.0 - u);
    double inv_d_minus_1 = u / ((1.0 + sq) * sq);
    double r0 = p->r_center_m + (double)(n - p->n_range / 2) * dr;
    return r0 * inv_d_minus_1 / dr;
}

/* The eight interpolator weights for fraction mu, taps j = -3..4 in w[0..7]. */
void oracle_sar_interp_weights(double mu, double *w)
{
    double s = 0.0;
    for (int j = -3; j <= 4; ++j) {
        w[j + 3] = sinc_pi(mu - (double)j);
        s += w[j + 3];
    }
    for (int j = 0; j < 8; ++j) w[j] /= s;
}

/* S1[k, n] = sum_j w_j(mu) S[k, n + i0 + j] */
int oracle_sar_rcmc(const oracle_sar_params *p, const double *S, double *S1)
{
    int64_t na = p->n_azimuth, nr = p->n_range;
    if (!p->rcmc_enabled) {
        memcpy(S1, S, sizeof(double) * 2 * (size_t)na * (size_t)nr);
        return 0;
    }
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < na; ++k) {
        for (int64_t n = 0; n < nr; ++n) {
            double dn = oracle_sar_migration_bins(p, k, n);
            double fl = floor(dn);
            int64_t i0 = (int64_t)fl;
            double mu = dn - fl;
            double w[8];
            oracle_sar_interp_weights(mu, w);
            double sr = 0.0, si = 0.0;
            for (int j = -3; j <= 4; ++j) {
                int64_t src = n + i0 + j;
                if (src < 0 || src >= nr) continue;
                sr += w[j + 3] * S[2 * (k * nr + src)];
                si += w[j + 3] * S[2 * (k * nr + src) + 1];
            }
            S1[2 * (k * nr + n)] = sr;
            S1[2 * (k * nr + n) + 1] = si;
        }
    }
    return 0;
}

/* Azimuth filter phase in radians for azimuth bin k, range bin n. */
double oracle_sar_filter_phase(const oracle_sar_params *p, int64_t k, int64_t n)
{
    double dr = ORACLE_C_LIGHT / (2.0 * p->fs_hz);
    double f = doppler_hz(p, k);
    double a = p->wavelength_m * f / (2.0 * p->velocity_mps);
    double u = a * a;
    double sq = sqrt(1.0 - u);
    double r0 = p->r_center_m + (double)(n - p->n_range / 2) * dr;
    double d_term = p->baseband_filter ? (-u / (1.0 + sq)) : sq;
    return 4.0 * M_PI * r0 * d_term / p->wavelength_m;
}

/* S2 = S1 * exp(+j phase); may run in place. */
int oracle_sar_azimuth_filter(const oracle_sar_params *p, const double *S1, double *S2)
{
    int64_t na = p->n_azimuth, nr = p->n_range;
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < na; ++k)
        for (int64_t n = 0; n < nr; ++n) {
            double ph = oracle_sar_filter_phase(p, k, n);
            double c = cos(ph), s = sin(ph);
            double ar = S1[2 * (k * nr + n)], ai = S1[2 * (k * nr + n) + 1];
            S2[2 * (k * nr + n)] = ar * c - ai * s;
            S2[2 * (k * nr + n) + 1] = ar * s + ai * c;
        }
    return 0;
}

/* image[:, n] = IFFT over azimuth of S2[:, n] (with 1/N_a) */
int oracle_sar_azimuth_ifft(const oracle_sar_params *p, const double *S2, double *image)
{
    return oracle_fft_c2c(p->n_azimuth, p->n_range, p->n_range, 1, +1, 0, S2, image);
}

/* The whole chain. stage_out, if not NULL, receives the range-compressed image
 * (same shape), for tests that pin the first step on its own. */
int oracle_sar_rda(const oracle_sar_params *p, const double *raw, double *image,
                   double *stage_out)
{
    size_t bytes = sizeof(double) * 2 * (size_t)p->n_azimuth * (size_t)p->n_range;
    double *a = (double *)malloc(bytes), *b = (double *)malloc(bytes);
    if (!a || !b) { free(a); free(b); return 2; }
    int rc = oracle_sar_range_compress(p, raw, a);
    if (!rc && stage_out) memcpy(stage_out, a, bytes);
    if (!rc) rc = oracle_sar_azimuth_fft(p, a, b);
    if (!rc) rc = oracle_sar_rcmc(p, b, a);
    if (!rc) rc = oracle_sar_azimuth_filter(p, a, a);
    if (!rc) rc = oracle_sar_azimuth_ifft(p, a, image);
    free(a);
    free(b);
    return rc;
}
