/*
 * TEST INFRASTRUCTURE -- not part of the product.
 *
 * Plain, slow, fp64 CPU definitions of the four steps of the augmentation and
 * feature path, written out from their definitions so that they can be checked
 * against the paper by eye.  Nothing here is blocked, fused or reordered beyond
 * an OpenMP loop over independent outputs, and nothing is shared with the CUDA
 * library: no headers, no tables, no helpers.
 *
 * Only the tests, the smoke check and the CPU-baseline timing may call this.
 *
 * The paper (Sections 1 and 2.3) names the blocks -- an acoustic simulator that
 * builds room impulse responses on the fly, reverberates speech and adds noise
 * at a random SNR, then mel filterbank features -- and leaves their formulas to
 * the cited simulator papers.  The conventions used here (image-source method,
 * windowed-sinc fractional delay, causal "same" convolution, periodic Hann
 * window, unscaled power spectrum) are this library's stated readings.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifndef M_PI
#define M_PI 3.14159265358979323846
#endif

/* sinc(x) = sin(pi x)/(pi x), sinc(0) = 1 */
static double sinc_pi(double x) {
    if (x == 0.0) return 1.0;
    double a = M_PI * x;
    return sin(a) / a;
}

/*
 * Image-source room impulse response of a shoebox room (simulator block of
 * Sections 1 and 2.3; method: image sources with fractional delays).
 *
 *   room[3]  side lengths in metres
 *   beta[6]  pressure reflection coefficients of the walls x=0, x=Lx, y=0, y=Ly, z=0, z=Lz
 *   order    largest total number of reflections |kx|+|ky|+|kz| kept (cube == 0), or
 *            largest per-axis index max(|kx|,|ky|,|kz|) (cube != 0)
 *   half_w   half width W_h (samples) of the Hann-windowed sinc that places a
 *            delay tau between sample points
 *   h[L]     output, overwritten
 *
 * Along one axis the images are indexed by an integer k = 2m - p, p in {0,1}:
 * position (1-2p)*src + 2m*L, reflected |m-p| times by the wall at 0 and |m|
 * times by the wall at L.  Each image adds  A * sinc(n-tau) * hann(n-tau)
 * with A = prod(beta^hits)/d and tau = d*fs/c.
 * Returns the number of images summed.
 */
int64_t orc_rir_image_method(const double *room, const double *beta, const double *mic,
                             const double *src, int order, int cube, double fs, double c,
                             int half_w, int L, double *h) {
    int64_t n_img = 0;
    memset(h, 0, sizeof(double) * (size_t)L);
    for (int kx = -order; kx <= order; ++kx)
        for (int ky = -order; ky <= order; ++ky)
            for (int kz = -order; kz <= order; ++kz) {
                if (!cube && abs(kx) + abs(ky) + abs(kz) > order) continue;
                int k[3] = {kx, ky, kz};
                double d2 = 0.0, gain = 1.0;
                for (int a = 0; a < 3; ++a) {
                    int p = ((k[a] % 2) + 2) % 2;       /* k = 2m - p */
                    int m = (k[a] + p) / 2;
                    double img = (1 - 2 * p) * src[a] + 2.0 * m * room[a];
                    double diff = img - mic[a];
                    d2 += diff * diff;
                    gain *= pow(beta[2 * a], abs(m - p)) * pow(beta[2 * a + 1], abs(m));
                }
                double d = sqrt(d2);
                double A = gain / d;
                double tau = d * fs / c;
                ++n_img;
                int64_t n_lo = (int64_t)ceil(tau - half_w);
                int64_t n_hi = (int64_t)floor(tau + half_w);
                if (n_lo < 0) n_lo = 0;
                if (n_hi > L - 1) n_hi = L - 1;
                for (int64_t n = n_lo; n <= n_hi; ++n) {
                    double x = (double)n - tau;
                    h[n] += A * sinc_pi(x) * 0.5 * (1.0 + cos(M_PI * x / half_w));
                }
            }
    return n_img;
}

/*
 * Causal convolution cut to the input length:
 *   y[n] = sum_{j=0}^{min(n, L-1)} h[j] * x[n-j],   0 <= n < N.
 */
__attribute__((target_clones("default", "avx2", "avx512f")))
static double dot_reversed(const double *h, const double *xr, int64_t count) {
    double s = 0.0;
#pragma omp simd reduction(+ : s)
    for (int64_t j = 0; j < count; ++j) s += h[j] * xr[-j];
    return s;
}

void orc_convolve_causal(const double *x, int64_t N, const double *h, int64_t L, double *y) {
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t n = 0; n < N; ++n) {
        int64_t jmax = n < L - 1 ? n : L - 1;
        y[n] = dot_reversed(h, x + n, jmax + 1);
    }
}

/* T = 1 + floor((N - win)/hop) if N >= win, else 0: no padding, no centring. */
int orc_frame_count(int64_t N, int win, int hop) {
    if (N < win) return 0;
    return (int)(1 + (N - win) / hop);
}

/*
 * Power spectrum of Hann-windowed frames by the DFT definition:
 *   w[n] = 1/2 - 1/2 cos(2 pi n / win)            (periodic Hann)
 *   X[t][k] = sum_{n<win} w[n] x[t*hop+n] exp(-2 pi i k n / K),  k = 0..K/2
 *   P[t][k] = |X[t][k]|^2                          (no scaling)
 * power is [T][K/2+1], row-major.
 */
void orc_stft_power(const double *x, int64_t N, int win, int hop, int K, double *power) {
    int T = orc_frame_count(N, win, hop);
    int nb = K / 2 + 1;
    double *cs = (double *)malloc(sizeof(double) * 2 * (size_t)K);
    double *w = (double *)malloc(sizeof(double) * (size_t)win);
    for (int j = 0; j < K; ++j) {           /* the K-th roots of unity, each evaluated once */
        cs[2 * j] = cos(2.0 * M_PI * j / K);
        cs[2 * j + 1] = sin(2.0 * M_PI * j / K);
    }
    for (int n = 0; n < win; ++n) w[n] = 0.5 - 0.5 * cos(2.0 * M_PI * n / win);
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        const double *f = x + (int64_t)t * hop;
        for (int k = 0; k < nb; ++k) {
            double re = 0.0, im = 0.0;
            for (int n = 0; n < win; ++n) {
                int j = (int)(((int64_t)k * n) % K);
                double v = w[n] * f[n];
                re += v * cs[2 * j];
                im -= v * cs[2 * j + 1];
            }
            power[(int64_t)t * nb + k] = re * re + im * im;
        }
    }
    free(cs);
    free(w);
}
