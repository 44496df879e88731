/*
 * Test-infrastructure oracle for low-bit convolution (plain C, int64, CPU only).
 *
 * This file is NOT part of the product library.  It is the slow, obviously
 * correct statement of what the packed GPU path must reproduce bit for bit.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may
 * call it.  It shares no code with the CUDA sources and includes none of
 * their headers.
 *
 * The packed method is an exact re-arrangement of plain convolution
 * (Theorems 1-3 are identities), so the oracle is the plain definition:
 *
 *   1-D (Eq. 2-4):  h = f extended with zeros,
 *                   y[m] = sum_{k=0}^{K-1} h[m-k] * g[k],  m = 0 .. len+K-2.
 *   2-D (Eq. 16, with zero padding as in the "0 otherwise" branch of Eq. 19):
 *                   O[b][co][h][w] = sum_{ci,kh,kw}
 *                       Ipad[b][ci][h+kh][w+kw] * W[co][ci][kh][kw]
 *                   stride 1, no kernel flip, H_o = H + 2*pad - K + 1.
 *   requantize:     clamp(acc >> shift, lo, hi), ">>" rounding toward -inf.
 *   max-pool:       2x2 window, stride 2, floor output size.
 *
 * All values are int64; there is no blocking, fusion or reordering.
 * The only concession to run time is an OpenMP "parallel for" over
 * independent outputs (one output element never depends on another).
 */
#include <stddef.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Eq. 2-4: full linear convolution, len+K-1 outputs. */
void oracle_conv1d_full(const int64_t *f, int64_t len, const int64_t *g, int64_t K, int64_t *y)
{
    const int64_t n_out = len + K - 1;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < n_out; ++m) {
        int64_t s = 0;
        for (int64_t k = 0; k < K; ++k) {
            const int64_t n = m - k;               /* index into h */
            const int64_t h = (n >= 0 && n < len) ? f[n] : 0;   /* Eq. 2 */
            s += h * g[k];                          /* Eq. 3 */
        }
        y[m] = s;
    }
}

/* Eq. 16 with zero padding; x is [B][Ci][H][W], w is [Co][Ci][K][K], out is [B][Co][Ho][Wo]. */
void oracle_conv2d_nchw(const int64_t *x, int64_t B, int64_t Ci, int64_t H, int64_t W,
                        const int64_t *w, int64_t Co, int64_t K, int64_t pad, int64_t *out)
{
    const int64_t Ho = H + 2 * pad - K + 1;
    const int64_t Wo = W + 2 * pad - K + 1;
    if (Ho <= 0 || Wo <= 0) return;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < B; ++b) {
        for (int64_t co = 0; co < Co; ++co) {
            for (int64_t h = 0; h < Ho; ++h) {
                for (int64_t ww = 0; ww < Wo; ++ww) {
                    int64_t s = 0;
                    for (int64_t ci = 0; ci < Ci; ++ci) {
                        for (int64_t kh = 0; kh < K; ++kh) {
                            for (int64_t kw = 0; kw < K; ++kw) {
                                const int64_t r = h + kh - pad;     /* row in the unpadded input */
                                const int64_t c = ww + kw - pad;    /* column in the unpadded input */
                                int64_t v = 0;
                                if (r >= 0 && r < H && c >= 0 && c < W)
                                    v = x[((b * Ci + ci) * H + r) * W + c];
                                s += v * w[((co * Ci + ci) * K + kh) * K + kw];
                            }
                        }
                    }
                    out[((b * Co + co) * Ho + h) * Wo + ww] = s;
                }
            }
        }
    }
}

/* floor(a / 2^shift) without relying on the implementation-defined ">>" of negative values. */
static int64_t floor_shift(int64_t a, int64_t shift)
{
    const int64_t d = (int64_t)1 << shift;
    int64_t qv = a / d;                 /* truncates toward zero */
    if ((a % d) != 0 && a < 0) qv -= 1; /* move to floor */
    return qv;
}

void oracle_requant(const int64_t *acc, int64_t n, int64_t shift, int64_t lo, int64_t hi, int64_t *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int64_t v = floor_shift(acc[i], shift);
        if (v < lo) v = lo;
        if (v > hi) v = hi;
        out[i] = v;
    }
}

/* 2x2 max-pool, stride 2, on [B*C][H][W] -> [B*C][H/2][W/2] (floor). */
void oracle_maxpool2x2(const int64_t *x, int64_t BC, int64_t H, int64_t W, int64_t *out)
{
    const int64_t Ho = H / 2, Wo = W / 2;
#pragma omp parallel for schedule(static)
    for (int64_t c = 0; c < BC; ++c) {
        for (int64_t h = 0; h < Ho; ++h) {
            for (int64_t ww = 0; ww < Wo; ++ww) {
                const int64_t *p = x + (c * H + 2 * h) * W + 2 * ww;
                int64_t m = p[0];
                if (p[1] > m) m = p[1];
                if (p[W] > m) m = p[W];
                if (p[W + 1] > m) m = p[W + 1];
                out[(c * Ho + h) * Wo + ww] = m;
            }
        }
    }
}
