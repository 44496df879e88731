/* Test and measurement infrastructure, not product code.
 *
 * The paper's CPU method for one signal (Section V-A, Algorithm 2, in the reading that resolves its
 * misprints): the input is cut into blocks of N elements; per block one packed word A (Eq. 5), ONE
 * multiplication with the packed kernel B, the product added to what the previous block left above
 * its N low segments (Theorem 2), N outputs split off (shift and mask; Eq. 29 for signed values),
 * and the rest carried to the next block.  A 32x32 -> 64-bit multiplier is assumed: the caller
 * passes N and S such that both operands fit 32 bits and S (N + K - 1) <= 64.
 *
 * It is written to be compared, in results and in run time, with the plain nested loops of
 * hikonv_oracle.c on the same int64 arrays: this is the experiment of the paper's CPU evaluation
 * (Section VI-A) restated on the host of the GPU machine.  It shares nothing with the CUDA code.
 */
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline int64_t seg_unsigned(uint64_t c, int S, int m, uint64_t mask) { return (int64_t)((c >> (S * m)) & mask); }

/* Eq. 29: the S-bit field plus the bit just below it, read as an S-bit two's-complement number */
static inline int64_t seg_signed(uint64_t c, int S, int m, uint64_t mask) {
    uint64_t field = (c >> (S * m)) & mask;
    uint64_t below = m > 0 ? (c >> (S * m - 1)) & 1u : 0u;
    uint64_t v = (field + below) & mask;
    return (v >> (S - 1)) ? (int64_t)v - ((int64_t)1 << S) : (int64_t)v;
}

static inline uint64_t pack_block(const int64_t *f, int64_t len, int64_t e0, int N, int S) {
    uint64_t a = 0;
    for (int n = 0; n < N; ++n) {
        int64_t e = e0 + n;
        if (e >= 0 && e < len) a += (uint64_t)f[e] << (S * n);   /* Eq. 5; two's complement does Eq. 28 */
    }
    return a;
}

/* Blocks [x0, x1) of the running loop, starting from the carry that `warm` earlier blocks leave. */
static void run_blocks(const int64_t *f, int64_t len, uint64_t B, int K, int S, int N, int is_signed, int64_t x0, int64_t x1,
                       int warm, int64_t n_out, int64_t *y, int last) {
    const uint64_t mask = S >= 64 ? ~0ull : (((uint64_t)1 << S) - 1);
    uint64_t carry = 0;
    for (int64_t x = x0 - warm; x < x1; ++x) {
        if (x < 0) continue;
        uint64_t A = pack_block(f, len, x * N, N, S);
        uint64_t C;
        if (is_signed) C = (uint64_t)((int64_t)(int32_t)(uint32_t)A * (int64_t)(int32_t)(uint32_t)B) + carry;
        else C = (uint64_t)(uint32_t)A * (uint64_t)(uint32_t)B + carry;
        if (x >= x0) {
            for (int m = 0; m < N; ++m) {
                int64_t o = x * N + m;
                if (o < n_out) y[o] = is_signed ? seg_signed(C, S, m, mask) : seg_unsigned(C, S, m, mask);
            }
        }
        /* what lies above the N low outputs: for signed values the arithmetic shift plus the borrow bit */
        if (is_signed) carry = (uint64_t)(((int64_t)C >> (S * N)) + (int64_t)((C >> (S * N - 1)) & 1u));
        else carry = C >> (S * N);
    }
    if (last) {
        for (int m = 0; m < K - 1; ++m) {
            int64_t o = x1 * N + m;
            if (o < n_out) y[o] = is_signed ? seg_signed(carry, S, m, mask) : seg_unsigned(carry, S, m, mask);
        }
    }
}

/* y[0 .. len+K-2] = f * g.  Returns 0, or -1 when the layout does not fit a 32x32 -> 64 multiplier. */
int alg2_conv1d(const int64_t *f, int64_t len, const int64_t *g, int K, int S, int N, int is_signed, int threads, int64_t *y) {
    if (len < 0 || K < 1 || N < 1 || S < 1 || S * (N + K - 1) > 64 || S * (K - 1) >= 32 || S * (N - 1) >= 32) return -1;
    const int64_t n_out = len + K - 1;
    uint64_t B = 0;
    for (int k = 0; k < K; ++k) B += (uint64_t)g[k] << (S * k);
    const int64_t X = (len + N - 1) / N;
    const int warm = (K - 1 + N - 1) / N + 1;        /* blocks whose products still reach the first block of a chunk */
    int T = 1;
#ifdef _OPENMP
    T = threads > 0 ? threads : omp_get_max_threads();
#endif
    if (T > X) T = X > 0 ? (int)X : 1;
    if (X == 0) {
        for (int64_t o = 0; o < n_out; ++o) y[o] = 0;
        return 0;
    }
#pragma omp parallel for num_threads(T) schedule(static)
    for (int t = 0; t < T; ++t) {
        const int64_t x0 = X * t / T, x1 = X * (t + 1) / T;
        run_blocks(f, len, B, K, S, N, is_signed, x0, x1, warm, n_out, y, t == T - 1);
    }
    return 0;
}
