// Fast 1-D kernels: each lane owns a contiguous run of outputs.
//
// A lane computes R consecutive blocks of N outputs (L = R N outputs, a multiple of 4) entirely in
// registers: it loads the L codes of its run plus the J N codes in front of it as aligned 32-bit words,
// extracts codes with one byte-permute each, packs the R + J words A_x (Eq. 5, by multiply-add),
// forms Q_x = bias + sum_j A_{x-j} B_j for x = -1 .. R-1 (Eq. 9; the extra product in front replaces the
// "prologue multiplication" of Algorithm 2), adds the part of Q_{x-1} above its N low slots to Q_x
// (Theorem 2: the previous product shifted right, the running loop of Algorithm 2 unrolled in
// registers), splits N outputs per block and writes its L outputs with 16-byte stores.  Tiles that
// touch the ends of the signal, and unaligned buffers, take a guarded byte-wise path in the same kernel.
// The comparator uses the same loads and stores with one 32-bit multiply-add per product.
#include <type_traits>

#include "hikonv_conv1d_run.cuh"

namespace hikonv {

__host__ __device__ constexpr int gcd_c(int a, int b) { return b == 0 ? a : gcd_c(b, a % b); }
// blocks per lane: L = R N is a multiple of 4 and at least kMinRun
constexpr int kMinRun = 24;
__host__ __device__ constexpr int blocks_per_lane(int N) {
    // N = 5 and 10 would get runs of 40 outputs, whose registers cost a resident CTA per SM: 20 instead
    if (N == 5 || N == 10) return 20 / N;
    const int step = 4 / gcd_c(N, 4);
    int r = step;
    while (r * N < kMinRun) r += step;
    return r;
}

// Dense input: P bits per code (1, 2 or 4), code e at bit (e P) % 8 of byte (e P) / 8.  Field `k` (a
// compile-time index) of a word array that starts at the lane's first code: one bit-field extract.
template <bool SIGNED, int P>
__device__ __forceinline__ uint32_t extract_dense(const uint32_t *v, int k) {
    constexpr int EPW = 32 / P;
    uint32_t r;
    if (SIGNED) asm("bfe.s32 %0, %1, %2, %3;" : "=r"(r) : "r"(v[k / EPW]), "r"((k % EPW) * P), "r"(P));
    else asm("bfe.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(v[k / EPW]), "r"((k % EPW) * P), "r"(P));
    return r;
}

// Loads the NE codes that start at code e_first into v[0 .. NV), code k at bit (k % EPW) P of v[k / EPW].
// Fast path: NV + 1 aligned words and a funnel shift each (the run of a lane starts at any bit of a word);
// guarded path: one byte load per code, zero outside [0, len) (Eq. 2).
template <int NV, int NE, int P>
__device__ __forceinline__ void load_dense(const int8_t *f, long long len, long long e_first, bool fast, uint32_t (&v)[NV]) {
    constexpr int EPW = 32 / P;
    if (fast) {
        const long long w0 = e_first / EPW;
        const int boff = (int)(e_first - w0 * EPW) * P;
        const uint32_t *src = reinterpret_cast<const uint32_t *>(f) + w0;
        uint32_t w[NV + 1];
#pragma unroll
        for (int i = 0; i < NV + 1; ++i) w[i] = __ldg(src + i);
#pragma unroll
        for (int i = 0; i < NV; ++i) v[i] = __funnelshift_r(w[i], w[i + 1], boff);
    } else {
#pragma unroll
        for (int i = 0; i < NV; ++i) v[i] = 0;
#pragma unroll
        for (int k = 0; k < NE; ++k) {
            const long long e = e_first + k;
            if (e >= 0 && e < len) {
                const uint32_t byte = (uint8_t)__ldg(f + (e * P) / 8);
                v[k / EPW] |= ((byte >> (int)((e * P) % 8)) & ((1u << P) - 1u)) << ((k % EPW) * P);
            }
        }
    }
}

// SC > 0 fixes the slot width at compile time (shifts and masks become immediates); SC == 0 reads it
// from the parameters.
// P == 0: one code per byte; P = 1, 2, 4: dense input with P bits per code.
template <int N, int J, int SC, bool SP, bool FS, int P = 0>
__global__ void __launch_bounds__(kThreadsTc, ((N >= 9 && P == 0) ? 3 : 4)) conv1d_packed_tc_kernel(const Conv1dTcParams p) {
    constexpr int R = blocks_per_lane(N);
    constexpr int L = R * N;
    constexpr int HW = (J * N + 3) / 4;          // words in front of the run (one code per byte)
    constexpr int NE = L + J * N;                // codes a lane needs
    constexpr int NWORDS = P == 0 ? HW + L / 4 : (NE * (P == 0 ? 8 : P) + 31) / 32;
    constexpr int FRONT = P == 0 ? 4 * HW : J * N;   // codes held in front of the run
    __shared__ __align__(16) int32_t s_stage[kWarpsTc][32 * stage_pitch(L)];

    const int S = SC > 0 ? SC : p.S;
    const uint32_t mask = SC > 0 ? ((1u << (SC > 0 ? SC : 1)) - 1u) : p.mask;
    const int hi_shift = SC > 0 ? SC * N : p.hi_shift;
    // the kernel chunks B_j (Eq. 5 on g); every lane builds them itself from warp-uniform loads
    uint32_t Bw[J];
#pragma unroll
    for (int j = 0; j < J; ++j) {
        uint32_t b = 0;
        for (int k = 0; k < p.Kc; ++k) {
            const int idx = j * p.Kc + k;
            if (idx < p.K) {
                const int8_t raw = __ldg(p.g + idx);
                const int32_t v = p.g_signed ? (int32_t)raw : (int32_t)(uint8_t)raw;
                b += (uint32_t)v << (S * k);
            }
        }
        Bw[j] = b;
    }
    uint32_t slot_pow[N];
#pragma unroll
    for (int n = 0; n < N; ++n) slot_pow[n] = 1u << (S * n);

    const int lane = threadIdx.x & 31;
    const long long stride = (long long)gridDim.x * kWarpsTc;
    long long t = (long long)blockIdx.x * kWarpsTc + (threadIdx.x >> 5);
    // a tile takes the fast path when all its loads and stores are aligned and inside the buffers
    auto tile_is_fast = [&](long long tile0) -> bool {
        if (!p.aligned || tile0 < FRONT || tile0 + 32 * L > p.len) return false;
        if (P == 0) return true;
        // dense: the last lane reads NWORDS + 1 words from the word that holds its first code
        const long long last_first = tile0 + 31 * L - J * N;
        return last_first / (32 / (P == 0 ? 8 : P)) + NWORDS + 1 <= p.dense_words;
    };
    auto load_tile = [&](long long tile0, bool fast, uint32_t (&dst)[NWORDS]) {
        if constexpr (P == 0) load_words<NWORDS, HW>(p.f, p.len, tile0 + lane * L, fast, dst);
        else load_dense<NWORDS, NE, (P == 0 ? 8 : P)>(p.f, p.len, tile0 + lane * L - J * N, fast, dst);
    };
    uint32_t wn[NWORDS];
    bool fast_n = false;
    if (t < p.n_tiles) {
        const long long tile0 = t * (32 * L);
        fast_n = tile_is_fast(tile0);
        load_tile(tile0, fast_n, wn);
    }
    while (t < p.n_tiles) {
        const long long tile0 = t * (32 * L);
        const bool fast = fast_n;
        uint32_t w[NWORDS];
#pragma unroll
        for (int i = 0; i < NWORDS; ++i) w[i] = wn[i];
        t += stride;
        if (t < p.n_tiles) {                       // next tile's codes are in flight while this one is computed
            const long long next0 = t * (32 * L);
            fast_n = tile_is_fast(next0);
            load_tile(next0, fast_n, wn);
        }

        // the arithmetic of one tile; `fast_c` is a compile-time copy of `fast`, so that on interior tiles the
        // staging stores can be issued while later blocks are still being computed (fewer live registers)
        auto tile_body = [&](auto fast_c) {
            // A_x for x = -J .. R-1 (index x + J); element n of block x is code FRONT + x N + n of w
            uint32_t A[R + J];
#pragma unroll
            for (int x = -J; x < R; ++x) {
                uint32_t a = 0;
#pragma unroll
                for (int n = 0; n < N; ++n) {
                    const int pos = FRONT + x * N + n;
                    uint32_t c;
                    if constexpr (P == 0) c = extract_code<FS>(w[pos / 4], pos % 4);
                    else c = extract_dense<FS, (P == 0 ? 8 : P)>(w, pos);
                    a = (n == 0) ? c : a + c * slot_pow[n];
                }
                A[x + J] = a;
            }
            // Q_x for x = -1 .. R-1, carry chain, split
            int32_t out[L];
            uint32_t carry = 0;
#pragma unroll
            for (int x = -1; x < R; ++x) {
                uint64_t Q = SP ? p.bias : 0;           // unsigned products are never negative: every slot bias is zero
#pragma unroll
                for (int j = 0; j < J; ++j) mad_wide<SP>(Q, A[x - j + J], Bw[j]);
                if (x >= 0) {
                    const uint64_t D = Q + (uint64_t)carry;
#pragma unroll
                    for (int m = 0; m < N; ++m) {
                        const int sh = SC > 0 ? SC * m : p.seg_shift[m];
                        const int32_t field = (int32_t)(shr64_lo(D, sh) & mask);
                        out[x * N + m] = SP ? field - p.carry_bias[m] : field;
                    }
                }
                carry = shr64_lo(Q, hi_shift);
            }
            store_run<L>(p.y, p.n_out, tile0, lane, decltype(fast_c)::value, s_stage[threadIdx.x >> 5], out);
        };
        if (fast) tile_body(std::true_type{});
        else tile_body(std::false_type{});
    }
}

// Comparator: runs of L outputs per lane, one product per 32-bit multiply-add.
template <int K, bool FS, int L, int MINB>
__global__ void __launch_bounds__(kThreadsTc, MINB) conv1d_unpacked_tc_kernel(const Conv1dTcParams p) {
    constexpr int HW = (K - 1 + 3) / 4;
    constexpr int NWORDS = HW + L / 4;
    __shared__ __align__(16) int32_t s_stage[kWarpsTc][32 * stage_pitch(L)];
    int32_t gk[K];
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const int8_t raw = __ldg(p.g + k);
        gk[k] = p.g_signed ? (int32_t)raw : (int32_t)(uint8_t)raw;
    }
    walk_tiles<L, HW>(p.f, p.y, p.len, p.n_out, (unsigned)p.n_tiles, p.fast_after_first, s_stage[threadIdx.x >> 5],
                      [&](const uint32_t (&w)[NWORDS], int32_t (&out)[L]) {
        int32_t e[L + K - 1];                       // e[i] = f[e0 - (K-1) + i]
#pragma unroll
        for (int i = 0; i < L + K - 1; ++i) {
            const int pos = 4 * HW - (K - 1) + i;
            e[i] = (int32_t)extract_code<FS>(w[pos / 4], pos % 4);
        }
#pragma unroll
        for (int o = 0; o < L; ++o) {
            int32_t s = 0;
#pragma unroll
            for (int k = 0; k < K; ++k) s += e[o + (K - 1) - k] * gk[k];      // y[m] = sum_k f[m-k] g[k]
            out[o] = s;
        }
    });
}

// Second comparator: the byte dot-product instruction (dp4a: four 8-bit products summed into 32 bits), the
// SIMD alternative to packing codes into a wide multiplier.  Output m needs the codes f[m-K+1 .. m]; tap word
// t holds the taps g[4t+3], g[4t+2], g[4t+1], g[4t] in its bytes 0..3 (zero past K-1), and the matching window
// f[m-4t-3 .. m-4t] is cut out of two neighbouring loaded words with one funnel shift.  32 outputs per lane.
template <bool FS, bool GS>
__device__ __forceinline__ int32_t dot4(uint32_t codes, uint32_t taps, int32_t acc) {
    int32_t d;
    if (FS && GS) asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(codes), "r"(taps), "r"(acc));
    else if (FS) asm("dp4a.s32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(codes), "r"(taps), "r"(acc));
    else if (GS) asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(codes), "r"(taps), "r"(acc));
    else asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(codes), "r"(taps), "r"(acc));
    return d;
}

template <int KW, bool FS, bool GS, int L, int MINB>
__global__ void __launch_bounds__(kThreadsTc, MINB) conv1d_dp4a_tc_kernel(const Conv1dTcParams p) {
    constexpr int HW = KW;                       // 4 KW codes in front of the run cover the K - 1 <= 4 KW - 1 it needs
    constexpr int NWORDS = HW + L / 4;
    __shared__ __align__(16) int32_t s_stage[kWarpsTc][32 * stage_pitch(L)];
    uint32_t gw[KW];
#pragma unroll
    for (int t = 0; t < KW; ++t) {
        uint32_t v = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int k = 4 * t + 3 - j;
            if (k < p.K) v |= (uint32_t)(uint8_t)__ldg(p.g + k) << (8 * j);
        }
        gw[t] = v;
    }
    walk_tiles<L, HW>(p.f, p.y, p.len, p.n_out, (unsigned)p.n_tiles, p.fast_after_first, s_stage[threadIdx.x >> 5],
                      [&](const uint32_t (&w)[NWORDS], int32_t (&out)[L]) {
#pragma unroll
        for (int o = 0; o < L; ++o) {
            int32_t acc = 0;
#pragma unroll
            for (int tw = 0; tw < KW; ++tw) {
                const int rel = o - 4 * tw - 3 + 4 * HW;      // first code of the window, counted from the first loaded code
                const int idx = rel / 4, r = rel % 4;
                const uint32_t window = r == 0 ? w[idx] : __funnelshift_r(w[idx], w[idx + 1], 8 * r);
                acc = dot4<FS, GS>(window, gw[tw], acc);
            }
            out[o] = acc;
        }
    });
}

int conv1d_tc_outputs_per_tile(int N) {
    switch (N) {
#define HK_CASE(n) case n: return 32 * blocks_per_lane(n) * n;
        HK_CASE(1) HK_CASE(2) HK_CASE(3) HK_CASE(4) HK_CASE(5) HK_CASE(6) HK_CASE(7) HK_CASE(8) HK_CASE(9) HK_CASE(10) HK_CASE(11) HK_CASE(12)
#undef HK_CASE
        default: return 0;
    }
}

template <int N, int J, int SC>
static int launch_packed_tc_njs(const Conv1dTcParams &p, bool sp, bool fs, cudaStream_t st) {
    if (!sp) return launch_persistent(conv1d_packed_tc_kernel<N, J, SC, false, false>, p, st);
    if (fs) return launch_persistent(conv1d_packed_tc_kernel<N, J, SC, true, true>, p, st);
    return launch_persistent(conv1d_packed_tc_kernel<N, J, SC, true, false>, p, st);
}

// The 1-D kernels are bound by HBM, not by the multiplier, and run fastest with per-lane runs of 24 to 28
// outputs at four resident CTAs per SM.  N = 5 (runs of 20) and N >= 9 (runs of 36 to 44, three CTAs) miss
// that; the block sizes 4 and 8 reach it with the same slot width and a few more multiplies.
int conv1d_tc_preferred_n(int N) {
    if (N == 5) return 4;
    if (N >= 9) return 8;
    return N;
}

bool conv1d_packed_tc_available(int N, int J) {
    if (J == 1) return N >= 1 && N <= 12;
    if (J == 2) return N >= 2 && N <= 6;
    if (J == 3) return N == 2 || N == 3;
    if (J == 4) return N == 2;
    return false;
}

int launch_conv1d_packed_tc(const Conv1dTcParams &p, int N, int J, bool sp, bool fs, cudaStream_t st) {
    // layouts of the p = q bitwidth sweep (K = 3, 5, 7) with the slot width as a compile-time constant
#define HK_NJS(n, j, sc) if (N == n && J == j && p.S == sc) return launch_packed_tc_njs<n, j, sc>(p, sp, fs, st);
    HK_NJS(11, 1, 3) HK_NJS(8, 1, 3) HK_NJS(8, 1, 4) HK_NJS(4, 1, 6) HK_NJS(4, 1, 7) HK_NJS(4, 2, 7) HK_NJS(6, 1, 6) HK_NJS(5, 1, 6) HK_NJS(5, 1, 7) HK_NJS(5, 2, 7) HK_NJS(4, 1, 8) HK_NJS(4, 2, 9)
    HK_NJS(3, 1, 10) HK_NJS(3, 2, 11) HK_NJS(3, 3, 11) HK_NJS(3, 1, 12) HK_NJS(3, 2, 13) HK_NJS(3, 3, 13)
    HK_NJS(2, 2, 14) HK_NJS(2, 3, 15) HK_NJS(2, 4, 15) HK_NJS(2, 2, 16) HK_NJS(2, 3, 17) HK_NJS(2, 4, 17)
    HK_NJS(2, 2, 18) HK_NJS(2, 3, 19) HK_NJS(2, 4, 19)
#undef HK_NJS
    // any other layout: slot width read at run time
#define HK_NJ(n, j) if (N == n && J == j) return launch_packed_tc_njs<n, j, 0>(p, sp, fs, st);
    HK_NJ(1, 1) HK_NJ(2, 1) HK_NJ(3, 1) HK_NJ(4, 1) HK_NJ(5, 1) HK_NJ(6, 1) HK_NJ(7, 1) HK_NJ(8, 1) HK_NJ(9, 1) HK_NJ(10, 1)
    HK_NJ(11, 1) HK_NJ(12, 1)
    HK_NJ(2, 2) HK_NJ(3, 2) HK_NJ(4, 2) HK_NJ(5, 2) HK_NJ(6, 2)
    HK_NJ(2, 3) HK_NJ(3, 3)
    HK_NJ(2, 4)
#undef HK_NJ
    return HIKONV_ERR_UNSUPPORTED;
}

// Dense input: the layouts of the 1-, 2- and 4-bit cases of the sweep (K = 3, 5, 7; any combination of signed and
// unsigned operands: the mixed cases take the same (N, J, S)), slot width at compile time.
#define HK_DENSE_LAYOUTS(X) X(1, 11, 1, 3) X(1, 8, 1, 4) X(2, 6, 1, 6) X(2, 5, 1, 6) X(2, 5, 1, 7) X(2, 5, 2, 7) \
                            X(4, 3, 1, 10) X(4, 3, 2, 11) X(4, 3, 3, 11)

bool conv1d_packed_dense_available(int P, int N, int J, int S, bool sp, bool fs) {
    (void)sp;
    (void)fs;
#define HK_X(pp, n, j, sc) if (P == pp && N == n && J == j && S == sc) return true;
    HK_DENSE_LAYOUTS(HK_X)
#undef HK_X
    return false;
}

int launch_conv1d_packed_dense(const Conv1dTcParams &p, int P, int N, int J, bool sp, bool fs, cudaStream_t st) {
#define HK_X(pp, n, j, sc)                                                                                       \
    if (P == pp && N == n && J == j && p.S == sc) {                                                              \
        if (fs) return launch_persistent(conv1d_packed_tc_kernel<n, j, sc, true, true, pp>, p, st);             \
        if (sp) return launch_persistent(conv1d_packed_tc_kernel<n, j, sc, true, false, pp>, p, st);            \
        return launch_persistent(conv1d_packed_tc_kernel<n, j, sc, false, false, pp>, p, st);                   \
    }
    HK_DENSE_LAYOUTS(HK_X)
#undef HK_X
    return HIKONV_ERR_UNSUPPORTED;
}

bool conv1d_unpacked_tc_available(int K) { return K == 3 || K == 5 || K == 7; }

int launch_conv1d_unpacked_tc(const Conv1dTcParams &p, int K, bool fs, int shape, cudaStream_t st) {
#define HK_K(k, shape_c, run_c, minb)                                                                    \
    if (K == k && shape == shape_c) {                                                                    \
        if (fs) return launch_persistent(conv1d_unpacked_tc_kernel<k, true, run_c, minb>, p, st);        \
        return launch_persistent(conv1d_unpacked_tc_kernel<k, false, run_c, minb>, p, st);               \
    }
    HK_K(3, 24, 24, 4) HK_K(5, 24, 24, 4) HK_K(7, 24, 24, 4) HK_K(3, 25, 24, 5) HK_K(5, 25, 24, 5) HK_K(7, 25, 24, 5)
    HK_K(3, 32, 32, 3) HK_K(5, 32, 32, 3) HK_K(7, 32, 32, 3)
#undef HK_K
    return HIKONV_ERR_UNSUPPORTED;
}

bool conv1d_dp4a_tc_available(int K) { return K >= 1 && K <= 8; }

int launch_conv1d_dp4a_tc(const Conv1dTcParams &p, int K, bool fs, bool gs, int shape, cudaStream_t st) {
#define HK_KW(kw, shape_c, run_c, minb)                                                                             \
    if ((K + 3) / 4 == kw && shape == shape_c) {                                                                    \
        if (fs && gs) return launch_persistent(conv1d_dp4a_tc_kernel<kw, true, true, run_c, minb>, p, st);          \
        if (fs) return launch_persistent(conv1d_dp4a_tc_kernel<kw, true, false, run_c, minb>, p, st);               \
        if (gs) return launch_persistent(conv1d_dp4a_tc_kernel<kw, false, true, run_c, minb>, p, st);               \
        return launch_persistent(conv1d_dp4a_tc_kernel<kw, false, false, run_c, minb>, p, st);                      \
    }
    HK_KW(1, 24, 24, 4) HK_KW(2, 24, 24, 4) HK_KW(1, 25, 24, 5) HK_KW(2, 25, 24, 5) HK_KW(1, 32, 32, 3) HK_KW(2, 32, 32, 3)
#undef HK_KW
    return HIKONV_ERR_UNSUPPORTED;
}

}  // namespace hikonv
