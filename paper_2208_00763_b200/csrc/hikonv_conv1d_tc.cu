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
#include "hikonv_cuda.cuh"
#include "hikonv_conv1d_tc.h"

namespace hikonv {

constexpr int kThreadsTc = 256;
constexpr int kWarpsTc = kThreadsTc / 32;

__host__ __device__ constexpr int gcd_c(int a, int b) { return b == 0 ? a : gcd_c(b, a % b); }
// blocks per lane: L = R N is a multiple of 4 and at least 12
__host__ __device__ constexpr int blocks_per_lane(int N) {
    const int step = 4 / gcd_c(N, 4);
    int r = step;
    while (r * N < 12) r += step;
    return r;
}

// Byte `b` (0..3) of w as a 32-bit value, sign- or zero-extended: one prmt.
template <bool SIGNED>
__device__ __forceinline__ uint32_t extract_code(uint32_t w, int b) {
    uint32_t r;
    // selector nibbles: low nibble picks byte b; in the upper three, bit 3 replicates that byte's sign,
    // or index 4 picks byte 0 of the zero second operand
    const uint32_t sel = SIGNED ? (uint32_t)(b | ((8 | b) << 4) | ((8 | b) << 8) | ((8 | b) << 12)) : (uint32_t)(b | 0x4440);
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(w), "r"(0u), "r"(sel));
    return r;
}

// Loads the words covering elements [e0 - 4 HW, e0 + 4 NWD - 4 HW) of f; e0 is a multiple of 4.
template <int NWORDS, int HW>
__device__ __forceinline__ void load_words(const int8_t *f, long long len, long long e0, bool fast, uint32_t (&w)[NWORDS]) {
    if (fast) {
        const uint32_t *src = reinterpret_cast<const uint32_t *>(f + e0) - HW;
#pragma unroll
        for (int i = 0; i < NWORDS; ++i) w[i] = __ldg(src + i);
    } else {
#pragma unroll
        for (int i = 0; i < NWORDS; ++i) {
            uint32_t v = 0;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const long long idx = e0 + 4 * (i - HW) + b;
                if (idx >= 0 && idx < len) v |= (uint32_t)(uint8_t)__ldg(f + idx) << (8 * b);   // Eq. 2: zero outside
            }
            w[i] = v;
        }
    }
}

// Row pitch (in words) of a lane's run in the warp's staging buffer: L padded so that the 16-byte
// stores of eight neighbouring lanes fall into different banks.
__host__ __device__ constexpr int stage_pitch(int L) { return (L % 8 == 0) ? L + 4 : L; }

// Writes a warp tile of 32 runs of L outputs.  Interior tiles go through the warp's shared-memory
// buffer so that every store instruction writes 512 contiguous bytes; edge tiles are stored guarded.
template <int L>
__device__ __forceinline__ void store_run(int32_t *y, long long n_out, long long tile0, int lane, bool fast, int32_t *stage,
                                          const int32_t (&out)[L]) {
    constexpr int P = stage_pitch(L);
    if (fast) {
        int4 *row = reinterpret_cast<int4 *>(stage + lane * P);
#pragma unroll
        for (int i = 0; i < L / 4; ++i) row[i] = make_int4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
        __syncwarp();
        int4 *dst = reinterpret_cast<int4 *>(y + tile0);
#pragma unroll
        for (int k = 0; k < L / 4; ++k) {
            const int idx = 4 * (lane + 32 * k);              // first output of this 16-byte piece within the tile
            const int src_lane = idx / L, src_off = idx % L;  // L is a multiple of 4: a piece never straddles two runs
            dst[lane + 32 * k] = *reinterpret_cast<const int4 *>(stage + src_lane * P + src_off);
        }
        __syncwarp();
    } else {
        const long long e0 = tile0 + lane * L;
#pragma unroll
        for (int i = 0; i < L; ++i)
            if (e0 + i < n_out) y[e0 + i] = out[i];
    }
}

template <int N, int J, bool SP, bool FS>
__global__ void __launch_bounds__(kThreadsTc) conv1d_packed_tc_kernel(const Conv1dTcParams p) {
    constexpr int R = blocks_per_lane(N);
    constexpr int L = R * N;
    constexpr int HW = (J * N + 3) / 4;          // words in front of the run
    constexpr int NWORDS = HW + L / 4;
    __shared__ uint32_t s_B[J];
    __shared__ __align__(16) int32_t s_stage[kWarpsTc][32 * stage_pitch(L)];
    if (threadIdx.x < J) {                        // pack the kernel chunk B_j (Eq. 5 on g)
        uint32_t b = 0;
        for (int k = 0; k < p.Kc; ++k) {
            const int idx = threadIdx.x * p.Kc + k;
            if (idx < p.K) {
                const int8_t raw = __ldg(p.g + idx);
                const int32_t v = p.g_signed ? (int32_t)raw : (int32_t)(uint8_t)raw;
                b += (uint32_t)v << (p.S * k);
            }
        }
        s_B[threadIdx.x] = b;
    }
    __syncthreads();
    uint32_t Bw[J];
#pragma unroll
    for (int j = 0; j < J; ++j) Bw[j] = s_B[j];
    uint32_t slot_pow[N];
#pragma unroll
    for (int n = 0; n < N; ++n) slot_pow[n] = 1u << (p.S * n);

    const int lane = threadIdx.x & 31;
    for (long long t = (long long)blockIdx.x * kWarpsTc + (threadIdx.x >> 5); t < p.n_tiles; t += (long long)gridDim.x * kWarpsTc) {
        const long long tile0 = t * (32 * L);
        const bool fast = p.aligned && tile0 >= 4 * HW && tile0 + 32 * L <= p.len;
        const long long e0 = tile0 + lane * L;
        uint32_t w[NWORDS];
        load_words<NWORDS, HW>(p.f, p.len, e0, fast, w);

        // A_x for x = -J .. R-1 (index x + J); element n of block x sits at byte 4 HW + x N + n of w
        uint32_t A[R + J];
#pragma unroll
        for (int x = -J; x < R; ++x) {
            uint32_t a = 0;
#pragma unroll
            for (int n = 0; n < N; ++n) {
                const int pos = 4 * HW + x * N + n;
                const uint32_t c = extract_code<FS>(w[pos / 4], pos % 4);
                a = (n == 0) ? c : a + c * slot_pow[n];
            }
            A[x + J] = a;
        }
        // Q_x for x = -1 .. R-1, carry chain, split
        int32_t out[L];
        uint32_t carry = 0;
#pragma unroll
        for (int x = -1; x < R; ++x) {
            uint64_t Q = p.bias;
#pragma unroll
            for (int j = 0; j < J; ++j) mad_wide<SP>(Q, A[x - j + J], Bw[j]);
            if (x >= 0) {
                const uint64_t D = Q + (uint64_t)carry;
#pragma unroll
                for (int m = 0; m < N; ++m)
                    out[x * N + m] = (int32_t)(shr64_lo(D, p.seg_shift[m]) & p.mask) - p.carry_bias[m];
            }
            carry = shr64_lo(Q, p.hi_shift);
        }
        store_run<L>(p.y, p.n_out, tile0, lane, fast, s_stage[threadIdx.x >> 5], out);
    }
}

// Comparator: 16 outputs per lane, one product per 32-bit multiply-add.
template <int K, bool FS>
__global__ void __launch_bounds__(kThreadsTc) conv1d_unpacked_tc_kernel(const Conv1dTcParams p) {
    constexpr int L = 16;
    constexpr int HW = (K - 1 + 3) / 4;
    constexpr int NWORDS = HW + L / 4;
    __shared__ int32_t s_g[K];
    __shared__ __align__(16) int32_t s_stage[kWarpsTc][32 * stage_pitch(L)];
    if (threadIdx.x < K) {
        const int8_t raw = __ldg(p.g + threadIdx.x);
        s_g[threadIdx.x] = p.g_signed ? (int32_t)raw : (int32_t)(uint8_t)raw;
    }
    __syncthreads();
    int32_t gk[K];
#pragma unroll
    for (int k = 0; k < K; ++k) gk[k] = s_g[k];
    const int lane = threadIdx.x & 31;
    for (long long t = (long long)blockIdx.x * kWarpsTc + (threadIdx.x >> 5); t < p.n_tiles; t += (long long)gridDim.x * kWarpsTc) {
        const long long tile0 = t * (32 * L);
        const bool fast = p.aligned && tile0 >= 4 * HW && tile0 + 32 * L <= p.len;
        const long long e0 = tile0 + lane * L;
        uint32_t w[NWORDS];
        load_words<NWORDS, HW>(p.f, p.len, e0, fast, w);
        int32_t e[L + K - 1];                       // e[i] = f[e0 - (K-1) + i]
#pragma unroll
        for (int i = 0; i < L + K - 1; ++i) {
            const int pos = 4 * HW - (K - 1) + i;
            e[i] = (int32_t)extract_code<FS>(w[pos / 4], pos % 4);
        }
        int32_t out[L];
#pragma unroll
        for (int o = 0; o < L; ++o) {
            int32_t s = 0;
#pragma unroll
            for (int k = 0; k < K; ++k) s += e[o + (K - 1) - k] * gk[k];      // y[m] = sum_k f[m-k] g[k]
            out[o] = s;
        }
        store_run<L>(p.y, p.n_out, tile0, lane, fast, s_stage[threadIdx.x >> 5], out);
    }
}

static unsigned tc_grid(long long n_tiles) {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long want = (n_tiles + kWarpsTc - 1) / kWarpsTc;
    const long long cap = (long long)sms * 32;
    return (unsigned)(want < cap ? want : cap);
}

int conv1d_tc_outputs_per_tile(int N) {
    switch (N) {
#define HK_CASE(n) case n: return 32 * blocks_per_lane(n) * n;
        HK_CASE(1) HK_CASE(2) HK_CASE(3) HK_CASE(4) HK_CASE(5) HK_CASE(6) HK_CASE(7) HK_CASE(8) HK_CASE(9) HK_CASE(10) HK_CASE(11) HK_CASE(12)
#undef HK_CASE
        default: return 0;
    }
}

template <int N, int J>
static int launch_packed_tc_nj(const Conv1dTcParams &p, bool sp, bool fs, cudaStream_t st) {
    const unsigned grid = tc_grid(p.n_tiles);
    if (!sp) conv1d_packed_tc_kernel<N, J, false, false><<<grid, kThreadsTc, 0, st>>>(p);
    else if (fs) conv1d_packed_tc_kernel<N, J, true, true><<<grid, kThreadsTc, 0, st>>>(p);
    else conv1d_packed_tc_kernel<N, J, true, false><<<grid, kThreadsTc, 0, st>>>(p);
    return launch_status();
}

bool conv1d_packed_tc_available(int N, int J) {
    if (J == 1) return N >= 1 && N <= 12;
    if (J == 2) return N >= 2 && N <= 6;
    if (J == 3) return N == 2 || N == 3;
    if (J == 4) return N == 2;
    return false;
}

int launch_conv1d_packed_tc(const Conv1dTcParams &p, int N, int J, bool sp, bool fs, cudaStream_t st) {
#define HK_NJ(n, j) if (N == n && J == j) return launch_packed_tc_nj<n, j>(p, sp, fs, st);
    HK_NJ(1, 1) HK_NJ(2, 1) HK_NJ(3, 1) HK_NJ(4, 1) HK_NJ(5, 1) HK_NJ(6, 1) HK_NJ(7, 1) HK_NJ(8, 1) HK_NJ(9, 1) HK_NJ(10, 1)
    HK_NJ(11, 1) HK_NJ(12, 1)
    HK_NJ(2, 2) HK_NJ(3, 2) HK_NJ(4, 2) HK_NJ(5, 2) HK_NJ(6, 2)
    HK_NJ(2, 3) HK_NJ(3, 3)
    HK_NJ(2, 4)
#undef HK_NJ
    return HIKONV_ERR_UNSUPPORTED;
}

bool conv1d_unpacked_tc_available(int K) { return K == 3 || K == 5 || K == 7; }

int launch_conv1d_unpacked_tc(const Conv1dTcParams &p, int K, bool fs, cudaStream_t st) {
    const unsigned grid = tc_grid(p.n_tiles);
#define HK_K(k)                                                                                   \
    if (K == k) {                                                                                 \
        if (fs) conv1d_unpacked_tc_kernel<k, true><<<grid, kThreadsTc, 0, st>>>(p);               \
        else conv1d_unpacked_tc_kernel<k, false><<<grid, kThreadsTc, 0, st>>>(p);                 \
        return launch_status();                                                                   \
    }
    HK_K(3) HK_K(5) HK_K(7)
#undef HK_K
    return HIKONV_ERR_UNSUPPORTED;
}

}  // namespace hikonv
