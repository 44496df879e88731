// HIKONV_ALGO_PACKED64EMU for hikonv_conv1d: the packed method on a 64x64 -> 128 multiplier that the
// GPU does not have, built from its 32-bit multiply pipe (the low and the high 64 bits of the product
// are each a short sequence of 32x32 multiply-adds).  The paper notes that a wider multiplier is used
// in the same way as the 32-bit one (Section V-A); this is that variant:
//   A_x = sum_n f[xN+n] 2^(S n)   in 64 bits  (Eq. 5; more codes per word than 32 bits hold)
//   Q_x = bias + sum_j A_{x-j} B_j in 128 bits (Eq. 9)
//   D_x = Q_x + (Q_{x-1} >> S N)               (Theorem 2)
//   y[xN+m] = ((D_x >> S m) & mask) - carry_bias[m],  m < N   (Algorithm 2's shift and mask on biased slots)
// One block of N outputs per lane, 32 consecutive blocks per warp step, neighbours by shuffle, outputs
// staged per warp in shared memory and written with coalesced 16-byte stores.
#include "hikonv_conv1d_emu64.h"
#include "hikonv_cuda.cuh"

namespace hikonv {

constexpr int kThreadsE = 256;
constexpr int kWarpsE = kThreadsE / 32;

typedef unsigned __int128 u128;

struct Emu64Params {
    const int8_t *f;
    const int8_t *g;
    int32_t *y;
    long long len;
    long long n_out;
    long long n_chunks;      // chunks of 32 blocks covering n_out outputs
    int K, S, J, Kc;
    int hi_shift;            // S * N
    int g_signed;
    int chunks_per_warp;
    int y_aligned16;
    uint32_t mask;
    uint64_t bias_lo, bias_hi;
    int32_t carry_bias[kMaxNEmu64];
};

// The full 128-bit product of two 64-bit words.
template <bool SIGNED>
__device__ __forceinline__ u128 mul_64x64(uint64_t a, uint64_t b) {
    const uint64_t lo = a * b;
    const uint64_t hi = SIGNED ? (uint64_t)__mul64hi((long long)a, (long long)b) : __umul64hi(a, b);
    return ((u128)hi << 64) | lo;
}

__device__ __forceinline__ u128 shuffle_128(u128 v, int src_lane) {
    const uint64_t lo = __shfl_sync(0xFFFFFFFFu, (uint64_t)v, src_lane);
    const uint64_t hi = __shfl_sync(0xFFFFFFFFu, (uint64_t)(v >> 64), src_lane);
    return ((u128)hi << 64) | lo;
}

template <int N, bool F_SIGNED>
__device__ __forceinline__ void load_codes_e(const Emu64Params &p, long long chunk, int lane, int32_t (&v)[N]) {
    const long long base = (chunk * 32 + lane) * (long long)N;
#pragma unroll
    for (int n = 0; n < N; ++n) {
        const long long idx = base + n;
        v[n] = (idx >= 0 && idx < p.len) ? load_code<F_SIGNED>(p.f + idx) : 0;   // Eq. 2: zero outside the signal
    }
}

__host__ __device__ constexpr int stage_chunks_e(int N) { return 16 / N > 0 ? 16 / N : 1; }

template <int N, bool SIGNED_PROD, bool F_SIGNED>
__global__ void __launch_bounds__(kThreadsE) conv1d_emu64_kernel(const Emu64Params p) {
    constexpr int G = stage_chunks_e(N);
    __shared__ uint64_t s_B[kMaxJ];
    __shared__ __align__(16) int32_t s_out[kWarpsE][G * 32 * N];

    if (threadIdx.x < p.J) {            // Eq. 5 on the kernel chunk B_j, 64 bits
        const int j = threadIdx.x;
        uint64_t b = 0;
        for (int k = 0; k < p.Kc; ++k) {
            const int idx = j * p.Kc + k;
            if (idx < p.K) {
                const int8_t raw = __ldg(p.g + idx);
                const long long v = p.g_signed ? (long long)raw : (long long)(uint8_t)raw;
                b += (uint64_t)v << (p.S * k);
            }
        }
        s_B[j] = b;
    }
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long c0 = ((long long)blockIdx.x * kWarpsE + warp) * p.chunks_per_warp;
    if (c0 >= p.n_chunks) return;
    const long long c1 = (c0 + p.chunks_per_warp < p.n_chunks) ? c0 + p.chunks_per_warp : p.n_chunks;

    const uint64_t B0 = s_B[0];
    const u128 bias = ((u128)p.bias_hi << 64) | p.bias_lo;
    int32_t *stage = s_out[warp];

    uint64_t prevA = 0;
    u128 prevHi = 0;
    long long group_c0 = c0;
    for (long long c = c0 - 1; c < c1; ++c) {       // the chunk before the run only seeds A_{x-j} and the carry
        int32_t v[N];
        load_codes_e<N, F_SIGNED>(p, c, lane, v);
        uint64_t A = 0;
#pragma unroll
        for (int n = 0; n < N; ++n) A += (uint64_t)(long long)v[n] << (p.S * n);

        u128 Q = bias + mul_64x64<SIGNED_PROD>(A, B0);
        for (int j = 1; j < p.J; ++j) {
            const uint64_t src = (lane >= 32 - j) ? prevA : A;      // block x-j: lane - j of this or the previous chunk
            const uint64_t Aj = __shfl_sync(0xFFFFFFFFu, src, (lane - j) & 31);
            Q += mul_64x64<SIGNED_PROD>(Aj, s_B[j]);
        }
        const u128 hi = Q >> p.hi_shift;                             // slots N.. of this block's product
        u128 carry = shuffle_128(hi, (lane + 31) & 31);
        if (lane == 0) carry = prevHi;
        prevHi = shuffle_128(hi, 31);
        prevA = A;
        if (c < c0) continue;

        const u128 D = Q + carry;
        const int slot = (int)(c - group_c0);
        int32_t *dst = stage + (slot * 32 + lane) * N;
#pragma unroll
        for (int m = 0; m < N; ++m) dst[m] = (int32_t)((uint32_t)(D >> (p.S * m)) & p.mask) - p.carry_bias[m];

        if (slot == G - 1 || c == c1 - 1) {         // write the staged group out, coalesced
            __syncwarp();
            const long long first = group_c0 * 32 * (long long)N;
            const int count = (slot + 1) * 32 * N;
            if (p.y_aligned16 && first + count <= p.n_out) {
                const int4 *s4 = reinterpret_cast<const int4 *>(stage);
                int4 *d4 = reinterpret_cast<int4 *>(p.y + first);
                for (int i = lane; i < count / 4; i += 32) d4[i] = s4[i];
            } else {
                for (int i = lane; i < count; i += 32)
                    if (first + i < p.n_out) p.y[first + i] = stage[i];
            }
            __syncwarp();
            group_c0 = c + 1;
        }
    }
}

template <int N>
static int launch_n(const Emu64Params &p, bool signed_prod, bool f_signed, unsigned grid, cudaStream_t st) {
    if (!signed_prod) return launch_plain(conv1d_emu64_kernel<N, false, false>, dim3(grid), dim3(kThreadsE), 0, st, p);
    if (f_signed) return launch_plain(conv1d_emu64_kernel<N, true, true>, dim3(grid), dim3(kThreadsE), 0, st, p);
    return launch_plain(conv1d_emu64_kernel<N, true, false>, dim3(grid), dim3(kThreadsE), 0, st, p);
}

int launch_conv1d_emu64(const int8_t *d_f, size_t len, const int8_t *d_g, int K, int p, int q, int f_signed, int g_signed,
                        int32_t *d_y, const hikonv_tuning_t *tune, cudaStream_t st) {
    hikonv_layout_t L;
    const int rc = make_layout_emu64(p, q, f_signed, g_signed, K, tune, &L);
    if (rc != HIKONV_OK) return rc;
    if (L.N > kMaxNEmu64) return HIKONV_ERR_UNSUPPORTED;
    const SplitConsts128 sc = make_split_consts128(L, p, q, f_signed, g_signed, K);
    Emu64Params kp;
    kp.f = d_f; kp.g = d_g; kp.y = d_y; kp.len = (long long)len; kp.n_out = (long long)len + K - 1;
    const long long n_blocks = (kp.n_out + L.N - 1) / L.N;
    kp.n_chunks = (n_blocks + 31) / 32;
    kp.K = K; kp.S = L.S; kp.J = L.J; kp.Kc = L.Kc; kp.hi_shift = L.S * L.N;
    kp.g_signed = g_signed ? 1 : 0;
    kp.y_aligned16 = ((uintptr_t)d_y % 16 == 0) ? 1 : 0;
    kp.mask = sc.slot_mask;
    kp.bias_lo = sc.bias_lo;
    kp.bias_hi = sc.bias_hi;
    for (int m = 0; m < kMaxNEmu64; ++m) kp.carry_bias[m] = m < L.N ? sc.carry_bias[m] : 0;
    // long runs amortise the one seeding chunk per warp; short problems spread over the SMs first
    long long cpw = tune && tune->tile > 0 ? tune->tile : 16;
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long want_warps = (long long)sms * kWarpsE * 4;
    if (kp.n_chunks / cpw < want_warps) cpw = kp.n_chunks / want_warps;
    if (cpw < 1) cpw = 1;
    kp.chunks_per_warp = (int)cpw;
    const long long warps = (kp.n_chunks + cpw - 1) / cpw;
    const long long grid = (warps + kWarpsE - 1) / kWarpsE;
    if (grid > 0x7FFFFFFFLL) return HIKONV_ERR_UNSUPPORTED;
    const bool sp = L.signed_prod != 0, fs = f_signed != 0;
    switch (L.N) {
        case 1: return launch_n<1>(kp, sp, fs, (unsigned)grid, st);
        case 2: return launch_n<2>(kp, sp, fs, (unsigned)grid, st);
        case 3: return launch_n<3>(kp, sp, fs, (unsigned)grid, st);
        case 4: return launch_n<4>(kp, sp, fs, (unsigned)grid, st);
        case 5: return launch_n<5>(kp, sp, fs, (unsigned)grid, st);
        case 6: return launch_n<6>(kp, sp, fs, (unsigned)grid, st);
        case 7: return launch_n<7>(kp, sp, fs, (unsigned)grid, st);
        case 8: return launch_n<8>(kp, sp, fs, (unsigned)grid, st);
        case 9: return launch_n<9>(kp, sp, fs, (unsigned)grid, st);
        case 10: return launch_n<10>(kp, sp, fs, (unsigned)grid, st);
        case 11: return launch_n<11>(kp, sp, fs, (unsigned)grid, st);
        case 12: return launch_n<12>(kp, sp, fs, (unsigned)grid, st);
        case 13: return launch_n<13>(kp, sp, fs, (unsigned)grid, st);
        case 14: return launch_n<14>(kp, sp, fs, (unsigned)grid, st);
        case 15: return launch_n<15>(kp, sp, fs, (unsigned)grid, st);
        case 16: return launch_n<16>(kp, sp, fs, (unsigned)grid, st);
        default: return HIKONV_ERR_UNSUPPORTED;
    }
}

}  // namespace hikonv
