// hikonv_conv1d: full 1-D convolution, packed (Theorems 1 and 2) and unpacked comparator.
//
// Packed kernel, per warp: a run of "chunks" of 32 consecutive blocks, one block of N outputs
// per lane.  For block x a lane
//   packs   A_x = sum_n f[xN+n] 2^(S n)                                  (Eq. 5)
//   forms   Q_x = bias + sum_j A_{x-j} * B_j                              (Eq. 9; J > 1 when the
//           kernel is cut into chunks of N taps, A_{x-j} comes from lane - j by shuffle)
//   adds    the carry of block x-1:  D_x = Q_x + (Q_{x-1} >> S N)         (Theorem 2, the
//           "previous product shifted right" step of Section V-A; lane - 1 by shuffle)
//   splits  y[xN+m] = ((D_x >> S m) & mask) - carry_bias[m],  m < N       (Algorithm 2's shift
//           and mask; the per-slot bias replaces the sign-borrow increment of Eq. 29)
// Outputs are staged per warp in shared memory and written with coalesced 16-byte stores.
// This file holds the argument checks, the layout choice and the general (any N, J, K) kernels; the
// register-resident kernels of the packed method and of the two comparators are in hikonv_conv1d_tc.cu,
// the variant on an emulated 64x64 multiplier in hikonv_conv1d_emu64.cu.
#include <cstring>

#include "hikonv_cuda.cuh"
#include "hikonv_conv1d_bs.h"
#include "hikonv_conv1d_emu64.h"
#include "hikonv_conv1d_run.cuh"
#include "hikonv_conv1d_tc.h"

namespace hikonv {

constexpr int kThreads1D = 256;
constexpr int kWarps1D = kThreads1D / 32;

struct Conv1dParams {
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
    uint64_t bias;
    int seg_shift[kMaxN1D];  // S * m
    int32_t carry_bias[kMaxN1D];
};

__host__ __device__ constexpr int stage_chunks(int N) { return N >= 16 ? 1 : (16 / N > 0 ? 16 / N : 1); }

template <int N, bool F_SIGNED>
__device__ __forceinline__ void load_block_codes(const Conv1dParams &p, long long chunk, int lane, int32_t (&v)[N]) {
    const long long base = (chunk * 32 + lane) * (long long)N;
    if (chunk >= 0 && (chunk * 32 + 32) * (long long)N <= p.len) {       // whole chunk inside the signal
        const int8_t *src = p.f + base;
#pragma unroll
        for (int n = 0; n < N; ++n) v[n] = load_code<F_SIGNED>(src + n);
    } else {
#pragma unroll
        for (int n = 0; n < N; ++n) {
            const long long idx = base + n;
            v[n] = (idx >= 0 && idx < p.len) ? load_code<F_SIGNED>(p.f + idx) : 0;   // Eq. 2: zero outside
        }
    }
}

template <int N, bool SIGNED_PROD, bool F_SIGNED>
__global__ void __launch_bounds__(kThreads1D) conv1d_packed_kernel(const Conv1dParams p) {
    constexpr int G = stage_chunks(N);
    __shared__ uint32_t s_B[kMaxJ];
    __shared__ __align__(16) int32_t s_out[kWarps1D][G * 32 * N];

    if (threadIdx.x < p.J) {            // pack the kernel chunk B_j (Eq. 5 on g)
        const int j = threadIdx.x;
        uint32_t b = 0;
        for (int k = 0; k < p.Kc; ++k) {
            const int idx = j * p.Kc + k;
            if (idx < p.K) {
                const int8_t raw = __ldg(p.g + idx);
                const int32_t v = p.g_signed ? (int32_t)raw : (int32_t)(uint8_t)raw;
                b += (uint32_t)v << (p.S * k);
            }
        }
        s_B[j] = b;
    }
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long c0 = ((long long)blockIdx.x * kWarps1D + warp) * p.chunks_per_warp;
    if (c0 >= p.n_chunks) return;
    const long long c1 = (c0 + p.chunks_per_warp < p.n_chunks) ? c0 + p.chunks_per_warp : p.n_chunks;

    uint32_t slot_pow[N];               // 2^(S n): packing by multiply-add
#pragma unroll
    for (int n = 0; n < N; ++n) slot_pow[n] = 1u << (p.S * n);
    const uint32_t B0 = s_B[0];
    int32_t *stage = s_out[warp];

    uint32_t prevA = 0, prevHi = 0;
    int32_t vnext[N];
    load_block_codes<N, F_SIGNED>(p, c0 - 1, lane, vnext);
    long long group_c0 = c0;
    for (long long c = c0 - 1; c < c1; ++c) {
        int32_t v[N];
#pragma unroll
        for (int n = 0; n < N; ++n) v[n] = vnext[n];
        if (c + 1 < c1) load_block_codes<N, F_SIGNED>(p, c + 1, lane, vnext);

        uint32_t A = (uint32_t)v[0];
#pragma unroll
        for (int n = 1; n < N; ++n) A += (uint32_t)v[n] * slot_pow[n];

        uint64_t Q = p.bias;
        mad_wide<SIGNED_PROD>(Q, A, B0);
        for (int j = 1; j < p.J; ++j) {
            const uint32_t src = (lane >= 32 - j) ? prevA : A;          // block x-j sits in lane-j of this or the previous chunk
            const uint32_t Aj = __shfl_sync(0xFFFFFFFFu, src, (lane - j) & 31);
            mad_wide<SIGNED_PROD>(Q, Aj, s_B[j]);
        }
        const uint32_t hi = shr64_lo(Q, p.hi_shift);                     // slots N.. of this block's product
        uint32_t carry = __shfl_up_sync(0xFFFFFFFFu, hi, 1);
        if (lane == 0) carry = prevHi;
        prevHi = __shfl_sync(0xFFFFFFFFu, hi, 31);
        prevA = A;
        if (c < c0) continue;           // the chunk before the run only seeds the carries

        const uint64_t D = Q + (uint64_t)carry;
        int32_t out[N];
#pragma unroll
        for (int m = 0; m < N; ++m) out[m] = (int32_t)(shr64_lo(D, p.seg_shift[m]) & p.mask) - p.carry_bias[m];

        const int slot = (int)(c - group_c0);
        int32_t *dst = stage + (slot * 32 + lane) * N;
        if (N % 4 == 0) {
#pragma unroll
            for (int m = 0; m < N; m += 4) *reinterpret_cast<int4 *>(dst + m) = make_int4(out[m], out[m + 1], out[m + 2], out[m + 3]);
        } else if (N % 2 == 0) {
#pragma unroll
            for (int m = 0; m < N; m += 2) *reinterpret_cast<int2 *>(dst + m) = make_int2(out[m], out[m + 1]);
        } else {
#pragma unroll
            for (int m = 0; m < N; ++m) dst[m] = out[m];
        }

        if (slot == G - 1 || c == c1 - 1) {     // write the staged group out, coalesced
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

// Comparator: one product per 32-bit multiply-add.  Each thread computes four consecutive outputs
// with a sliding window over f.
struct Conv1dUnpackedParams {
    const int8_t *f;
    const int8_t *g;
    int32_t *y;
    long long len;
    long long n_out;
    int K;
    int g_signed;
    int y_aligned16;
};

// One kernel tap for four neighbouring outputs: y[t0+o] += f[t0+o-k] g[k], then slide the window
// one element towards lower indices for the next tap.
template <bool F_SIGNED>
__device__ __forceinline__ void unpacked_tap(const Conv1dUnpackedParams &p, long long t0, int k, int K, bool interior,
                                             int32_t gk, int32_t (&w)[4], int32_t (&acc)[4]) {
#pragma unroll
    for (int o = 0; o < 4; ++o) acc[o] += w[o] * gk;
    if (k + 1 < K) {
        const long long idx = t0 - (k + 1);
        w[3] = w[2];
        w[2] = w[1];
        w[1] = w[0];
        w[0] = (interior || (idx >= 0 && idx < p.len)) ? load_code<F_SIGNED>(p.f + idx) : 0;
    }
}

template <int KT, bool F_SIGNED>
__global__ void __launch_bounds__(kThreads1D) conv1d_unpacked_kernel(const Conv1dUnpackedParams p) {
    __shared__ int32_t s_g[kMaxK];
    const int K = KT > 0 ? KT : p.K;
    if (threadIdx.x < K) {
        const int8_t raw = __ldg(p.g + threadIdx.x);
        s_g[threadIdx.x] = p.g_signed ? (int32_t)raw : (int32_t)(uint8_t)raw;
    }
    __syncthreads();
    const long long t0 = ((long long)blockIdx.x * kThreads1D + threadIdx.x) * 4;
    if (t0 >= p.n_out) return;
    const bool interior = (t0 - (K - 1) >= 0) && (t0 + 3 < p.len);
    int32_t w[4];
#pragma unroll
    for (int o = 0; o < 4; ++o) {
        const long long idx = t0 + o;
        w[o] = (interior || idx < p.len) ? load_code<F_SIGNED>(p.f + idx) : 0;
    }
    int32_t acc[4] = {0, 0, 0, 0};
    if (KT > 0) {
#pragma unroll
        for (int k = 0; k < KT; ++k) unpacked_tap<F_SIGNED>(p, t0, k, KT, interior, s_g[k], w, acc);
    } else {
        for (int k = 0; k < K; ++k) unpacked_tap<F_SIGNED>(p, t0, k, K, interior, s_g[k], w, acc);
    }
    if (p.y_aligned16 && t0 + 3 < p.n_out) {
        *reinterpret_cast<int4 *>(p.y + t0) = make_int4(acc[0], acc[1], acc[2], acc[3]);
    } else {
#pragma unroll
        for (int o = 0; o < 4; ++o)
            if (t0 + o < p.n_out) p.y[t0 + o] = acc[o];
    }
}

template <int N>
static int launch_packed_n(const Conv1dParams &p, bool signed_prod, bool f_signed, unsigned grid, cudaStream_t st) {
    if (!signed_prod) return launch_plain(conv1d_packed_kernel<N, false, false>, dim3(grid), dim3(kThreads1D), 0, st, p);
    if (f_signed) return launch_plain(conv1d_packed_kernel<N, true, true>, dim3(grid), dim3(kThreads1D), 0, st, p);
    return launch_plain(conv1d_packed_kernel<N, true, false>, dim3(grid), dim3(kThreads1D), 0, st, p);
}

static int launch_packed(int N, const Conv1dParams &p, bool sp, bool fs, unsigned grid, cudaStream_t st) {
    switch (N) {
        case 1: return launch_packed_n<1>(p, sp, fs, grid, st);
        case 2: return launch_packed_n<2>(p, sp, fs, grid, st);
        case 3: return launch_packed_n<3>(p, sp, fs, grid, st);
        case 4: return launch_packed_n<4>(p, sp, fs, grid, st);
        case 5: return launch_packed_n<5>(p, sp, fs, grid, st);
        case 6: return launch_packed_n<6>(p, sp, fs, grid, st);
        case 7: return launch_packed_n<7>(p, sp, fs, grid, st);
        case 8: return launch_packed_n<8>(p, sp, fs, grid, st);
        case 9: return launch_packed_n<9>(p, sp, fs, grid, st);
        case 10: return launch_packed_n<10>(p, sp, fs, grid, st);
        case 11: return launch_packed_n<11>(p, sp, fs, grid, st);
        case 12: return launch_packed_n<12>(p, sp, fs, grid, st);
        default: return HIKONV_ERR_UNSUPPORTED;
    }
}

template <bool F_SIGNED>
static int launch_unpacked(const Conv1dUnpackedParams &p, unsigned grid, cudaStream_t st) {
    switch (p.K) {
        case 3: return launch_plain(conv1d_unpacked_kernel<3, F_SIGNED>, dim3(grid), dim3(kThreads1D), 0, st, p);
        case 5: return launch_plain(conv1d_unpacked_kernel<5, F_SIGNED>, dim3(grid), dim3(kThreads1D), 0, st, p);
        case 7: return launch_plain(conv1d_unpacked_kernel<7, F_SIGNED>, dim3(grid), dim3(kThreads1D), 0, st, p);
        default: return launch_plain(conv1d_unpacked_kernel<0, F_SIGNED>, dim3(grid), dim3(kThreads1D), 0, st, p);
    }
}

// The layout hikonv_conv1d runs with on one-code-per-byte input.  The path is HBM-bound, so the layout with the
// fewest instructions per output wins, not the one with the most outputs per multiply:
//   1. byte-aligned slots (S = 8, 16, 24 with N S = 32) when the sums fit them and K <= 8 (*slot_bytes > 0);
//   2. else the planner's choice, with N lowered to the block size the register-resident kernel streams fastest
//      with when that needs the same slot width and no more kernel chunks.
// A forced N or S (tune) is taken as it is; tune->tile == -1 skips step 1, tune->tile > 0 both.
static int layout_for_byte_input(int p, int q, int f_signed, int g_signed, int K, const hikonv_tuning_t *tune,
                                 hikonv_layout_t *L, int *slot_bytes) {
    *slot_bytes = 0;
    const bool forced = tune && (tune->N > 0 || tune->S > 0 || tune->tile > 0);
    if (!forced && !(tune && tune->tile == -1)) {
        if (validate_codes(p, q) != HIKONV_OK || K < 1 || K > kMaxK) return HIKONV_ERR_INVALID_ARG;
        const int sb = make_layout_byte_slots(p, q, f_signed, g_signed, K, L);
        if (sb > 0) {
            *slot_bytes = sb;
            return HIKONV_OK;
        }
    }
    int rc = make_layout(p, q, f_signed, g_signed, K, 1, 0, 0, tune, L);
    if (rc != HIKONV_OK) return rc;
    if (forced) return rc;
    const int n_pref = conv1d_tc_preferred_n(L->N);
    if (n_pref == L->N) return rc;
    hikonv_tuning_t forced_n = {n_pref, L->S, 0, 0};
    hikonv_layout_t alt;
    if (make_layout(p, q, f_signed, g_signed, K, 1, 0, 0, &forced_n, &alt) == HIKONV_OK && alt.J <= L->J &&
        conv1d_packed_tc_available(alt.N, alt.J))
        *L = alt;
    return HIKONV_OK;
}

static int check_conv1d_args(const void *f, size_t len, const void *g, int K, int p, int q, const void *y, int algo) {
    if (!f || !g || !y || len < 1 || K < 1 || K > kMaxK) return HIKONV_ERR_INVALID_ARG;
    if (validate_codes(p, q) != HIKONV_OK) return HIKONV_ERR_INVALID_ARG;
    if (len > (size_t)1 << 40) return HIKONV_ERR_UNSUPPORTED;
    if (algo != HIKONV_ALGO_PACKED32 && algo != HIKONV_ALGO_PACKED64EMU && algo != HIKONV_ALGO_UNPACKED_IMAD &&
        algo != HIKONV_ALGO_DP4A)
        return HIKONV_ERR_INVALID_ARG;
    if (((uintptr_t)y) % 4 != 0) return HIKONV_ERR_INVALID_ARG;
    return HIKONV_OK;
}

}  // namespace hikonv

using namespace hikonv;

extern "C" int hikonv_conv1d(const int8_t *d_f, size_t len, const int8_t *d_g, int K, int p, int q, int f_signed,
                             int g_signed, int32_t *d_y, int algo, const hikonv_tuning_t *tune, void *stream) {
    int rc = check_conv1d_args(d_f, len, d_g, K, p, q, d_y, algo);
    if (rc != HIKONV_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (algo == HIKONV_ALGO_PACKED64EMU)
        return launch_conv1d_emu64(d_f, len, d_g, K, p, q, f_signed, g_signed, d_y, tune, st);
    const long long n_out = (long long)len + K - 1;
    const int y_aligned16 = ((uintptr_t)d_y % 16 == 0) ? 1 : 0;

    // tune->tile > 0 selects the shuffle-based kernels below (any N, J, K); otherwise the
    // register-resident kernels are used whenever they are instantiated for the layout
    const bool want_tc = !(tune && tune->tile > 0);
    Conv1dTcParams tp;
    std::memset(&tp, 0, sizeof(tp));
    tp.f = d_f; tp.g = d_g; tp.y = d_y; tp.len = (long long)len; tp.n_out = n_out; tp.K = K;
    tp.g_signed = g_signed ? 1 : 0;
    tp.aligned = (y_aligned16 && ((uintptr_t)d_f % 4 == 0)) ? 1 : 0;

    if (algo == HIKONV_ALGO_DP4A) {
        if (!conv1d_dp4a_tc_available(K)) return HIKONV_ERR_UNSUPPORTED;
        // one tap word (K <= 4) leaves registers for five resident CTAs per SM, which stream 2-3 % faster; two do not
        const int forced = tune ? -tune->tile : 0;
        const int shape = (forced == 32 || forced == 25 || forced == 24) ? forced : (K <= 4 ? 25 : 24);
        const int run = shape == 32 ? 32 : 24;
        tp.n_tiles = (n_out + 32 * run - 1) / (32 * run);
        tp.fast_after_first = fast_tiles_after_first((long long)len, run, tp.aligned != 0);
        return launch_conv1d_dp4a_tc(tp, K, f_signed != 0, g_signed != 0, shape, st);
    }
    if (algo == HIKONV_ALGO_UNPACKED_IMAD && want_tc && conv1d_unpacked_tc_available(K)) {
        // runs of 24 outputs per lane stream fastest (as for the packed kernels): with the register budget of five
        // resident CTAs per SM up to five taps, of four beyond (seven taps spill at five); -32 keeps the longer runs
        // reachable, -24 / -25 force a budget
        const int forced = tune ? -tune->tile : 0;
        const int shape = (forced == 32 || forced == 25 || forced == 24) ? forced : (K <= 5 ? 25 : 24);
        const int run = shape == 32 ? 32 : 24;
        tp.n_tiles = (n_out + 32 * run - 1) / (32 * run);
        tp.fast_after_first = fast_tiles_after_first((long long)len, run, tp.aligned != 0);
        return launch_conv1d_unpacked_tc(tp, K, f_signed != 0, shape, st);
    }
    if (algo == HIKONV_ALGO_UNPACKED_IMAD) {
        Conv1dUnpackedParams up;
        up.f = d_f; up.g = d_g; up.y = d_y; up.len = (long long)len; up.n_out = n_out; up.K = K;
        up.g_signed = g_signed ? 1 : 0; up.y_aligned16 = y_aligned16;
        const long long threads = (n_out + 3) / 4;
        const long long grid = (threads + kThreads1D - 1) / kThreads1D;
        if (grid > 0x7FFFFFFFLL) return HIKONV_ERR_UNSUPPORTED;
        return f_signed ? launch_unpacked<true>(up, (unsigned)grid, st) : launch_unpacked<false>(up, (unsigned)grid, st);
    }

    hikonv_layout_t L;
    int slot_bytes = 0;
    rc = layout_for_byte_input(p, q, f_signed, g_signed, K, tune, &L, &slot_bytes);
    if (rc != HIKONV_OK) return rc;
    if (slot_bytes > 0) {           // register-aligned slots: mode 1, 2 or 3
        Conv1dBsParams bp;
        std::memset(&bp, 0, sizeof(bp));
        bp.f = d_f; bp.g = d_g; bp.y = d_y; bp.len = (long long)len; bp.n_out = n_out; bp.K = K;
        bp.g_signed = g_signed ? 1 : 0;
        bp.aligned = tp.aligned;
        if (f_signed) {
            bp.code_xor = 0x01010101u * (1u << (p - 1));
            bp.code_and = 0x01010101u * ((1u << p) - 1u);
        }
        bp.S = L.S;
        bp.mask3 = (1u << L.S) - 1u;
        if (slot_bytes == 3 && L.signed_prod) {
            // slot 2 receives floor(K / 2) products: its bias lifts their most negative sum to zero, slot 0 takes the rest
            const SplitConsts sc3 = make_split_consts(L, p, q, f_signed, g_signed, K, 1);
            const uint64_t half = 1ull << (L.S - 1), b2 = (uint64_t)sc3.seg_bias[2];
            bp.bias3 = (half - b2) + (half << L.S) + (b2 << (2 * L.S));
        }
        bp.n_tiles = (unsigned)((n_out + 32 * kBsRun - 1) / (32 * kBsRun));
        bp.fast_after_first = fast_tiles_after_first((long long)len, kBsRun, tp.aligned != 0);
        return launch_conv1d_bs(bp, slot_bytes, L.J, f_signed != 0, L.signed_prod != 0, tune ? -tune->tile : 0, st);
    }
    if (L.N > kMaxN1D) return HIKONV_ERR_UNSUPPORTED;
    const SplitConsts sc = make_split_consts(L, p, q, f_signed, g_signed, K, 1);

    if (want_tc && conv1d_packed_tc_available(L.N, L.J)) {
        const int per_tile = conv1d_tc_outputs_per_tile(L.N);
        tp.n_tiles = (n_out + per_tile - 1) / per_tile;
        tp.S = L.S; tp.Kc = L.Kc; tp.hi_shift = L.S * L.N; tp.mask = sc.slot_mask; tp.bias = sc.bias;
        for (int m = 0; m < kMaxN1D; ++m) {
            tp.seg_shift[m] = m < L.N ? L.S * m : 0;
            tp.carry_bias[m] = m < L.N ? sc.carry_bias[m] : 0;
        }
        return launch_conv1d_packed_tc(tp, L.N, L.J, L.signed_prod != 0, f_signed != 0, st);
    }

    Conv1dParams kp;
    kp.f = d_f; kp.g = d_g; kp.y = d_y; kp.len = (long long)len; kp.n_out = n_out;
    const long long n_blocks = (n_out + L.N - 1) / L.N;
    kp.n_chunks = (n_blocks + 31) / 32;
    kp.K = K; kp.S = L.S; kp.J = L.J; kp.Kc = L.Kc; kp.hi_shift = L.S * L.N;
    kp.g_signed = g_signed ? 1 : 0;
    kp.y_aligned16 = y_aligned16;
    kp.mask = sc.slot_mask;
    kp.bias = sc.bias;
    for (int m = 0; m < kMaxN1D; ++m) {
        kp.seg_shift[m] = m < L.N ? L.S * m : 0;
        kp.carry_bias[m] = m < L.N ? sc.carry_bias[m] : 0;
    }
    // long runs amortise the one seeding chunk per warp; short problems spread over the SMs first
    long long cpw = tune && tune->tile > 0 ? tune->tile : 16;
    int sms = 148;
    {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    const long long want_warps = (long long)sms * kWarps1D * 4;
    if (kp.n_chunks / cpw < want_warps) cpw = kp.n_chunks / want_warps;
    if (cpw < 1) cpw = 1;
    kp.chunks_per_warp = (int)cpw;
    const long long warps = (kp.n_chunks + cpw - 1) / cpw;
    const long long grid = (warps + kWarps1D - 1) / kWarps1D;
    if (grid > 0x7FFFFFFFLL) return HIKONV_ERR_UNSUPPORTED;
    return launch_packed(L.N, kp, L.signed_prod != 0, f_signed != 0, (unsigned)grid, st);
}

extern "C" int hikonv_conv1d_layout(int p, int q, int f_signed, int g_signed, int K, const hikonv_tuning_t *tune,
                                    hikonv_layout_t *out) {
    if (!out) return HIKONV_ERR_INVALID_ARG;
    int slot_bytes = 0;
    return layout_for_byte_input(p, q, f_signed, g_signed, K, tune, out, &slot_bytes);
}

extern "C" int hikonv_conv1d_dense(const uint8_t *d_f_dense, size_t len, const int8_t *d_g, int K, int p, int q, int f_signed,
                                   int g_signed, int32_t *d_y, const hikonv_tuning_t *tune, void *stream) {
    int rc = check_conv1d_args(d_f_dense, len, d_g, K, p, q, d_y, HIKONV_ALGO_PACKED32);
    if (rc != HIKONV_OK) return rc;
    if (p != 1 && p != 2 && p != 4) return HIKONV_ERR_UNSUPPORTED;      // codes must not straddle bytes
    hikonv_layout_t L;
    rc = make_layout(p, q, f_signed, g_signed, K, 1, 0, 0, tune, &L);
    if (rc != HIKONV_OK) return rc;
    if (!conv1d_packed_dense_available(p, L.N, L.J, L.S, L.signed_prod != 0, f_signed != 0)) return HIKONV_ERR_UNSUPPORTED;
    const SplitConsts sc = make_split_consts(L, p, q, f_signed, g_signed, K, 1);
    Conv1dTcParams tp;
    std::memset(&tp, 0, sizeof(tp));
    const long long n_out = (long long)len + K - 1;
    tp.f = reinterpret_cast<const int8_t *>(d_f_dense); tp.g = d_g; tp.y = d_y; tp.len = (long long)len; tp.n_out = n_out; tp.K = K;
    tp.g_signed = g_signed ? 1 : 0;
    tp.aligned = (((uintptr_t)d_y % 16 == 0) && ((uintptr_t)d_f_dense % 4 == 0)) ? 1 : 0;
    tp.dense_words = (long long)(((unsigned long long)len * (unsigned)p + 7) / 8 / 4);
    const int per_tile = conv1d_tc_outputs_per_tile(L.N);
    tp.n_tiles = (n_out + per_tile - 1) / per_tile;
    tp.S = L.S; tp.Kc = L.Kc; tp.hi_shift = L.S * L.N; tp.mask = sc.slot_mask; tp.bias = sc.bias;
    for (int m = 0; m < kMaxN1D; ++m) {
        tp.seg_shift[m] = m < L.N ? L.S * m : 0;
        tp.carry_bias[m] = m < L.N ? sc.carry_bias[m] : 0;
    }
    return launch_conv1d_packed_dense(tp, p, L.N, L.J, L.signed_prod != 0, f_signed != 0, (cudaStream_t)stream);
}

extern "C" size_t hikonv_conv1d_host_workspace_bytes(size_t len, int K) {
    if (K < 1) return 0;
    return align_up(len, 256) + align_up((size_t)K, 256) + align_up((len + (size_t)K - 1) * sizeof(int32_t), 256);
}

extern "C" int hikonv_conv1d_host(const int8_t *h_f, size_t len, const int8_t *h_g, int K, int p, int q, int f_signed,
                                  int g_signed, int32_t *h_y, void *d_workspace, size_t workspace_bytes, int algo,
                                  const hikonv_tuning_t *tune, void *stream) {
    if (!h_f || !h_g || !h_y || len < 1 || K < 1 || K > kMaxK) return HIKONV_ERR_INVALID_ARG;
    if (!d_workspace || ((uintptr_t)d_workspace % 256) != 0 || workspace_bytes < hikonv_conv1d_host_workspace_bytes(len, K))
        return HIKONV_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    int8_t *d_f = (int8_t *)d_workspace;
    int8_t *d_g = d_f + align_up(len, 256);
    int32_t *d_y = (int32_t *)(d_g + align_up((size_t)K, 256));
    HIKONV_CUDA_TRY(cudaMemcpyAsync(d_f, h_f, len, cudaMemcpyHostToDevice, st));
    HIKONV_CUDA_TRY(cudaMemcpyAsync(d_g, h_g, (size_t)K, cudaMemcpyHostToDevice, st));
    const int rc = hikonv_conv1d(d_f, len, d_g, K, p, q, f_signed, g_signed, d_y, algo, tune, st);
    if (rc != HIKONV_OK) return rc;
    HIKONV_CUDA_TRY(cudaMemcpyAsync(h_y, d_y, (len + (size_t)K - 1) * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    return HIKONV_OK;
}

extern "C" double hikonv_conv1d_multiplies(size_t len, int K, int p, int q, int f_signed, int g_signed, int algo,
                                           const hikonv_tuning_t *tune) {
    if (len < 1 || K < 1) return 0.0;
    const double n_out = (double)len + K - 1;
    if (algo == HIKONV_ALGO_UNPACKED_IMAD) return n_out * K;
    if (algo == HIKONV_ALGO_DP4A) return n_out * ((K + 3) / 4);
    hikonv_layout_t L;
    if (algo == HIKONV_ALGO_PACKED64EMU) {
        if (make_layout_emu64(p, q, f_signed, g_signed, K, tune, &L) != HIKONV_OK) return 0.0;
    } else {
        int slot_bytes = 0;
        if (layout_for_byte_input(p, q, f_signed, g_signed, K, tune, &L, &slot_bytes) != HIKONV_OK) return 0.0;
    }
    const double blocks = (double)(((long long)n_out + L.N - 1) / L.N);
    return blocks * L.J;
}
