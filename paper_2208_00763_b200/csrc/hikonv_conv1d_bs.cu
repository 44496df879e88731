// 1-D packed kernels with register-aligned slots.
//
// The 1-D path is bound by HBM, so what counts is instructions per output, not outputs per multiply.  When the
// slot width is a whole number of bytes and N S = 32 (MODE 1: S = 8, N = 4; MODE 2: S = 16, N = 2),
//   - a loaded 32-bit word of one-byte codes IS the packed operand A of Eq. 5 (S = 8), or becomes one with a
//     single byte permute (S = 16);
//   - the slots above the N low ones of a product are exactly its high register, so the overlap-add of
//     Theorem 2 is one 32-bit add of the previous product's high half to this product's low half;
//   - every output is one byte permute of that sum (zero- or sign-extending), in place of shift and mask.
// Sums that need 17 to 21 bits (8-bit codes, unsigned 7-bit codes with K >= 5) take MODE 3: N = 2, Kc = 2 with
// the slot width S as a run-time value.  There the carry of block x-1 (slot 2 of its sum) enters block x as
// the start value of its multiply-add chain, so no separate 64-bit add is needed, and the outputs are read with
// one mask and one funnel shift plus mask.
//
// Signed codes are handled without Eq. 29's per-slot increment: the stored codes are lifted to non-negative
// values with one logic operation per loaded word (f + c per slot), the constant c sum_j B_j that this adds to
// every product is taken out of the chain's start value (exact in 64 bits), and the start value also holds a
// bias per slot (2^(S-1) per output slot in total) so that every field of the sum is non-negative and no slot
// borrows from its neighbour.  MODE 1, 2: one exclusive-or per word turns the fields into two's complement and
// the permute sign-extends them; MODE 3: the bias is subtracted after the mask.
//   MODE 1: S = 8,  N = 4, Kc = 4 taps per kernel word B_j, J = ceil(K / 4)   (1- and 2-bit codes, most 3-bit)
//   MODE 2: S = 16, N = 2, Kc = 2, J = ceil(K / 2)                            (4- to 6-bit codes, most 7-bit)
//   MODE 3: S = 17 .. 21, N = 2, Kc = 2, J = ceil(K / 2)                      (8-bit codes)
// Launch shape, loads, staging and stores are those of the other register-resident 1-D kernels.
#include "hikonv_conv1d_bs.h"
#include "hikonv_conv1d_run.cuh"

namespace hikonv {

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

// MODE 1 (S = 8): the N = 4 outputs of every block x = 0 .. R-1 from the loaded words.
template <int J, bool FS, bool SP, int L, int NW>
__device__ __forceinline__ void compute_s8(const Conv1dBsParams &p, const uint32_t (&Bw)[J], uint64_t init, const uint32_t (&w)[NW],
                                           int32_t (&out)[L]) {
    constexpr int R = L / 4, HW = J;
    constexpr uint32_t BIAS = SP ? 0x80808080u : 0u;
    // A_x = word HW + x (x = -J .. R-1); signed codes lifted to f + 2^(p-1) per byte
    uint32_t a[NW];
#pragma unroll
    for (int i = 0; i < NW; ++i) a[i] = FS ? ((w[i] ^ p.code_xor) & p.code_and) : w[i];
    uint32_t carry = 0;
#pragma unroll
    for (int x = -1; x < R; ++x) {
        uint64_t Q = init;
#pragma unroll
        for (int j = 0; j < J; ++j) Q = mul_wide_add<SP>(a[HW + x - j], Bw[j], Q);      // Eq. 9 over the kernel words
        if (x >= 0) {
            uint32_t D = (uint32_t)Q + carry;                                       // Theorem 2: + slots N.. of block x-1
            if (SP) D ^= BIAS;
#pragma unroll
            for (int m = 0; m < 4; ++m)
                out[4 * x + m] = (int32_t)prmt(D, 0u, SP ? (uint32_t)(m | ((8 | m) * 0x1110)) : (uint32_t)(m | 0x4440));
        }
        carry = (uint32_t)(Q >> 32);
    }
}

// MODE 2 (S = 16) and MODE 3 (S = 17 .. 21): N = 2, the two outputs of every block x = 0 .. R-1.
template <int MODE, int J, bool FS, bool SP, int L, int NW>
__device__ __forceinline__ void compute_n2(int S, uint32_t mask3, int32_t half3, const uint32_t (&Bw)[J], uint64_t init,
                                           const uint32_t (&w)[NW], int32_t (&out)[L]) {
    constexpr int R = L / 2, HW = (2 * J + 3) / 4, FRONT = 4 * HW;
    constexpr uint32_t BIAS = SP ? 0x80008000u : 0u;
    uint32_t s[NW];
#pragma unroll
    for (int i = 0; i < NW; ++i) s[i] = FS ? (w[i] ^ 0x80808080u) : w[i];      // signed codes lifted to f + 128
    // A_x = code(2x) + code(2x+1) 2^S, x = -J .. R-1 at index x + J
    uint32_t A[R + J];
#pragma unroll
    for (int x = -J; x < R; ++x) {
        const int pos = FRONT + 2 * x;
        if constexpr (MODE == 2) {
            A[x + J] = prmt(s[pos / 4], 0u, pos % 4 == 0 ? 0x4140u : 0x4342u);
        } else {
            const uint32_t c0 = prmt(s[pos / 4], 0u, pos % 4 == 0 ? 0x4440u : 0x4442u);
            const uint32_t c1 = prmt(s[pos / 4], 0u, pos % 4 == 0 ? 0x4441u : 0x4443u);
            A[x + J] = c0 + (c1 << S);
        }
    }
    uint32_t carry = 0;
    if constexpr (MODE == 2) {
#pragma unroll
        for (int x = -1; x < R; ++x) {
            uint64_t Q = init;
#pragma unroll
            for (int j = 0; j < J; ++j) Q = mul_wide_add<SP>(A[x - j + J], Bw[j], Q);
            if (x >= 0) {
                uint32_t D = (uint32_t)Q + carry;
                if (SP) D ^= BIAS;
                out[2 * x] = (int32_t)prmt(D, 0u, SP ? 0x9910u : 0x4410u);
                out[2 * x + 1] = (int32_t)prmt(D, 0u, SP ? 0xBB32u : 0x4432u);
            }
            carry = (uint32_t)(Q >> 32);
        }
    } else {
        // D_x = start + c_{x-1} + sum_j A_{x-j} B_j with c_{x-1} = slot 2 of D_{x-1}: adding c (below 2^S, into a slot
        // that has room for it) never carries out of slot 0, so slot 2 of D_x is that of the bare product sum
#pragma unroll
        for (int x = -1; x < R; ++x) {
            uint64_t D = init + (uint64_t)carry;
#pragma unroll
            for (int j = 0; j < J; ++j) D = mul_wide_add<SP>(A[x - j + J], Bw[j], D);
            if (x >= 0) {
                out[2 * x] = (int32_t)((uint32_t)D & mask3) - half3;
                out[2 * x + 1] = (int32_t)((uint32_t)(D >> S) & mask3) - half3;
            }
            carry = (uint32_t)(D >> 32) >> (2 * S - 32);
        }
    }
}

// MODE: see above.  J: words B_j per kernel.  FS: f is signed.  SP: signed product (f or g signed).
// L: outputs per lane and tile.  MINB: resident CTAs per SM the register budget is cut for.
template <int MODE, int J, bool FS, bool SP, int L, int MINB>
__global__ void __launch_bounds__(kThreadsTc, MINB) conv1d_bs_kernel(const Conv1dBsParams p) {
    static_assert(!FS || SP, "a signed operand makes the product signed");
    constexpr int N = MODE == 1 ? 4 : 2;
    constexpr int HW = (J * N + 3) / 4;          // words in front of the run: the J blocks its first products read
    constexpr int NW = HW + L / 4;
    const int S = MODE == 1 ? 8 : MODE == 2 ? 16 : p.S;
    __shared__ __align__(16) int32_t s_stage[kWarpsTc][32 * stage_pitch(L)];

    // kernel words B_j (Eq. 5 on g), built by every lane from warp-uniform loads
    uint32_t Bw[J];
#pragma unroll
    for (int j = 0; j < J; ++j) {
        uint32_t b = 0;
#pragma unroll
        for (int k = 0; k < N; ++k) {
            const int idx = j * N + k;
            if (idx < p.K) {
                const int8_t raw = __ldg(p.g + idx);
                const int32_t v = p.g_signed ? (int32_t)raw : (int32_t)(uint8_t)raw;
                b += (uint32_t)v << (S * k);
            }
        }
        Bw[j] = b;
    }
    // start value of every product chain: the slot biases (MODE 1, 2: 2^(S-1) in every output slot of the low half),
    // minus what the lifted codes add (A' = A + CA in every word)
    uint64_t init = !SP ? 0ull : MODE == 1 ? 0x80808080ull : MODE == 2 ? 0x80008000ull : p.bias3;
    if (FS) {
        const uint32_t CA = MODE == 1 ? p.code_xor : MODE == 2 ? 0x00800080u : (0x80u + (0x80u << S));
#pragma unroll
        for (int j = 0; j < J; ++j) init -= (uint64_t)((int64_t)CA * (int64_t)(int32_t)Bw[j]);
    }
    const uint32_t mask3 = MODE == 3 ? p.mask3 : 0u;
    const int32_t half3 = (MODE == 3 && SP) ? (int32_t)(1u << (S - 1)) : 0;

    walk_tiles<L, HW>(p.f, p.y, p.len, p.n_out, p.n_tiles, p.fast_after_first, s_stage[threadIdx.x >> 5],
                      [&](const uint32_t (&w)[NW], int32_t (&out)[L]) {
        if constexpr (MODE == 1) compute_s8<J, FS, SP, L, NW>(p, Bw, init, w, out);
        else compute_n2<MODE, J, FS, SP, L, NW>(S, mask3, half3, Bw, init, w, out);
    });
}

template <int MODE, int J, int L, int MINB>
static int launch_bs_sign(const Conv1dBsParams &p, bool fs, bool sp, cudaStream_t st) {
    if (fs) return launch_persistent(conv1d_bs_kernel<MODE, J, true, true, L, MINB>, p, st);
    if (sp) return launch_persistent(conv1d_bs_kernel<MODE, J, false, true, L, MINB>, p, st);
    return launch_persistent(conv1d_bs_kernel<MODE, J, false, false, L, MINB>, p, st);
}

int launch_conv1d_bs(const Conv1dBsParams &p, int mode, int J, bool fs, bool sp, int variant, cudaStream_t st) {
    // Measured over the 48 sweep cases at 2^24 codes: kernels with one or two kernel words per block fit the
    // register budget of five resident CTAs per SM and stream 2-3 % faster with them; with three or four words
    // that budget spills, and four CTAs are faster.
    const bool five = variant == 25 || (variant != 24 && (mode == 1 || J <= 2));
#define HK_BS(m, j)                                                                          \
    if (mode == m && J == j) {                                                               \
        if (five) return launch_bs_sign<m, j, 24, 5>(p, fs, sp, st);                        \
        return launch_bs_sign<m, j, 24, 4>(p, fs, sp, st);                                  \
    }
    HK_BS(1, 1) HK_BS(1, 2)
    HK_BS(2, 1) HK_BS(2, 2) HK_BS(2, 3) HK_BS(2, 4)
    HK_BS(3, 1) HK_BS(3, 2) HK_BS(3, 3) HK_BS(3, 4)
#undef HK_BS
    return HIKONV_ERR_UNSUPPORTED;
}

}  // namespace hikonv
