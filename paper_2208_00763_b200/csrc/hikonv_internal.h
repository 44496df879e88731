// Internal declarations shared by the translation units of the library (not installed).
#pragma once

#include <cstddef>
#include <cstdint>

#include "hikonv.h"

namespace hikonv {

constexpr int kMaxN1D = 12;     // largest N the 1-D kernels are instantiated for
constexpr int kMaxN2D = 4;      // largest N the 2-D kernels are instantiated for
constexpr int kMaxNEmu64 = 16;  // largest N the emulated 64x64 1-D kernel is instantiated for
constexpr int kMaxSegments = 24;
constexpr int kMaxK = 64;       // longest kernel accepted
constexpr int kMaxJ = 16;       // most weight chunks per kernel row

// Constants of the biased split.  Every slot m of the 64-bit accumulator starts at
// seg_bias[m] = -(smallest sum the slot can receive), so every stored field is non-negative and
// slots never borrow from each other; the bias is subtracted after extraction.
struct SplitConsts {
    uint64_t bias;                      // sum_m seg_bias[m] 2^(S m): initial accumulator value
    int32_t seg_bias[kMaxSegments];     // per product slot
    int32_t carry_bias[kMaxSegments];   // slot m of (product + carry of the previous block), m < N
    uint32_t slot_mask;                 // 2^S - 1
    uint64_t mask_low;                  // the low h bits of every slot (h = carry_bits)
    uint64_t mask_high;                 // the remaining bits of every slot, moved down by h
};

// Cost-model constants for the 2-D planner, in scheduler cycles per warp instruction.
struct CostModel {
    double mul_cycles = 4.0;        // one 32x32->64 multiply-accumulate (half the rate of a 32-bit one)
    double carry_save_cycles = 10.0; // moving the upper slot bits to the second accumulator, per accumulator
};

// Constants of the biased split for the 128-bit product of the emulated 64x64 multiplier (1-D only).
struct SplitConsts128 {
    uint64_t bias_lo, bias_hi;          // sum_m seg_bias[m] 2^(S m), low and high halves
    int32_t carry_bias[kMaxSegments];   // slot m of (product + carry of the previous block), m < N
    uint32_t slot_mask;                 // 2^S - 1
};

int validate_codes(int p, int q);
// Exact-range layout search; `packed_overlap` selects the 1-D rule (block carries are added
// before the split, so a slot holds all K terms).
int make_layout(int p, int q, int f_signed, int g_signed, int K, int dims, int total_terms,
                int row_outputs, const hikonv_tuning_t *tune, hikonv_layout_t *out);
// Layout for 64-bit operands and a 128-bit product (1-D rule); fields as in hikonv_layout_t with
// 64 / 128 in place of 32 / 64.
int make_layout_emu64(int p, int q, int f_signed, int g_signed, int K, const hikonv_tuning_t *tune, hikonv_layout_t *out);
// 1-D layout with register-aligned slots, the narrowest that holds every sum of K products: returns the kernel
// mode (1: S = 8, N = 4; 2: S = 16, N = 2; 3: S = 17 .. 21, N = 2) and fills `out`, or returns 0 when none applies
// (K > 8, an operand that does not fit its register, sums beyond 21 bits).
int make_layout_byte_slots(int p, int q, int f_signed, int g_signed, int K, hikonv_layout_t *out);
SplitConsts128 make_split_consts128(const hikonv_layout_t &L, int p, int q, int f_signed, int g_signed, int K);
SplitConsts make_split_consts(const hikonv_layout_t &L, int p, int q, int f_signed, int g_signed, int K, int M);

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Words per packed kernel row in the 2-D kernels' shared memory, and the cap on channels per stage that
// keeps one staged weight tile within 24 KB (two of them and the activation tiles share 72 KB).
constexpr int kBPitch = 64;
inline int stage_channel_cap(int K, int J) {
    const int c = 6144 / (K * J * kBPitch);
    return c < 1 ? 1 : (c > 8 ? 8 : c);
}

// 2-D kernels stage CK input channels at a time and move the upper slot bits to the second
// accumulator every `fc` stages.  Given the number of channels CF that may be accumulated between two
// such moves, picks CK <= ck_cap and fc with CK * fc <= CF as large as possible (stages of fewer than
// three channels are avoided when something close is available).  Returns CK * fc.
inline int pick_chunking(int CF, int Ci, int *CK, int *fc, int ck_cap = 8) {
    if (CF >= Ci) {
        *CK = Ci < ck_cap ? Ci : ck_cap;
        *fc = 1 << 30;
        return Ci;
    }
    int best = 0;
    double best_score = -1.0;
    for (int ck = (CF < ck_cap ? CF : ck_cap); ck >= 1; --ck) {
        const int f = CF / ck, eff = ck * f;
        const double score = ck >= 3 ? eff : 0.7 * eff;
        if (score > best_score) {
            best_score = score;
            best = eff;
            *CK = ck;
            *fc = f;
        }
    }
    return best;
}
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace hikonv
