// Host-side planning: the paper's throughput search (Algorithm 1) and the exact-range layout
// the CUDA kernels run with.
#include <algorithm>
#include <cstring>
#include <mutex>
#include <vector>

#include "hikonv_internal.h"

namespace hikonv {

typedef __int128 i128;

static int ceil_log2(long long v) {
    int b = 0;
    while ((1LL << b) < v) ++b;
    return b;
}

// Eq. 11, the 1-D rule and the DNN rule.
static int guard_bits(int mode, int N, int K, int M) {
    switch (mode) {
        case HIKONV_GB_SINGLE: return ceil_log2(std::min(K, N));
        case HIKONV_GB_1D: return ceil_log2(K);
        case HIKONV_GB_DNN: return ceil_log2((long long)M * std::min(K, N));
        default: return -1;
    }
}

// Eq. 6.
static int slice_bits(int p, int q, int Gb) {
    if (p == 1) return q + Gb;
    if (q == 1) return p + Gb;
    return p + q + Gb;
}

int validate_codes(int p, int q) {
    if (p < 1 || p > 8 || q < 1 || q > 8) return HIKONV_ERR_INVALID_ARG;
    return HIKONV_OK;
}

struct Range {
    long long lo, hi;
};

static Range code_range(int bits, int is_signed) {
    if (is_signed) return {-(1LL << (bits - 1)), (1LL << (bits - 1)) - 1};
    return {0, (1LL << bits) - 1};
}

// Largest and smallest value of sum_{n<count} v 2^(S n) over codes v in r.
static void packed_range(Range r, int count, int S, i128 *lo, i128 *hi) {
    i128 geo = 0;
    for (int n = 0; n < count; ++n) geo += (i128)1 << (S * n);
    *lo = (i128)r.lo * geo;
    *hi = (i128)r.hi * geo;
}

static bool operand_fits(Range r, int count, int S, bool signed_mul) {
    if ((long long)S * (count - 1) > 60) return false;
    i128 lo, hi;
    packed_range(r, count, S, &lo, &hi);
    if (signed_mul) return lo >= -((i128)1 << 31) && hi <= ((i128)1 << 31) - 1;
    return lo >= 0 && hi <= ((i128)1 << 32) - 1;
}

// Number of (n, k) pairs with n + k == m, 0 <= n < N, 0 <= k < kc.
static int pair_count(int m, int N, int kc) {
    int lo = std::max(0, m - kc + 1), hi = std::min(m, N - 1);
    return hi >= lo ? hi - lo + 1 : 0;
}

// Does a value range fit a w-bit slot once it is biased by -lo (so that the stored field is >= 0)?
static bool slot_fits(i128 lo, i128 hi, int w) {
    if (w < 1) return lo == 0 && hi == 0;
    if (w > 62) w = 62;
    return hi - lo <= ((i128)1 << w) - 1;
}

// Checks one candidate (N, S) and fills Kc, J, segments, top_bits and the largest M (capped).
// `packed_overlap`: the carry of block x-1 is added to block x's product before the split (1-D).
// `carry_save_total` > 0 selects the 2-D rule: after every M accumulated products the part of each
// slot above its low h bits is moved to a second packed accumulator, so a slot must hold
// (2^h - 1) + bias + M T pmax with the bias a multiple of 2^h, and the second accumulator must
// survive ceil(total / M) such moves (at most 2^h of them).
static bool check_candidate(int p, int q, int fs, int gs, int K, int N, int S, bool packed_overlap,
                            long long M_cap, long long carry_save_total, long long force_M, hikonv_layout_t *L) {
    if (S < 1 || S > 31 || N < 1) return false;
    const bool sp = fs || gs;
    const Range fr = code_range(p, fs), gr = code_range(q, gs);
    if (!operand_fits(fr, N, S, sp)) return false;
    // weights: one word if the whole kernel fits and its carry reaches only the next block,
    // else chunks of N taps (Theorem 2 applied to the kernel)
    int Kc, J;
    if (K <= N + 1 && operand_fits(gr, K, S, sp)) {
        Kc = K;
        J = 1;
    } else {
        Kc = N;
        J = ceil_div(K, N);
        if (!operand_fits(gr, Kc, S, sp)) return false;
    }
    if (J > kMaxJ) return false;
    const int NS = N + Kc - 1;
    if (NS > kMaxSegments) return false;
    if ((long long)S * (NS - 1) >= 64) return false;
    const int top_bits = std::min(S, 64 - S * (NS - 1));
    const long long prods[4] = {fr.lo * gr.lo, fr.lo * gr.hi, fr.hi * gr.lo, fr.hi * gr.hi};
    const long long pmin = *std::min_element(prods, prods + 4), pmax = *std::max_element(prods, prods + 4);
    // term counts per slot
    int T[kMaxSegments] = {0};
    for (int j = 0; j < J; ++j) {
        const int kc = std::min(Kc, K - j * Kc);
        for (int m = 0; m < NS; ++m) T[m] += pair_count(m, N, kc);
    }
    auto fits_with = [&](long long M) {
        for (int m = 0; m < NS; ++m) {
            const int w = (m == NS - 1) ? top_bits : S;
            if (!slot_fits((i128)M * T[m] * pmin, (i128)M * T[m] * pmax, w)) return false;
        }
        if (packed_overlap) {
            for (int m = 0; m < N; ++m) {
                const int t = T[m] + (m + N < NS ? T[m + N] : 0);
                if (!slot_fits((i128)M * t * pmin, (i128)M * t * pmax, S)) return false;
            }
        }
        return true;
    };
    long long lo = 1;
    int carry_bits = 0;
    if (carry_save_total > 0) {
        auto fits_cs = [&](long long M, int h) {
            for (int m = 0; m < NS; ++m) {
                const int w = (m == NS - 1) ? top_bits : S;
                if (h >= w) return false;
                const i128 unit = (i128)1 << h;
                i128 bias = (i128)M * T[m] * (-pmin);
                bias = (bias + unit - 1) / unit * unit;
                const i128 low = (h > 0 && M < carry_save_total) ? unit - 1 : 0;
                if (low + bias + (i128)M * T[m] * pmax > ((i128)1 << w) - 1) return false;
            }
            return true;
        };
        long long bestM = 0;
        for (int h = 0; h < S; ++h) {
            long long a = 1, b = force_M > 0 ? force_M : std::max(1LL, M_cap);
            if (force_M > 0) a = force_M;
            if (!fits_cs(a, h)) continue;
            while (a < b) {
                const long long mid = (a + b + 1) / 2;
                if (fits_cs(mid, h)) a = mid; else b = mid - 1;
            }
            if (a < carry_save_total) {
                // the kernel moves bits at channel-stage borders: whole channels, in the staging it can realise
                const int Ci = (int)(carry_save_total / K);
                if (a < K) continue;
                int ck, fc;
                const int eff = pick_chunking((int)(a / K), Ci, &ck, &fc, stage_channel_cap(K, J));
                if (ceil_div(Ci, eff) > (1LL << h)) continue;
                a = (long long)eff * K;
            }
            if (a > bestM) { bestM = a; carry_bits = h; }
        }
        if (bestM < 1) return false;
        lo = bestM;
    } else {
        if (!fits_with(1)) return false;
        long long hi = std::max(1LL, M_cap);           // largest M in [1, M_cap] that fits (monotone)
        while (lo < hi) {
            const long long mid = (lo + hi + 1) / 2;
            if (fits_with(mid)) lo = mid; else hi = mid - 1;
        }
    }
    L->N = N;
    L->S = S;
    L->Kc = Kc;
    L->J = J;
    L->segments = NS;
    L->top_bits = top_bits;
    L->M = (int)lo;
    L->signed_prod = sp ? 1 : 0;
    L->carry_bits = carry_bits;
    return true;
}

static int search_layout(int p, int q, int fs, int gs, int K, int dims, int total_terms, int row_outputs,
                         const hikonv_tuning_t *tune, hikonv_layout_t *out) {
    if (validate_codes(p, q) != HIKONV_OK || K < 1 || K > kMaxK || !out || (dims != 1 && dims != 2))
        return HIKONV_ERR_INVALID_ARG;
    fs = fs ? 1 : 0;
    gs = gs ? 1 : 0;
    const int forceN = tune ? tune->N : 0, forceS = tune ? tune->S : 0, forceM = tune ? tune->M : 0;
    if (forceN < 0 || forceS < 0 || forceM < 0) return HIKONV_ERR_INVALID_ARG;
    std::memset(out, 0, sizeof(*out));
    hikonv_layout_t best;
    bool found = false;
    if (dims == 1) {
        // Theorem 2: Gb = ceil(log2 K); widen S until the exact ranges fit
        const int S_paper = slice_bits(p, q, guard_bits(HIKONV_GB_1D, 1, K, 1));
        const int maxN = forceN ? forceN : kMaxN1D;
        for (int S = forceS ? forceS : S_paper; S <= (forceS ? forceS : 31) && !found; ++S) {
            double best_rate = 0.0;
            for (int N = forceN ? forceN : 1; N <= maxN; ++N) {
                hikonv_layout_t c;
                if (!check_candidate(p, q, fs, gs, K, N, S, true, 1, 0, 0, &c)) continue;
                const double rate = (double)c.N / c.J;   // outputs per multiply
                if (rate > best_rate + 1e-9) {
                    best_rate = rate;
                    best = c;
                    found = true;
                }
            }
        }
        if (found) best.S_paper = S_paper;
    } else {
        if (total_terms < 1) return HIKONV_ERR_INVALID_ARG;
        const CostModel cm;
        double best_cost = 0.0;
        const int maxN = forceN ? forceN : kMaxN2D;
        const int wo = row_outputs > 0 ? row_outputs : 64;
        for (int N = forceN ? forceN : 1; N <= maxN; ++N) {
            // a wider slot allows more accumulations between two splits, but may push the kernel
            // row into several chunks: score every feasible (N, S)
            for (int S = forceS ? forceS : 31; S >= (forceS ? forceS : 1); --S) {
                hikonv_layout_t c;
                if (!check_candidate(p, q, fs, gs, K, N, S, false, total_terms, total_terms, forceM, &c)) continue;
                const double blocks = (double)(ceil_div(wo, N) + c.J);   // words per output row, halo included
                const double per_mul = cm.mul_cycles + cm.carry_save_cycles / (double)c.M;
                const double cost = blocks * c.J * per_mul / (double)wo; // cycles per output pixel and (ci, kh)
                if (!found || cost <= best_cost + 1e-12) {      // ties: the narrower slot
                    best_cost = cost;
                    best = c;
                    found = true;
                }
            }
        }
        if (found) {
            // reference value of the printed rule for the chosen N (DNN guard bits with the chosen M)
            best.S_paper = slice_bits(p, q, guard_bits(HIKONV_GB_DNN, best.N, std::min(K, best.Kc), best.M));
        }
    }
    if (!found) return HIKONV_ERR_NO_FIT;
    if (forceM && dims == 1) {
        if (forceM > best.M) return HIKONV_ERR_NO_FIT;
        best.M = forceM;
    }
    *out = best;
    return HIKONV_OK;
}

// ---- the 64x64 -> 128 multiplier (the paper's remark that wider multipliers are handled the same way) ----
// Same rules as the 1-D search above with 64-bit operands and a 128-bit product: both packed operands
// must fit a 64-bit register, the N + Kc - 1 slots must fit 128 bits, and every slot must hold the
// extreme sum it can receive once the carry of the previous block has been added (Theorem 2).
static bool operand_fits64(Range r, int count, int S, bool signed_mul) {
    if ((long long)S * (count - 1) > 63) return false;
    i128 lo, hi;
    packed_range(r, count, S, &lo, &hi);
    if (signed_mul) return lo >= -((i128)1 << 63) && hi <= ((i128)1 << 63) - 1;
    return lo >= 0 && hi <= ((i128)1 << 64) - 1;
}

static bool check_candidate_emu64(int p, int q, int fs, int gs, int K, int N, int S, hikonv_layout_t *L) {
    if (S < 1 || S > 31 || N < 1) return false;
    const bool sp = fs || gs;
    const Range fr = code_range(p, fs), gr = code_range(q, gs);
    if (!operand_fits64(fr, N, S, sp)) return false;
    int Kc, J;
    if (K <= N + 1 && operand_fits64(gr, K, S, sp)) {
        Kc = K;
        J = 1;
    } else {
        Kc = N;
        J = ceil_div(K, N);
        if (!operand_fits64(gr, Kc, S, sp)) return false;
    }
    if (J > kMaxJ) return false;
    const int NS = N + Kc - 1;
    if (NS > kMaxSegments) return false;
    if ((long long)S * (NS - 1) >= 128) return false;
    const int top_bits = std::min(S, 128 - S * (NS - 1));
    const long long prods[4] = {fr.lo * gr.lo, fr.lo * gr.hi, fr.hi * gr.lo, fr.hi * gr.hi};
    const long long pmin = *std::min_element(prods, prods + 4), pmax = *std::max_element(prods, prods + 4);
    int T[kMaxSegments] = {0};
    for (int j = 0; j < J; ++j) {
        const int kc = std::min(Kc, K - j * Kc);
        for (int m = 0; m < NS; ++m) T[m] += pair_count(m, N, kc);
    }
    for (int m = 0; m < NS; ++m) {
        const int w = (m == NS - 1) ? top_bits : S;
        if (!slot_fits((i128)T[m] * pmin, (i128)T[m] * pmax, w)) return false;
    }
    for (int m = 0; m < N; ++m) {       // after the carry of the previous block has been added
        const int t = T[m] + (m + N < NS ? T[m + N] : 0);
        if (!slot_fits((i128)t * pmin, (i128)t * pmax, S)) return false;
    }
    L->N = N;
    L->S = S;
    L->Kc = Kc;
    L->J = J;
    L->segments = NS;
    L->top_bits = top_bits;
    L->M = 1;
    L->signed_prod = sp ? 1 : 0;
    L->carry_bits = 0;
    return true;
}

int make_layout_emu64(int p, int q, int fs, int gs, int K, const hikonv_tuning_t *tune, hikonv_layout_t *out) {
    if (validate_codes(p, q) != HIKONV_OK || K < 1 || K > kMaxK || !out) return HIKONV_ERR_INVALID_ARG;
    fs = fs ? 1 : 0;
    gs = gs ? 1 : 0;
    const int forceN = tune ? tune->N : 0, forceS = tune ? tune->S : 0;
    if (forceN < 0 || forceS < 0) return HIKONV_ERR_INVALID_ARG;
    std::memset(out, 0, sizeof(*out));
    const int S_paper = slice_bits(p, q, guard_bits(HIKONV_GB_1D, 1, K, 1));
    hikonv_layout_t best;
    bool found = false;
    for (int S = forceS ? forceS : S_paper; S <= (forceS ? forceS : 31) && !found; ++S) {
        double best_rate = 0.0;
        for (int N = forceN ? forceN : 1; N <= (forceN ? forceN : kMaxNEmu64); ++N) {
            hikonv_layout_t c;
            if (!check_candidate_emu64(p, q, fs, gs, K, N, S, &c)) continue;
            const double rate = (double)c.N / c.J;      // outputs per 64x64 multiply
            if (rate > best_rate + 1e-9) {
                best_rate = rate;
                best = c;
                found = true;
            }
        }
    }
    if (!found) return HIKONV_ERR_NO_FIT;
    best.S_paper = S_paper;
    *out = best;
    return HIKONV_OK;
}

// Register-aligned slots for the 1-D kernels.  Mode 1: S = 8, N = 4, four taps per kernel word; mode 2: S = 16,
// N = 2, two taps; mode 3: the narrowest S in 17 .. 21 with N = 2, two taps.  The conditions are those of the
// exact-range rule above, specialised: both operands fit a 32-bit register (31 bits plus sign for a signed
// multiply; signed codes enter the multiplier lifted to non-negative values -- by 2^(p-1) in mode 1, by 128 in
// modes 2 and 3 -- so only their lifted width counts), the N + Kc - 1 slots fit 64 bits, and every output, a sum
// of at most K products, fits its S-bit slot: as an unsigned value, or as a two's-complement one when either
// operand is signed (modes 1 and 2 read signed slots with a sign-extending permute, mode 3 subtracts 2^(S-1)).
int make_layout_byte_slots(int p, int q, int fs, int gs, int K, hikonv_layout_t *out) {
    if (validate_codes(p, q) != HIKONV_OK || K < 1 || K > 8) return 0;
    fs = fs ? 1 : 0;
    gs = gs ? 1 : 0;
    const bool sp = fs || gs;
    const Range fr = code_range(p, fs), gr = code_range(q, gs);
    const long long prods[4] = {fr.lo * gr.lo, fr.lo * gr.hi, fr.hi * gr.lo, fr.hi * gr.hi};
    const long long pmin = *std::min_element(prods, prods + 4), pmax = *std::max_element(prods, prods + 4);
    const long long lo = (long long)K * pmin, hi = (long long)K * pmax;
    for (int S = 8; S <= 21; S = (S == 8 ? 16 : S + 1)) {
        const int mode = S == 8 ? 1 : S == 16 ? 2 : 3;
        const int N = mode == 1 ? 4 : 2;
        const int Kc = std::min(K, N), J = ceil_div(K, Kc);
        const Range lifted = {0, (mode == 1 || !fs) ? (1LL << p) - 1 : 255};
        if (!operand_fits(lifted, N, S, sp)) continue;
        if (!operand_fits(gr, Kc, S, sp)) continue;
        if (S * (N + Kc - 1) > 63) continue;
        if (sp ? (lo < -(1LL << (S - 1)) || hi > (1LL << (S - 1)) - 1) : (hi > (1LL << S) - 1)) continue;
        if (out) {
            std::memset(out, 0, sizeof(*out));
            out->N = N;
            out->S = S;
            out->Kc = Kc;
            out->J = J;
            out->segments = N + Kc - 1;
            out->top_bits = std::min(S, 64 - S * (N + Kc - 2));
            out->M = 1;
            out->signed_prod = sp ? 1 : 0;
            out->S_paper = slice_bits(p, q, guard_bits(HIKONV_GB_1D, 1, K, 1));
            out->carry_bits = 0;
        }
        return mode;
    }
    return 0;
}

SplitConsts128 make_split_consts128(const hikonv_layout_t &L, int p, int q, int fs, int gs, int K) {
    SplitConsts128 c;
    std::memset(&c, 0, sizeof(c));
    c.slot_mask = (1u << L.S) - 1u;
    const Range fr = code_range(p, fs ? 1 : 0), gr = code_range(q, gs ? 1 : 0);
    const long long prods[4] = {fr.lo * gr.lo, fr.lo * gr.hi, fr.hi * gr.lo, fr.hi * gr.hi};
    const long long pmin = *std::min_element(prods, prods + 4);
    int T[kMaxSegments] = {0};
    for (int j = 0; j < L.J; ++j) {
        const int kc = std::min(L.Kc, K - j * L.Kc);
        for (int m = 0; m < L.segments; ++m) T[m] += pair_count(m, L.N, kc);
    }
    int32_t seg_bias[kMaxSegments];
    unsigned __int128 bias = 0;
    for (int m = 0; m < L.segments; ++m) {
        seg_bias[m] = (int32_t)(-(long long)T[m] * pmin);     // >= 0: lifts the most negative sum to 0
        bias += (unsigned __int128)(uint32_t)seg_bias[m] << (L.S * m);
    }
    c.bias_lo = (uint64_t)bias;
    c.bias_hi = (uint64_t)(bias >> 64);
    for (int m = 0; m < L.N; ++m)
        c.carry_bias[m] = seg_bias[m] + (m + L.N < L.segments ? seg_bias[m + L.N] : 0);
    return c;
}

// The search above costs about a hundred microseconds of host time, as much as a layer takes on the
// device, and its result depends on its arguments alone: keep the most recent results.
namespace {
struct LayoutKey {
    int v[11];
    bool operator==(const LayoutKey &o) const { return std::memcmp(v, o.v, sizeof(v)) == 0; }
};
struct LayoutEntry {
    LayoutKey key;
    int status;
    hikonv_layout_t layout;
};
constexpr size_t kLayoutCacheEntries = 128;
std::mutex g_layout_mutex;
std::vector<LayoutEntry> g_layout_cache;
size_t g_layout_next = 0;
}  // namespace

int make_layout(int p, int q, int fs, int gs, int K, int dims, int total_terms, int row_outputs,
                const hikonv_tuning_t *tune, hikonv_layout_t *out) {
    if (!out) return HIKONV_ERR_INVALID_ARG;
    LayoutKey key = {{p, q, fs ? 1 : 0, gs ? 1 : 0, K, dims, total_terms, row_outputs, tune ? tune->N : 0,
                      tune ? tune->S : 0, tune ? tune->M : 0}};
    {
        std::lock_guard<std::mutex> lock(g_layout_mutex);
        for (const LayoutEntry &e : g_layout_cache)
            if (e.key == key) {
                *out = e.layout;
                return e.status;
            }
    }
    LayoutEntry e;
    e.key = key;
    std::memset(&e.layout, 0, sizeof(e.layout));
    e.status = search_layout(p, q, fs, gs, K, dims, total_terms, row_outputs, tune, &e.layout);
    *out = e.layout;
    std::lock_guard<std::mutex> lock(g_layout_mutex);
    if (g_layout_cache.size() < kLayoutCacheEntries) g_layout_cache.push_back(e);
    else g_layout_cache[g_layout_next++ % kLayoutCacheEntries] = e;
    return e.status;
}

// Term counts per product slot for a layout: T[m] = number of code products that land in slot m
// of one accumulated product (all J chunks).
static void term_counts(const hikonv_layout_t &L, int K, int *T) {
    for (int m = 0; m < L.segments; ++m) T[m] = 0;
    for (int j = 0; j < L.J; ++j) {
        const int kc = std::min(L.Kc, K - j * L.Kc);
        for (int m = 0; m < L.segments; ++m) T[m] += pair_count(m, L.N, kc);
    }
}

SplitConsts make_split_consts(const hikonv_layout_t &L, int p, int q, int fs, int gs, int K, int M) {
    SplitConsts c;
    std::memset(&c, 0, sizeof(c));
    c.slot_mask = (L.S >= 32) ? 0xFFFFFFFFu : ((1u << L.S) - 1u);
    const Range fr = code_range(p, fs ? 1 : 0), gr = code_range(q, gs ? 1 : 0);
    const long long prods[4] = {fr.lo * gr.lo, fr.lo * gr.hi, fr.hi * gr.lo, fr.hi * gr.hi};
    const long long pmin = *std::min_element(prods, prods + 4);
    int T[kMaxSegments];
    term_counts(L, K, T);
    const int h = L.carry_bits;
    const long long unit = 1LL << h;
    for (int m = 0; m < L.segments; ++m) {
        long long b = -(long long)M * T[m] * pmin;            // >= 0: lifts the most negative sum to 0
        b = (b + unit - 1) / unit * unit;                     // a multiple of 2^h (2-D carry-save; h = 0 otherwise)
        const int w = (m == L.segments - 1) ? L.top_bits : L.S;
        c.seg_bias[m] = (int32_t)b;
        c.bias += (uint64_t)b << (L.S * m);
        c.mask_low += (uint64_t)(unit - 1) << (L.S * m);
        c.mask_high += (uint64_t)((1LL << (w - h)) - 1) << (L.S * m);
    }
    for (int m = 0; m < L.N; ++m)
        c.carry_bias[m] = c.seg_bias[m] + (m + L.N < L.segments ? c.seg_bias[m + L.N] : 0);
    return c;
}

}  // namespace hikonv

using namespace hikonv;

extern "C" int hikonv_plan(int p, int q, int LA, int LB, int mode, int M, int K_fixed, hikonv_plan_t *out) {
    if (!out || p < 1 || q < 1 || p > 32 || q > 32 || LA < 1 || LB < 1 || LA > 64 || LB > 64) return HIKONV_ERR_INVALID_ARG;
    if (mode != HIKONV_GB_SINGLE && mode != HIKONV_GB_1D && mode != HIKONV_GB_DNN) return HIKONV_ERR_INVALID_ARG;
    if (M < 1 || K_fixed < 0) return HIKONV_ERR_INVALID_ARG;
    hikonv_plan_t best = {0, 0, 0, 0, 0};
    const int k_lo = K_fixed ? K_fixed : 1, k_hi = K_fixed ? K_fixed : LB;
    for (int k = k_lo; k <= k_hi; ++k) {
        for (int n = 1; n <= LA; ++n) {
            const int Gb = guard_bits(mode, n, k, M);
            const int S = slice_bits(p, q, Gb);
            if (p + (long long)(n - 1) * S > LA) break;          // Eq. 7 (monotone in n up to the Gb steps)
            if (q + (long long)(k - 1) * S > LB) continue;       // Eq. 8
            const int ops = n * k + (n - 1) * (k - 1);           // Eq. 24
            if (ops > best.ops) best = {n, k, S, Gb, ops};
        }
    }
    if (best.ops == 0) return HIKONV_ERR_NO_FIT;
    *out = best;
    return HIKONV_OK;
}

extern "C" int hikonv_layout(int p, int q, int f_signed, int g_signed, int K, int dims, int total_terms,
                             const hikonv_tuning_t *tune, hikonv_layout_t *out) {
    return make_layout(p, q, f_signed, g_signed, K, dims, total_terms, 0, tune, out);
}

extern "C" int hikonv_layout_emu64(int p, int q, int f_signed, int g_signed, int K, const hikonv_tuning_t *tune,
                                   hikonv_layout_t *out) {
    return make_layout_emu64(p, q, f_signed, g_signed, K, tune, out);
}

extern "C" const char *hikonv_status_string(int status) {
    switch (status) {
        case HIKONV_OK: return "ok";
        case HIKONV_ERR_INVALID_ARG: return "invalid argument";
        case HIKONV_ERR_UNSUPPORTED: return "unsupported configuration";
        case HIKONV_ERR_NO_FIT: return "no packed layout fits the multiplier";
        case HIKONV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case HIKONV_ERR_CUDA: return "CUDA runtime error";
        case HIKONV_ERR_TOO_LARGE: return "layer needs more scratch than the built-in static buffer holds";
        case HIKONV_ERR_RANGE: return "a stored code lies outside its bit range";
        default: return "unknown status";
    }
}
