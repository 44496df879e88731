// hikonv_conv2d: a convolution layer as row-wise packed 1-D convolutions (Theorem 3), with the
// products of all input channels and kernel rows summed in the 64-bit packed accumulator before
// the split (Eq. 23), plus the one-product-per-multiply comparator on the same tiling.
//
// Work decomposition.  Output row R = (b, h) is cut into blocks of N pixels; block x and its J
// "halo" predecessors form the positions xb = x + J of the row.  For position (R, xb) and output
// channel co the kernel keeps
//     Q = bias + sum_{ci, kh, j} A[b][ci][h+kh][xb - j] * Bw[co][ci][kh][j]
// where A packs N neighbouring input pixels (Eq. 5) and Bw packs N (or all K) taps of the REVERSED
// kernel row (g = W[co][ci][kh][K-1:0], Theorem 3).  Slot m < N of Q holds partial sums of pixel
// xN + m, slot m >= N those of pixel (x+1)N + (m-N): the overlap-add of Theorem 2.
//
// Activations are packed once per layer by pack_operands_kernel into Ap[ci][b*Hp + hp][xb] (zero padding
// rows and halo words materialised), weights by the same launch into Bw[(ci,kh,j)][co]; the layer
// kernel streams both with 16-byte asynchronous copies into double-buffered shared memory.  Deep layers with
// unsigned activations and signed weights are packed as x - 2^(p-1), padding included, and get the constant
// 2^(p-1) sum(W[co]) back in the epilogue (make_setup says when and why).
//
// A CTA computes TR consecutive output rows (one row segment each) times TCO output channels; it
// is a register-tiled integer "GEMM" over packed words: each thread owns TM positions times TN
// channels (a warp's consecutive positions are dealt round-robin to its lanes), the k dimension runs
// over (ci, kh, j).
//
// Split.  Every slot starts at a bias that makes its running sum non-negative, so slots never borrow
// from each other (this replaces the sign-borrow increment of Eq. 29).  After at most M accumulated
// (ci, kh) pairs a slot would overflow; instead of splitting all slots into int32 sums there (the
// shift-and-mask of Algorithm 2, N + K - 1 extractions per accumulator), the kernel moves the bits of
// every slot above its low h bits into a SECOND packed accumulator with the same slot layout,
//     E += (Q >> h) & mask_high;      Q = (Q & mask_low) | bias;
// eight logic/shift/add instructions per accumulator whatever N is.  E can take 2^h such moves.  The
// slots are extracted once, at the end: slot m holds 2^h E_m + Q_m - (moves + 1) bias_m, the low N
// slots belong to this block and the upper ones are added to the next block of the row (Theorem 2).
#include <algorithm>
#include <cstring>
#include <mutex>
#include <type_traits>

#include "hikonv_cuda.cuh"

namespace hikonv {

constexpr int kMaxThreads2D = 256;
constexpr int kMaxN2DSeg = 8;      // N + Kc - 1 <= 2 N <= 8
constexpr int kCopyPieces = 4;     // 16-byte activation pieces per thread and stage whose offsets are kept in registers
constexpr int kEPitch = 17;        // 8-byte entries per thread in the second-accumulator area (16 used)

struct Conv2dParams {
    const int8_t *x;
    const uint32_t *ap;        // packed activations [Ci][B*Hp][XBT]
    const uint32_t *wp;        // packed weights [Ci*K*J][CoP]
    void *out;
    int B, Ci, H, W, Co, CoP, K, pad, Ho, Wo, Hp;
    int S, J, Kc, M;
    int X;                     // output blocks per row
    int XBT;                   // words per packed activation row (halo + blocks, rounded up so that every tile row can be read in 16-byte pieces)
    int NSEG, XO, XB;          // row segments, output blocks per segment (a multiple of 4 when NSEG > 1), positions per segment (XO + J)
    int XBS;                   // words per activation row in shared memory (XB rounded up to a multiple of 4)
    int TR, TMX, TNX, TCO, CK;
    int NRmax, a_plane, lead;  // staged rows per channel; words per channel in shared memory; words before the first row
    int a_words;               // words per activation tile (CK * a_plane)
    int b_off;                 // word offset of the first weight tile in shared memory
    int b_words;               // words per weight tile (CK * K * J rows of 64 words)
    int e_off;                 // word offset of the second accumulators in shared memory (after the tiles and the exchange area)
    int requant, shift, lo, hi;
    int total_rows;            // B * Ho
    int flush_chunks;          // channel stages accumulated between two carry-save moves (CK * K * flush_chunks <= M)
    int move_every;            // > 0: every accumulator row moves once per this many channels, at a fixed place of an unrolled group (CK a multiple of it)
    int hbits, nslots;         // carry-save: low bits kept per slot; number of slots N + Kc - 1
    uint64_t bias, mask_low, mask_high;
    uint32_t slot_mask, top_mask;
    int32_t slot_bias[kMaxN2DSeg];
    // requantised output: the CTA's codes are staged as bytes in shared memory ([channel][row][column], WTP bytes
    // per row) and leave in pieces of `vec` bytes along a row; with pool != 0 rows and columns are first reduced
    // by a 2x2 maximum (output [B][Co][Ho/2][Wo/2]; TR and Ho are even then)
    int stage_out;             // 1: staged (every requantised layer), 0: direct stores
    int tile_off;              // word offset of the byte tile in shared memory
    int WTP;                   // bytes per tile row (a multiple of 16)
    int vec;                   // bytes per output piece: 16, 8, 4 or 1
    int pool;                  // 2x2 max-pool fused into the copy-out
    int out_signed;            // pooled codes compare as signed bytes
    int out_bits;              // 8: one code per byte; 1 / 2 / 4: dense output, 8 / out_bits codes per byte (vec: 4 or 1 bytes)
    // multipliers of fast_div() for the divisors fixed per launch: XB, Ho, 16-byte pieces per activation row, CK, NSEG
    uint32_t mg_xb, mg_ho, mg_xq, mg_ck, mg_nseg;
    // unsigned activations run as signed ones: every packed code is x - x_off (also outside the image, where x = 0),
    // and corr[co] = x_off * (sum of all weights of channel co) is added back to every output (0: not used)
    int x_off;
    const int32_t *corr;
};

template <bool UNPACKED>
struct AccType {
    typedef uint64_t type;
};
template <>
struct AccType<true> {
    typedef int32_t type;
};

// n / d for 0 <= n < 2^22 and d > 0 with inv_d = 1.0f / d: the float quotient is off by at most one.
// (The per-thread index arithmetic of a tile would otherwise be some thirty integer divisions.)
__device__ __forceinline__ int small_div(int n, int d, float inv_d) {
    int q = (int)((float)n * inv_d);
    const int r = n - q * d;
    if (r < 0) --q;
    else if (r >= d) ++q;
    return q;
}

// n / d for 0 <= n < 2^16 and 0 < d < 2^16 with magic = ceil(2^32 / d) mod 2^32 (0 stands for d == 1): the high
// word of n * magic is the exact quotient because n (d - 1) < 2^32.
__device__ __forceinline__ int fast_div(int n, uint32_t magic) {
    return magic ? (int)__umulhi((uint32_t)n, magic) : n;
}

// n / d for any 32-bit n and a divisor d >= 1 fixed per launch (division by invariant integers using
// multiplication, Granlund and Montgomery 1994): with L = ceil(log2 d) and m = floor(2^32 (2^L - d) / d) + 1,
// t = mulhi(m, n) and n / d = (t + ((n - t) >> min(L, 1))) >> max(L - 1, 0).  Five instructions instead of the
// twenty-odd of a hardware-less 32-bit division.
struct Div32 {
    uint32_t m, s1, s2;
};
__host__ inline Div32 make_div32(uint32_t d) {
    uint32_t L = 0;
    while (L < 32 && (1ull << L) < d) ++L;
    Div32 r;
    r.m = (uint32_t)(((1ull << 32) * ((1ull << L) - d)) / d + 1);
    r.s1 = L < 1 ? L : 1;
    r.s2 = L > 1 ? L - 1 : 0;
    return r;
}
__device__ __forceinline__ uint32_t div32(uint32_t n, const Div32 &d) {
    const uint32_t t = __umulhi(d.m, n);
    return (t + ((n - t) >> d.s1)) >> d.s2;
}

// One multiply-accumulate of the k loop: the packed 32x32->64 product of Eq. 9 added to the 64-bit
// accumulator, or (comparator) one 32-bit product added to an int32 sum.
template <bool UNPACKED, bool SP>
__device__ __forceinline__ void mac(typename AccType<UNPACKED>::type &acc, uint32_t a, uint32_t b) {
    if constexpr (UNPACKED) {
        acc += (int32_t)a * (int32_t)b;
    } else if constexpr (SP) {
        acc += (uint64_t)((int64_t)(int32_t)a * (int64_t)(int32_t)b);
    } else {
        acc += (uint64_t)a * (uint64_t)b;
    }
}

// VEC input bytes of two rows per thread (VEC = 8: two 8-byte loads, one 4-byte store; VEC = 16: two
// 16-byte loads, one 8-byte store), per-byte maxima; needs W % VEC == 0 and VEC-byte aligned input,
// VEC/2-byte aligned output.
template <bool SIGNED>
__device__ __forceinline__ uint32_t pool_pairs(uint32_t a0, uint32_t a1, uint32_t b0, uint32_t b1) {
    uint32_t v0 = SIGNED ? __vmaxs4(a0, b0) : __vmaxu4(a0, b0);     // the two rows
    uint32_t v1 = SIGNED ? __vmaxs4(a1, b1) : __vmaxu4(a1, b1);
    v0 = SIGNED ? __vmaxs4(v0, v0 >> 8) : __vmaxu4(v0, v0 >> 8);    // bytes 0 and 2 hold the pair maxima
    v1 = SIGNED ? __vmaxs4(v1, v1 >> 8) : __vmaxu4(v1, v1 >> 8);
    return __byte_perm(v0, v1, 0x6420);
}

// N: pixels per packed word; SC: slot width when known at compile time (0: read from the parameters);
// TM x TN: per-thread tile (positions x channels); UNPACKED: comparator (N == 1, one tap per word,
// 32-bit multiply-add, int32 accumulators); SP: signed product;
// KT, JT: kernel size and chunks per kernel row when known at compile time (0, 0: read from the
// parameters; the (kh, j) loops are then not unrolled);
// PITCH: words per activation row in shared memory when known at compile time (then every operand load
// of the unrolled loops has an immediate offset), 0: read from the parameters.
// U > 0: the channel loop runs in unrolled groups of U channels in which accumulator row i does its
// carry-save move after channel (i U) / TM of the group, so that the moves of different rows sit between
// the multiplies of the others instead of forming one burst per stage (channels past Ci carry zero weights).
template <int N, int SC, int TM, int TN, bool UNPACKED, bool SP, int KT, int JT, int PITCH, int U>
__global__ void __launch_bounds__(kMaxThreads2D, 2) conv2d_kernel(const Conv2dParams p) {
    typedef typename AccType<UNPACKED>::type acc_t;
    extern __shared__ __align__(16) uint32_t smem[];
    grid_dependency_release();
    uint32_t *As = smem;                                   // two tiles [CK][a_plane]
    uint32_t *Bs = smem + p.b_off;                         // two tiles [CK*K*J][TCO]

    const int tid = threadIdx.x, nthreads = blockDim.x;
    const int tnx_log2 = 31 - __clz(p.TNX);                 // TNX is a power of two
    const int tn = tid & (p.TNX - 1);
    const int row_tile = p.NSEG > 1 ? (int)(blockIdx.x / (unsigned)p.NSEG) : (int)blockIdx.x;
    const int seg = blockIdx.x - row_tile * p.NSEG;
    const int R0 = row_tile * p.TR;
    const int co0 = blockIdx.y * p.TCO;
    const int TRe = min(p.TR, p.total_rows - R0);
    const int b0 = R0 / p.Ho, h0 = R0 - b0 * p.Ho;
    const int Rp0 = b0 * p.Hp + h0;                         // first staged padded row
    const int Rlast = R0 + TRe - 1;
    const int bl = b0 + fast_div(h0 + TRe - 1, p.mg_ho);
    const int NR = (bl * p.Hp + (Rlast - bl * p.Ho) + p.K - 1) - Rp0 + 1;
    const int TP = TRe * p.XB;                              // positions of this tile
    const int S = SC > 0 ? SC : p.S;

    // A warp owns 32 / TNX * TM consecutive positions, dealt round-robin to its 32 / TNX position lanes:
    // the lanes of one operand load then read consecutive words (no bank conflicts), and the block in
    // front of a lane's position sits in the lane before it.
    const int lane = tid & 31, warp = tid >> 5;
    const int lanes_m = 32 >> tnx_log2, lm = lane >> tnx_log2;
    const int wpos0 = warp * lanes_m * TM;
    // this thread's positions: shared-memory address of the packed word for (ci = 0, kh = 0, j = 0)
    const uint32_t *aptr[TM];
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        // an idle position (past the tile) reads the words of position 0; its result is dropped
        const int pos = wpos0 + i * lanes_m + lm, pc = pos < TP ? pos : 0;
        const int r = fast_div(pc, p.mg_xb), xb = pc - r * p.XB;
        const int db = fast_div(h0 + r, p.mg_ho);                    // images past the tile's first one: K - 1 more padded rows each
        aptr[i] = As + p.lead + (r + db * (p.K - 1)) * p.XBS + xb;
    }

    constexpr bool NOE = U < 0;          // the whole (ci, kh) sum fits the slots: no second accumulator at all
    static_assert(UNPACKED || NOE || TM * TN <= kEPitch, "second-accumulator pitch too small for the thread tile");
    acc_t acc[TM][TN];
    // second packed accumulator (upper slot bits): in shared memory, TM * TN 8-byte entries per thread with
    // a pitch of kEPitch entries per thread (odd, so that the lanes of a warp fall into different banks
    // and every access has an immediate offset); only read-modify-written every M products, it would
    // otherwise hold half of the thread's registers
    uint2 *Es = reinterpret_cast<uint2 *>(smem + p.e_off) + tid * kEPitch;
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int t = 0; t < TN; ++t) acc[i][t] = UNPACKED ? (acc_t)0 : (acc_t)p.bias;
    if constexpr (!UNPACKED && !NOE) {
#pragma unroll
        for (int k = 0; k < TM * TN; ++k) Es[k] = make_uint2(0u, 0u);
    }
    int nmoves = 0, chunks_since_move = 0;

    // move the upper bits of every slot to E and restart the slots at their bias (on 32-bit halves, so
    // that it is two funnel/plain shifts, four logic operations and one add with carry per accumulator)
    auto carry_save_row = [&](int i) {
        if constexpr (!UNPACKED) {
            const uint32_t mh_lo = (uint32_t)p.mask_high, mh_hi = (uint32_t)(p.mask_high >> 32);
            const uint32_t ml_lo = (uint32_t)p.mask_low, ml_hi = (uint32_t)(p.mask_low >> 32);
            const uint32_t b_lo = (uint32_t)p.bias, b_hi = (uint32_t)(p.bias >> 32);
            const int h = p.hbits;                                   // 1 .. 31 whenever a move happens
#pragma unroll
            for (int t = 0; t < TN; ++t) {
                uint32_t qlo = (uint32_t)acc[i][t], qhi = (uint32_t)((uint64_t)acc[i][t] >> 32);
                uint2 e = Es[i * TN + t];
                uint32_t elo = e.x, ehi = e.y;
                const uint32_t hlo = __funnelshift_r(qlo, qhi, h) & mh_lo;
                const uint32_t hhi = (qhi >> h) & mh_hi;
                asm("add.cc.u32 %0, %0, %2;\n\taddc.u32 %1, %1, %3;" : "+r"(elo), "+r"(ehi) : "r"(hlo), "r"(hhi));
                qlo = (qlo & ml_lo) | b_lo;
                qhi = (qhi & ml_hi) | b_hi;
                Es[i * TN + t] = make_uint2(elo, ehi);
                acc[i][t] = (acc_t)(((uint64_t)qhi << 32) | qlo);
            }
        }
    };
    auto carry_save = [&]() {
#pragma unroll
        for (int i = 0; i < TM; ++i) carry_save_row(i);
        ++nmoves;
    };

    const int KJ = p.K * p.J;
    const int xq = (p.XB + 3) / 4;                                   // 16-byte pieces per activation row
    const int ap_plane = p.B * p.Hp * p.XBT;                         // words per channel of Ap
    const uint32_t *ap_tile = p.ap + (size_t)Rp0 * p.XBT + seg * p.XO;   // first word this tile reads (16-byte aligned)

    // The 16-byte pieces of an activation stage this thread copies: the same ones every stage, so their
    // offsets are worked out once (channel in the top byte of the destination offset, -1: none).
    constexpr int kPieces = kCopyPieces;
    int piece_src[kPieces], piece_dst[kPieces];
#pragma unroll
    for (int k = 0; k < kPieces; ++k) {
        const int q = tid + k * nthreads;                            // pieces numbered [row][channel][piece of the row]
        const int rc = fast_div(q, p.mg_xq), qd = q - rc * xq;
        const int rl = fast_div(rc, p.mg_ck), cl = rc - rl * p.CK;
        piece_src[k] = cl * ap_plane + rl * p.XBT + 4 * qd;
        piece_dst[k] = q < p.CK * NR * xq ? ((cl << 24) | (cl * p.a_plane + p.lead + rl * p.XBS + 4 * qd)) : -1;
    }
    const bool pieces_in_regs = p.CK * NR * xq <= kPieces * nthreads;
    const int tco4 = p.TCO / 4, tco4_log2 = 31 - __clz(tco4);        // TCO / 4 is a power of two

    // Asynchronous fetch of one stage: NR packed rows of ckn channels and the packed kernel rows of the
    // same channels for TCO output channels, all in 16-byte pieces.
    auto fetch = [&](int ci0, int ckn, uint32_t *Adst, uint32_t *Bdst) {
        const uint32_t *asrc = ap_tile + (size_t)ci0 * ap_plane;
        if (pieces_in_regs) {
#pragma unroll
            for (int k = 0; k < kPieces; ++k)
                if (piece_dst[k] >= 0 && (piece_dst[k] >> 24) < ckn) cp_async_16(Adst + (piece_dst[k] & 0xFFFFFF), asrc + piece_src[k]);
        } else {
            const int per_ch = NR * xq;
            for (int cl = 0; cl < ckn; ++cl) {
                const uint32_t *src = asrc + (size_t)cl * ap_plane;
                uint32_t *dst = Adst + cl * p.a_plane + p.lead;
                for (int idx = tid; idx < per_ch; idx += nthreads) {
                    const int rl = fast_div(idx, p.mg_xq), qd = idx - rl * xq;
                    cp_async_16(dst + rl * p.XBS + 4 * qd, src + (size_t)rl * p.XBT + 4 * qd);
                }
            }
        }
        const uint32_t *bsrc = p.wp + (size_t)ci0 * KJ * p.CoP + co0;
        const int rows_b = (U > 0 ? p.CK : ckn) * KJ;                // grouped mode multiplies all CK channels of a stage
        for (int idx = tid; idx < rows_b << tco4_log2; idx += nthreads) {
            const int kr = idx >> tco4_log2, c4 = idx & (tco4 - 1);
            uint32_t *dst = Bdst + kr * kBPitch + c4 * 4;
            if (co0 + c4 * 4 < p.CoP && kr < ckn * KJ) cp_async_16(dst, bsrc + kr * p.CoP + c4 * 4);
            else *reinterpret_cast<uint4 *>(dst) = make_uint4(0, 0, 0, 0);
        }
        cp_async_commit();
    };

    grid_dependency_wait();                                          // everything above touched no global memory
    fetch(0, min(p.CK, p.Ci), As, Bs);
    int stage = 0;
    for (int ci0 = 0; ci0 < p.Ci; ci0 += p.CK, stage ^= 1) {
        const int ckn = min(p.CK, p.Ci - ci0);
        cp_async_wait_all();
        __syncthreads();                                             // this stage has landed; the previous one is fully consumed
        if (ci0 + p.CK < p.Ci)
            fetch(ci0 + p.CK, min(p.CK, p.Ci - ci0 - p.CK), As + (stage ^ 1) * p.a_words, Bs + (stage ^ 1) * p.b_words);
        const int astage = stage * p.a_words;
        const uint32_t *bptr = Bs + stage * p.b_words + tn * TN;
        // ---- multiply-accumulate over (ci, kh, j)
        if constexpr (KT > 0 && PITCH > 0) {
            const uint32_t *ap[TM];
#pragma unroll
            for (int i = 0; i < TM; ++i) ap[i] = aptr[i] + astage;
            const uint32_t *bp = bptr;
            if constexpr (U > 0 && !UNPACKED) {
#pragma unroll 2
                for (int c0 = 0; c0 < p.CK; c0 += U) {
#pragma unroll
                    for (int u = 0; u < U; ++u) {
#pragma unroll
                        for (int kh = 0; kh < KT; ++kh) {
#pragma unroll
                            for (int j = 0; j < JT; ++j) {
                                uint32_t a[TM], b[TN];
#pragma unroll
                                for (int i = 0; i < TM; ++i) a[i] = ap[i][kh * PITCH - j];
#pragma unroll
                                for (int t = 0; t < TN; t += 4) {
                                    const uint4 v = *reinterpret_cast<const uint4 *>(bp + (kh * JT + j) * kBPitch + t);
                                    b[t] = v.x; b[t + 1] = v.y; b[t + 2] = v.z; b[t + 3] = v.w;
                                }
#pragma unroll
                                for (int i = 0; i < TM; ++i)
#pragma unroll
                                    for (int t = 0; t < TN; ++t) mac<UNPACKED, SP>(acc[i][t], a[i], b[t]);
                            }
                        }
#pragma unroll
                        for (int i = 0; i < TM; ++i) ap[i] += p.a_plane;
                        bp += KT * JT * kBPitch;
#pragma unroll
                        for (int i = 0; i < TM; ++i)
                            if ((i * U) / TM == u) carry_save_row(i);
                    }
                    ++nmoves;
                }
            } else {
            // two channels per iteration: the operand loads of the next step then rotate through register
            // names instead of being copied at the loop edge
#pragma unroll 2
            for (int cl = 0; cl < ckn; ++cl) {
#pragma unroll
                for (int kh = 0; kh < KT; ++kh) {
#pragma unroll
                    for (int j = 0; j < JT; ++j) {
                        uint32_t a[TM], b[TN];
#pragma unroll
                        for (int i = 0; i < TM; ++i) a[i] = ap[i][kh * PITCH - j];
#pragma unroll
                        for (int t = 0; t < TN; t += 4) {
                            const uint4 v = *reinterpret_cast<const uint4 *>(bp + (kh * JT + j) * kBPitch + t);
                            b[t] = v.x; b[t + 1] = v.y; b[t + 2] = v.z; b[t + 3] = v.w;
                        }
#pragma unroll
                        for (int i = 0; i < TM; ++i)
#pragma unroll
                            for (int t = 0; t < TN; ++t) mac<UNPACKED, SP>(acc[i][t], a[i], b[t]);
                    }
                }
#pragma unroll
                for (int i = 0; i < TM; ++i) ap[i] += p.a_plane;
                bp += KT * JT * kBPitch;
            }
            }
        } else {
            for (int cl = 0; cl < ckn; ++cl) {
                for (int kh = 0; kh < p.K; ++kh) {
                    for (int j = 0; j < p.J; ++j) {
                        const int aoff = astage + cl * p.a_plane + kh * p.XBS - j;
                        const uint32_t *brow = bptr + ((cl * p.K + kh) * p.J + j) * kBPitch;
                        uint32_t a[TM], b[TN];
#pragma unroll
                        for (int i = 0; i < TM; ++i) a[i] = aptr[i][aoff];
#pragma unroll
                        for (int t = 0; t < TN; t += 4) {
                            const uint4 v = *reinterpret_cast<const uint4 *>(brow + t);
                            b[t] = v.x; b[t + 1] = v.y; b[t + 2] = v.z; b[t + 3] = v.w;
                        }
#pragma unroll
                        for (int i = 0; i < TM; ++i)
#pragma unroll
                            for (int t = 0; t < TN; ++t) mac<UNPACKED, SP>(acc[i][t], a[i], b[t]);
                    }
                }
            }
        }
        // at most M (ci, kh) pairs between two moves; none is needed after the last stage
        if constexpr (!UNPACKED && !NOE) {
            if (++chunks_since_move == p.flush_chunks && ci0 + p.CK < p.Ci) { carry_save(); chunks_since_move = 0; }
        }
    }

    // ---- extract the slots: slot m holds 2^h E_m + Q_m - (moves + 1) bias_m (uint32 arithmetic wraps by design)
    // slots per accumulator, N + Kc - 1: a constant of the unrolled kernels (Kc = K when the kernel row is one word, else N)
    constexpr int NS_CT = (!UNPACKED && KT > 0) ? N + (JT == 1 ? KT : N) - 1 : 0;
    const int nslots = NS_CT > 0 ? NS_CT : p.nslots;
    uint32_t slot_sub[2 * N], slot_msk[2 * N];                        // per slot: (moves + 1) bias_m and the field mask
#pragma unroll
    for (int m = 0; m < 2 * N; ++m) {
        slot_sub[m] = ((uint32_t)nmoves + 1u) * (uint32_t)p.slot_bias[m];
        slot_msk[m] = (m == nslots - 1) ? p.top_mask : p.slot_mask;
    }
    auto slot_value = [&](uint64_t Q, uint64_t Ev, int m) -> uint32_t {
        // a top slot that ends at bit 63 or beyond needs no mask: the shift leaves nothing above it
        const bool open_top = SC > 0 && NS_CT > 0 && m == NS_CT - 1 && SC * NS_CT >= 64;
        uint32_t qv = (uint32_t)(Q >> (S * m));
        if (!open_top) qv &= slot_msk[m];
        if constexpr (NOE) return qv - slot_sub[m];
        uint32_t ev = (uint32_t)(Ev >> (S * m));
        if (!open_top) ev &= slot_msk[m];
        return (ev << p.hbits) + qv - slot_sub[m];
    };
    auto load_e = [&](int i, int t) -> uint64_t {
        if constexpr (NOE) return 0;
        const uint2 e = Es[i * TN + t];
        return ((uint64_t)e.y << 32) | e.x;
    };
    // The upper slots of a position belong to the next position (Theorem 2), which the next lane holds:
    // they travel by a rotating shuffle, in which the last lane hands over those of its previous
    // position; a warp's first position takes them from the warp before through shared memory.
    if constexpr (!UNPACKED) {
        __syncthreads();
        uint32_t *xch = smem;                                        // [warp][N][TCO]
        if (lm == lanes_m - 1) {
#pragma unroll
            for (int m = 0; m < N; ++m)
#pragma unroll
                for (int t = 0; t < TN; ++t)
                    xch[(warp * N + m) * p.TCO + tn * TN + t] =
                        (N + m < nslots) ? slot_value((uint64_t)acc[TM - 1][t], load_e(TM - 1, t), N + m) : 0u;
        }
        __syncthreads();
    }

    // where each position's pixels go: element offset relative to the CTA's first output (image b0, channel co0),
    // which fits 32 bits (checked on the host), and number of pixels to store (0: none)
    uint32_t pix_rel[TM];
    int pix_n[TM];
    int tile_pos[TM];                                                // staged output: byte offset of the position's first pixel in a channel's tile
    const uint32_t chan_stride = (uint32_t)(p.Ho * p.Wo);
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int pos = wpos0 + i * lanes_m + lm, pc = pos < TP ? pos : 0;
        const int r = fast_div(pc, p.mg_xb), xbl = pc - r * p.XB;
        const int xg = seg * p.XO + xbl - p.J;                       // output block in the row; halo positions give no pixels
        const int db = fast_div(h0 + r, p.mg_ho);
        const int h = h0 + r - db * p.Ho;
        const bool valid = pos < TP && xbl >= p.J && xg < p.X;
        pix_rel[i] = (uint32_t)(db * p.Co) * chan_stride + (uint32_t)(h * p.Wo + xg * N);
        pix_n[i] = valid ? min(N, p.Wo - xg * N) : 0;
        tile_pos[i] = r * p.WTP + (xbl - p.J) * N;
    }
    const size_t cta_off = ((size_t)b0 * p.Co + co0) * chan_stride;

    if (UNPACKED && p.requant && p.stage_out) __syncthreads();     // the staged tile reuses the operand buffers of the main loop
    int8_t *tile = reinterpret_cast<int8_t *>(smem + p.tile_off);
    const int tile_chan = p.TR * p.WTP;                              // bytes per channel of the staged tile
    // ---- overlap-add, optional requantisation (arithmetic shift, clamp), store
    auto finish = [&](auto requant_tag, auto staged_tag) {
        constexpr bool REQ = decltype(requant_tag)::value, STAGED = decltype(staged_tag)::value;
        int8_t *out8 = (int8_t *)p.out + cta_off;
        int32_t *out32 = (int32_t *)p.out + cta_off;
#pragma unroll
        for (int t = 0; t < TN; ++t) {
            const int cl = tn * TN + t;
            const uint32_t chan_rel = (uint32_t)cl * chan_stride;
            const bool chan_ok = co0 + cl < p.Co;
            const uint32_t cadd = (p.x_off != 0 && chan_ok) ? (uint32_t)__ldg(p.corr + co0 + cl) : 0u;
            uint32_t up_prev[N];                                     // upper slots of this lane's previous position
#pragma unroll
            for (int m = 0; m < N; ++m) up_prev[m] = 0u;
#pragma unroll
            for (int i = 0; i < TM; ++i) {
                uint32_t Y[N];
                if constexpr (!UNPACKED) {
                    const uint64_t ev = load_e(i, t);
#pragma unroll
                    for (int m = 0; m < N; ++m) Y[m] = slot_value((uint64_t)acc[i][t], ev, m) + cadd;
#pragma unroll
                    for (int m = 0; m < N; ++m) {
                        if (N + m < nslots) {                        // uniform over the launch
                            const uint32_t up = slot_value((uint64_t)acc[i][t], ev, N + m);
                            uint32_t in = __shfl_sync(0xFFFFFFFFu, lm == lanes_m - 1 ? up_prev[m] : up, (lane - p.TNX) & 31);
                            if (i == 0 && lm == 0) in = warp > 0 ? smem[((warp - 1) * N + m) * p.TCO + cl] : 0u;
                            Y[m] += in;
                            up_prev[m] = up;
                        }
                    }
                } else {
                    Y[0] = (uint32_t)acc[i][t];
                }
                const uint32_t o = pix_rel[i] + chan_rel;
                const int n_store = chan_ok ? pix_n[i] : 0;
#pragma unroll
                for (int m = 0; m < N; ++m) {
                    int32_t v = (int32_t)Y[m];
                    if constexpr (REQ) {
                        v = max(p.lo, min(p.hi, v >> p.shift));
                        if (m < n_store) {
                            if constexpr (STAGED) tile[cl * tile_chan + tile_pos[i] + m] = (int8_t)v;
                            else out8[o + m] = (int8_t)v;
                        }
                    } else {
                        if (m < n_store) out32[o + m] = v;
                    }
                }
            }
        }
    };
    if (!p.requant) finish(std::false_type(), std::false_type());
    else if (p.stage_out) finish(std::true_type(), std::true_type());
    else finish(std::true_type(), std::false_type());
    if (!(p.requant && p.stage_out)) return;

    // ---- staged codes leave the CTA: whole rows in pieces of `vec` bytes, optionally max-pooled 2x2 on the way
    __syncthreads();
    const int col0 = seg * p.XO * N;                                 // first output column of this row segment
    const int wn = min(p.Wo - col0, p.XO * N);                       // columns of this segment
    const int ncv = min(p.TCO, p.Co - co0);                          // channels of this tile that exist
    if (p.out_bits < 8) {
        // dense codes: every output byte gathers 8 / out_bits neighbouring codes of a row (rows and segments start on
        // byte boundaries, checked on the host); with pool each code is the maximum of a 2x2 window first
        const int ob = p.out_bits, cpb = 8 / ob, sh = p.pool ? 1 : 0;
        const uint32_t cmask = (1u << ob) - 1u;
        const int Hq = p.Ho >> sh, Wq = p.Wo >> sh, TRq = TRe >> sh;
        const int ppr = ((((wn >> sh) * ob) >> 3)) / p.vec;          // pieces of `vec` dense bytes per row
        const float inv_ppr = 1.0f / (float)ppr, inv_tr = 1.0f / (float)TRq;
        for (int idx = tid; idx < ncv * TRq * ppr; idx += nthreads) {
            const int rr = small_div(idx, ppr, inv_ppr), piece = idx - rr * ppr;
            const int cl = small_div(rr, TRq, inv_tr), rq = rr - cl * TRq;
            const int r = rq << sh;
            const int db = fast_div(h0 + r, p.mg_ho);
            const int b = b0 + db, h = h0 + r - db * p.Ho;
            const int8_t *src = tile + cl * tile_chan + r * p.WTP;
            const size_t e0 = ((((size_t)b * p.Co + co0 + cl) * Hq + (h >> sh)) * Wq + (col0 >> sh));   // first code of this segment's row
            uint8_t *dst = (uint8_t *)p.out + ((e0 * ob) >> 3) + piece * p.vec;
            uint32_t word = 0;
            for (int u = 0; u < p.vec; ++u) {
                uint32_t byte = 0;
                for (int c = 0; c < cpb; ++c) {
                    const int col = (piece * p.vec + u) * cpb + c;           // code index within the segment's (pooled) row
                    int v;
                    if (p.pool) {
                        int a0 = src[2 * col], a1 = src[2 * col + 1], c0 = src[p.WTP + 2 * col], c1 = src[p.WTP + 2 * col + 1];
                        if (!p.out_signed) { a0 &= 0xFF; a1 &= 0xFF; c0 &= 0xFF; c1 &= 0xFF; }
                        v = max(max(a0, a1), max(c0, c1));
                    } else {
                        v = src[col];
                    }
                    byte |= ((uint32_t)v & cmask) << (ob * c);
                }
                word |= byte << (8 * u);
            }
            if (p.vec == 4) *reinterpret_cast<uint32_t *>(dst) = word;
            else *dst = (uint8_t)word;
        }
    } else if (!p.pool) {
        const int ppr = wn / p.vec;                                  // pieces per row (vec divides Wo and col0)
        const float inv_ppr = 1.0f / (float)ppr, inv_tr = 1.0f / (float)TRe;
        for (int idx = tid; idx < ncv * TRe * ppr; idx += nthreads) {
            const int rr = small_div(idx, ppr, inv_ppr), piece = idx - rr * ppr;
            const int cl = small_div(rr, TRe, inv_tr), r = rr - cl * TRe;
            const int db = fast_div(h0 + r, p.mg_ho);
            const int b = b0 + db, h = h0 + r - db * p.Ho;
            const int8_t *src = tile + cl * tile_chan + r * p.WTP + piece * p.vec;
            int8_t *dst = (int8_t *)p.out + (((size_t)b * p.Co + co0 + cl) * p.Ho + h) * p.Wo + col0 + piece * p.vec;
            if (p.vec == 16) *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(src);
            else if (p.vec == 8) *reinterpret_cast<uint2 *>(dst) = *reinterpret_cast<const uint2 *>(src);
            else if (p.vec == 4) *reinterpret_cast<uint32_t *>(dst) = *reinterpret_cast<const uint32_t *>(src);
            else *dst = *src;
        }
    } else {
        const int Hq = p.Ho >> 1, Wq = p.Wo >> 1, TRq = TRe >> 1;
        const int ppr = (wn >> 1) / p.vec;                           // pooled pieces per row
        const float inv_ppr = 1.0f / (float)ppr, inv_tr = 1.0f / (float)TRq;
        for (int idx = tid; idx < ncv * TRq * ppr; idx += nthreads) {
            const int rr = small_div(idx, ppr, inv_ppr), piece = idx - rr * ppr;
            const int cl = small_div(rr, TRq, inv_tr), rq = rr - cl * TRq;
            const int r = 2 * rq;
            const int db = fast_div(h0 + r, p.mg_ho);
            const int b = b0 + db, h = h0 + r - db * p.Ho;
            const int8_t *src = tile + cl * tile_chan + r * p.WTP + piece * 2 * p.vec;
            int8_t *dst = (int8_t *)p.out + (((size_t)b * p.Co + co0 + cl) * Hq + (h >> 1)) * Wq + (col0 >> 1) + piece * p.vec;
            if (p.vec == 8) {
                const uint4 r0 = *reinterpret_cast<const uint4 *>(src), r1 = *reinterpret_cast<const uint4 *>(src + p.WTP);
                const uint2 v = p.out_signed ? make_uint2(pool_pairs<true>(r0.x, r0.y, r1.x, r1.y), pool_pairs<true>(r0.z, r0.w, r1.z, r1.w))
                                             : make_uint2(pool_pairs<false>(r0.x, r0.y, r1.x, r1.y), pool_pairs<false>(r0.z, r0.w, r1.z, r1.w));
                *reinterpret_cast<uint2 *>(dst) = v;
            } else if (p.vec == 4) {
                const uint2 r0 = *reinterpret_cast<const uint2 *>(src), r1 = *reinterpret_cast<const uint2 *>(src + p.WTP);
                *reinterpret_cast<uint32_t *>(dst) = p.out_signed ? pool_pairs<true>(r0.x, r0.y, r1.x, r1.y) : pool_pairs<false>(r0.x, r0.y, r1.x, r1.y);
            } else {
                int a0 = src[0], a1 = src[1], c0 = src[p.WTP], c1 = src[p.WTP + 1];
                if (!p.out_signed) { a0 &= 0xFF; a1 &= 0xFF; c0 &= 0xFF; c1 &= 0xFF; }
                *dst = (int8_t)max(max(a0, a1), max(c0, c1));
            }
        }
    }
}

// Reversed, packed kernel rows (Theorem 3: g = W[co][ci][kh][K-1:0], then Eq. 5 per chunk of Kc taps).
// wp[((ci*K + kh)*J + j)*CoP + co] = sum_{k' < Kc} g[j Kc + k'] 2^(S k').  For the comparator S == 0,
// Kc == 1: one int32 weight per word.
struct WeightPackParams {
    const int8_t *w;
    uint32_t *wp;
    int Co, Ci, K, J, Kc, S, w_signed, CoP, total;
    int w_bits;                // storage: 8 = one code per byte, 1 / 2 / 4 = dense (8 / w_bits codes per byte)
    int w_blocks;              // CTAs that pack kernel rows; the CTAs after them sum the weights of a channel (x_off != 0)
    Div32 d_cop, d_j, d_k;     // divisions of pack_weight_word
    int x_off;                 // offset taken from every activation code (0: none)
    int32_t *corr;             // corr[co] = x_off * sum of the weights of channel co, CoP entries
};

// Code number e of a tensor stored densely with `bits` (1, 2, 4 or 8) bits per code: code e occupies bits
// [(e bits) % 8, (e bits) % 8 + bits) of byte (e bits) / 8, two's complement when signed (Section V-B: weights and
// features kept compressed in memory and unpacked as they are read).
__device__ __forceinline__ int32_t load_dense_code(const int8_t *base, size_t e, int bits, bool is_signed) {
    const size_t bit = e * (size_t)bits;
    const uint32_t byte = (uint8_t)__ldg(base + (bit >> 3));
    const uint32_t v = (byte >> (int)(bit & 7)) & ((1u << bits) - 1u);
    const uint32_t sb = 1u << (bits - 1);
    return is_signed ? (int32_t)((v ^ sb) - sb) : (int32_t)v;
}

__device__ __forceinline__ void pack_weight_word(const WeightPackParams &q, int idx) {
    if (idx >= q.total) return;
    uint32_t rest = div32((uint32_t)idx, q.d_cop);
    const int co = idx - (int)rest * q.CoP;
    uint32_t up = div32(rest, q.d_j);
    const int j = (int)(rest - up * q.J);
    rest = up;
    up = div32(rest, q.d_k);
    const int kh = (int)(rest - up * q.K);
    const int ci = (int)up;
    uint32_t word = 0;
    if (co < q.Co) {
        const size_t row_e = (((size_t)co * q.Ci + ci) * q.K + kh) * q.K;       // first code of the kernel row
        for (int k = 0; k < q.Kc; ++k) {
            const int g_idx = j * q.Kc + k;              // index into the reversed row
            if (g_idx < q.K) {
                int32_t v;
                if (q.w_bits == 8) {
                    const int8_t raw = __ldg(q.w + row_e + (q.K - 1 - g_idx));
                    v = q.w_signed ? (int32_t)raw : (int32_t)(uint8_t)raw;
                } else {
                    v = load_dense_code(q.w, row_e + (q.K - 1 - g_idx), q.w_bits, q.w_signed != 0);
                }
                word += (uint32_t)v << (q.S * k);
            }
        }
    }
    q.wp[idx] = word;
}

// corr[co] = x_off * sum_{ci, kh, kw} W[co][ci][kh][kw]: one warp per output channel (its Ci K K codes are contiguous).
__device__ __forceinline__ void sum_channel_weights(const WeightPackParams &q, int co, int lane) {
    if (co >= q.CoP) return;
    int32_t sum = 0;
    if (co < q.Co) {
        const int per_co = q.Ci * q.K * q.K;
        const size_t e0 = (size_t)co * per_co;
        for (int e = lane; e < per_co; e += 32) {
            if (q.w_bits == 8) {
                const int8_t raw = __ldg(q.w + e0 + e);
                sum += q.w_signed ? (int32_t)raw : (int32_t)(uint8_t)raw;
            } else {
                sum += load_dense_code(q.w, e0 + e, q.w_bits, q.w_signed != 0);
            }
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, d);
    }
    if (lane == 0) q.corr[co] = sum * q.x_off;
}

// Packed activation rows (Eq. 5): ap[(ci * B*Hp + b*Hp + hp) * XBT + xb] packs the N input pixels of block
// x = xb - J of padded row hp, i.e. columns (xb - J) N + K - 1 - pad + n of input row hp - pad, zero where the
// row or a column lies in the padding.  For the comparator S == 0 and N == 1: one int32 code per word.
// One thread packs four consecutive words of a row (one 16-byte store); threads are numbered through all
// (ci, b) planes, so that small maps still fill their CTAs.  The first CTAs of the launch sum the channels' weights
// (when the layer runs on shifted codes) and pack the kernel rows (one word per thread), so that a layer needs one
// packing launch and its longest serial work starts first.
// x_bits: storage of the activations, 8 = one code per byte, 1 / 2 / 4 = dense.
// With wq.x_off != 0 every slot holds code - x_off, the slots outside the image included (code 0 there).
struct ActPackDivs {
    Div32 per_plane, b, xq;    // pieces per (ci, b) plane, images, 16-byte pieces per packed row
};

template <bool XS, int N>
__global__ void __launch_bounds__(256) pack_operands_kernel(const int8_t *__restrict__ x, int B, int Ci, int H, int W, int Hp,
                                                            int pad, int K, int J, int S, int XBT,
                                                            uint32_t *__restrict__ ap, int weight_blocks, const WeightPackParams wq,
                                                            int x_bits, const ActPackDivs dv, unsigned act_items) {
    grid_dependency_release();
    grid_dependency_wait();                                          // the input may come from the kernel before; the workspace may still be read by it
    // the first CTAs sum the channels' weights (the longest serial work of the launch) and pack the kernel rows
    if ((int)blockIdx.x < weight_blocks) {
        const int cb = weight_blocks - wq.w_blocks;                  // CTAs that sum weights (0 unless x_off != 0)
        if ((int)blockIdx.x < cb) sum_channel_weights(wq, (int)blockIdx.x * 8 + ((int)threadIdx.x >> 5), (int)threadIdx.x & 31);
        else pack_weight_word(wq, ((int)blockIdx.x - cb) * 256 + (int)threadIdx.x);
        return;
    }
    // the (plane, piece) pairs are numbered through: a CTA may span several small planes (ci * B + b)
    const int xq = XBT / 4;                                          // 16-byte pieces per packed row
    const int per_plane = Hp * xq;
    const unsigned item = (blockIdx.x - (unsigned)weight_blocks) * 256u + threadIdx.x;
    if (item >= act_items) return;
    const int plane = (int)div32(item, dv.per_plane);
    const int piece = (int)(item - (unsigned)plane * (unsigned)per_plane);
    const int ci = (int)div32((uint32_t)plane, dv.b), b = plane - ci * B;
    const int hp = (int)div32((uint32_t)piece, dv.xq), q = piece - hp * xq;
    const int hi = hp - pad;
    uint32_t fill = 0u;                                              // a word whose N slots all hold -x_off
    if (wq.x_off != 0) {
#pragma unroll
        for (int n = 0; n < N; ++n) fill += (uint32_t)(-wq.x_off) << (S * n);
    }
    uint32_t word[4] = {fill, fill, fill, fill};
    if (hi >= 0 && hi < H) {
        const size_t row_e = (((size_t)b * Ci + ci) * H + hi) * W;  // first code of the input row
        const int col0 = (4 * q - J) * N + K - 1 - pad;              // input column of slot 0 of the first word
        if (x_bits == 8) {
            const int8_t *row = x + row_e;
#pragma unroll
            for (int w = 0; w < 4; ++w)
#pragma unroll
                for (int n = 0; n < N; ++n) {
                    const int col = col0 + w * N + n;
                    if (col >= 0 && col < W) word[w] += (uint32_t)load_code<XS>(row + col) << (S * n);
                }
        } else {
#pragma unroll
            for (int w = 0; w < 4; ++w)
#pragma unroll
                for (int n = 0; n < N; ++n) {
                    const int col = col0 + w * N + n;
                    if (col >= 0 && col < W) word[w] += (uint32_t)load_dense_code(x, row_e + col, x_bits, XS) << (S * n);
                }
        }
    }
    *reinterpret_cast<uint4 *>(ap + ((size_t)plane * Hp + hp) * XBT + 4 * q) = make_uint4(word[0], word[1], word[2], word[3]);
}

template <bool SIGNED, int VEC>
__global__ void __launch_bounds__(256) maxpool2x2_vec_kernel(const int8_t *__restrict__ in, long long items, int H, int W,
                                                             int8_t *__restrict__ out) {
    grid_dependency_release();
    grid_dependency_wait();
    const int Ho = H / 2, WV = W / VEC;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < items; idx += (long long)gridDim.x * blockDim.x) {
        const int wv = (int)(idx % WV);
        const long long rest = idx / WV;
        const int ho = (int)(rest % Ho);
        const long long c = rest / Ho;
        const int8_t *src = in + (c * H + 2 * ho) * (long long)W + VEC * wv;
        int8_t *dst = out + (c * Ho + ho) * (long long)(W / 2) + (VEC / 2) * wv;
        if constexpr (VEC == 16) {
            const uint4 r0 = __ldg(reinterpret_cast<const uint4 *>(src));
            const uint4 r1 = __ldg(reinterpret_cast<const uint4 *>(src + W));
            *reinterpret_cast<uint2 *>(dst) = make_uint2(pool_pairs<SIGNED>(r0.x, r0.y, r1.x, r1.y), pool_pairs<SIGNED>(r0.z, r0.w, r1.z, r1.w));
        } else {
            const uint2 r0 = __ldg(reinterpret_cast<const uint2 *>(src));
            const uint2 r1 = __ldg(reinterpret_cast<const uint2 *>(src + W));
            *reinterpret_cast<uint32_t *>(dst) = pool_pairs<SIGNED>(r0.x, r0.y, r1.x, r1.y);
        }
    }
}

__global__ void __launch_bounds__(256) maxpool2x2_kernel(const int8_t *__restrict__ in, int BC, int H, int W, int is_signed,
                                                         int8_t *__restrict__ out) {
    const int Ho = H / 2, Wo = W / 2;
    const long long total = (long long)BC * Ho * Wo;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
        const int wo = (int)(idx % Wo);
        const long long rest = idx / Wo;
        const int ho = (int)(rest % Ho);
        const long long c = rest / Ho;
        const int8_t *src = in + (c * H + 2 * ho) * W + 2 * wo;
        int v[4] = {src[0], src[1], src[W], src[W + 1]};
        if (!is_signed) {
#pragma unroll
            for (int i = 0; i < 4; ++i) v[i] &= 0xFF;
        }
        out[idx] = (int8_t)max(max(v[0], v[1]), max(v[2], v[3]));
    }
}

// ------------------------------------------------------------------ host side

struct Conv2dSetup {
    hikonv_layout_t L;
    Conv2dParams kp;
    size_t smem_bytes;
    size_t wp_bytes;      // packed weights and the per-channel correction in the workspace (256-byte multiple), packed activations follow
    size_t corr_off;      // byte offset of the correction (CoP int32) in the workspace
    size_t ap_words;      // packed activation words
    dim3 grid;
    int threads;
    bool unpacked;
    int tm;               // positions per thread of the packed kernel
};

static int sm_count() {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms;
}

template <int N, int SC, int TM, int TN, bool UNPACKED, int KT, int JT, int PITCH, int U>
static int launch_pitch(const Conv2dSetup &s, bool sp, cudaStream_t st) {
#define HK_LAUNCH(SPV)                                                                                           \
    do {                                                                                                         \
        auto kern = conv2d_kernel<N, SC, TM, TN, UNPACKED, SPV, KT, JT, PITCH, U>;                               \
        if (s.smem_bytes > 48 * 1024)                                                                            \
            HIKONV_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s.smem_bytes)); \
        const int launch_rc = launch_dependent(kern, s.grid, dim3(s.threads), s.smem_bytes, st, s.kp);          \
        if (launch_rc != HIKONV_OK) return launch_rc;                                                            \
    } while (0)
    if (!sp) HK_LAUNCH(false);
    else HK_LAUNCH(true);
#undef HK_LAUNCH
    return HIKONV_OK;
}

// KT > 0: the kernel with unrolled (kh, j) loops and a compile-time row pitch; KT == 0: everything at run time.
// U: channels per unrolled group with placed carry-save moves (0: moves at stage ends).
template <int N, int SC, int TM, int TN, bool UNPACKED, int KT, int JT, int U>
static int launch_variant_u(const Conv2dSetup &s, bool sp, cudaStream_t st) {
    if constexpr (KT == 0) {
        return launch_pitch<N, SC, TM, TN, UNPACKED, 0, 0, 0, 0>(s, sp, st);
    } else {
        switch (s.kp.XBS) {
            case 8: return launch_pitch<N, SC, TM, TN, UNPACKED, KT, JT, 8, U>(s, sp, st);
            case 16: return launch_pitch<N, SC, TM, TN, UNPACKED, KT, JT, 16, U>(s, sp, st);
            case 32: return launch_pitch<N, SC, TM, TN, UNPACKED, KT, JT, 32, U>(s, sp, st);
            case 64: return launch_pitch<N, SC, TM, TN, UNPACKED, KT, JT, 64, U>(s, sp, st);
            default: return HIKONV_ERR_UNSUPPORTED;
        }
    }
}

// GROUPED: also instantiate the kernels with placed moves (groups of 3 and 4 channels).
template <int N, int SC, int TM, int TN, bool UNPACKED, int KT, int JT, bool GROUPED = false, bool SHALLOW = false>
static int launch_variant(const Conv2dSetup &s, bool sp, cudaStream_t st) {
    // SHALLOW: instantiated for layers whose whole (ci, kh) sum fits the slots (no second accumulator)
    if constexpr (SHALLOW) {
        return launch_variant_u<N, SC, TM, TN, UNPACKED, KT, JT, -1>(s, sp, st);
    } else {
        if constexpr (GROUPED) {
            if (s.kp.move_every == 3) return launch_variant_u<N, SC, TM, TN, UNPACKED, KT, JT, 3>(s, sp, st);
            if (s.kp.move_every == 4) return launch_variant_u<N, SC, TM, TN, UNPACKED, KT, JT, 4>(s, sp, st);
        }
        if (s.kp.move_every != 0) return HIKONV_ERR_UNSUPPORTED;
        return launch_variant_u<N, SC, TM, TN, UNPACKED, KT, JT, 0>(s, sp, st);
    }
}

constexpr int kTM = 4, kTN = 4;          // per-thread tile of the packed kernels
constexpr int kTNShallow = 8;            // channels per thread of the kernel without second accumulators
constexpr int kTMU = 8, kTNU = 4;        // per-thread tile of the comparator

// Tile shape of one candidate and its modelled cost.
struct TileChoice {
    int TNX, TMX, TR, NSEG, XO, XB;
    double cost;
};

// Chooses channels per CTA (TNX * TN), rows per CTA (TR) and row segments so that the device is
// evenly loaded.  The model charges each "wave" of resident CTAs max(resident threads, 256) per SM
// (an SM with fewer threads than that cannot fill the multiply pipe), adds the staging work of a
// tile relative to its multiply work, and divides by the useful work.
static TileChoice choose_tiles(int total_rows, int Ho, int X, int N, int K, int J, int Co, int TM, int TN, int sms,
                               int force_tr, bool even_rows = false, int xo_mult = 4, int force_tnx = 0) {
    TileChoice best;
    best.cost = -1.0;
    // More than four channel lanes (16 channels per CTA) never measured faster than four on the benchmark layers
    // (sweeps over every TNX and tile height: 10x20 to 160x320 maps, 3 to 256 input channels); the automatic choice
    // stays within 1 .. 4, a forced value may go up to 16.
    for (int TNX = 1; TNX <= (force_tnx > 0 ? 16 : 4); TNX *= 2) {
        if (force_tnx > 0 && TNX != force_tnx) continue;
        const int TCO = TNX * TN;
        if (TNX > 1 && TCO / 2 >= Co) break;                       // more channel lanes than channels
        const int gy = ceil_div(Co, TCO);
        const int max_tmx = kMaxThreads2D / TNX;
        const int maxpos = max_tmx * TM;
        // rows wider than a tile are cut into segments of XO blocks (a multiple of 4, so that every tile
        // row starts on a 16-byte boundary of the packed activations), each with its own J halo positions
        const int rowmax = std::min(maxpos, 64);                  // a staged row holds at most 64 words
        int NSEG = 1, XO = X;
        if (X + J > rowmax) {
            // xo_mult: a multiple of 4 (16-byte pieces of the packed rows); larger when the segments of a dense output
            // row have to start on byte boundaries
            XO = (rowmax - J) / xo_mult * xo_mult;
            if (XO < xo_mult) continue;
            NSEG = ceil_div(X, XO);
            XO = std::min(XO, (ceil_div(X, NSEG) + xo_mult - 1) / xo_mult * xo_mult);
            NSEG = ceil_div(X, XO);
        }
        const int XB = XO + J;
        const int tr_hi = std::max(1, std::min(maxpos / XB, total_rows));
        const int tr_lo = force_tr > 0 ? std::min(force_tr, tr_hi) : 1;
        const int tr_end = force_tr > 0 ? tr_lo : tr_hi;
        for (int TR = tr_lo; TR <= tr_end; ++TR) {
            if (even_rows && (TR & 1)) continue;                      // a fused 2x2 pool needs both rows of a pair in one CTA
            int TMX = ceil_div(TR * XB, TM);
            int threads = (TMX * TNX + 31) / 32 * 32;               // whole warps
            if (threads > kMaxThreads2D) continue;
            TMX = threads / TNX;
            const long long tiles = (long long)ceil_div(total_rows, TR) * NSEG * gy;
            // shared memory of the two double-buffered tiles (8 channels per stage at most)
            const int pitch = XB <= 8 ? 8 : XB <= 16 ? 16 : XB <= 32 ? 32 : 64;
            const int span_s = (TR + Ho - 2) / Ho + 1;
            const int ckc = stage_channel_cap(K, J);
            const size_t smem = 2 * 4 * ((size_t)ckc * ((TR + (K - 1) * span_s) * pitch + 8) + (size_t)ckc * K * J * kBPitch);
            if (smem > 72 * 1024) continue;                            // plus the second accumulators, 136 bytes per thread
            // (the model keeps charging 32 KB for them: with their true size it preferred tiles that measured slower)
            const int per_sm = std::max(1, std::min(std::min(2048 / threads, 65536 / (threads * 128)), (int)(220 * 1024 / (smem + 32 * 1024))));
            const long long slots = (long long)per_sm * sms;
            const long long full_waves = tiles / slots;
            const long long rest = tiles - full_waves * slots;
            double time = (double)full_waves * std::max(per_sm * threads, 256);
            if (rest > 0) time += std::max((int)((rest + sms - 1) / sms) * threads, 256);
            const int span = (TR + Ho - 2) / Ho + 1;
            const double NR = TR + (K - 1) * span;
            const double work = (double)K * J * (TM * TN + 8) * threads;
            const double stage = 0.5 * NR * XB + 0.5 * K * J * TCO;   // a few instructions per 16-byte piece
            time *= 1.0 + stage / work;
            const double useful = (double)total_rows * X * Co;     // output blocks x channels
            const double cost = time * sms / useful;
            if (best.cost < 0 || cost < best.cost - 1e-12) best = {TNX, TMX, TR, NSEG, XO, XB, cost};
        }
    }
    return best;
}

static int make_setup(int B, int Ci, int H, int W, int Co, int K, int stride, int pad, int p, int q, int xs, int ws,
                      int requant, int shift, int lo, int hi, int algo, const hikonv_tuning_t *tune, Conv2dSetup *s,
                      int pool = 0, const void *d_out = nullptr, int out_bits = 8) {
    if (B < 1 || Ci < 1 || H < 1 || W < 1 || Co < 1 || K < 1 || K > kMaxK) return HIKONV_ERR_INVALID_ARG;
    if (validate_codes(p, q) != HIKONV_OK) return HIKONV_ERR_INVALID_ARG;
    if (stride != 1 || pad < 0 || pad >= K) return HIKONV_ERR_UNSUPPORTED;
    if (algo == HIKONV_ALGO_PACKED64EMU || algo == HIKONV_ALGO_DP4A) return HIKONV_ERR_UNSUPPORTED;
    if (algo != HIKONV_ALGO_PACKED32 && algo != HIKONV_ALGO_UNPACKED_IMAD) return HIKONV_ERR_INVALID_ARG;
    if (requant && (shift < 0 || shift > 31 || lo < -128 || hi > 255 || lo > hi)) return HIKONV_ERR_INVALID_ARG;
    const int Ho = H + 2 * pad - K + 1, Wo = W + 2 * pad - K + 1;
    if (Ho < 1 || Wo < 1) return HIKONV_ERR_INVALID_ARG;
    if (Ho >= 60000) return HIKONV_ERR_UNSUPPORTED;              // the kernel divides row numbers below 2^16 by a multiply (fast_div)
    if ((double)B * Ci * H * W >= 2147483647.0 || (double)B * Ho >= 2147483647.0) return HIKONV_ERR_UNSUPPORTED;
    // the exact sums must fit int32
    const double max_code = (double)(1 << p) * (double)(1 << q);
    if ((double)Ci * K * K * max_code >= 1073741824.0) return HIKONV_ERR_UNSUPPORTED;

    s->unpacked = (algo == HIKONV_ALGO_UNPACKED_IMAD);
    Conv2dParams &kp = s->kp;
    std::memset(&kp, 0, sizeof(kp));
    hikonv_layout_t &L = s->L;
    int TM, TN, N;
    if (s->unpacked) {
        L.N = 1; L.S = 0; L.Kc = 1; L.J = K; L.segments = 1; L.top_bits = 32; L.M = Ci * K; L.signed_prod = (xs || ws) ? 1 : 0;
        L.S_paper = 0;
        TM = kTMU; TN = kTNU; N = 1;
        s->tm = TM;
        if (K > kMaxJ) return HIKONV_ERR_UNSUPPORTED;
    } else {
        int rc = make_layout(p, q, xs, ws, K, 2, Ci * K, Wo, tune, &L);
        if (rc != HIKONV_OK) return rc;
        // Unsigned activations against signed weights: the products of codes x - 2^(p-1) span about half the range,
        // so a slot takes nearly twice as many of them between two carry-save moves, or a word one more pixel (5-bit
        // codes: three instead of two).  Layers whose signed layout is cheaper by the estimate below run on the shifted codes and get
        // 2^(p-1) * (sum of the channel's weights) added back in the epilogue: from 128 input channels on always
        // (measured: 256 channels on 14x14 maps 239 -> 218 us), from 32 on when the layer is large enough to keep four
        // positions per thread (32 channels on 40x80 maps 112 -> 106 us; the 64-channel layers on 10x20 maps, bound by
        // the latency of one thread's work, lose 2 us to the longer packing launch and keep their own codes).
        const double threads4_own = (double)B * Ho * (ceil_div(Wo, L.N) + L.J) / kTM * ceil_div(Co, kTN);
        const bool small_layer = threads4_own <= 1.1 * sm_count() * 2 * kMaxThreads2D;
        if (!xs && ws) {
            hikonv_layout_t Ls;
            // issue cycles per pixel and (ci, kh) pair: J multiplies of about four cycles and, every M pairs, a move of
            // about thirteen, shared by the N pixels of a word; the shifted codes are taken for a gain of 7 % or more,
            // always when they put more pixels into a word, else under the depth conditions above
            auto cycles = [&](const hikonv_layout_t &l) { return (l.J * 4.1 + 13.0 / std::min(l.M, Ci * K)) / l.N; };
            if (make_layout(p, q, 1, ws, K, 2, Ci * K, Wo, tune, &Ls) == HIKONV_OK && cycles(Ls) <= 0.93 * cycles(L) &&
                (Ls.N > L.N || (L.M < Ci * K && (Ci >= 128 || (Ci >= 32 && !small_layer))))) {
                L = Ls;
                xs = 1;
                kp.x_off = 1 << (p - 1);
            }
        }
        if (L.N > kMaxN2D || L.segments > kMaxN2DSeg) return HIKONV_ERR_UNSUPPORTED;
        TM = kTM; TN = kTN; N = L.N;
        // A first layer (8-bit activations, few input channels: no second accumulator) spends most of its instructions
        // on the per-position work around a short multiply loop; with eight channels per thread instead of four that
        // work is shared by twice the outputs (3 -> 16 channels on 160x320 maps: 179 -> 161 us).
        if (L.N == 2 && L.S == 17 && K == 3 && L.J == 2 && L.M >= Ci * K && Co % 8 == 0) TN = kTNShallow;
        // Small layers are bound by the serial work of a thread, not by the multiplier: when four positions per thread
        // would not even fill the resident thread slots of the device once (about 1.1 times, measured on the benchmark
        // network: 10x20 maps 56 -> 32 us, 20x40 maps 83 -> 68 us; larger layers lose 2-10 %), threads take two
        // positions and there are twice as many of them.  Built for the 3x3 kernel on N = 3, S = 13.
        if (L.N == 3 && L.S == 13 && K == 3 && L.J == 1) {
            const double threads4 = (double)B * Ho * (ceil_div(Wo, N) + L.J) / kTM * ceil_div(Co, kTN);
            if (threads4 <= 1.1 * sm_count() * 2 * kMaxThreads2D) TM = 2;
        }
        if (tune && tune->tile >= 100000) TM = tune->tile / 100000;          // forced: 100000 x positions per thread
        if (TM != kTM && !(TM == 2 && L.N == 3 && L.S == 13 && K == 3 && L.J == 1)) return HIKONV_ERR_UNSUPPORTED;
        s->tm = TM;
        const SplitConsts sc = make_split_consts(L, p, q, xs, ws, K, L.M);
        kp.bias = sc.bias; kp.mask_low = sc.mask_low; kp.mask_high = sc.mask_high;
        kp.hbits = L.carry_bits; kp.nslots = L.segments;
        kp.slot_mask = sc.slot_mask;
        kp.top_mask = (L.top_bits >= 32) ? 0xFFFFFFFFu : ((1u << L.top_bits) - 1u);
        for (int m = 0; m < kMaxN2DSeg; ++m) kp.slot_bias[m] = m < L.segments ? sc.seg_bias[m] : 0;
    }
    kp.B = B; kp.Ci = Ci; kp.H = H; kp.W = W; kp.Co = Co; kp.K = K; kp.pad = pad; kp.Ho = Ho; kp.Wo = Wo; kp.Hp = Ho + K - 1;
    kp.CoP = (Co + 3) / 4 * 4;
    kp.S = L.S; kp.J = L.J; kp.Kc = L.Kc; kp.M = L.M;
    kp.requant = requant ? 1 : 0; kp.shift = shift; kp.lo = lo; kp.hi = hi;
    kp.total_rows = B * Ho;
    kp.X = ceil_div(Wo, N);
    int xo_mult = 4;
    if (requant && out_bits < 8 && out_bits > 0) {
        // segment width in codes (halved by the pool) times out_bits must be a multiple of 8
        const int unit = pool ? 16 : 8;
        int g = N * out_bits, a = unit;
        while (a) { const int t = g % a; g = a; a = t; }               // g = gcd(N out_bits, unit)
        const int need = unit / g;
        while (xo_mult % need != 0) xo_mult += 4;
    }
    // tune->tile > 0: rows per CTA, plus 1000 x channel lanes per CTA (1, 2, 4, 8, 16) when those are forced too
    const int tile_arg = (tune && tune->tile > 0) ? tune->tile % 100000 : 0;
    const TileChoice tc = choose_tiles(kp.total_rows, Ho, kp.X, N, K, L.J, Co, TM, TN, sm_count(), tile_arg % 1000,
                                       requant && pool, xo_mult, tile_arg / 1000);
    if (tc.cost < 0) return HIKONV_ERR_UNSUPPORTED;
    kp.TNX = tc.TNX; kp.TMX = tc.TMX; kp.TCO = tc.TNX * TN;
    kp.NSEG = tc.NSEG; kp.XO = tc.XO; kp.XB = tc.XB; kp.TR = tc.TR;
    s->threads = tc.TMX * tc.TNX;
    const int span = (kp.TR + Ho - 2) / Ho + 1;              // images a tile can touch
    // output offsets relative to a CTA's first image and channel are kept in 32 bits
    if ((double)(span + 1) * std::max(Co, kp.TCO) * Ho * Wo >= 4294967296.0) return HIKONV_ERR_UNSUPPORTED;
    kp.NRmax = kp.TR + (K - 1) * span;
    // words per activation row in shared memory: 8, 16, 32 or 64 (the unrolled kernels have them as constants)
    kp.XBS = kp.XB <= 8 ? 8 : kp.XB <= 16 ? 16 : kp.XB <= 32 ? 32 : 64;
    kp.XBT = (kp.NSEG - 1) * kp.XO + (kp.XB + 3) / 4 * 4;
    kp.lead = (L.J + 3) / 4 * 4;                             // room for the xb - j reads in front of the first row
    kp.a_plane = kp.NRmax * kp.XBS + kp.lead;
    // channels per stage and stages between two carry-save moves (at most M (ci, kh) pairs)
    const int ck_cap = stage_channel_cap(K, L.J);
    int CK = std::min(ck_cap, Ci);
    kp.flush_chunks = 1 << 30;
    kp.move_every = 0;
    if (!s->unpacked && L.M < Ci * K) {
        if (L.M < K) return HIKONV_ERR_NO_FIT;               // not even one channel's kernel rows between two moves
        // the 3x3 kernel with N = 3, S = 13 has variants whose moves are placed inside unrolled groups of
        // 3 or 4 channels, for layers that have to move that often (stages then hold two groups instead of one);
        // it needs room for one move per group in the second accumulator.  With six or more channels between
        // moves the stage-end form measured faster.
        const int CF = L.M / K;
        int U = 0;
        if (L.N == 3 && L.S == 13 && K == 3 && L.J == 1 && !(tune && tune->tile < 0)) U = CF >= 6 ? 0 : CF >= 4 ? 4 : CF == 3 ? 3 : 0;
        if (U > 0 && ck_cap < U) U = 0;
        if (U > 0) {
            CK = ck_cap / U * U;
            // a stage's activation pieces should fit the per-thread copy descriptors (kPieces each): small CTAs
            // stage one group at a time
            const int pieces_per_channel = kp.NRmax * ((kp.XB + 3) / 4);
            while (CK > U && CK * pieces_per_channel > kCopyPieces * s->threads) CK -= U;
            // every group of every stage moves once, the zero-weight channels that fill the last stage included
            if (ceil_div(Ci, CK) * (CK / U) > (1 << L.carry_bits)) {
                U = 0;
                CK = std::min(ck_cap, Ci);
            }
        }
        if (U > 0) {
            kp.move_every = U;
        } else {
            int fc = 1;
            const int eff = pick_chunking(CF, Ci, &CK, &fc, ck_cap);
            if (ceil_div(Ci, eff) > (1 << L.carry_bits)) return HIKONV_ERR_NO_FIT;
            kp.flush_chunks = fc;
        }
    }
    kp.CK = CK;
    {
        auto magic = [](int d) -> uint32_t { return d <= 1 ? 0u : (uint32_t)((0x100000000ull + (unsigned)d - 1) / (unsigned)d); };
        kp.mg_xb = magic(kp.XB); kp.mg_ho = magic(Ho); kp.mg_xq = magic((kp.XB + 3) / 4); kp.mg_ck = magic(CK); kp.mg_nseg = magic(kp.NSEG);
    }
    kp.a_words = CK * kp.a_plane;
    kp.b_off = 2 * kp.a_words;
    kp.b_words = CK * K * L.J * kBPitch;
    const size_t words = (size_t)kp.b_off + 2 * (size_t)kp.b_words;
    const size_t xch_words = s->unpacked ? 0 : (size_t)kp.TMX * N * kp.TCO;
    // requantised codes are staged per CTA ([channel][row][column] bytes, behind the exchange area) and written in
    // the widest pieces that divide every row start: Wo, the segment width and the output address
    size_t stage_words = 0;
    kp.stage_out = 0;
    kp.pool = 0;
    kp.out_bits = 8;
    if (!requant && (pool || out_bits != 8)) return HIKONV_ERR_INVALID_ARG;
    if (requant && (pool || out_bits != 8)) {
        // (plain byte output keeps direct stores: staged, it measured 3 % slower on the 56x56 layer)
        if (out_bits != 8 && out_bits != 4 && out_bits != 2 && out_bits != 1) return HIKONV_ERR_INVALID_ARG;
        if (pool && ((Ho | Wo) & 1)) return HIKONV_ERR_UNSUPPORTED;        // the fused 2x2 pool wants even output sizes
        if (out_bits < 8 && (lo < (lo < 0 ? -(1 << (out_bits - 1)) : 0) || hi > (lo < 0 ? (1 << (out_bits - 1)) - 1 : (1 << out_bits) - 1)))
            return HIKONV_ERR_INVALID_ARG;                                  // the clamp range must fit the stored width
        kp.stage_out = 1;
        kp.pool = pool ? 1 : 0;
        kp.out_signed = lo < 0 ? 1 : 0;
        kp.out_bits = out_bits;
        kp.WTP = (kp.XO * N + 15) / 16 * 16;
        kp.tile_off = (int)((xch_words + 3) / 4 * 4);
        stage_words = (size_t)kp.tile_off + (size_t)kp.TCO * kp.TR * kp.WTP / 4;
        const int w_out = pool ? Wo / 2 : Wo, seg_out = pool ? kp.XO * N / 2 : kp.XO * N;
        if (pool && kp.NSEG > 1 && ((kp.XO * N) & 1)) return HIKONV_ERR_UNSUPPORTED;
        if (out_bits == 8) {
            int vec = pool ? 8 : 16;
            while (vec > 1 && (w_out % vec != 0 || (kp.NSEG > 1 && seg_out % vec != 0) || ((uintptr_t)d_out % vec) != 0)) vec /= 2;
            kp.vec = vec == 2 ? 1 : vec;
        } else {
            // rows and row segments must start on byte boundaries of the dense output
            if ((w_out * out_bits) % 8 != 0 || (kp.NSEG > 1 && (seg_out * out_bits) % 8 != 0)) return HIKONV_ERR_UNSUPPORTED;
            const int row_bytes = w_out * out_bits / 8, seg_bytes = seg_out * out_bits / 8;
            kp.vec = (row_bytes % 4 == 0 && (kp.NSEG == 1 || seg_bytes % 4 == 0) && ((uintptr_t)d_out % 4) == 0) ? 4 : 1;
        }
    }
    kp.e_off = (int)((std::max(std::max(words, xch_words), stage_words) + 3) / 4 * 4);
    const size_t e_words = s->unpacked ? 0 : (size_t)kEPitch * s->threads * 2;
    s->smem_bytes = ((size_t)kp.e_off + e_words) * 4 + 16;
    s->corr_off = align_up((size_t)Ci * K * L.J * kp.CoP * sizeof(uint32_t), 256);
    s->wp_bytes = s->corr_off + align_up((size_t)kp.CoP * sizeof(int32_t), 256);
    s->ap_words = (size_t)Ci * B * kp.Hp * kp.XBT;
    if (s->ap_words >= 0x7FFFFFFFull || (size_t)Ci * K * L.J * kp.CoP >= 0x7FFFFFFFull) return HIKONV_ERR_UNSUPPORTED;
    if (s->smem_bytes > 200 * 1024) return HIKONV_ERR_UNSUPPORTED;
    const long long row_tiles = ((long long)kp.total_rows + kp.TR - 1) / kp.TR;
    const long long gx = row_tiles * kp.NSEG;
    const int gy = ceil_div(Co, kp.TCO);
    if (gx > 0x7FFFFFFFLL || gy > 65535) return HIKONV_ERR_UNSUPPORTED;
    s->grid = dim3((unsigned)gx, (unsigned)gy, 1);
    return HIKONV_OK;
}

static int launch_conv2d(const Conv2dSetup &s, cudaStream_t st) {
    const bool sp = s.L.signed_prod != 0;
    const int K = s.kp.K, J = s.L.J;
    if (s.unpacked) {
        if (K == 3) return launch_variant<1, 0, kTMU, kTNU, true, 3, 3>(s, sp, st);
        if (K == 1) return launch_variant<1, 0, kTMU, kTNU, true, 1, 1>(s, sp, st);
        return launch_variant<1, 0, kTMU, kTNU, true, 0, 0>(s, sp, st);
    }
    // the layouts of 3x3 and 1x1 layers with the slot width and loop bounds as compile-time constants
    if (s.L.N == 3 && s.L.S == 13 && K == 3 && J == 1 && s.tm == 2) return launch_variant<3, 13, 2, kTN, false, 3, 1, true>(s, sp, st);
    if (s.L.N == 3 && s.L.S == 13 && K == 3 && J == 1) return launch_variant<3, 13, kTM, kTN, false, 3, 1, true>(s, sp, st);
    if (s.L.N == 3 && s.L.S == 13 && K == 1 && J == 1) return launch_variant<3, 13, kTM, kTN, false, 1, 1>(s, sp, st);
    // 8-bit activations x 4-bit weights with few input channels (a network's first layer): no moves at all
    if (s.L.N == 2 && s.L.S == 17 && K == 3 && J == 2 && s.L.M >= s.kp.Ci * K && s.kp.move_every == 0)
        return s.kp.TCO == s.kp.TNX * kTNShallow ? launch_variant<2, 17, kTM, kTNShallow, false, 3, 2, false, true>(s, sp, st)
                                                 : launch_variant<2, 17, kTM, kTN, false, 3, 2, false, true>(s, sp, st);
    if (s.kp.TCO != s.kp.TNX * kTN) return HIKONV_ERR_UNSUPPORTED;       // every other packed kernel holds four channels per thread
    // 1- and 2-bit codes: four pixels per word, the whole 3x3 kernel row in one word
    if (s.L.N == 4 && K == 3 && J == 1)
        return (s.L.M >= s.kp.Ci * K && s.kp.move_every == 0) ? launch_variant<4, 0, kTM, kTN, false, 3, 1, false, true>(s, sp, st)
                                                              : launch_variant<4, 0, kTM, kTN, false, 3, 1>(s, sp, st);
    if (s.L.N == 2 && K == 3 && J == 2)
        return (s.L.M >= s.kp.Ci * K && s.kp.move_every == 0) ? launch_variant<2, 0, kTM, kTN, false, 3, 2, false, true>(s, sp, st)
                                                              : launch_variant<2, 0, kTM, kTN, false, 3, 2>(s, sp, st);
    if (s.L.N == 2 && K == 3 && J == 1) return launch_variant<2, 0, kTM, kTN, false, 3, 1>(s, sp, st);
    // pointwise layers at the other widths
    if (s.L.N == 4 && K == 1 && J == 1) return launch_variant<4, 0, kTM, kTN, false, 1, 1>(s, sp, st);
    if (s.L.N == 2 && K == 1 && J == 1) return launch_variant<2, 0, kTM, kTN, false, 1, 1>(s, sp, st);
    switch (s.L.N) {
        case 1: return launch_variant<1, 0, kTM, kTN, false, 0, 0>(s, sp, st);
        case 2: return launch_variant<2, 0, kTM, kTN, false, 0, 0>(s, sp, st);
        case 3: return launch_variant<3, 0, kTM, kTN, false, 0, 0>(s, sp, st);
        case 4: return launch_variant<4, 0, kTM, kTN, false, 0, 0>(s, sp, st);
        default: return HIKONV_ERR_UNSUPPORTED;
    }
}

}  // namespace hikonv

using namespace hikonv;

extern "C" size_t hikonv_conv2d_workspace_bytes(int B, int Ci, int H, int W, int Co, int K, int pad) {
    if (B < 1 || Ci < 1 || H < 1 || W < 1 || Co < 1 || K < 1 || pad < 0) return 0;
    const long long Ho = (long long)H + 2 * pad - K + 1, Wo = (long long)W + 2 * pad - K + 1;
    if (Ho < 1 || Wo < 1) return 0;
    // packed kernel rows: at most K words per (ci, kh) row (one tap per word in the comparator), Co rounded up to 4
    // (plus one int32 per channel: the correction of layers that run unsigned activations as signed ones)
    const size_t weights = align_up((size_t)Ci * K * K * ((Co + 3) / 4 * 4) * sizeof(uint32_t), 256) +
                           align_up((size_t)((Co + 3) / 4 * 4) * sizeof(int32_t), 256);
    // packed activation rows: at most one word per output pixel plus K halo words per row (the comparator's
    // layout), rounded up to 16-byte pieces, with one more piece per row segment (segments hold >= 32 blocks)
    const size_t row_words = (size_t)(Wo + K + 3) / 4 * 4 + 16 + (size_t)(Wo + K) / 8;
    const size_t acts = (size_t)Ci * B * (size_t)(Ho + K - 1) * row_words * sizeof(uint32_t);
    return weights + align_up(acts, 256);
}

// One layer: packing launch, then the layer kernel.  x_bits / w_bits: storage of activations and weights (8 = one code
// per byte, else dense); out_bits and pool describe the requantised output (see make_setup).
static int conv2d_run(const void *d_x, int x_bits, int B, int Ci, int H, int W, const void *d_w, int w_bits, int Co, int K,
                      int stride, int pad, int p, int q, int x_signed, int w_signed, void *d_out, int out_bits, int requant,
                      int shift, int lo, int hi, int pool, void *d_workspace, size_t workspace_bytes, int algo,
                      const hikonv_tuning_t *tune, void *stream) {
    if (!d_x || !d_w || !d_out) return HIKONV_ERR_INVALID_ARG;
    Conv2dSetup s;
    int rc = make_setup(B, Ci, H, W, Co, K, stride, pad, p, q, x_signed ? 1 : 0, w_signed ? 1 : 0, requant, shift, lo, hi, algo,
                        tune, &s, pool, d_out, out_bits);
    if (rc != HIKONV_OK) return rc;
    if (!requant && ((uintptr_t)d_out % 4) != 0) return HIKONV_ERR_INVALID_ARG;
    const size_t need = s.wp_bytes + s.ap_words * sizeof(uint32_t);
    if (!d_workspace || ((uintptr_t)d_workspace % 256) != 0 || workspace_bytes < need ||
        workspace_bytes < hikonv_conv2d_workspace_bytes(B, Ci, H, W, Co, K, pad))
        return HIKONV_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    uint32_t *d_wp = (uint32_t *)d_workspace;
    uint32_t *d_ap = (uint32_t *)((char *)d_workspace + s.wp_bytes);
    int32_t *d_corr = (int32_t *)((char *)d_workspace + s.corr_off);
    s.kp.corr = d_corr;
    s.kp.x = (const int8_t *)d_x;
    s.kp.wp = d_wp;
    s.kp.ap = d_ap;
    s.kp.out = d_out;
    // a2: reversed kernel rows packed per (ci, kh, chunk); a3: activation rows packed per block; one launch
    {
        WeightPackParams wq;
        wq.w = (const int8_t *)d_w; wq.wp = d_wp; wq.Co = Co; wq.Ci = Ci; wq.K = K; wq.J = s.L.J; wq.Kc = s.L.Kc; wq.S = s.L.S;
        wq.w_signed = w_signed ? 1 : 0; wq.CoP = s.kp.CoP; wq.total = Ci * K * s.L.J * s.kp.CoP; wq.w_bits = w_bits;
        wq.x_off = s.kp.x_off; wq.corr = d_corr;
        wq.d_cop = make_div32((uint32_t)s.kp.CoP); wq.d_j = make_div32((uint32_t)s.L.J); wq.d_k = make_div32((uint32_t)K);
        const size_t act_items = (size_t)Ci * B * s.kp.Hp * (s.kp.XBT / 4);              // below 2^29: ap_words is below 2^31
        const size_t act_blocks = (act_items + 255) / 256, w_blocks = (size_t)ceil_div(wq.total, 256);
        const size_t corr_blocks = s.kp.x_off ? (size_t)ceil_div(s.kp.CoP, 8) : 0;      // one warp per channel
        wq.w_blocks = (int)w_blocks;
        if (act_blocks + w_blocks + corr_blocks > 0x7FFFFFFFull) return HIKONV_ERR_UNSUPPORTED;
        const unsigned grid = (unsigned)(act_blocks + w_blocks + corr_blocks);
        ActPackDivs dv;
        dv.per_plane = make_div32((uint32_t)(s.kp.Hp * (s.kp.XBT / 4)));
        dv.b = make_div32((uint32_t)B);
        dv.xq = make_div32((uint32_t)(s.kp.XBT / 4));
#define HK_PACK(XSIGN, NN)                                                                                                 \
    rc = launch_dependent(pack_operands_kernel<XSIGN, NN>, dim3(grid), dim3(256), 0, st, (const int8_t *)d_x, B, Ci, H, W, s.kp.Hp, \
                          pad, K, s.L.J, s.L.S, s.kp.XBT, d_ap, (int)(w_blocks + corr_blocks), wq, x_bits, dv, (unsigned)act_items)
        switch (s.L.N * 2 + (x_signed ? 1 : 0)) {
            case 2: HK_PACK(false, 1); break;
            case 3: HK_PACK(true, 1); break;
            case 4: HK_PACK(false, 2); break;
            case 5: HK_PACK(true, 2); break;
            case 6: HK_PACK(false, 3); break;
            case 7: HK_PACK(true, 3); break;
            case 8: HK_PACK(false, 4); break;
            case 9: HK_PACK(true, 4); break;
            default: return HIKONV_ERR_UNSUPPORTED;
        }
#undef HK_PACK
    }
    if (rc != HIKONV_OK) return rc;
    return launch_conv2d(s, st);
}

extern "C" int hikonv_conv2d(const int8_t *d_x, int B, int Ci, int H, int W, const int8_t *d_w, int Co, int K, int stride,
                             int pad, int p, int q, int x_signed, int w_signed, void *d_out, int requant, int shift, int lo,
                             int hi, void *d_workspace, size_t workspace_bytes, int algo, const hikonv_tuning_t *tune,
                             void *stream) {
    return conv2d_run(d_x, 8, B, Ci, H, W, d_w, 8, Co, K, stride, pad, p, q, x_signed, w_signed, d_out, 8, requant, shift, lo, hi, 0,
                      d_workspace, workspace_bytes, algo, tune, stream);
}

static bool storage_bits_ok(int store_bits, int code_bits) {
    return store_bits == 8 || (store_bits == code_bits && (code_bits == 1 || code_bits == 2 || code_bits == 4));
}

extern "C" int hikonv_conv2d_dense(const void *d_x, int x_store_bits, int B, int Ci, int H, int W, const void *d_w,
                                   int w_store_bits, int Co, int K, int stride, int pad, int p, int q, int x_signed,
                                   int w_signed, void *d_out, int out_store_bits, int requant, int shift, int lo, int hi,
                                   int pool, void *d_workspace, size_t workspace_bytes, int algo,
                                   const hikonv_tuning_t *tune, void *stream) {
    if (validate_codes(p, q) != HIKONV_OK) return HIKONV_ERR_INVALID_ARG;
    if (!storage_bits_ok(x_store_bits, p) || !storage_bits_ok(w_store_bits, q)) return HIKONV_ERR_UNSUPPORTED;
    if (!requant && out_store_bits != 32) return HIKONV_ERR_INVALID_ARG;
    if (requant && out_store_bits != 8 && out_store_bits != 4 && out_store_bits != 2 && out_store_bits != 1)
        return HIKONV_ERR_INVALID_ARG;
    return conv2d_run(d_x, x_store_bits, B, Ci, H, W, d_w, w_store_bits, Co, K, stride, pad, p, q, x_signed, w_signed, d_out,
                      requant ? out_store_bits : 8, requant, shift, lo, hi, pool, d_workspace, workspace_bytes, algo, tune, stream);
}

// Times the layer with the library's own tile and with every forced tile shape (positions per thread x channel lanes x
// rows per CTA), `batch` launches between two events, best of `repeats`; the result of every launch is the layer's output.
extern "C" int hikonv_conv2d_tune(const void *d_x, int x_store_bits, int B, int Ci, int H, int W, const void *d_w,
                                  int w_store_bits, int Co, int K, int stride, int pad, int p, int q, int x_signed,
                                  int w_signed, void *d_out, int out_store_bits, int requant, int shift, int lo, int hi,
                                  int pool, void *d_workspace, size_t workspace_bytes, int algo, int repeats, int *h_tile,
                                  double *h_us, double *h_default_us, void *stream) {
    if (!h_tile || repeats < 1 || repeats > 100) return HIKONV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    cudaEvent_t e0, e1;
    HIKONV_CUDA_TRY(cudaEventCreate(&e0));
    if (cudaEventCreate(&e1) != cudaSuccess) {
        cudaEventDestroy(e0);
        return HIKONV_ERR_CUDA;
    }
    constexpr int kBatch = 4;
    // best time in microseconds per launch with this tuning record; negative: the library refused it; rc_cuda set on a CUDA error
    int rc_cuda = HIKONV_OK;
    auto run = [&](const hikonv_tuning_t *tune) {
        return hikonv_conv2d_dense(d_x, x_store_bits, B, Ci, H, W, d_w, w_store_bits, Co, K, stride, pad, p, q, x_signed, w_signed,
                                   d_out, out_store_bits, requant, shift, lo, hi, pool, d_workspace, workspace_bytes, algo, tune, stream);
    };
    auto time_of = [&](const hikonv_tuning_t *tune, double give_up_above) -> double {
        float ms = 0.0f;
        if (cudaEventRecord(e0, st) != cudaSuccess) { rc_cuda = HIKONV_ERR_CUDA; return -1.0; }
        const int rc = run(tune);
        if (rc != HIKONV_OK) {
            if (rc == HIKONV_ERR_CUDA) rc_cuda = rc;
            return -1.0;
        }
        if (cudaEventRecord(e1, st) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess ||
            cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) { rc_cuda = HIKONV_ERR_CUDA; return -1.0; }
        if (ms * 1e3 > give_up_above) return ms * 1e3;               // a first launch this slow cannot win
        double best = 1e30;
        for (int rep = 0; rep < repeats; ++rep) {
            if (cudaEventRecord(e0, st) != cudaSuccess) { rc_cuda = HIKONV_ERR_CUDA; return -1.0; }
            for (int k = 0; k < kBatch; ++k)
                if (run(tune) != HIKONV_OK) { rc_cuda = HIKONV_ERR_CUDA; return -1.0; }
            if (cudaEventRecord(e1, st) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess ||
                cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) { rc_cuda = HIKONV_ERR_CUDA; return -1.0; }
            best = std::min(best, (double)ms * 1e3 / kBatch);
        }
        return best;
    };
    int rc = run(nullptr);                                            // argument errors surface here, before any timing
    double base = -1.0;
    if (rc == HIKONV_OK) {
        base = time_of(nullptr, 1e30);
        if (base < 0.0) rc = rc_cuda != HIKONV_OK ? rc_cuda : HIKONV_ERR_CUDA;
    }
    double best = base;
    int best_tile = 0;
    if (rc == HIKONV_OK) {
        const long long rows = (long long)B * ((long long)H + 2 * pad - K + 1);
        for (int tm = 4; tm >= 2 && rc_cuda == HIKONV_OK; tm -= 2)
            for (int tnx = 1; tnx <= 8 && rc_cuda == HIKONV_OK; tnx *= 2)
                for (int tr = 1; tr <= 48 && tr <= rows && rc_cuda == HIKONV_OK; ++tr) {
                    hikonv_tuning_t tune;
                    std::memset(&tune, 0, sizeof(tune));
                    tune.tile = tr + 1000 * tnx + 100000 * tm;
                    const double t = time_of(&tune, 2.0 * best);
                    if (t >= 0.0 && t < best) { best = t; best_tile = tune.tile; }
                }
        if (rc_cuda != HIKONV_OK) rc = rc_cuda;
    }
    if (rc == HIKONV_OK && best_tile != 0 && best > 0.97 * base) { best = base; best_tile = 0; }   // not worth forcing
    if (rc == HIKONV_OK && best_tile != 0) {
        hikonv_tuning_t tune;                                          // leave d_out written by a complete, untimed launch
        std::memset(&tune, 0, sizeof(tune));
        tune.tile = best_tile;
        rc = run(&tune);
    } else if (rc == HIKONV_OK) {
        rc = run(nullptr);
    }
    if (rc == HIKONV_OK && cudaStreamSynchronize(st) != cudaSuccess) rc = HIKONV_ERR_CUDA;
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (rc != HIKONV_OK) return rc;
    *h_tile = best_tile;
    if (h_us) *h_us = best;
    if (h_default_us) *h_default_us = base;
    return HIKONV_OK;
}

// ---- scratch that needs no allocation: a fixed buffer inside the library image, one copy per GPU
static __device__ __align__(256) unsigned char g_static_scratch[HIKONV_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void *g_scratch_ptr[kMaxDevices] = {nullptr};

// Is `ptr` device memory of GPU `dev`?  (A query of the pointer's attributes; nothing is allocated.)
bool on_device(const void *ptr, int dev) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, ptr) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return (attr.type == cudaMemoryTypeDevice || attr.type == cudaMemoryTypeManaged) && attr.device == dev;
}

// Device address of g_static_scratch on the current device.  In host code the array's name is only
// a handle, so the address is asked for once per device and cached.  The buffer of the CURRENT device is
// used, so the operands must live there: a buffer of one GPU must not reach kernels that run on another.
int static_scratch_address(void **out, const void *d_x, const void *d_out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return HIKONV_ERR_CUDA;
    if (!d_x || !d_out || !on_device(d_x, dev) || !on_device(d_out, dev)) return HIKONV_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return HIKONV_ERR_CUDA;
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return HIKONV_OK;
}
}  // namespace

extern "C" int hikonv_conv2d_static_scratch(const int8_t *d_x, int B, int Ci, int H, int W, const int8_t *d_w, int Co, int K,
                                            int stride, int pad, int p, int q, int x_signed, int w_signed, void *d_out,
                                            int requant, int shift, int lo, int hi, int algo, const hikonv_tuning_t *tune,
                                            void *stream) {
    const size_t need = hikonv_conv2d_workspace_bytes(B, Ci, H, W, Co, K, pad);
    if (need == 0) return HIKONV_ERR_INVALID_ARG;
    if (need > (size_t)HIKONV_STATIC_SCRATCH_BYTES) return HIKONV_ERR_TOO_LARGE;
    void *scratch = nullptr;
    const int rc = static_scratch_address(&scratch, d_x, d_out);
    if (rc != HIKONV_OK) return rc;
    // the packing kernels write every word the layer kernel reads, so stale contents are harmless
    return hikonv_conv2d(d_x, B, Ci, H, W, d_w, Co, K, stride, pad, p, q, x_signed, w_signed, d_out, requant, shift, lo, hi,
                         scratch, (size_t)HIKONV_STATIC_SCRATCH_BYTES, algo, tune, stream);
}

extern "C" size_t hikonv_conv2d_host_workspace_bytes(int B, int Ci, int H, int W, int Co, int K, int pad, int requant) {
    if (B < 1 || Ci < 1 || H < 1 || W < 1 || Co < 1 || K < 1 || pad < 0) return 0;
    const long long Ho = H + 2 * pad - K + 1, Wo = W + 2 * pad - K + 1;
    if (Ho < 1 || Wo < 1) return 0;
    const size_t out_bytes = (size_t)B * Co * Ho * Wo * (requant ? 1 : 4);
    return align_up((size_t)B * Ci * H * W, 256) + align_up((size_t)Co * Ci * K * K, 256) + align_up(out_bytes, 256) +
           hikonv_conv2d_workspace_bytes(B, Ci, H, W, Co, K, pad);
}

extern "C" int hikonv_conv2d_host(const int8_t *h_x, int B, int Ci, int H, int W, const int8_t *h_w, int Co, int K, int stride,
                                  int pad, int p, int q, int x_signed, int w_signed, void *h_out, int requant, int shift, int lo,
                                  int hi, void *d_workspace, size_t workspace_bytes, int algo, const hikonv_tuning_t *tune,
                                  void *stream) {
    if (!h_x || !h_w || !h_out) return HIKONV_ERR_INVALID_ARG;
    const size_t need = hikonv_conv2d_host_workspace_bytes(B, Ci, H, W, Co, K, pad, requant);
    if (need == 0) return HIKONV_ERR_INVALID_ARG;
    if (!d_workspace || ((uintptr_t)d_workspace % 256) != 0 || workspace_bytes < need) return HIKONV_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t x_bytes = (size_t)B * Ci * H * W, w_bytes = (size_t)Co * Ci * K * K;
    const size_t Ho = H + 2 * pad - K + 1, Wo = W + 2 * pad - K + 1;
    const size_t out_bytes = (size_t)B * Co * Ho * Wo * (requant ? 1 : 4);
    int8_t *d_x = (int8_t *)d_workspace;
    int8_t *d_w = d_x + align_up(x_bytes, 256);
    int8_t *d_out = d_w + align_up(w_bytes, 256);
    int8_t *d_ws = d_out + align_up(out_bytes, 256);
    HIKONV_CUDA_TRY(cudaMemcpyAsync(d_x, h_x, x_bytes, cudaMemcpyHostToDevice, st));
    HIKONV_CUDA_TRY(cudaMemcpyAsync(d_w, h_w, w_bytes, cudaMemcpyHostToDevice, st));
    const int rc = hikonv_conv2d(d_x, B, Ci, H, W, d_w, Co, K, stride, pad, p, q, x_signed, w_signed, d_out, requant, shift, lo,
                                 hi, d_ws, hikonv_conv2d_workspace_bytes(B, Ci, H, W, Co, K, pad), algo, tune, st);
    if (rc != HIKONV_OK) return rc;
    HIKONV_CUDA_TRY(cudaMemcpyAsync(h_out, d_out, out_bytes, cudaMemcpyDeviceToHost, st));
    return HIKONV_OK;
}

extern "C" int hikonv_maxpool2x2_i8(const int8_t *d_in, int B, int C, int H, int W, int is_signed, int8_t *d_out, void *stream) {
    if (!d_in || !d_out || B < 1 || C < 1 || H < 1 || W < 1) return HIKONV_ERR_INVALID_ARG;
    const long long total = (long long)B * C * (H / 2) * (W / 2);
    if (total == 0) return HIKONV_OK;
    if ((double)B * C >= 2147483647.0) return HIKONV_ERR_UNSUPPORTED;
    const long long cap = (long long)sm_count() * 32;
    const cudaStream_t pst = (cudaStream_t)stream;
    if (W % 16 == 0 && ((uintptr_t)d_in % 16) == 0 && ((uintptr_t)d_out % 8) == 0) {
        const long long items = total / 8;
        const unsigned grid = (unsigned)std::min((items + 255) / 256, cap);
        if (is_signed) return launch_dependent(maxpool2x2_vec_kernel<true, 16>, dim3(grid), dim3(256), 0, pst, d_in, items, H, W, d_out);
        return launch_dependent(maxpool2x2_vec_kernel<false, 16>, dim3(grid), dim3(256), 0, pst, d_in, items, H, W, d_out);
    }
    if (W % 8 == 0 && ((uintptr_t)d_in % 8) == 0 && ((uintptr_t)d_out % 4) == 0) {
        const long long items = total / 4;
        const unsigned grid = (unsigned)std::min((items + 255) / 256, cap);
        if (is_signed) return launch_dependent(maxpool2x2_vec_kernel<true, 8>, dim3(grid), dim3(256), 0, pst, d_in, items, H, W, d_out);
        return launch_dependent(maxpool2x2_vec_kernel<false, 8>, dim3(grid), dim3(256), 0, pst, d_in, items, H, W, d_out);
    }
    long long blocks = (total + 255) / 256;
    if (blocks > cap) blocks = cap;
    return launch_plain(maxpool2x2_kernel, dim3((unsigned)blocks), dim3(256), 0, (cudaStream_t)stream, d_in, B * C, H, W,
                        is_signed ? 1 : 0, d_out);
}

extern "C" int hikonv_conv2d_layout(int B, int Ci, int H, int W, int Co, int K, int pad, int p, int q, int x_signed,
                                    int w_signed, const hikonv_tuning_t *tune, hikonv_layout_t *out, int *x_shift) {
    if (!out) return HIKONV_ERR_INVALID_ARG;
    Conv2dSetup s;
    const int rc = make_setup(B, Ci, H, W, Co, K, 1, pad, p, q, x_signed ? 1 : 0, w_signed ? 1 : 0, 0, 0, 0, 0,
                              HIKONV_ALGO_PACKED32, tune, &s);
    if (rc != HIKONV_OK) return rc;
    *out = s.L;
    if (x_shift) *x_shift = s.kp.x_off;
    return HIKONV_OK;
}

extern "C" double hikonv_conv2d_multiplies(int B, int Ci, int H, int W, int Co, int K, int pad, int p, int q, int x_signed,
                                           int w_signed, int algo, const hikonv_tuning_t *tune) {
    Conv2dSetup s;
    if (make_setup(B, Ci, H, W, Co, K, 1, pad, p, q, x_signed ? 1 : 0, w_signed ? 1 : 0, 0, 0, 0, 0, algo, tune, &s) != HIKONV_OK)
        return 0.0;
    // one multiply per position, channel pair and (kh, j): halo positions included, idle threads not
    const double positions = (double)s.kp.total_rows * s.kp.NSEG * s.kp.XB;
    return positions * (double)Co * Ci * K * s.L.J;
}
