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
// A CTA computes TR consecutive output rows (one row segment each) times TCO output channels; it
// is a register-tiled integer "GEMM" over packed words: each thread owns TM consecutive positions
// times TN channels, the k dimension runs over (ci, kh, j).
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

#include "hikonv_cuda.cuh"

namespace hikonv {

constexpr int kMaxThreads2D = 256;
constexpr int kMaxN2DSeg = 8;      // N + Kc - 1 <= 2 N <= 8

struct Conv2dParams {
    const int8_t *x;
    const uint32_t *wp;        // packed weights [Ci*K*J][CoP]
    void *out;
    int B, Ci, H, W, Co, CoP, K, pad, Ho, Wo, Hp;
    int S, J, Kc, M;
    int X;                     // output blocks per row
    int NSEG, XO, XB;          // row segments, output blocks per segment, positions per segment (XO + J)
    int TR, TMX, TNX, TCO, CK;
    int NRmax, a_plane, lead;
    int b_off;                 // word offset of the two weight tiles in shared memory (multiple of 4: 16-byte loads)
    int b_words;               // words per weight tile (CK * K * J * TCO)
    int raw_off, RPW;          // word offset of the raw activation rows, and their pitch in words
    int async_ok;              // x is 4-byte aligned: rows can be fetched with 4-byte asynchronous copies
    int x_bytes;               // B * Ci * H * W
    int requant, shift, lo, hi;
    int total_rows;            // B * Ho
    int flush_chunks;          // channel chunks accumulated between two splits (CK * K * flush_chunks <= M)
    int hbits, nslots;         // carry-save: low bits kept per slot; number of slots N + Kc - 1
    uint64_t bias, mask_low, mask_high;
    uint32_t slot_mask, top_mask;
    int32_t slot_bias[kMaxN2DSeg];
};

template <bool UNPACKED>
struct AccType {
    typedef uint64_t type;
};
template <>
struct AccType<true> {
    typedef int32_t type;
};

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

// N: pixels per packed word; SC: slot width when known at compile time (0: read from the parameters);
// TM x TN: per-thread tile (positions x channels); UNPACKED: comparator (N == 1, one tap per word,
// 32-bit multiply-add, int32 accumulators); SP: signed product; XS: signed activations;
// KT, JT: kernel size and chunks per kernel row when known at compile time (0, 0: read from the
// parameters; the (kh, j) loops are then not unrolled).
template <int N, int SC, int TM, int TN, bool UNPACKED, bool SP, bool XS, int KT, int JT>
__global__ void __launch_bounds__(kMaxThreads2D, 2) conv2d_kernel(const Conv2dParams p) {
    typedef typename AccType<UNPACKED>::type acc_t;
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t *As = smem;                                   // [CK][a_plane]
    uint32_t *Bs = As + p.b_off;                           // two tiles [CK*K*J][TCO], 16-byte aligned
    uint32_t *raw = As + p.raw_off;                        // [CK][NR][RPW] input rows as fetched (bytes, 4-byte granules)
    int *s_row = (int *)(raw + p.CK * p.NRmax * p.RPW);    // [NRmax] input offset of each staged row, -1 = zero row

    const int tid = threadIdx.x, nthreads = blockDim.x;
    const int warp = tid >> 5, lane = tid & 31, nwarps = nthreads >> 5;
    const int tn = tid % p.TNX, tm = tid / p.TNX;
    const int seg = blockIdx.x % p.NSEG;
    const int R0 = (blockIdx.x / p.NSEG) * p.TR;
    const int co0 = blockIdx.y * p.TCO;
    const int TRe = min(p.TR, p.total_rows - R0);
    const int b0 = R0 / p.Ho, h0 = R0 - b0 * p.Ho;
    const int Rp0 = b0 * p.Hp + h0;                         // first staged padded row
    const int Rlast = R0 + TRe - 1;
    const int bl = Rlast / p.Ho;
    const int NR = (bl * p.Hp + (Rlast - bl * p.Ho) + p.K - 1) - Rp0 + 1;
    const int TP = TRe * p.XB;                              // positions of this tile
    const int S = SC > 0 ? SC : p.S;

    for (int rl = tid; rl < NR; rl += nthreads) {
        const int rp = Rp0 + rl;
        const int b = rp / p.Hp, hi = rp - b * p.Hp - p.pad;
        s_row[rl] = (b < p.B && hi >= 0 && hi < p.H) ? (b * p.Ci * p.H + hi) * p.W : -1;
    }

    // this thread's positions: shared-memory address of the packed word for (ci = 0, kh = 0, j = 0)
    const uint32_t *aptr[TM];
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int pos = tm * TM + i;
        int off = p.lead;                                    // idle position: reads valid memory, result dropped
        if (pos < TP) {
            const int r = pos / p.XB, xb = pos - r * p.XB;
            const int R = R0 + r;
            const int b = R / p.Ho;
            off = p.lead + ((b * p.Hp + (R - b * p.Ho)) - Rp0) * p.XB + xb;
        }
        aptr[i] = As + off;
    }

    acc_t acc[TM][TN];
    acc_t E[UNPACKED ? 1 : TM][UNPACKED ? 1 : TN];     // second packed accumulator (upper slot bits)
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int t = 0; t < TN; ++t) acc[i][t] = UNPACKED ? (acc_t)0 : (acc_t)p.bias;
    if constexpr (!UNPACKED) {
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int t = 0; t < TN; ++t) E[i][t] = 0;
    }
    int nmoves = 0, chunks_since_move = 0;

    // move the upper bits of every slot to E and restart the slots at their bias
    auto carry_save = [&]() {
        if constexpr (!UNPACKED) {
            const uint64_t mask_high = p.mask_high, mask_low = p.mask_low, bias = p.bias;
            const int h = p.hbits;
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int t = 0; t < TN; ++t) {
                    const uint64_t Q = (uint64_t)acc[i][t];
                    E[i][t] += (Q >> h) & mask_high;
                    acc[i][t] = (acc_t)((Q & mask_low) | bias);
                }
            ++nmoves;
        }
    };

    const int HW = p.H * p.W;
    const int KJ = p.K * p.J;
    uint32_t slot_pow[N];
#pragma unroll
    for (int n = 0; n < N; ++n) slot_pow[n] = UNPACKED ? 1u : (1u << (S * n));
    const int col_seg0 = (seg * p.XO - p.J) * N + p.K - 1 - p.pad;   // input column of slot 0 at xb = 0
    const int c_lo = max(col_seg0, 0), c_hi = min(p.W, col_seg0 + p.XB * N);   // input columns this row segment reads
    const unsigned long long xaddr = (unsigned long long)p.x;

    // Asynchronous fetch of one stage: the input rows of ckn channels as they are (4-byte granules that
    // cover the needed columns, whatever the row's alignment) and the packed kernel rows for TCO channels.
    auto fetch = [&](int ci0, int ckn, uint32_t *Bdst) {
        if (c_hi > c_lo) {
            for (int cl = 0; cl < ckn; ++cl) {
                for (int rl = warp; rl < NR; rl += nwarps) {
                    const int base = s_row[rl];
                    if (base < 0) continue;
                    const int first = base + (ci0 + cl) * HW + c_lo;          // byte offset of the first needed code
                    const int phase = (int)((xaddr + (unsigned long long)first) & 3ull);
                    const int nwords = (phase + (c_hi - c_lo) + 3) >> 2;
                    uint32_t *dst = raw + (cl * NR + rl) * p.RPW;
                    if (p.async_ok) {
                        const int8_t *src = p.x + (first - phase);
                        for (int wd = lane; wd < nwords; wd += 32) {
                            const int left = p.x_bytes - (first - phase + 4 * wd);  // bytes up to the end of the tensor
                            cp_async_4(dst + wd, src + 4 * wd, left >= 4 ? 4 : left);
                        }
                    } else {
                        for (int wd = lane; wd < nwords; wd += 32) {
                            uint32_t v = 0;
#pragma unroll
                            for (int bb = 0; bb < 4; ++bb) {
                                const int off = first - phase + 4 * wd + bb;
                                if (off >= 0 && off < p.x_bytes) v |= (uint32_t)(uint8_t)__ldg(p.x + off) << (8 * bb);
                            }
                            dst[wd] = v;
                        }
                    }
                }
            }
        }
        const int tco4 = p.TCO / 4;
        const int rows = ckn * KJ;
        for (int idx = tid; idx < rows * tco4; idx += nthreads) {
            const int kr = idx / tco4, c4 = idx - kr * tco4;
            const int co = co0 + c4 * 4;
            uint32_t *dst = Bdst + (kr * tco4 + c4) * 4;
            if (co < p.CoP) cp_async_16(dst, p.wp + (size_t)(ci0 * KJ + kr) * p.CoP + co);
            else *reinterpret_cast<uint4 *>(dst) = make_uint4(0, 0, 0, 0);
        }
        cp_async_commit();
    };

    // Packs the fetched rows into A words (Eq. 5): a warp per row, a lane per word.
    auto pack_rows = [&](int ci0, int ckn) {
        for (int cl = 0; cl < ckn; ++cl) {
            for (int rl = warp; rl < NR; rl += nwarps) {
                const int base = s_row[rl];
                uint32_t *dst = As + cl * p.a_plane + p.lead + rl * p.XB;
                if (base < 0 || c_hi <= c_lo) {
                    for (int xb = lane; xb < p.XB; xb += 32) dst[xb] = 0;
                    continue;
                }
                const int first = base + (ci0 + cl) * HW + c_lo;
                const int phase = (int)((xaddr + (unsigned long long)first) & 3ull);
                const int8_t *rb = reinterpret_cast<const int8_t *>(raw + (cl * NR + rl) * p.RPW) + phase - c_lo;   // rb[col]
                for (int xb = lane; xb < p.XB; xb += 32) {
                    const int col0 = col_seg0 + xb * N;
                    uint32_t word = 0;
                    if (col0 >= c_lo && col0 + N <= c_hi) {
#pragma unroll
                        for (int n = 0; n < N; ++n) {
                            const uint32_t c = (uint32_t)code_value<XS>(rb[col0 + n]);
                            word = (n == 0) ? c : word + c * slot_pow[n];
                        }
                    } else {
#pragma unroll
                        for (int n = 0; n < N; ++n) {
                            const int col = col0 + n;
                            if (col >= c_lo && col < c_hi) word += (uint32_t)code_value<XS>(rb[col]) * slot_pow[n];
                        }
                    }
                    dst[xb] = word;
                }
            }
        }
    };

    __syncthreads();                                                 // s_row is written
    fetch(0, min(p.CK, p.Ci), Bs);
    int stage = 0;
    for (int ci0 = 0; ci0 < p.Ci; ci0 += p.CK, stage ^= 1) {
        const int ckn = min(p.CK, p.Ci - ci0);
        cp_async_wait_all();
        __syncthreads();                                             // this stage has landed; the previous one is fully consumed
        pack_rows(ci0, ckn);
        __syncthreads();                                             // A words ready; the raw rows may be overwritten
        if (ci0 + p.CK < p.Ci) fetch(ci0 + p.CK, min(p.CK, p.Ci - ci0 - p.CK), Bs + (stage ^ 1) * p.b_words);
        const uint32_t *bptr = Bs + stage * p.b_words + tn * TN;
        // ---- multiply-accumulate over (ci, kh, j)
        if constexpr (KT > 0) {
            for (int cl = 0; cl < ckn; ++cl) {
                const int abase = cl * p.a_plane;
                const int bbase = cl * (KT * JT) * p.TCO;
#pragma unroll
                for (int kh = 0; kh < KT; ++kh) {
#pragma unroll
                    for (int j = 0; j < JT; ++j) {
                        const int aoff = abase + kh * p.XB - j;
                        const uint32_t *brow = bptr + bbase + (kh * JT + j) * p.TCO;
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
        } else {
            for (int cl = 0; cl < ckn; ++cl) {
                for (int kh = 0; kh < p.K; ++kh) {
                    for (int j = 0; j < p.J; ++j) {
                        const int aoff = cl * p.a_plane + kh * p.XB - j;
                        const uint32_t *brow = bptr + ((cl * p.K + kh) * p.J + j) * p.TCO;
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
        if (!UNPACKED && ++chunks_since_move == p.flush_chunks && ci0 + p.CK < p.Ci) { carry_save(); chunks_since_move = 0; }
    }

    // ---- extract the slots: slot m holds 2^h E_m + Q_m - (moves + 1) bias_m (uint32 arithmetic wraps by design)
    const uint32_t nb = (uint32_t)nmoves + 1u;
    auto slot_value = [&](uint64_t Q, uint64_t Ev, int m) -> uint32_t {
        const uint32_t msk = (m == p.nslots - 1) ? p.top_mask : p.slot_mask;
        const uint32_t qv = (uint32_t)(Q >> (S * m)) & msk;
        const uint32_t ev = (uint32_t)(Ev >> (S * m)) & msk;
        return (ev << p.hbits) + qv - nb * (uint32_t)p.slot_bias[m];
    };
    // the upper slots of a thread's last position belong to the next thread's first position (Theorem 2)
    if constexpr (!UNPACKED) {
        __syncthreads();
        uint32_t *xch = smem;                                        // [TMX][N][TCO]
#pragma unroll
        for (int m = 0; m < N; ++m)
#pragma unroll
            for (int t = 0; t < TN; ++t)
                xch[(tm * N + m) * p.TCO + tn * TN + t] =
                    (N + m < p.nslots) ? slot_value((uint64_t)acc[TM - 1][t], (uint64_t)E[TM - 1][t], N + m) : 0u;
        __syncthreads();
    }

    // ---- overlap-add, optional requantisation (arithmetic shift, clamp), store
#pragma unroll
    for (int t = 0; t < TN; ++t) {
        const int co = co0 + tn * TN + t;
        uint32_t upper[N];                                           // upper slots of the previous position
        if constexpr (!UNPACKED) {
#pragma unroll
            for (int m = 0; m < N; ++m) upper[m] = (tm > 0) ? smem[((tm - 1) * N + m) * p.TCO + tn * TN + t] : 0u;
        }
#pragma unroll
        for (int i = 0; i < TM; ++i) {
            uint32_t Y[N];
            if constexpr (!UNPACKED) {
#pragma unroll
                for (int m = 0; m < N; ++m) Y[m] = slot_value((uint64_t)acc[i][t], (uint64_t)E[i][t], m) + upper[m];
#pragma unroll
                for (int m = 0; m < N; ++m)
                    upper[m] = (N + m < p.nslots) ? slot_value((uint64_t)acc[i][t], (uint64_t)E[i][t], N + m) : 0u;
            } else {
                Y[0] = (uint32_t)acc[i][t];
            }
            const int pos = tm * TM + i;
            if (pos >= TP || co >= p.Co) continue;
            const int r = pos / p.XB, xbl = pos - r * p.XB;
            if (xbl < p.J) continue;                                 // halo positions produce no pixels
            const int xg = seg * p.XO + xbl - p.J;                   // output block in the row
            if (xg >= p.X) continue;
            const int R = R0 + r;
            const int b = R / p.Ho, h = R - b * p.Ho;
            const size_t row_off = (((size_t)b * p.Co + co) * p.Ho + h) * p.Wo;
#pragma unroll
            for (int m = 0; m < N; ++m) {
                const int w = xg * N + m;
                if (w >= p.Wo) continue;
                int32_t v = (int32_t)Y[m];
                if (p.requant) {
                    v >>= p.shift;
                    v = max(p.lo, min(p.hi, v));
                    ((int8_t *)p.out)[row_off + w] = (int8_t)v;
                } else {
                    ((int32_t *)p.out)[row_off + w] = v;
                }
            }
        }
    }
}

// Reversed, packed kernel rows (Theorem 3: g = W[co][ci][kh][K-1:0], then Eq. 5 per chunk of Kc taps).
// wp[((ci*K + kh)*J + j)*CoP + co] = sum_{k' < Kc} g[j Kc + k'] 2^(S k').  For the comparator S == 0,
// Kc == 1: one int32 weight per word.
__global__ void __launch_bounds__(256) pack_weights_kernel(const int8_t *__restrict__ w, int Co, int Ci, int K, int J, int Kc,
                                                           int S, int w_signed, int CoP, uint32_t *__restrict__ wp, int total) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int co = idx % CoP;
    int rest = idx / CoP;
    const int j = rest % J;
    rest /= J;
    const int kh = rest % K;
    const int ci = rest / K;
    uint32_t word = 0;
    if (co < Co) {
        const int8_t *row = w + (((size_t)co * Ci + ci) * K + kh) * K;
        for (int k = 0; k < Kc; ++k) {
            const int g_idx = j * Kc + k;                // index into the reversed row
            if (g_idx < K) {
                const int8_t raw = __ldg(row + (K - 1 - g_idx));
                const int32_t v = w_signed ? (int32_t)raw : (int32_t)(uint8_t)raw;
                word += (uint32_t)v << (S * k);
            }
        }
    }
    wp[idx] = word;
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
    dim3 grid;
    int threads;
    bool unpacked;
};

static int sm_count() {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms;
}

template <int N, int SC, int TM, int TN, bool UNPACKED, int KT, int JT>
static int launch_variant(const Conv2dSetup &s, bool sp, bool xs, cudaStream_t st) {
#define HK_LAUNCH(SPV, XSV)                                                                                      \
    do {                                                                                                         \
        auto kern = conv2d_kernel<N, SC, TM, TN, UNPACKED, SPV, XSV, KT, JT>;                                    \
        if (s.smem_bytes > 48 * 1024)                                                                            \
            HIKONV_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s.smem_bytes)); \
        kern<<<s.grid, s.threads, s.smem_bytes, st>>>(s.kp);                                                     \
    } while (0)
    if (!sp) HK_LAUNCH(false, false);
    else if (xs) HK_LAUNCH(true, true);
    else HK_LAUNCH(true, false);
#undef HK_LAUNCH
    return launch_status();
}

constexpr int kTM = 4, kTN = 4;          // per-thread tile of the packed kernels
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
                               int force_tr) {
    TileChoice best;
    best.cost = -1.0;
    for (int TNX = 1; TNX <= 16; TNX *= 2) {
        const int TCO = TNX * TN;
        if (TNX > 1 && TCO / 2 >= Co) break;                       // more channel lanes than channels
        const int gy = ceil_div(Co, TCO);
        const int max_tmx = kMaxThreads2D / TNX;
        const int maxpos = max_tmx * TM;
        int NSEG = 1;
        while (ceil_div(X, NSEG) + J > maxpos) ++NSEG;
        const int XO = ceil_div(X, NSEG), XB = XO + J;
        const int tr_hi = std::max(1, std::min(maxpos / XB, total_rows));
        const int tr_lo = force_tr > 0 ? std::min(force_tr, tr_hi) : 1;
        const int tr_end = force_tr > 0 ? tr_lo : tr_hi;
        for (int TR = tr_lo; TR <= tr_end; ++TR) {
            int TMX = ceil_div(TR * XB, TM);
            int threads = (TMX * TNX + 31) / 32 * 32;               // whole warps
            if (threads > kMaxThreads2D) continue;
            TMX = threads / TNX;
            const long long tiles = (long long)ceil_div(total_rows, TR) * NSEG * gy;
            const int per_sm = std::max(1, std::min(2048 / threads, 65536 / (threads * 128)));
            const long long slots = (long long)per_sm * sms;
            const long long full_waves = tiles / slots;
            const long long rest = tiles - full_waves * slots;
            double time = (double)full_waves * std::max(per_sm * threads, 256);
            if (rest > 0) time += std::max((int)((rest + sms - 1) / sms) * threads, 256);
            const int span = (TR + Ho - 2) / Ho + 1;
            const double NR = TR + (K - 1) * span;
            const double work = (double)K * J * (TM * TN + 8) * threads;
            const double stage = NR * XB * (4.0 * N + 10.0) + (double)K * J * TCO;
            time *= 1.0 + stage / work;
            const double useful = (double)total_rows * X * Co;     // output blocks x channels
            const double cost = time * sms / useful;
            if (best.cost < 0 || cost < best.cost - 1e-12) best = {TNX, TMX, TR, NSEG, XO, XB, cost};
        }
    }
    return best;
}

static int make_setup(int B, int Ci, int H, int W, int Co, int K, int stride, int pad, int p, int q, int xs, int ws,
                      int requant, int shift, int lo, int hi, int algo, const hikonv_tuning_t *tune, Conv2dSetup *s) {
    if (B < 1 || Ci < 1 || H < 1 || W < 1 || Co < 1 || K < 1 || K > kMaxK) return HIKONV_ERR_INVALID_ARG;
    if (validate_codes(p, q) != HIKONV_OK) return HIKONV_ERR_INVALID_ARG;
    if (stride != 1 || pad < 0 || pad >= K) return HIKONV_ERR_UNSUPPORTED;
    if (algo == HIKONV_ALGO_PACKED64EMU) return HIKONV_ERR_UNSUPPORTED;
    if (algo != HIKONV_ALGO_PACKED32 && algo != HIKONV_ALGO_UNPACKED_IMAD) return HIKONV_ERR_INVALID_ARG;
    if (requant && (shift < 0 || shift > 31 || lo < -128 || hi > 255 || lo > hi)) return HIKONV_ERR_INVALID_ARG;
    const int Ho = H + 2 * pad - K + 1, Wo = W + 2 * pad - K + 1;
    if (Ho < 1 || Wo < 1) return HIKONV_ERR_INVALID_ARG;
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
        if (K > kMaxJ) return HIKONV_ERR_UNSUPPORTED;
    } else {
        int rc = make_layout(p, q, xs, ws, K, 2, Ci * K, Wo, tune, &L);
        if (rc != HIKONV_OK) return rc;
        if (L.N > kMaxN2D || L.segments > kMaxN2DSeg) return HIKONV_ERR_UNSUPPORTED;
        TM = kTM; TN = kTN; N = L.N;
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
    const TileChoice tc = choose_tiles(kp.total_rows, Ho, kp.X, N, K, L.J, Co, TM, TN, sm_count(), tune ? tune->tile : 0);
    if (tc.cost < 0) return HIKONV_ERR_UNSUPPORTED;
    kp.TNX = tc.TNX; kp.TMX = tc.TMX; kp.TCO = tc.TNX * TN;
    kp.NSEG = tc.NSEG; kp.XO = tc.XO; kp.XB = tc.XB; kp.TR = tc.TR;
    s->threads = tc.TMX * tc.TNX;
    const int span = (kp.TR + Ho - 2) / Ho + 1;              // images a tile can touch
    kp.NRmax = kp.TR + (K - 1) * span;
    kp.lead = L.J;                                           // room for the xb - j reads at the front
    kp.a_plane = kp.NRmax * kp.XB + kp.lead;
    // channels per stage and stages between two carry-save moves (at most M (ci, kh) pairs)
    int CK = std::min(8, Ci);
    kp.flush_chunks = 1 << 30;
    if (!s->unpacked && L.M < Ci * K) {
        if (L.M < K) return HIKONV_ERR_NO_FIT;               // not even one channel's kernel rows between two moves
        int fc = 1;
        const int eff = pick_chunking(L.M / K, Ci, &CK, &fc);
        if (ceil_div(Ci, eff) > (1 << L.carry_bits)) return HIKONV_ERR_NO_FIT;
        kp.flush_chunks = fc;
    }
    kp.CK = CK;
    kp.b_off = (CK * kp.a_plane + 3) / 4 * 4;
    kp.b_words = CK * K * L.J * kp.TCO;
    kp.raw_off = kp.b_off + 2 * kp.b_words;
    kp.RPW = (std::min(W, kp.XB * N) + 6) / 4 + 1;
    kp.x_bytes = B * Ci * H * W;
    size_t words = (size_t)kp.raw_off + (size_t)CK * kp.NRmax * kp.RPW + (size_t)kp.NRmax;
    size_t xch_words = s->unpacked ? 0 : (size_t)kp.TMX * N * kp.TCO;
    s->smem_bytes = std::max(words, xch_words) * 4 + 16;
    if (s->smem_bytes > 200 * 1024) return HIKONV_ERR_UNSUPPORTED;
    const long long row_tiles = ((long long)kp.total_rows + kp.TR - 1) / kp.TR;
    const long long gx = row_tiles * kp.NSEG;
    const int gy = ceil_div(Co, kp.TCO);
    if (gx > 0x7FFFFFFFLL || gy > 65535) return HIKONV_ERR_UNSUPPORTED;
    s->grid = dim3((unsigned)gx, (unsigned)gy, 1);
    return HIKONV_OK;
}

static int launch_conv2d(const Conv2dSetup &s, bool xs, cudaStream_t st) {
    const bool sp = s.L.signed_prod != 0;
    const int K = s.kp.K, J = s.L.J;
    if (s.unpacked) {
        if (K == 3) return launch_variant<1, 0, kTMU, kTNU, true, 3, 3>(s, sp, xs, st);
        if (K == 1) return launch_variant<1, 0, kTMU, kTNU, true, 1, 1>(s, sp, xs, st);
        return launch_variant<1, 0, kTMU, kTNU, true, 0, 0>(s, sp, xs, st);
    }
    // the layouts of 3x3 and 1x1 layers with the slot width and loop bounds as compile-time constants
    if (s.L.N == 3 && s.L.S == 13 && K == 3 && J == 1) return launch_variant<3, 13, kTM, kTN, false, 3, 1>(s, sp, xs, st);
    if (s.L.N == 3 && s.L.S == 13 && K == 1 && J == 1) return launch_variant<3, 13, kTM, kTN, false, 1, 1>(s, sp, xs, st);
    if (s.L.N == 2 && K == 3 && J == 2) return launch_variant<2, 0, kTM, kTN, false, 3, 2>(s, sp, xs, st);
    if (s.L.N == 2 && K == 3 && J == 1) return launch_variant<2, 0, kTM, kTN, false, 3, 1>(s, sp, xs, st);
    switch (s.L.N) {
        case 1: return launch_variant<1, 0, kTM, kTN, false, 0, 0>(s, sp, xs, st);
        case 2: return launch_variant<2, 0, kTM, kTN, false, 0, 0>(s, sp, xs, st);
        case 3: return launch_variant<3, 0, kTM, kTN, false, 0, 0>(s, sp, xs, st);
        case 4: return launch_variant<4, 0, kTM, kTN, false, 0, 0>(s, sp, xs, st);
        default: return HIKONV_ERR_UNSUPPORTED;
    }
}

}  // namespace hikonv

using namespace hikonv;

extern "C" size_t hikonv_conv2d_workspace_bytes(int Ci, int Co, int K) {
    if (Ci < 1 || Co < 1 || K < 1) return 0;
    // at most K words per (ci, kh) row (one tap per word in the comparator), Co rounded up to 4
    return align_up((size_t)Ci * K * K * ((Co + 3) / 4 * 4) * sizeof(uint32_t), 256);
}

extern "C" int hikonv_conv2d(const int8_t *d_x, int B, int Ci, int H, int W, const int8_t *d_w, int Co, int K, int stride,
                             int pad, int p, int q, int x_signed, int w_signed, void *d_out, int requant, int shift, int lo,
                             int hi, void *d_workspace, size_t workspace_bytes, int algo, const hikonv_tuning_t *tune,
                             void *stream) {
    if (!d_x || !d_w || !d_out) return HIKONV_ERR_INVALID_ARG;
    Conv2dSetup s;
    int rc = make_setup(B, Ci, H, W, Co, K, stride, pad, p, q, x_signed ? 1 : 0, w_signed ? 1 : 0, requant, shift, lo, hi, algo,
                        tune, &s);
    if (rc != HIKONV_OK) return rc;
    if (!requant && ((uintptr_t)d_out % 4) != 0) return HIKONV_ERR_INVALID_ARG;
    if (!d_workspace || ((uintptr_t)d_workspace % 256) != 0 || workspace_bytes < hikonv_conv2d_workspace_bytes(Ci, Co, K))
        return HIKONV_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    s.kp.x = d_x;
    s.kp.async_ok = ((uintptr_t)d_x % 4 == 0) ? 1 : 0;
    s.kp.wp = (const uint32_t *)d_workspace;
    s.kp.out = d_out;
    const int total = Ci * K * s.L.J * s.kp.CoP;
    pack_weights_kernel<<<ceil_div(total, 256), 256, 0, st>>>(d_w, Co, Ci, K, s.L.J, s.L.Kc, s.L.S, w_signed ? 1 : 0, s.kp.CoP,
                                                             (uint32_t *)d_workspace, total);
    rc = launch_status();
    if (rc != HIKONV_OK) return rc;
    return launch_conv2d(s, x_signed != 0, st);
}

// ---- scratch that needs no allocation: a fixed buffer inside the library image, one copy per GPU
static __device__ __align__(256) unsigned char g_static_scratch[HIKONV_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void *g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of g_static_scratch on the current device.  In host code the array's name is only
// a handle, so the address is asked for once per device and cached.
int static_scratch_address(void **out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return HIKONV_ERR_CUDA;
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
    if (Ci < 1 || Co < 1 || K < 1) return HIKONV_ERR_INVALID_ARG;
    const size_t need = hikonv_conv2d_workspace_bytes(Ci, Co, K);
    if (need > (size_t)HIKONV_STATIC_SCRATCH_BYTES) return HIKONV_ERR_TOO_LARGE;
    void *scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != HIKONV_OK) return rc;
    // the packing kernel writes every word the layer kernel reads, so stale contents are harmless
    return hikonv_conv2d(d_x, B, Ci, H, W, d_w, Co, K, stride, pad, p, q, x_signed, w_signed, d_out, requant, shift, lo, hi,
                         scratch, (size_t)HIKONV_STATIC_SCRATCH_BYTES, algo, tune, stream);
}

extern "C" size_t hikonv_conv2d_host_workspace_bytes(int B, int Ci, int H, int W, int Co, int K, int pad, int requant) {
    if (B < 1 || Ci < 1 || H < 1 || W < 1 || Co < 1 || K < 1 || pad < 0) return 0;
    const long long Ho = H + 2 * pad - K + 1, Wo = W + 2 * pad - K + 1;
    if (Ho < 1 || Wo < 1) return 0;
    const size_t out_bytes = (size_t)B * Co * Ho * Wo * (requant ? 1 : 4);
    return align_up((size_t)B * Ci * H * W, 256) + align_up((size_t)Co * Ci * K * K, 256) + align_up(out_bytes, 256) +
           hikonv_conv2d_workspace_bytes(Ci, Co, K);
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
                                 hi, d_ws, hikonv_conv2d_workspace_bytes(Ci, Co, K), algo, tune, st);
    if (rc != HIKONV_OK) return rc;
    HIKONV_CUDA_TRY(cudaMemcpyAsync(h_out, d_out, out_bytes, cudaMemcpyDeviceToHost, st));
    return HIKONV_OK;
}

extern "C" int hikonv_maxpool2x2_i8(const int8_t *d_in, int B, int C, int H, int W, int is_signed, int8_t *d_out, void *stream) {
    if (!d_in || !d_out || B < 1 || C < 1 || H < 1 || W < 1) return HIKONV_ERR_INVALID_ARG;
    const long long total = (long long)B * C * (H / 2) * (W / 2);
    if (total == 0) return HIKONV_OK;
    if ((double)B * C >= 2147483647.0) return HIKONV_ERR_UNSUPPORTED;
    long long blocks = (total + 255) / 256;
    const long long cap = (long long)sm_count() * 32;
    if (blocks > cap) blocks = cap;
    maxpool2x2_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(d_in, B * C, H, W, is_signed ? 1 : 0, d_out);
    return launch_status();
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
