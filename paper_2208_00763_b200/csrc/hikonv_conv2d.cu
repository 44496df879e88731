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
// xN + m, slot m >= N those of pixel (x+1)N + (m-N): the overlap-add of Theorem 2.  After at most
// M accumulated (ci, kh) pairs the slots are extracted into int32 sums and Q restarts at `bias`.
//
// A CTA computes TR consecutive output rows (one row segment each) times TCO output channels; it
// is a register-tiled integer "GEMM" over packed words: each thread owns TM consecutive positions
// times TN channels, the k dimension runs over (ci, kh, j).
#include <algorithm>
#include <cstring>
#include <mutex>

#include "hikonv_cuda.cuh"

namespace hikonv {

constexpr int kThreads2D = 256;
constexpr int kMaxN2DSeg = 8;      // N + Kc - 1 <= 2 N <= 8

struct Conv2dParams {
    const int8_t *x;
    const uint32_t *wp;        // packed weights [Ci*K*J][CoP]
    void *out;
    int B, Ci, H, W, Co, CoP, K, pad, Ho, Wo, Hp;
    int S, J, Kc, nhi, M;      // nhi = Kc - 1 slots above the N low ones
    int X;                     // output blocks per row
    int NSEG, XO, XB;          // row segments, output blocks per segment, positions per segment (XO + J)
    int TR, TMX, TNX, TCO, CK;
    int NRmax, a_plane, lead;
    int b_off;                 // word offset of the weight tile in shared memory (multiple of 4: 16-byte loads)
    int requant, shift, lo, hi;
    int total_rows;            // B * Ho
    uint32_t mask;
    uint64_t bias;
    int seg_shift[kMaxN2DSeg];
    int32_t carry_bias[kMaxN2D];
};

template <bool UNPACKED>
struct AccType {
    typedef uint64_t type;
};
template <>
struct AccType<true> {
    typedef int32_t type;
};

// N: pixels per packed word; TM x TN: per-thread tile (positions x channels); UNPACKED: comparator
// (N == 1, one tap per word, 32-bit multiply-add, int32 accumulators); SP: signed product;
// XS: signed activations.
template <int N, int TM, int TN, bool UNPACKED, bool SP, bool XS>
__global__ void __launch_bounds__(kThreads2D) conv2d_kernel(const Conv2dParams p) {
    typedef typename AccType<UNPACKED>::type acc_t;
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t *As = smem;                                   // [CK][a_plane]
    uint32_t *Bs = As + p.b_off;                           // [CK*K*J][TCO], 16-byte aligned
    int *s_row = (int *)(Bs + p.CK * p.K * p.J * p.TCO);   // [NRmax] input offset of each staged row, -1 = zero row

    const int tid = threadIdx.x;
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

    for (int rl = tid; rl < NR; rl += kThreads2D) {
        const int rp = Rp0 + rl;
        const int b = rp / p.Hp, hi = rp - b * p.Hp - p.pad;
        s_row[rl] = (b < p.B && hi >= 0 && hi < p.H) ? (b * p.Ci * p.H + hi) * p.W : -1;
    }

    // this thread's positions: smem offset of the packed word for (kh = 0, j = 0), and validity
    int off[TM];
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int pos = tm * TM + i;
        if (pos < TP) {
            const int r = pos / p.XB, xb = pos - r * p.XB;
            const int R = R0 + r;
            const int b = R / p.Ho;
            off[i] = p.lead + ((b * p.Hp + (R - b * p.Ho)) - Rp0) * p.XB + xb;
        } else {
            off[i] = p.lead;                                 // idle position: reads valid memory, result dropped
        }
    }

    acc_t acc[TM][TN];
    // int32 sums kept as uint32: the biased partial sums may wrap, the final difference is exact
    uint32_t outv[UNPACKED ? 1 : TM][UNPACKED ? 1 : N][UNPACKED ? 1 : TN];
    uint32_t carry[UNPACKED ? 1 : N][UNPACKED ? 1 : TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int t = 0; t < TN; ++t) acc[i][t] = UNPACKED ? (acc_t)0 : (acc_t)p.bias;
    if constexpr (!UNPACKED) {
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int m = 0; m < N; ++m)
#pragma unroll
                for (int t = 0; t < TN; ++t) outv[i][m][t] = 0;
#pragma unroll
        for (int m = 0; m < N; ++m)
#pragma unroll
            for (int t = 0; t < TN; ++t) carry[m][t] = 0;
    }
    int cnt = 0, nflush = 0;

    // Split of the 64-bit accumulators (Algorithm 2's shift-and-mask on biased slots): slots
    // 0..N-1 go to this position, slots N.. to the next position of the row (Theorem 2).
    auto flush = [&]() {
        if constexpr (!UNPACKED) {
#pragma unroll
        for (int t = 0; t < TN; ++t) {
#pragma unroll
            for (int i = 0; i < TM; ++i) {
                const uint64_t Q = (uint64_t)acc[i][t];
#pragma unroll
                for (int m = 0; m < N; ++m) outv[i][m][t] += shr64_lo(Q, p.seg_shift[m]) & p.mask;
#pragma unroll
                for (int m = 0; m < N; ++m) {
                    if (m < p.nhi) {
                        const uint32_t f = shr64_lo(Q, p.seg_shift[N + m < kMaxN2DSeg ? N + m : 0]) & p.mask;
                        if (i + 1 < TM) outv[i + 1 < TM ? i + 1 : 0][m][t] += f;
                        else carry[m][t] += f;
                    }
                }
                acc[i][t] = (acc_t)p.bias;
            }
        }
        ++nflush;
        }
    };

    const int HW = p.H * p.W;
    const int KJ = p.K * p.J;
    const int words_per_plane = NR * p.XB;
    uint32_t slot_pow[N];
#pragma unroll
    for (int n = 0; n < N; ++n) slot_pow[n] = UNPACKED ? 1u : (1u << (p.S * n));
    const int col_seg0 = (seg * p.XO - p.J) * N + p.K - 1 - p.pad;   // input column of slot 0 at xb = 0

    for (int ci0 = 0; ci0 < p.Ci; ci0 += p.CK) {
        const int ckn = min(p.CK, p.Ci - ci0);
        __syncthreads();                                             // previous chunk fully consumed (and s_row written)
        // ---- stage the packed activation rows of ckn channels (Eq. 5, built from int8 codes)
        for (int idx = tid; idx < ckn * words_per_plane; idx += kThreads2D) {
            const int cl = idx / words_per_plane;
            const int rem = idx - cl * words_per_plane;
            const int rl = rem / p.XB, xb = rem - rl * p.XB;
            const int base = s_row[rl];
            uint32_t word = 0;
            if (base >= 0) {
                const int8_t *src = p.x + base + (ci0 + cl) * HW;
                const int col0 = col_seg0 + xb * N;
#pragma unroll
                for (int n = 0; n < N; ++n) {
                    const int col = col0 + n;
                    if (col >= 0 && col < p.W) word += (uint32_t)load_code<XS>(src + col) * slot_pow[n];
                }
            }
            As[cl * p.a_plane + p.lead + rem] = word;
        }
        // ---- stage the packed kernel rows of the same channels for TCO output channels
        {
            const int tco4 = p.TCO / 4;
            const int rows = ckn * KJ;
            for (int idx = tid; idx < rows * tco4; idx += kThreads2D) {
                const int kr = idx / tco4, c4 = idx - kr * tco4;
                const int co = co0 + c4 * 4;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (co < p.CoP) v = __ldg(reinterpret_cast<const uint4 *>(p.wp + (size_t)(ci0 * KJ + kr) * p.CoP + co));
                reinterpret_cast<uint4 *>(Bs)[kr * tco4 + c4] = v;
            }
        }
        __syncthreads();
        // ---- multiply-accumulate over (ci, kh, j)
        for (int cl = 0; cl < ckn; ++cl) {
            for (int kh = 0; kh < p.K; ++kh) {
                for (int j = 0; j < p.J; ++j) {
                    const uint32_t *arow = As + cl * p.a_plane + kh * p.XB - j;
                    const uint32_t *brow = Bs + ((cl * p.K + kh) * p.J + j) * p.TCO + tn * TN;
                    uint32_t a[TM], b[TN];
#pragma unroll
                    for (int i = 0; i < TM; ++i) a[i] = arow[off[i]];
#pragma unroll
                    for (int t = 0; t < TN; t += 4) {
                        const uint4 v = *reinterpret_cast<const uint4 *>(brow + t);
                        b[t] = v.x; b[t + 1] = v.y; b[t + 2] = v.z; b[t + 3] = v.w;
                    }
#pragma unroll
                    for (int i = 0; i < TM; ++i)
#pragma unroll
                        for (int t = 0; t < TN; ++t) {
                            if (UNPACKED) acc[i][t] = (acc_t)((int32_t)acc[i][t] + (int32_t)a[i] * (int32_t)b[t]);
                            else { uint64_t q = (uint64_t)acc[i][t]; mad_wide<SP>(q, a[i], b[t]); acc[i][t] = (acc_t)q; }
                        }
                }
                if (!UNPACKED && ++cnt == p.M) { flush(); cnt = 0; }
            }
        }
    }
    if (!UNPACKED && cnt > 0) flush();

    // ---- hand the slots that belong to the next thread's first position across (Theorem 2 at thread borders)
    if constexpr (!UNPACKED) {
        __syncthreads();
        uint32_t *xch = smem;                              // [TMX][N][TCO]
#pragma unroll
        for (int m = 0; m < N; ++m)
#pragma unroll
            for (int t = 0; t < TN; ++t) xch[(tm * N + m) * p.TCO + tn * TN + t] = carry[m][t];
        __syncthreads();
        if (tm > 0) {
#pragma unroll
            for (int m = 0; m < N; ++m)
#pragma unroll
                for (int t = 0; t < TN; ++t) outv[0][m][t] += xch[((tm - 1) * N + m) * p.TCO + tn * TN + t];
        }
    }

    // ---- bias removal, optional requantisation (arithmetic shift, clamp), store
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int pos = tm * TM + i;
        if (pos >= TP) continue;
        const int r = pos / p.XB, xbl = pos - r * p.XB;
        if (xbl < p.J) continue;                                     // halo positions produce no pixels
        const int xg = seg * p.XO + xbl - p.J;                       // output block in the row
        if (xg >= p.X) continue;
        const int R = R0 + r;
        const int b = R / p.Ho, h = R - b * p.Ho;
#pragma unroll
        for (int t = 0; t < TN; ++t) {
            const int co = co0 + tn * TN + t;
            if (co >= p.Co) continue;
            const size_t row_off = (((size_t)b * p.Co + co) * p.Ho + h) * p.Wo;
#pragma unroll
            for (int m = 0; m < N; ++m) {
                const int w = xg * N + m;
                if (w >= p.Wo) continue;
                int32_t v;
                if (UNPACKED) v = (int32_t)acc[i][t];
                else v = (int32_t)(outv[UNPACKED ? 0 : i][UNPACKED ? 0 : m][UNPACKED ? 0 : t] - (uint32_t)nflush * (uint32_t)p.carry_bias[m]);
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
    int variant;          // index into the launch table
    size_t smem_bytes;
    dim3 grid;
    bool unpacked;
};

static int sm_count() {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms;
}

template <int N, int TM, int TN, bool UNPACKED>
static int launch_variant(const Conv2dSetup &s, bool sp, bool xs, cudaStream_t st) {
#define HK_LAUNCH(SPV, XSV)                                                                                      \
    do {                                                                                                         \
        auto kern = conv2d_kernel<N, TM, TN, UNPACKED, SPV, XSV>;                                                \
        if (s.smem_bytes > 48 * 1024)                                                                            \
            HIKONV_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s.smem_bytes)); \
        kern<<<s.grid, kThreads2D, s.smem_bytes, st>>>(s.kp);                                                    \
    } while (0)
    if (!sp) HK_LAUNCH(false, false);
    else if (xs) HK_LAUNCH(true, true);
    else HK_LAUNCH(true, false);
#undef HK_LAUNCH
    return launch_status();
}

constexpr int kTM = 4, kTN = 4;          // per-thread tile of the packed kernels
constexpr int kTMU = 8, kTNU = 4;        // per-thread tile of the comparator

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
        kp.mask = sc.slot_mask;
        kp.bias = sc.bias;
        for (int m = 0; m < kMaxN2DSeg; ++m) kp.seg_shift[m] = m < L.segments ? L.S * m : 0;
        for (int m = 0; m < kMaxN2D; ++m) kp.carry_bias[m] = m < L.N ? sc.carry_bias[m] : 0;
    }
    kp.B = B; kp.Ci = Ci; kp.H = H; kp.W = W; kp.Co = Co; kp.K = K; kp.pad = pad; kp.Ho = Ho; kp.Wo = Wo; kp.Hp = Ho + K - 1;
    kp.CoP = (Co + 3) / 4 * 4;
    kp.S = L.S; kp.J = L.J; kp.Kc = L.Kc; kp.nhi = L.segments - L.N; kp.M = L.M;
    kp.requant = requant ? 1 : 0; kp.shift = shift; kp.lo = lo; kp.hi = hi;
    kp.total_rows = B * Ho;
    kp.X = ceil_div(Wo, N);
    // channels per CTA: up to 64, thread grid TMX x TNX = 256
    int TNX = 1;
    while (TNX * TN < Co && TNX * TN < 64) TNX *= 2;
    kp.TNX = TNX; kp.TMX = kThreads2D / TNX; kp.TCO = TNX * TN;
    const int maxpos = kp.TMX * TM;
    // rows wider than a tile are cut into segments, each with its own J halo positions
    kp.NSEG = 1;
    while (ceil_div(kp.X, kp.NSEG) + L.J > maxpos) ++kp.NSEG;
    kp.XO = ceil_div(kp.X, kp.NSEG);
    kp.XB = kp.XO + L.J;
    int TR = maxpos / kp.XB;
    if (tune && tune->tile > 0 && tune->tile < TR) TR = tune->tile;
    if (TR > kp.total_rows) TR = kp.total_rows;
    kp.TR = TR;
    const int span = (TR + Ho - 2) / Ho + 1;                 // images a tile can touch
    kp.NRmax = TR + (K - 1) * span;
    kp.lead = L.J;                                           // room for the xb - j reads at the front
    kp.a_plane = kp.NRmax * kp.XB + kp.lead;
    // channels per stage: a multiple of the split period when that is short, about 8 otherwise
    int CK = 8;
    if (!s->unpacked && L.M < Ci * K) CK = std::max(1, std::min(8, L.M / K));
    if (CK > Ci) CK = Ci;
    kp.CK = CK;
    kp.b_off = (CK * kp.a_plane + 3) / 4 * 4;
    size_t words = (size_t)kp.b_off + (size_t)CK * K * L.J * kp.TCO;
    size_t xch_words = s->unpacked ? 0 : (size_t)kp.TMX * N * kp.TCO;
    s->smem_bytes = std::max(words + (size_t)kp.NRmax, xch_words) * 4 + 16;
    if (s->smem_bytes > 200 * 1024) return HIKONV_ERR_UNSUPPORTED;
    const long long row_tiles = ((long long)kp.total_rows + TR - 1) / TR;
    const long long gx = row_tiles * kp.NSEG;
    const int gy = ceil_div(Co, kp.TCO);
    if (gx > 0x7FFFFFFFLL || gy > 65535) return HIKONV_ERR_UNSUPPORTED;
    s->grid = dim3((unsigned)gx, (unsigned)gy, 1);
    return HIKONV_OK;
}

static int launch_conv2d(const Conv2dSetup &s, bool xs, cudaStream_t st) {
    const bool sp = s.L.signed_prod != 0;
    if (s.unpacked) return launch_variant<1, kTMU, kTNU, true>(s, sp, xs, st);
    switch (s.L.N) {
        case 1: return launch_variant<1, kTM, kTN, false>(s, sp, xs, st);
        case 2: return launch_variant<2, kTM, kTN, false>(s, sp, xs, st);
        case 3: return launch_variant<3, kTM, kTN, false>(s, sp, xs, st);
        case 4: return launch_variant<4, kTM, kTN, false>(s, sp, xs, st);
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
