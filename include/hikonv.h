/*
 * hikonv.h - C interface of the packed low-bit convolution library for NVIDIA B200 (sm_100a).
 *
 * The library computes 1-D and 2-D convolutions of 1..8-bit quantised codes by packing
 * N activations and K weights into two 32-bit words with S-bit slots, so that ONE
 * 32x32->64 multiply yields N+K-1 partial convolution sums (Theorem 1), which are
 * overlap-added across blocks (Theorem 2), accumulated over input channels and kernel
 * rows while still packed (Theorem 3, the DNN guard-bit rule), then split into int32
 * (Algorithm 2 / Eq. 29) and optionally requantised.
 *
 * Conventions for every entry point
 *   - Codes are stored one per byte (int8_t; hikonv_conv1d_dense alone reads a denser format).  A signed p-bit code is its int8 value; an
 *     unsigned p-bit code is the byte read as uint8 (so unsigned 8-bit codes use all 256
 *     byte values).  Codes are ASSUMED to lie in their p-bit range; a code outside it
 *     silently breaks the guard bits (hikonv_check_range is the debug pass that looks).
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  All memory is owned
 *     by the caller; the library allocates nothing and keeps no pointer after a call.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Device
 *     entry points enqueue their kernels on it and return without synchronising.
 *   - Every function returns a hikonv_status (as int); nothing aborts, nothing traps on
 *     the device.  Arguments are validated on the host before any launch.  HIKONV_ERR_CUDA
 *     reports what the call's own launches and copies returned; an error that earlier,
 *     unrelated CUDA calls left unread in the thread's error state is neither reported nor
 *     cleared.
 *   - There is no CPU fallback: without a CUDA device the device entry points return
 *     HIKONV_ERR_CUDA.
 */
#ifndef HIKONV_H
#define HIKONV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    HIKONV_OK = 0,
    HIKONV_ERR_INVALID_ARG = 1, /* null pointer, p/q outside 1..8, K < 1, sizes < 0, bad enum        */
    HIKONV_ERR_UNSUPPORTED = 2, /* stride != 1, an algorithm that is not built, pad >= K               */
    HIKONV_ERR_NO_FIT = 3,      /* no (N >= 1, S) satisfies the operand, slot and accumulator bounds   */
    HIKONV_ERR_WORKSPACE = 4,   /* workspace pointer null/misaligned or workspace_bytes too small      */
    HIKONV_ERR_CUDA = 5,        /* a CUDA runtime call failed (see cudaGetLastError)                   */
    HIKONV_ERR_TOO_LARGE = 6,   /* the layer needs more scratch than the built-in static buffer holds  */
    HIKONV_ERR_RANGE = 7        /* hikonv_check_range: a stored code lies outside its p-bit range      */
} hikonv_status;

typedef enum {
    HIKONV_ALGO_PACKED32 = 0,      /* packed operands, 32x32->64 multiply (mad.wide)                    */
    HIKONV_ALGO_PACKED64EMU = 1,   /* packed operands of 64 bits, 64x64->128 product built from 32-bit
                                      multiplies (Section V-A's wider multiplier); hikonv_conv1d only */
    HIKONV_ALGO_UNPACKED_IMAD = 2, /* comparator: one product per 32-bit multiply-add, int32 accumulate */
    HIKONV_ALGO_DP4A = 3           /* second comparator: four products per byte dot-product instruction
                                      (dp4a), int32 accumulate; hikonv_conv1d only, K <= 8               */
} hikonv_algo;

typedef enum {
    HIKONV_GB_SINGLE = 0, /* Eq. 11: Gb = ceil(log2 min(K, N))          */
    HIKONV_GB_1D = 1,     /* 1-D extension: Gb = ceil(log2 K)            */
    HIKONV_GB_DNN = 2     /* DNN extension: Gb = ceil(log2(M min(K, N))) */
} hikonv_gb_mode;

/* Result of the paper's throughput search (Algorithm 1). */
typedef struct {
    int N;   /* activations per packed word            */
    int K;   /* weights per packed word                */
    int S;   /* slot width in bits (Eq. 6)             */
    int Gb;  /* guard bits of the chosen pair          */
    int ops; /* N K + (N-1)(K-1), Eq. 24               */
} hikonv_plan_t;

/* The layout the CUDA kernels actually run with (exact value-range analysis, see below). */
typedef struct {
    int N;           /* activations per 32-bit word A                                        */
    int S;           /* slot width                                                            */
    int Kc;          /* weights per 32-bit word B (taps per chunk)                            */
    int J;           /* number of weight chunks, ceil(K / Kc); J > 1 implies Kc == N          */
    int segments;    /* N + Kc - 1 slots of the 64-bit product                                */
    int top_bits;    /* width of the highest slot, 64 - S (segments - 1), capped at S         */
    int M;           /* products that may be summed in the 64-bit accumulator before a split  */
    int signed_prod; /* 1 when either operand is signed (signed multiply, biased split)       */
    int S_paper;     /* Eq. 6 with the mode's guard bits, for reference                       */
    int carry_bits;  /* 2-D: every M products the slot bits above this many low bits move to a
                        second packed accumulator (0: never, M covers the whole layer; 1-D: 0)   */
} hikonv_layout_t;

/* Optional overrides for experiments and tests; zero in a field means "choose automatically".
 * Pass NULL for fully automatic behaviour. */
typedef struct {
    int N;          /* force activations per word                                   */
    int S;          /* force slot width                                             */
    int M;          /* force the number of accumulated products between two splits  */
    int tile;       /* kernel-specific tile selector (0 = automatic); conv2d: > 0 output
                       rows per CTA + 1000 x channel lanes per CTA (1, 2, 4, 8, 16) + 100000 x
                       positions per thread (2 or 4), each part 0 = automatic; < 0 carry-save moves
                       at stage ends instead of at fixed places inside channel groups; conv1d: > 0 the general kernel, -1 the
                       planner's layout instead of register-aligned slots; -24 / -25 force the
                       register budget of four / five resident CTAs per SM in the register-aligned
                       kernels and the two comparators (default: whichever measured faster for the
                       kernel), -32 runs of 32 outputs per lane (default 24) in the two comparators */
} hikonv_tuning_t;

/*
 * hikonv_plan - the paper's configuration search (Section IV-D, Algorithm 1; host only).
 * Maximises Eq. 24 over (N, K) subject to Eq. 7-8 with S from Eq. 6 and the guard bits of
 * `mode` (hikonv_gb_mode; M is the number of accumulated feature maps, used by the DNN rule).
 * K_fixed > 0 fixes the kernel length and searches N only.  LA, LB are the multiplier's
 * operand widths (1..64).  The search ranges are inclusive (the printed strict bounds cannot
 * reproduce the paper's own counts).  Returns HIKONV_ERR_NO_FIT when not even N = K = 1 fits.
 */
int hikonv_plan(int p, int q, int LA, int LB, int mode, int M, int K_fixed, hikonv_plan_t *out);

/*
 * hikonv_layout - the packed layout used by the CUDA kernels for a 32x32->64 multiplier (host only).
 * Starts from the paper's slot width (Eq. 6 with Gb = ceil(log2 K) for dims == 1, Theorem 2) and
 * verifies it against the exact value ranges of the codes: both packed operands must fit a 32-bit
 * register (31 bits for an unsigned operand of a signed multiply), every slot must hold the
 * extreme sum it can receive, and the top slot must fit what is left of 64 bits.  S is widened
 * when the printed rule is too small (signed 1-bit codes).  For dims == 2 (Theorem 3, Eq. 23)
 * S is chosen as large as N allows so that M, the number of (channel, kernel-row) products
 * accumulated before a split, is as large as possible, and N is chosen by a cost model.
 * K taps that do not fit one word are cut into J chunks of N taps (Theorem 2 applied to the
 * kernel).  `total_terms` is Ci*K for dims == 2 (ignored for dims == 1); `tune` may be NULL.
 */
int hikonv_layout(int p, int q, int f_signed, int g_signed, int K, int dims, int total_terms,
                  const hikonv_tuning_t *tune, hikonv_layout_t *out);

/*
 * hikonv_layout_emu64 - the 1-D layout for a 64x64->128 multiplier (HIKONV_ALGO_PACKED64EMU; host only).
 * The rules of hikonv_layout with dims == 1 and 64 / 128 bits in place of 32 / 64: Eq. 6 with
 * Gb = ceil(log2 K) as the starting slot width, widened until both packed operands fit 64 bits
 * (63 for an unsigned operand of a signed multiply), the N + Kc - 1 slots fit 128 bits and every slot
 * holds the extreme sum it can receive after the overlap-add of Theorem 2.  N is at most 16.
 * Fields of `out` as in hikonv_layout_t (M = 1, carry_bits = 0).  Only tune->N and tune->S are used.
 */
int hikonv_layout_emu64(int p, int q, int f_signed, int g_signed, int K, const hikonv_tuning_t *tune,
                        hikonv_layout_t *out);

/*
 * hikonv_pack - Eq. 5: words[x] = sum_{n<N} in[x N + n] * 2^(S n), modulo 2^word_bits.
 * d_in: n codes (device, int8 storage, `bits` wide, signed or not).  The tail of the last word is
 * zero-filled.  d_words: ceil(n / N) words of word_bits (32 or 64) bits, device, naturally aligned.
 * For signed codes the word is the two's-complement sum, which equals the slot-by-slot
 * decrementer form of Eq. 28.  Requires bits + (N-1) S <= word_bits.
 */
int hikonv_pack(const int8_t *d_in, size_t n, int bits, int is_signed, int S, int N, int word_bits,
                void *d_words, void *stream);

/*
 * hikonv_check_range - debug pass: do all n stored codes lie in their range?
 * The slot width of Eq. 6 and the operand bounds of Eq. 7-8 are derived from the code ranges
 * [0, 2^bits - 1] (unsigned) and [-2^(bits-1), 2^(bits-1) - 1] (signed); the convolution entry points
 * assume them and do not look.  This call counts the codes of d_in (device, one code per byte, n of them,
 * any alignment) outside that range.  d_count: one 8-byte-aligned device word owned by the caller; the
 * call zeroes it, adds the violations, copies it to *h_count (host, may be NULL) and SYNCHRONISES
 * `stream` before it returns.  Returns HIKONV_OK when every code is in range, HIKONV_ERR_RANGE when at
 * least one is not (the count is in *h_count and *d_count).  With bits == 8 every byte is a valid code.
 */
int hikonv_check_range(const int8_t *d_in, size_t n, int bits, int is_signed, unsigned long long *d_count,
                       unsigned long long *h_count, void *stream);

/*
 * hikonv_conv1d - full 1-D convolution F_{len,K}(f, g) (Eq. 2-4 via Theorems 1 and 2).
 * d_f: len codes of p bits; d_g: K codes of q bits; d_y: len + K - 1 int32 outputs (device, 4-byte
 * aligned), y[m] = sum_k f[m-k] g[k] with f zero outside [0, len).
 * algo: HIKONV_ALGO_PACKED32, HIKONV_ALGO_UNPACKED_IMAD, HIKONV_ALGO_PACKED64EMU (64-bit packed
 * words, layout of hikonv_layout_emu64; same results, kept as the wider-multiplier variant), or
 * HIKONV_ALGO_DP4A (the SIMD byte dot product, reported beside the packed method; K <= 8, else
 * HIKONV_ERR_UNSUPPORTED).
 * tune may be NULL.  len >= 1, 1 <= K <= 64.
 * The packed algorithm is bound by HBM on this input format, not by the multiplier, so without a forced
 * layout the call does not run the planner's layout (most outputs per multiply) but the one with the fewest
 * instructions per output: hikonv_conv1d_layout returns it, hikonv_conv1d_multiplies counts its multiplies.
 */
int hikonv_conv1d(const int8_t *d_f, size_t len, const int8_t *d_g, int K, int p, int q,
                  int f_signed, int g_signed, int32_t *d_y, int algo, const hikonv_tuning_t *tune,
                  void *stream);

/*
 * hikonv_conv1d_layout - the packed layout hikonv_conv1d(HIKONV_ALGO_PACKED32) runs with for these arguments
 * (host only; hikonv_layout reports the planner's choice, which maximises outputs per multiply).
 * On one-code-per-byte input the path is bound by HBM, so the call prefers the layout with the fewest
 * instructions per output: slots of 8 or 16 bits with N S = 32 whenever every sum of K products fits such a
 * slot and K <= 8 (the packed operand of Eq. 5 is then the loaded word itself or one byte permute of it, the
 * carry of Theorem 2 is the high register of the previous product, and every output is one byte permute);
 * sums of 17 to 21 bits (8-bit codes) run with N = 2 and two taps per kernel word at the narrowest such S.
 * Otherwise it takes the planner's layout with N lowered to 8 (from 9..12) or 4 (from 5) when that keeps S
 * and J.  tune: a forced N or S is taken as it is, tile == -1 keeps the planner's layout, tile > 0 the
 * general kernel.
 */
int hikonv_conv1d_layout(int p, int q, int f_signed, int g_signed, int K, const hikonv_tuning_t *tune,
                         hikonv_layout_t *out);

/*
 * hikonv_conv1d_dense - hikonv_conv1d (packed algorithm) on a signal stored without its unused bits
 * (Section V-B, "Single convolver architecture": weights and features kept compressed in memory and
 * unpacked into the multiplier's slices as they are read).
 * d_f_dense: len codes of p bits, p in {1, 2, 4}, 8 / p codes per byte: code e occupies bits
 * [(e p) % 8, (e p) % 8 + p) of byte (e p) / 8 (two's complement when f_signed); the unused bits of the
 * last byte are ignored.  ceil(len p / 8) bytes, device, caller-owned; any alignment is accepted, 4-byte
 * alignment takes the fast path.  d_g, d_y, q, K, tune, stream as for hikonv_conv1d.
 * Built for the layouts of K in {3, 5, 7} with q == p (signed or unsigned operands in any combination); any
 * other combination returns HIKONV_ERR_UNSUPPORTED (nothing is launched).
 */
int hikonv_conv1d_dense(const uint8_t *d_f_dense, size_t len, const int8_t *d_g, int K, int p, int q,
                        int f_signed, int g_signed, int32_t *d_y, const hikonv_tuning_t *tune,
                        void *stream);

/* Device scratch needed by hikonv_conv1d_host: room for f, g and y on the device. */
size_t hikonv_conv1d_host_workspace_bytes(size_t len, int K);

/*
 * hikonv_conv1d_host - the same convolution with HOST buffers: copies h_f and h_g to the device
 * workspace, runs hikonv_conv1d, copies len + K - 1 int32 results back to h_y, all on `stream`
 * (asynchronous when the host buffers are pinned; the caller synchronises the stream).
 * d_workspace: device memory of at least hikonv_conv1d_host_workspace_bytes(len, K) bytes,
 * 256-byte aligned.
 */
int hikonv_conv1d_host(const int8_t *h_f, size_t len, const int8_t *h_g, int K, int p, int q,
                       int f_signed, int g_signed, int32_t *h_y, void *d_workspace,
                       size_t workspace_bytes, int algo, const hikonv_tuning_t *tune, void *stream);

/*
 * hikonv_conv2d - one convolution layer (Eq. 16 through Theorem 3 and Eq. 23), stride 1, zero padding.
 * d_x: [B][Ci][H][W] codes of p bits; d_w: [Co][Ci][K][K] codes of q bits;
 * output [B][Co][Ho][Wo], Ho = H + 2 pad - K + 1, Wo = W + 2 pad - K + 1:
 *   requant == 0: d_out is int32, the exact sums;
 *   requant != 0: d_out is int8, clamp(sum >> shift, lo, hi) with an arithmetic (floor) shift,
 *                 0 <= shift <= 31, -128 <= lo <= hi <= 255 (values above 127 are stored as the
 *                 byte of the unsigned code).
 * Two kernels run on `stream`: the reversed kernel rows (g = W[co][ci][kh][K-1:0], Theorem 3) and the
 * activation rows are packed (Eq. 5) into d_workspace, then the layer kernel streams the packed words.
 * d_workspace: hikonv_conv2d_workspace_bytes(...) bytes of device memory, 256-byte aligned; the call
 * overwrites it and needs nothing from it afterwards.  The unpacked comparator uses the same workspace for
 * int32 copies of the weights and codes.
 * stride must be 1 and 0 <= pad < K.  Limits (HIKONV_ERR_UNSUPPORTED beyond them): Ho < 60000; B Ci H W and B Ho
 * below 2^31; (images a tile of rows can touch + 1) x Co x Ho x Wo below 2^32 (output offsets inside a CTA are 32-bit).
 * Layers with unsigned activations and signed weights may run on activation codes shifted by 2^(p-1) where that
 * saves carry-save moves or puts one more pixel into a word (see hikonv_conv2d_layout); results are the same exact sums.
 */
int hikonv_conv2d(const int8_t *d_x, int B, int Ci, int H, int W, const int8_t *d_w, int Co, int K,
                  int stride, int pad, int p, int q, int x_signed, int w_signed, void *d_out,
                  int requant, int shift, int lo, int hi, void *d_workspace, size_t workspace_bytes,
                  int algo, const hikonv_tuning_t *tune, void *stream);

/*
 * hikonv_conv2d_tune - times the tile shapes of one layer on the device and returns the fastest (a set-up aid with no
 * counterpart in the paper: the automatic choice comes from a cost model, which on small layers misses tiles that
 * measure 10-20 % faster).  Arguments up to `algo` are those of hikonv_conv2d_dense (one code per byte: storage 8 / 8,
 * out_store_bits 8, or 32 without requant).  The call runs the layer with the library's own tile and with every forced
 * tile (positions per thread 4 and 2 x channel lanes 1, 2, 4, 8 x output rows per CTA 1 .. 48; shapes the layer does not
 * support are skipped), each as groups of four launches between two CUDA events on `stream`, best of `repeats` (1 .. 100)
 * groups, and SYNCHRONISES.  Every launch writes the layer's complete, correct output to d_out.
 * *h_tile: the value for hikonv_tuning_t.tile in later calls on this shape, or 0 when no forced tile is at least 3 %
 * faster than the automatic one.  *h_us / *h_default_us (may be NULL): microseconds per launch of the winner and of
 * the automatic choice.  Errors as for hikonv_conv2d_dense; results never depend on the tile.
 */
int hikonv_conv2d_tune(const void *d_x, int x_store_bits, int B, int Ci, int H, int W, const void *d_w,
                       int w_store_bits, int Co, int K, int stride, int pad, int p, int q, int x_signed,
                       int w_signed, void *d_out, int out_store_bits, int requant, int shift, int lo, int hi,
                       int pool, void *d_workspace, size_t workspace_bytes, int algo, int repeats, int *h_tile,
                       double *h_us, double *h_default_us, void *stream);

/*
 * hikonv_conv2d_layout - the packed layout hikonv_conv2d(HIKONV_ALGO_PACKED32) runs this layer with (host only).
 * *out: N, S, Kc, J, slots, M (accumulated (ci, kh) pairs between two carry-save moves), as hikonv_layout reports them.
 * *x_shift (may be NULL): 0, or 2^(p-1) when the layer runs its unsigned activations as signed codes x - 2^(p-1):
 * the span of a product halves, a slot takes about twice as many products between moves (or the word one more
 * pixel), and the epilogue adds
 * 2^(p-1) x (sum of the output channel's weights) back.  *out is then the layout for signed activations, which is
 * not what hikonv_layout reports for the layer's own signs.  Arguments and errors as for hikonv_conv2d.
 */
int hikonv_conv2d_layout(int B, int Ci, int H, int W, int Co, int K, int pad, int p, int q, int x_signed,
                         int w_signed, const hikonv_tuning_t *tune, hikonv_layout_t *out, int *x_shift);

/*
 * hikonv_conv2d_dense - hikonv_conv2d on tensors stored without their unused bits (Section V-B, single convolver
 * architecture: the weights sit in memory in compressed form, and the section notes that features can be kept
 * that way at run time too), with the layer's requantised output written in the same compressed form and,
 * optionally, max-pooled on the way out.
 *   Dense storage of a tensor of b-bit codes, b in {1, 2, 4}: the codes in their NCHW (OIHW) order, 8 / b per
 *   byte, code e in bits [(e b) % 8, (e b) % 8 + b) of byte (e b) / 8, two's complement when signed;
 *   ceil(count b / 8) bytes.
 *   x_store_bits: 8 (one code per byte, as hikonv_conv2d reads) or p (dense, p in {1, 2, 4});
 *   w_store_bits: 8 or q (dense, q in {1, 2, 4});
 *   out_store_bits: 32 with requant == 0 (int32 sums, 4-byte aligned);
 *                   with requant != 0: 8 (one code per byte) or 1 / 2 / 4 (dense; [lo, hi] must lie in the
 *                   code range of that width, signed when lo < 0, and every output row must fill whole bytes:
 *                   Wo' * out_store_bits a multiple of 8, else HIKONV_ERR_UNSUPPORTED);
 *   pool: 0, or 1 = 2x2 maximum with stride 2 after requantisation (requant != 0, Ho and Wo even); the output is
 *         then [B][Co][Ho / 2][Wo / 2] (Ho' = Ho / 2, Wo' = Wo / 2), else [B][Co][Ho][Wo].
 * The packing stage unpacks dense codes as it reads them; the layer kernel stages a CTA's requantised codes in
 * shared memory and writes whole bytes.  All other arguments, the workspace and the error behaviour are those of
 * hikonv_conv2d; combinations that are not built return HIKONV_ERR_UNSUPPORTED and launch nothing.
 */
int hikonv_conv2d_dense(const void *d_x, int x_store_bits, int B, int Ci, int H, int W, const void *d_w,
                        int w_store_bits, int Co, int K, int stride, int pad, int p, int q, int x_signed,
                        int w_signed, void *d_out, int out_store_bits, int requant, int shift, int lo, int hi,
                        int pool, void *d_workspace, size_t workspace_bytes, int algo,
                        const hikonv_tuning_t *tune, void *stream);

/* Workspace needed by hikonv_conv2d for this layer shape (an upper bound over all layouts and both algorithms). */
size_t hikonv_conv2d_workspace_bytes(int B, int Ci, int H, int W, int Co, int K, int pad);

/*
 * hikonv_conv2d_static_scratch - hikonv_conv2d for callers that cannot provide device scratch.
 * (The paper has no counterpart; this is a deployment convenience of this library.)
 *
 * Some callers cannot allocate device memory at the point where they run a layer: code that runs
 * inside a memory-capped serving process whose pool is owned by another component, plug-ins that are
 * handed input and output tensors only, and real-time loops where cudaMalloc (which synchronises the
 * device and can fail late) is forbidden after start-up.  For them the packed kernel and activation rows
 * go to a fixed buffer of HIKONV_STATIC_SCRATCH_BYTES that lives inside the library image on every GPU that
 * loads it, from load until the process exits.  Arguments are those of hikonv_conv2d without the
 * workspace pair; results are identical.
 *
 *   - Limit: hikonv_conv2d_workspace_bytes(B, Ci, H, W, Co, K, pad) must not exceed HIKONV_STATIC_SCRATCH_BYTES,
 *     otherwise HIKONV_ERR_TOO_LARGE is returned and nothing is launched.
 *   - The function calls no cudaMalloc/cudaFree and no allocating library routine.
 *   - The buffer that is used is the CURRENT device's.  d_x and d_out must be memory of the current device
 *     (checked with a pointer-attribute query; otherwise HIKONV_ERR_INVALID_ARG and nothing is launched) and
 *     `stream` must belong to it.
 *   - The first call on each device looks up the buffer's device address (once per device, with that
 *     device current) and keeps it for the life of the process; cudaDeviceReset invalidates it.  Make that
 *     first call during start-up, before any stream capture.
 *   - All calls on a device share the one buffer and it keeps the previous call's contents.  Nothing
 *     in it has to start at zero: every call rewrites all words it later reads.  Two calls whose
 *     kernels can overlap on the GPU (different streams, no dependency between them) race on the
 *     buffer; order them on one stream or with events.
 */
#define HIKONV_STATIC_SCRATCH_BYTES (4u << 20)
int hikonv_conv2d_static_scratch(const int8_t *d_x, int B, int Ci, int H, int W, const int8_t *d_w, int Co, int K,
                                 int stride, int pad, int p, int q, int x_signed, int w_signed, void *d_out,
                                 int requant, int shift, int lo, int hi, int algo, const hikonv_tuning_t *tune,
                                 void *stream);

/* Device scratch needed by hikonv_conv2d_host: x, w, out and the kernel workspace. */
size_t hikonv_conv2d_host_workspace_bytes(int B, int Ci, int H, int W, int Co, int K, int pad, int requant);

/* hikonv_conv2d with HOST buffers (copies in, runs, copies out, all on `stream`). */
int hikonv_conv2d_host(const int8_t *h_x, int B, int Ci, int H, int W, const int8_t *h_w, int Co, int K,
                       int stride, int pad, int p, int q, int x_signed, int w_signed, void *h_out,
                       int requant, int shift, int lo, int hi, void *d_workspace, size_t workspace_bytes,
                       int algo, const hikonv_tuning_t *tune, void *stream);

/*
 * hikonv_maxpool2x2_i8 - 2x2 max-pool, stride 2, on [B][C][H][W] byte codes -> [B][C][H/2][W/2].
 * Not part of the paper's method (its pooling is not accelerated); glue for the full-network
 * workload.  is_signed selects int8 or uint8 comparison.
 */
int hikonv_maxpool2x2_i8(const int8_t *d_in, int B, int C, int H, int W, int is_signed, int8_t *d_out,
                         void *stream);

/* Number of wide multiplies (packed) or 32-bit multiply-adds (unpacked) the last-planned launch of
 * the given problem executes, for roofline accounting.  Host only. */
double hikonv_conv1d_multiplies(size_t len, int K, int p, int q, int f_signed, int g_signed, int algo,
                                const hikonv_tuning_t *tune);
double hikonv_conv2d_multiplies(int B, int Ci, int H, int W, int Co, int K, int pad, int p, int q,
                                int x_signed, int w_signed, int algo, const hikonv_tuning_t *tune);

/*
 * hikonv_pipe_rate - measured issue rate of one integer instruction, for the rooflines of the packed kernels.
 * (A measurement aid; the paper has no counterpart.)  The 2-D layer kernels are bound by the 32x32->64
 * multiply-add that implements Eq. 9, and no public table gives its rate on this GPU.  The call runs a
 * register-only kernel (four CTAs of 256 threads per SM, eight independent dependency chains per thread whose
 * operands depend on the previous result, so nothing is loop-invariant), times it with CUDA events on `stream`
 * (best of three launches after a warm-up; the call SYNCHRONISES) and returns instructions x 32 lanes per second
 * in *h_ops_per_second and, if h_lanes_per_clock_per_sm is not NULL, that rate divided by (SM count x the device's
 * maximum SM clock).  d_scratch_word: one 4-byte device word owned by the caller.  iters: loop trips of 64
 * instructions per thread (1 .. 2^20; the mixed kind runs 32 logic instructions on top, which are not counted).
 */
typedef enum {
    HIKONV_PIPE_MAD_WIDE_U32 = 0, /* mad.wide.u32: the packed multiply of unsigned layouts       */
    HIKONV_PIPE_MAD_WIDE_S32 = 1, /* mad.wide.s32: the packed multiply of signed layouts         */
    HIKONV_PIPE_MAD_LO_S32 = 2,   /* mad.lo.s32: the comparator's 32-bit multiply-add            */
    HIKONV_PIPE_LOGIC = 3,        /* lop3.b32: masks of the split and of the carry-save moves    */
    HIKONV_PIPE_SHIFT = 4,        /* shf.r: the funnel shifts of the split                       */
    HIKONV_PIPE_PRMT = 5,         /* prmt.b32: code extraction and byte-aligned slot extraction  */
    HIKONV_PIPE_MAD_WIDE_WITH_LOGIC = 6 /* mad.wide.u32 with one lop3.b32 (on other registers) per two of them:
                                     the rate of the multiply-adds alone in that mix; against kind 0 it tells what an
                                     instruction of another pipe costs the stream of packed multiplies              */
} hikonv_pipe_kind;
int hikonv_pipe_rate(int kind, int iters, uint32_t *d_scratch_word, double *h_ops_per_second,
                     double *h_lanes_per_clock_per_sm, void *stream);

const char *hikonv_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* HIKONV_H */
