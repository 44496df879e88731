// Pieces shared by the register-resident 1-D kernels: each lane owns a contiguous run of L outputs, loads the
// codes of its run (plus a few in front) as aligned 32-bit words, and the warp writes its 32 runs through a
// shared-memory transpose so that every store instruction covers 512 contiguous bytes.
#pragma once

#include <mutex>
#include <unordered_map>

#include "hikonv_cuda.cuh"
#include "hikonv_conv1d_tc.h"

namespace hikonv {

constexpr int kThreadsTc = 256;
constexpr int kWarpsTc = kThreadsTc / 32;

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
            __stcs(dst + lane + 32 * k, *reinterpret_cast<const int4 *>(stage + src_lane * P + src_off));   // written once, never re-read
        }
        __syncwarp();
    } else {
        const long long e0 = tile0 + lane * L;
#pragma unroll
        for (int i = 0; i < L; ++i)
            if (e0 + i < n_out) y[e0 + i] = out[i];
    }
}

// The tile loop of a persistent warp: tiles t = first, first + stride, ... of 32 L outputs; the codes of the next
// tile are loaded before this tile's arithmetic.  `compute(w, out)` turns the NW = HW + L/4 loaded words of a lane
// (the 4 HW codes in front of its run, then its run) into its L outputs.  Tiles 1 .. fast_after_first lie inside
// aligned buffers and take 32-bit word loads and staged 16-byte stores, addressed as base + t * constant (one
// multiply-add each); tile 0, the tail and unaligned buffers take the guarded byte path.
template <int L, int HW, bool PREFETCH = true, typename Compute>
__device__ __forceinline__ void walk_tiles(const int8_t *f, int32_t *y, long long len, long long n_out, unsigned n_tiles,
                                           unsigned fast_after_first, int32_t *stage, Compute compute) {
    constexpr int NW = HW + L / 4;
    constexpr int P = stage_pitch(L);
    const unsigned lane = threadIdx.x & 31;
    const unsigned stride = gridDim.x * kWarpsTc;
    unsigned t = blockIdx.x * kWarpsTc + (threadIdx.x >> 5);
    const uint32_t *f_lane = reinterpret_cast<const uint32_t *>(f) + (int)(lane * (L / 4)) - HW;
    int4 *y_lane = reinterpret_cast<int4 *>(y) + lane;
    int4 *st_row = reinterpret_cast<int4 *>(stage + lane * P);
    // 16-byte piece g = lane + 32 k of the tile sits in row g / (L / 4) at word 4 (g % (L / 4)).  When L / 4 divides
    // 32 that is one base per lane plus a constant per k; otherwise the L / 4 offsets are worked out once, here.
    constexpr bool LINEAR = 32 % (L / 4) == 0;
    constexpr int PIECE_STEP = (32 / (L / 4)) * P / 4;                     // 16-byte units per k (LINEAR)
    const int4 *st_piece = reinterpret_cast<const int4 *>(stage + (lane / (L / 4)) * P + 4 * (lane % (L / 4)));
    int piece_off[LINEAR ? 1 : L / 4];
    if (!LINEAR) {
#pragma unroll
        for (int k = 0; k < L / 4; ++k) {
            const int g = lane + 32 * k;
            piece_off[k] = ((g / (L / 4)) * P + 4 * (g % (L / 4))) / 4;
        }
    }

    auto fetch = [&](unsigned tt, bool &fast, uint32_t (&dst)[NW]) {
        fast = (tt - 1u) < fast_after_first;
        if (fast) {
            const uint32_t *src = f_lane + (size_t)tt * (8 * L);
#pragma unroll
            for (int i = 0; i < NW; ++i) dst[i] = __ldg(src + i);
        } else {
            load_words<NW, HW>(f, len, (long long)tt * (32 * L) + lane * L, false, dst);
        }
    };
    uint32_t wn[NW];
    bool fast_n = false;
    if (PREFETCH && t < n_tiles) fetch(t, fast_n, wn);
    while (t < n_tiles) {
        const unsigned tc = t;
        uint32_t w[NW];
        bool fast;
        if (PREFETCH) {
            fast = fast_n;
#pragma unroll
            for (int i = 0; i < NW; ++i) w[i] = wn[i];
            t += stride;
            if (t < n_tiles) fetch(t, fast_n, wn);
        } else {                                   // without the prefetch the other resident warps cover the load latency
            fetch(t, fast, w);
            t += stride;
        }
        int32_t out[L];
        if (fast) {
            compute(w, out);
#pragma unroll
            for (int i = 0; i < L / 4; ++i) st_row[i] = make_int4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
            __syncwarp();
            int4 *dst = y_lane + (size_t)tc * (8 * L);
#pragma unroll
            for (int k = 0; k < L / 4; ++k)                                                     // written once, never re-read
                __stcs(dst + 32 * k, LINEAR ? st_piece[k * PIECE_STEP] : reinterpret_cast<const int4 *>(stage)[piece_off[LINEAR ? 0 : k]]);
            __syncwarp();
        } else {
            compute(w, out);
            const long long e0 = (long long)tc * (32 * L) + lane * L;
#pragma unroll
            for (int i = 0; i < L; ++i)
                if (e0 + i < n_out) y[e0 + i] = out[i];
        }
    }
}

// Tiles after tile 0 that take the fast path (see walk_tiles); 0 when the buffers are not aligned.
inline unsigned fast_tiles_after_first(long long len, int run, bool aligned) {
    const long long whole = len / (32LL * run);
    return (aligned && whole > 1) ? (unsigned)(whole - 1) : 0u;
}

// Persistent launch: as many CTAs as fit on the device at once (occupancy query, cached per kernel),
// fewer when the problem is small; each warp then walks tiles with a grid-wide stride.
// CTAs of `kernel` that fit one SM, asked once per kernel (all instantiations share one function-pointer
// type, so the answer is kept per pointer, not per template instance of the launcher).
inline int resident_ctas(const void *kernel) {
    static std::mutex mutex;
    static std::unordered_map<const void *, int> known;
    std::lock_guard<std::mutex> lock(mutex);
    auto it = known.find(kernel);
    if (it != known.end()) return it->second;
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kThreadsTc, 0) != cudaSuccess || occ < 1) occ = 1;
    known[kernel] = occ;
    return occ;
}

template <typename Kernel, typename Params>
inline int launch_persistent(Kernel kernel, const Params &p, cudaStream_t st) {
    const int resident = resident_ctas(reinterpret_cast<const void *>(kernel));
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long want = (p.n_tiles + kWarpsTc - 1) / kWarpsTc;
    const long long cap = (long long)sms * resident;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    return launch_plain(kernel, dim3(grid), dim3(kThreadsTc), 0, st, p);
}

}  // namespace hikonv
