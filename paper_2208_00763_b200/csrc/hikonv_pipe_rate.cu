// hikonv_pipe_rate: measured issue rate of the integer instructions the packed kernels are made of.
//
// The roofline of the 2-D layer kernels is the rate of the 32x32->64 multiply-add (Eq. 9 is one such
// instruction).  No public table gives that rate for this GPU, so the library measures it: every thread runs
// eight independent dependency chains of the instruction in registers; the multiplicand of each step is the
// low half of the NEXT chain's accumulator, so no product is loop-invariant and nothing can be hoisted or folded.
// The wide multiply-adds use the library's own helper (mad_wide), so the measurement counts what the kernels run.
// HIKONV_PIPE_MAD_WIDE_WITH_LOGIC interleaves one three-input logic instruction (on registers of its own) per two
// wide multiply-adds and reports the rate of the multiply-adds alone: what an instruction of another pipe costs
// the multiply-add stream (the layer kernels spend one to two such instructions per multiply-add on loads, carry-save
// moves and the split).
// Grid: four CTAs of 256 threads per SM (eight warps per scheduler, 64 independent instructions in flight on
// each), timed with CUDA events around the launch.
#include "hikonv_cuda.cuh"

namespace hikonv {

constexpr int kChains = 8;
constexpr int kUnroll = 8;

template <int KIND>
__global__ void __launch_bounds__(256) pipe_rate_kernel(int iters, uint32_t seed, uint32_t *sink) {
    const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t b = seed | 1u;                              // an odd multiplier: the chain never collapses to zero
    uint64_t acc[kChains];
    uint32_t side[kChains / 2];                                // the logic instructions of the mixed kind work on these
#pragma unroll
    for (int c = 0; c < kChains; ++c) acc[c] = ((uint64_t)(tid + 1) << 20) + 977u * c + seed;
#pragma unroll
    for (int c = 0; c < kChains / 2; ++c) side[c] = tid * 2654435761u + c;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                const uint32_t lo = (uint32_t)acc[c];
                const uint32_t hi = (uint32_t)(acc[c] >> 32);
                const uint32_t other = (uint32_t)acc[(c + 1) % kChains];
                if (KIND == HIKONV_PIPE_MAD_WIDE_WITH_LOGIC) {
                    mad_wide<false>(acc[c], other, b);
                    if (c & 1) {
                        const int j = c >> 1;
                        asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(side[j]) : "r"(b), "r"(side[(j + 1) % (kChains / 2)]));
                    }
                } else if (KIND == HIKONV_PIPE_MAD_WIDE_U32) {
                    mad_wide<false>(acc[c], other, b);
                } else if (KIND == HIKONV_PIPE_MAD_WIDE_S32) {
                    mad_wide<true>(acc[c], other, b);
                } else if (KIND == HIKONV_PIPE_MAD_LO_S32) {
                    uint32_t r;
                    asm volatile("mad.lo.s32 %0, %1, %2, %3;" : "=r"(r) : "r"(lo), "r"(b), "r"(hi));
                    acc[c] = ((uint64_t)hi << 32) | r;
                } else if (KIND == HIKONV_PIPE_LOGIC) {
                    uint32_t r;
                    asm volatile("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(r) : "r"(lo), "r"(b), "r"(hi));   // three-input xor
                    acc[c] = ((uint64_t)hi << 32) | r;
                } else if (KIND == HIKONV_PIPE_SHIFT) {
                    uint32_t r;
                    asm volatile("shf.r.wrap.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(lo), "r"(hi), "r"(b));
                    acc[c] = ((uint64_t)hi << 32) | r;
                } else {                                                                                   // byte permute
                    uint32_t r;
                    asm volatile("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(lo), "r"(hi), "r"(0x5140u));
                    acc[c] = ((uint64_t)hi << 32) | r;
                }
            }
        }
    }
    uint32_t x = 0;
#pragma unroll
    for (int c = 0; c < kChains; ++c) x ^= (uint32_t)acc[c] ^ (uint32_t)(acc[c] >> 32);
#pragma unroll
    for (int c = 0; c < kChains / 2; ++c) x ^= side[c];
    if (x == 0x9E3779B9u) sink[0] = x;                          // keeps the chains alive; practically never true
}

template <int KIND>
static int run_kind(int iters, unsigned grid, cudaStream_t st, uint32_t *d_sink) {
    return launch_plain(pipe_rate_kernel<KIND>, dim3(grid), dim3(256), 0, st, iters, 12345u, d_sink);
}

static int launch_kind(int kind, int iters, unsigned grid, cudaStream_t st, uint32_t *d_sink) {
    switch (kind) {
        case HIKONV_PIPE_MAD_WIDE_U32: return run_kind<HIKONV_PIPE_MAD_WIDE_U32>(iters, grid, st, d_sink);
        case HIKONV_PIPE_MAD_WIDE_S32: return run_kind<HIKONV_PIPE_MAD_WIDE_S32>(iters, grid, st, d_sink);
        case HIKONV_PIPE_MAD_LO_S32: return run_kind<HIKONV_PIPE_MAD_LO_S32>(iters, grid, st, d_sink);
        case HIKONV_PIPE_LOGIC: return run_kind<HIKONV_PIPE_LOGIC>(iters, grid, st, d_sink);
        case HIKONV_PIPE_SHIFT: return run_kind<HIKONV_PIPE_SHIFT>(iters, grid, st, d_sink);
        case HIKONV_PIPE_PRMT: return run_kind<HIKONV_PIPE_PRMT>(iters, grid, st, d_sink);
        case HIKONV_PIPE_MAD_WIDE_WITH_LOGIC: return run_kind<HIKONV_PIPE_MAD_WIDE_WITH_LOGIC>(iters, grid, st, d_sink);
        default: return HIKONV_ERR_INVALID_ARG;
    }
}

}  // namespace hikonv

using namespace hikonv;

extern "C" int hikonv_pipe_rate(int kind, int iters, uint32_t *d_scratch_word, double *h_ops_per_second,
                                double *h_lanes_per_clock_per_sm, void *stream) {
    if (!d_scratch_word || !h_ops_per_second || iters < 1 || iters > (1 << 20)) return HIKONV_ERR_INVALID_ARG;
    if (kind < HIKONV_PIPE_MAD_WIDE_U32 || kind > HIKONV_PIPE_MAD_WIDE_WITH_LOGIC) return HIKONV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    int dev = 0, sms = 0, khz = 0;
    HIKONV_CUDA_TRY(cudaGetDevice(&dev));
    HIKONV_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    HIKONV_CUDA_TRY(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev));
    const unsigned grid = (unsigned)sms * 4u;
    cudaEvent_t e0, e1;
    HIKONV_CUDA_TRY(cudaEventCreate(&e0));
    if (cudaEventCreate(&e1) != cudaSuccess) {
        cudaEventDestroy(e0);
        return HIKONV_ERR_CUDA;
    }
    int rc = launch_kind(kind, iters, grid, st, d_scratch_word);         // warm-up (clocks, instruction cache)
    float best_ms = 0.0f;
    for (int rep = 0; rep < 3 && rc == HIKONV_OK; ++rep) {
        if (cudaEventRecord(e0, st) != cudaSuccess) { rc = HIKONV_ERR_CUDA; break; }
        rc = launch_kind(kind, iters, grid, st, d_scratch_word);
        if (rc != HIKONV_OK) break;
        float ms = 0.0f;
        if (cudaEventRecord(e1, st) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess ||
            cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) { rc = HIKONV_ERR_CUDA; break; }
        if (rep == 0 || ms < best_ms) best_ms = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (rc != HIKONV_OK) return rc;
    if (best_ms <= 0.0f) return HIKONV_ERR_CUDA;
    const double ops = (double)grid * 256.0 * (double)iters * kUnroll * kChains;
    *h_ops_per_second = ops / (best_ms * 1e-3);
    if (h_lanes_per_clock_per_sm) *h_lanes_per_clock_per_sm = *h_ops_per_second / ((double)sms * (double)khz * 1e3);
    return HIKONV_OK;
}
