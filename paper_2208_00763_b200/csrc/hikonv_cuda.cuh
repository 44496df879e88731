// Small device/host helpers shared by the CUDA translation units.
#pragma once

#include <cuda_runtime.h>

#include <cstdint>

#include "hikonv_internal.h"

namespace hikonv {

// Evaluates a CUDA runtime call; on failure returns HIKONV_ERR_CUDA from the enclosing function.
#define HIKONV_CUDA_TRY(expr)                                 \
    do {                                                      \
        cudaError_t _e = (expr);                              \
        if (_e != cudaSuccess) return HIKONV_ERR_CUDA;        \
    } while (0)

// Plain launch that is judged by its own result: the status is what cudaLaunchKernelEx returns for THIS launch,
// so an error that an earlier, unrelated call left unread in the thread's error state is neither reported here
// nor cleared.
template <typename... Params, typename... Args>
inline int launch_plain(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = nullptr;
    cfg.numAttrs = 0;
    return cudaLaunchKernelEx(&cfg, kernel, args...) == cudaSuccess ? HIKONV_OK : HIKONV_ERR_CUDA;
}

// Programmatic dependent launch.  A kernel launched with launch_dependent() may be scheduled while the
// kernel before it on the stream is still running; it must call grid_dependency_wait() before its first
// access to global memory (the wait returns once the earlier kernel has finished and its writes are
// visible).  grid_dependency_release() lets the NEXT kernel of the stream be scheduled early; it takes
// effect once every CTA of this grid has called it or exited.  Every CTA of every such kernel waits, so
// completion of a kernel still implies completion of all kernels before it.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;"); }

template <typename... Params, typename... Args>
inline int launch_dependent(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...) == cudaSuccess ? HIKONV_OK : HIKONV_ERR_CUDA;
}

// The 32x32->64 product of two packed words (Eq. 9).  The multiply is given as inline PTX (mul.wide) and the
// 64-bit add is left to the compiler, which fuses the pair into one wide multiply-add.  Two other spellings were
// tried and dropped after counting instructions per opcode in the profiler: mad.wide as inline PTX came out as a
// multiply plus separate 64-bit additions, and the plain C++ expression (int64)a * (int64)b + c becomes a full
// 64-bit multiply (three multiplies and adds) whenever the optimiser has hoisted or combined one of the sign
// extensions.
template <bool SIGNED>
__device__ __forceinline__ uint64_t mul_wide(uint32_t a, uint32_t b) {
    uint64_t r;
    if (SIGNED)
        asm("mul.wide.s32 %0, %1, %2;" : "=l"(r) : "r"(a), "r"(b));
    else
        asm("mul.wide.u32 %0, %1, %2;" : "=l"(r) : "r"(a), "r"(b));
    return r;
}

// acc += a * b.
template <bool SIGNED>
__device__ __forceinline__ void mad_wide(uint64_t &acc, uint32_t a, uint32_t b) {
    acc += mul_wide<SIGNED>(a, b);
}

// a * b + c with the addend as an operand of its own.
template <bool SIGNED>
__device__ __forceinline__ uint64_t mul_wide_add(uint32_t a, uint32_t b, uint64_t c) {
    return c + mul_wide<SIGNED>(a, b);
}

// Low 32 bits of (v >> sh) for 0 <= sh < 64.
__device__ __forceinline__ uint32_t shr64_lo(uint64_t v, int sh) { return (uint32_t)(v >> sh); }

// A code byte as a 32-bit value (sign- or zero-extended).
template <bool SIGNED>
__device__ __forceinline__ int32_t code_value(int8_t b) {
    return SIGNED ? (int32_t)b : (int32_t)(uint8_t)b;
}

template <bool SIGNED>
__device__ __forceinline__ int32_t load_code(const int8_t *p) {
    return code_value<SIGNED>(__ldg(p));
}

// Asynchronous global -> shared copies (cp.async); src_bytes < 4 zero-fills the rest of the 4-byte word.
__device__ __forceinline__ void cp_async_4(void *smem_dst, const void *gmem_src, int src_bytes) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(gmem_src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_16(void *smem_dst, const void *gmem_src) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

}  // namespace hikonv
