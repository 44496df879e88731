// hikonv_check_range: debug pass over stored codes.  The packed method assumes that every code lies in
// its p-bit range (the operand bounds of Eq. 7-8 and the guard bits of Eq. 11 are derived from that
// range); a code outside it overflows its slot without any error.  This pass counts such codes.
#include "hikonv_cuda.cuh"

namespace hikonv {

// Number of bytes of `w` whose bits selected by `high` are not all zero after adding `lift` to each byte.
// Signed codes: lift = 2^(p-1) maps the range [-2^(p-1), 2^(p-1) - 1] onto [0, 2^p - 1]; unsigned: lift = 0.
__device__ __forceinline__ unsigned bad_bytes(uint32_t w, uint32_t lift, uint32_t high) {
    const uint32_t t = __vadd4(w, lift) & high;
    return __popc(__vcmpne4(t, 0u)) >> 3;
}

__global__ void __launch_bounds__(256) check_range_kernel(const uint8_t *__restrict__ in, size_t n, size_t head, size_t n_vec,
                                                          uint32_t lift, uint32_t high, unsigned long long *count) {
    // [0, head): bytes before the first 16-byte boundary; n_vec 16-byte pieces; then the tail
    const uint4 *vec = reinterpret_cast<const uint4 *>(in + head);
    unsigned bad = 0;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += stride) {
        const uint4 v = __ldg(vec + i);
        bad += bad_bytes(v.x, lift, high) + bad_bytes(v.y, lift, high) + bad_bytes(v.z, lift, high) + bad_bytes(v.w, lift, high);
    }
    if (blockIdx.x == 0) {
        const size_t tail0 = head + n_vec * 16;
        const size_t edge = head + (n - tail0);            // fewer than 32 bytes in all
        for (size_t e = threadIdx.x; e < edge; e += blockDim.x) {
            const size_t idx = e < head ? e : tail0 + (e - head);
            bad += bad_bytes((uint32_t)in[idx], lift & 0xFFu, high & 0xFFu);
        }
    }
    bad = __reduce_add_sync(0xFFFFFFFFu, bad);
    if ((threadIdx.x & 31) == 0 && bad) atomicAdd(count, (unsigned long long)bad);
}

}  // namespace hikonv

using namespace hikonv;

extern "C" int hikonv_check_range(const int8_t *d_in, size_t n, int bits, int is_signed, unsigned long long *d_count,
                                  unsigned long long *h_count, void *stream) {
    if (!d_in || !d_count || bits < 1 || bits > 8 || ((uintptr_t)d_count % 8) != 0) return HIKONV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned long long found = 0;
    HIKONV_CUDA_TRY(cudaMemsetAsync(d_count, 0, sizeof(unsigned long long), st));
    if (bits < 8 && n > 0) {                    // every byte value is a valid 8-bit code, signed or not
        const uint32_t high1 = (0xFFu << bits) & 0xFFu, lift1 = is_signed ? (1u << (bits - 1)) : 0u;
        const uint32_t high = high1 * 0x01010101u, lift = lift1 * 0x01010101u;
        size_t head = (16 - ((uintptr_t)d_in % 16)) % 16;
        if (head > n) head = n;
        const size_t n_vec = (n - head) / 16;
        int sms = 148, dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        size_t blocks = (n_vec + 255) / 256;
        if (blocks > (size_t)sms * 8) blocks = (size_t)sms * 8;
        if (blocks < 1) blocks = 1;
        if (launch_plain(check_range_kernel, dim3((unsigned)blocks), dim3(256), 0, st, reinterpret_cast<const uint8_t *>(d_in), n, head,
                         n_vec, lift, high, d_count) != HIKONV_OK)
            return HIKONV_ERR_CUDA;
    }
    HIKONV_CUDA_TRY(cudaMemcpyAsync(&found, d_count, sizeof(found), cudaMemcpyDeviceToHost, st));
    HIKONV_CUDA_TRY(cudaStreamSynchronize(st));
    if (h_count) *h_count = found;
    return found ? HIKONV_ERR_RANGE : HIKONV_OK;
}
