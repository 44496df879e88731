// hikonv_pack: Eq. 5, codes -> packed 32- or 64-bit words (one thread per word).
#include "hikonv_cuda.cuh"

namespace hikonv {

template <bool SIGNED, typename WORD>
__global__ void __launch_bounds__(256) pack_kernel(const int8_t *__restrict__ in, size_t n, int S, int N,
                                                   WORD *__restrict__ words, size_t n_words) {
    const size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= n_words) return;
    const size_t base = x * (size_t)N;
    WORD a = 0;
    for (int i = 0; i < N; ++i) {
        const size_t idx = base + i;
        if (idx < n) {
            // two's-complement sum: a negative code borrows from the slots above it, which is
            // what the slot-by-slot decrementer of Eq. 28 builds
            const long long v = code_value<SIGNED>(__ldg(in + idx));
            a += (WORD)((unsigned long long)v << (S * i));
        }
    }
    words[x] = a;
}

}  // namespace hikonv

using namespace hikonv;

extern "C" int hikonv_pack(const int8_t *d_in, size_t n, int bits, int is_signed, int S, int N, int word_bits,
                           void *d_words, void *stream) {
    if (!d_in || !d_words) return HIKONV_ERR_INVALID_ARG;
    if (bits < 1 || bits > 8 || S < 1 || N < 1 || (word_bits != 32 && word_bits != 64)) return HIKONV_ERR_INVALID_ARG;
    if (S < bits) return HIKONV_ERR_INVALID_ARG;
    if ((long long)bits + (long long)(N - 1) * S > word_bits) return HIKONV_ERR_NO_FIT;
    if (((uintptr_t)d_words) % (word_bits / 8) != 0) return HIKONV_ERR_INVALID_ARG;
    if (n == 0) return HIKONV_OK;
    const size_t n_words = (n + N - 1) / N;
    const unsigned threads = 256;
    const size_t blocks = (n_words + threads - 1) / threads;
    if (blocks > 0x7FFFFFFFull) return HIKONV_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const dim3 grid((unsigned)blocks), block(threads);
    if (word_bits == 32) {
        if (is_signed) return launch_plain(pack_kernel<true, uint32_t>, grid, block, 0, st, d_in, n, S, N, (uint32_t *)d_words, n_words);
        return launch_plain(pack_kernel<false, uint32_t>, grid, block, 0, st, d_in, n, S, N, (uint32_t *)d_words, n_words);
    }
    if (is_signed) return launch_plain(pack_kernel<true, uint64_t>, grid, block, 0, st, d_in, n, S, N, (uint64_t *)d_words, n_words);
    return launch_plain(pack_kernel<false, uint64_t>, grid, block, 0, st, d_in, n, S, N, (uint64_t *)d_words, n_words);
}
