// Interface between hikonv_conv1d.cu and the 1-D kernels with byte-aligned slots (hikonv_conv1d_bs.cu).
#pragma once

#include <cuda_runtime.h>

#include "hikonv_internal.h"

namespace hikonv {

struct Conv1dBsParams {
    const int8_t *f;
    const int8_t *g;
    int32_t *y;
    long long len;
    long long n_out;
    unsigned n_tiles;        // warp tiles of 32 * L outputs covering n_out
    unsigned fast_after_first;   // tiles 1 .. this many lie inside aligned buffers (0 when f or y is not aligned)
    int K;
    int g_signed;
    int aligned;             // f is 4-byte aligned and y is 16-byte aligned
    uint32_t code_xor;       // one-byte slots, signed f: 2^(p-1) in every byte (lifts a stored code to f + 2^(p-1))
    uint32_t code_and;       // one-byte slots, signed f: 2^p - 1 in every byte
    int S;                   // mode 3: slot width, 17 .. 21
    uint32_t mask3;          // mode 3: 2^S - 1
    uint64_t bias3;          // mode 3, signed product: b0 + 2^(S-1) 2^S + b2 2^(2S) with b0 + b2 = 2^(S-1)
};

constexpr int kBsRun = 24;   // outputs per lane and tile
// mode: 1 (S = 8, N = 4), 2 (S = 16, N = 2), 3 (S = 17 .. 21, N = 2); J = kernel words.  variant 24 / 25: register
// budget for four / five resident CTAs per SM; anything else: the faster of the two for (mode, J).
int launch_conv1d_bs(const Conv1dBsParams &p, int mode, int J, bool f_signed, bool signed_prod, int variant,
                     cudaStream_t st);

}  // namespace hikonv
