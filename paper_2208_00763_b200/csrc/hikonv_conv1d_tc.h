// Interface between hikonv_conv1d.cu (argument checks, layout) and the register-resident 1-D kernels.
#pragma once

#include <cuda_runtime.h>

#include "hikonv_internal.h"

namespace hikonv {

struct Conv1dTcParams {
    const int8_t *f;
    const int8_t *g;
    int32_t *y;
    long long len;
    long long n_out;
    long long n_tiles;       // warp tiles of 32 * L outputs covering n_out
    unsigned fast_after_first;   // comparators: tiles 1 .. this many lie inside aligned buffers (0: f or y unaligned)
    int K, S, Kc;
    int hi_shift;            // S * N
    int g_signed;
    int aligned;             // f is 4-byte aligned and y is 16-byte aligned
    long long dense_words;   // dense input only: whole 32-bit words in the input buffer
    uint32_t mask;
    uint64_t bias;
    int seg_shift[kMaxN1D];
    int32_t carry_bias[kMaxN1D];
};

int conv1d_tc_outputs_per_tile(int N);
// Block size the register-resident kernel runs fastest with when the planner chose N (N itself, or a smaller one).
int conv1d_tc_preferred_n(int N);
bool conv1d_packed_tc_available(int N, int J);
int launch_conv1d_packed_tc(const Conv1dTcParams &p, int N, int J, bool signed_prod, bool f_signed, cudaStream_t st);
// Dense input (P = 1, 2 or 4 bits per code, 8 / P codes per byte): the layouts that are instantiated.
bool conv1d_packed_dense_available(int P, int N, int J, int S, bool signed_prod, bool f_signed);
int launch_conv1d_packed_dense(const Conv1dTcParams &p, int P, int N, int J, bool signed_prod, bool f_signed, cudaStream_t st);
bool conv1d_unpacked_tc_available(int K);
int launch_conv1d_unpacked_tc(const Conv1dTcParams &p, int K, bool f_signed, int shape /* 24: runs of 24 outputs per lane, four CTAs per SM; 25: the same with five CTAs; 32: runs of 32, three CTAs */, cudaStream_t st);
// Byte dot-product comparator (four products per dp4a): kernels of up to eight taps.
bool conv1d_dp4a_tc_available(int K);
int launch_conv1d_dp4a_tc(const Conv1dTcParams &p, int K, bool f_signed, bool g_signed, int shape /* 24: runs of 24 outputs per lane, four CTAs per SM; 25: the same with five CTAs; 32: runs of 32, three CTAs */,
                          cudaStream_t st);

}  // namespace hikonv
