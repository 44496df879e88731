// Launcher of the 1-D kernel that runs the packed method on an emulated 64x64 -> 128 multiplier.
#pragma once

#include <cuda_runtime.h>

#include "hikonv_internal.h"

namespace hikonv {

// Plans the 64-bit layout, then enqueues one launch on `st`.  Arguments as for hikonv_conv1d (already validated).
int launch_conv1d_emu64(const int8_t *d_f, size_t len, const int8_t *d_g, int K, int p, int q, int f_signed, int g_signed,
                        int32_t *d_y, const hikonv_tuning_t *tune, cudaStream_t st);

}  // namespace hikonv
