// Shared declarations of the Parle CUDA library (host context + small helpers).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/parle.h"

namespace parle {

// Slots of the status block (pinned host memory mapped into the device; the
// kernels store 1 into a slot, the host reads the block without synchronising).
enum StatusSlot { SLOT_NONFINITE = 0, SLOT_WAIT_LIMIT = 1, SLOT_BAD_LABEL = 2, SLOT_COUNT = 16 };

__host__ __device__ inline size_t round_up(size_t v, size_t m) { return (v + m - 1) / m * m; }

struct LayerPlan {
    int d_in, d_out;
    size_t w_off, b_off;          // element offsets inside one replica's vector
};

}  // namespace parle
