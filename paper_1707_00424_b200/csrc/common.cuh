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

// fp32 -> pair of tf32-exact floats (low 13 mantissa bits zero) with v = hi + lo up to 2^-22 |v|:
// hi = v rounded to tf32 (nearest, ties away from zero), lo = the exact remainder v - hi rounded the same way.
// Rounding to nearest keeps both errors centred on zero, so they do not add up over a long reduction.
__device__ __forceinline__ float round_tf32(float v) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
    return __uint_as_float(r);
}
__device__ __forceinline__ void split_tf32(float v, float &hi, float &lo) {
    hi = round_tf32(v);
    lo = round_tf32(v - hi);
}

// bf16 operand copy of a weight: the upper half of the fp32 word after adding 0x8000, i.e. rounded to nearest with
// ties away from zero.  Written this way (rather than ties-to-even) because the same addition splits the word into
// two 16-bit halves from which it can be put together again exactly: word = ((upper << 16) | lower) - 0x8000.
__device__ __forceinline__ uint32_t bf16_split_word(float v) { return __float_as_uint(v) + 0x8000u; }
__device__ __forceinline__ __nv_bfloat16 bf16_weight(float v) {
    return __ushort_as_bfloat16((unsigned short)(bf16_split_word(v) >> 16));
}

struct LayerPlan {
    int d_in, d_out;
    size_t w_off, b_off;          // element offsets inside one replica's vector
};

}  // namespace parle
