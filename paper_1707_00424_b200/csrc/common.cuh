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

// Mean loss of a replica, formed by whichever warp finishes the replica's last rows.  `count` rows of replica g (their
// losses already stored in row_loss by this warp) are reported; rows_done[g] (zero between launches) counts them, and
// the warp that completes the B rows adds all B row losses up in one fixed order (256 strided partial sums, then a
// binary tree), stores loss[g] and puts the counter back to zero.  Called by all 32 lanes.
static __device__ __noinline__ void replica_loss_finish(const float *row_loss, float *loss, int *rows_done,
                                                    int g, int B, int count, int lane) {
    int before = 0;
    if (lane == 0 && count > 0) {
        __threadfence();                                     // the row losses are visible before they are counted
        before = atomicAdd(rows_done + g, count);
    }
    before = __shfl_sync(0xffffffffu, before, 0);
    if (count <= 0 || before + count != B) return;
    __threadfence();
    const float *rl = row_loss + (size_t)g * B;
    float part[8];                                           // partial sums of "threads" lane, lane + 32, ..., lane + 224 of a 256-wide sum
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        part[k] = 0.f;
        for (int r = lane + 32 * k; r < B; r += 256) part[k] += __ldcg(rl + r);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) part[k] += part[k + 4];      // tree step 128
    part[0] += part[2]; part[1] += part[3];                   // 64
    float t = part[0] + part[1];                              // 32
    for (int o = 16; o > 0; o >>= 1) t += __shfl_down_sync(0xffffffffu, t, o);
    if (lane == 0) { loss[g] = t / (float)B; rows_done[g] = 0; }
}

struct LayerPlan {
    int d_in, d_out;
    size_t w_off, b_off;          // element offsets inside one replica's vector
};

}  // namespace parle
