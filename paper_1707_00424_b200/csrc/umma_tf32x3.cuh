// fp32 configurations of the replica-grouped MLP forward / backward (Section 1.1 / 2.1: the minibatch
// gradient of f) on the sm_100a tensor cores, at fp32 accuracy.
//
// tcgen05.mma has no fp32-operand mode; kind::tf32 keeps 10 mantissa bits of each operand.  Every fp32 operand
// v is therefore stored as two tf32-exact arrays
//     hi = v rounded to tf32,   lo = (v - hi) rounded to tf32,
// (v - hi is exact in fp32; |v - hi - lo| <= 2^-22 |v|), and every product is accumulated as
//     A B^T  ~=  A_lo B_hi^T + A_hi B_lo^T + A_hi B_hi^T          (fp32 accumulators in tensor memory),
// which drops only the lo x lo term (2^-22 relative) -- the same order as fp32 rounding of a long sum.
// The tensor cores add into their fp32 accumulator with truncation, which over a long reduction drifts by about
// 2^-24 of the running sum per instruction (1e-5 relative at K = 784, measured).  So the accumulator in tensor
// memory only ever holds ONE 32-deep k-block (the eight small products first, then the four hi x hi ones); the
// epilogue warps read it back after every k-block and add it to fp32 register accumulators with round-to-nearest.
// Four accumulator buffers rotate, so the MMAs of the next k-blocks run meanwhile.
//
// kind::tf32 takes K-major operands only (an MN-major descriptor yields zeros), so every operand exists in the
// layout whose contiguous direction is the reduction index of the product that reads it:
//   forward      H_l      : A = H_{l-1}   [B, d_in],     B = W_l    [d_out, d_in]   (K = d_in)
//   data grad    dH_{l-1} : A = dH_l      [B, d_out],    B = W_l^T  [d_in, d_out]   (K = d_out; transposed weight copy)
//   weight grad  dW_l^T   : A = H_{l-1}^T [d_in, B],     B = dH_l^T [d_out, B]      (K = batch)
//                (accumulator rows = d_in, the contiguous direction of W, so the store is coalesced)
// i.e. activations and their gradients are kept as hi/lo pairs in both layouts, written by the epilogue that
// produces them (tensor-memory lanes = batch rows: the transposed store is the coalesced one, the row-major one
// writes 128 contiguous bytes per thread).  Rows whose length is not a multiple of 4 floats are padded (TMA wants
// 16-byte pitches); the reduction length in the tensor map is the true one, so padding is never read.
// One persistent CTA per SM walks (replica, m-tile, n-tile) work items: warp 0 = TMA producer (128-byte swizzled
// 32-column fp32 boxes), warp 1 = MMA issuer (M = 128, N = BN, K = 8 per instruction, 12 instructions per 32-deep
// k-block), warps 2..9 = accumulation + epilogue (two per 32-lane quarter of tensor memory, each taking half of the
// tile's columns).  Every wait is bounded.
#pragma once

#include "umma_gemm.cuh"

namespace parle {

constexpr int T3_BM = 128, T3_BK = 32;                     // 32 fp32 = one 128-byte swizzle row
constexpr int T3_A_BYTES = T3_BM * T3_BK * 4;              // 16 KiB per hi (or lo) tile of A
constexpr int T3_RING_BYTES = 192 * 1024;
constexpr int T3_EPI_WARPS = 8;
constexpr int T3_ACC_BUFS = 4;                             // accumulator buffers of 128 columns: all 512 columns of tensor memory
constexpr int T3_THREADS = 32 * (2 + T3_EPI_WARPS);

template <int BN>
struct T3Shape {
    static_assert(BN == 64 || BN == 128, "tile width");
    static constexpr int B_BYTES = BN * T3_BK * 4;
    static constexpr int STAGE_BYTES = 2 * T3_A_BYTES + 2 * B_BYTES;     // A_hi | A_lo | B_hi | B_lo
    static constexpr int STAGES = T3_RING_BYTES / STAGE_BYTES;           // 3 (BN = 128) or 4 (BN = 64)
    static constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

enum T3Epilogue {
    T3_FWD_HIDDEN = 0,     // + bias[n], ReLU; hi/lo out, row-major [m * ld + n] and transposed [n * ldT + m]
    T3_FWD_LAST = 1,       // + bias[n]; fp32 out [m * ld + n]
    T3_DGRAD = 2,          // * (mask[n, m] > 0); hi/lo out, both layouts
    T3_WGRAD = 3           // fp32 out, transposed: element (m, n) -> outf[n * ld + m]
};

struct T3Params {
    int M, N, K;                 // per-replica problem: D[M,N] = A[M,K] * B[N,K]^T
    int groups, tiles_m, tiles_n;
    const float *bias; long long bias_gs;
    float *out_hi, *out_lo; long long out_gs; int out_ld;          // row-major pair (out_ld % 4 == 0)
    float *outT_hi, *outT_lo; long long outT_gs; int outT_ld;       // transposed pair
    float *outf; long long outf_gs; int outf_ld;
    const float *mask_hi; long long mask_gs; int mask_ld;   // hi part of the layer input, transposed: [n * mask_ld + m]
                                                             // (rounding to tf32 keeps the sign: H > 0 exactly when its hi part is)
    // split-K (T3_FWD_LAST only): each tile's k-blocks are divided among ksplit work items, each of which stores its raw
    // partial sums (no bias) at outf + split * part_ss; the softmax kernel adds them up in fixed order
    int ksplit; long long part_ss;
    int *status;
};

__device__ __forceinline__ void tc_mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                            uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// Instruction descriptor: tf32 x tf32 -> fp32, M = 128, N = bn.
__host__ __device__ constexpr uint32_t make_idesc_tf32(bool a_mn_major, bool b_mn_major, int bn) {
    return (1u << 4)                       // D format fp32
         | (2u << 7) | (2u << 10)          // A, B format tf32
         | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16)
         | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(T3_BM >> 4) << 24);
}

// Operand tiles in shared memory (K-major, 128-byte swizzle): rows of 32 fp32 (128 B), 8-row groups 1024 B apart;
// one instruction (K = 8) reads 32 B of every row.
template <int EPI, int BN>
__global__ void __launch_bounds__(T3_THREADS, 1)
umma_tf32x3_kernel(const __grid_constant__ CUtensorMap tmAhi, const __grid_constant__ CUtensorMap tmAlo,
                   const __grid_constant__ CUtensorMap tmBhi, const __grid_constant__ CUtensorMap tmBlo,
                   const T3Params p) {
    using SH = T3Shape<BN>;
    constexpr int STAGES = SH::STAGES, B_BYTES = SH::B_BYTES, STAGE_BYTES = SH::STAGE_BYTES;
    constexpr uint32_t TMEM_COLS = 128 * T3_ACC_BUFS;                   // accumulator buffers of BN <= 128 columns
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;
    uint8_t *ctl = smem_raw + (tiles_base - raw) + (size_t)STAGES * STAGE_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(ctl);                  // full[S], empty[S], tfull[T3_ACC_BUFS], tempty[T3_ACC_BUFS]
    constexpr int NBARS = 2 * STAGES + 2 * T3_ACC_BUFS;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(ctl + 8 * NBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * STAGES, bar_tempty = bar_tfull + 8 * T3_ACC_BUFS;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int per_g = p.tiles_m * p.tiles_n;
    const int num_kb = (p.K + T3_BK - 1) / T3_BK;
    const int ksplit = (EPI == T3_FWD_LAST && p.ksplit > 1) ? p.ksplit : 1;
    const int total_items = p.groups * per_g * ksplit;     // work item = (tile, k range)

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int s = 0; s < T3_ACC_BUFS; ++s) { mbar_init(bar_tfull + 8 * s, 1); mbar_init(bar_tempty + 8 * s, T3_EPI_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    auto coords = [&](int t, int &g, int &m0, int &n0) {
        g = t / per_g;
        const int r = t - g * per_g;
        m0 = (r % p.tiles_m) * T3_BM;
        n0 = (r / p.tiles_m) * BN;
    };

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            for (int it = blockIdx.x; it < total_items && ok; it += gridDim.x) {
                const int t = it / ksplit, split = it - t * ksplit;
                const int kb_lo = split * num_kb / ksplit, kb_hi = (split + 1) * num_kb / ksplit;
                int g, m0, n0; coords(t, g, m0, n0);
                for (int kb = kb_lo; kb < kb_hi; ++kb) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t sa = tiles_base + stage * STAGE_BYTES, sb = sa + 2 * T3_A_BYTES;
                    const uint32_t fb = bar_full + 8 * stage;
                    mbar_expect_tx(fb, STAGE_BYTES);
                    const int k0 = kb * T3_BK;
                    tma_load_3d(sa, &tmAhi, fb, k0, m0, g);
                    tma_load_3d(sa + T3_A_BYTES, &tmAlo, fb, k0, m0, g);
                    tma_load_3d(sb, &tmBhi, fb, k0, n0, g);
                    tma_load_3d(sb + B_BYTES, &tmBlo, fb, k0, n0, g);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // gave up: let the copies already issued land before the CTA exits
                for (int s = 0; s < STAGES; ++s) {
                    const uint32_t armed_parity = (s < stage) ? phase : (phase ^ 1u);
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_full + 8 * s, armed_parity) && global_ns() - t0 < 20000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_tf32(false, false, BN);
            int stage = 0; uint32_t phase = 0; int acc = 0; uint32_t acc_phase = 0; bool ok = true;
            for (int it = blockIdx.x; it < total_items && ok; it += gridDim.x) {
                const int split = it % ksplit;
                const int kb_lo = split * num_kb / ksplit, kb_hi = (split + 1) * num_kb / ksplit;
                for (int kb = kb_lo; kb < kb_hi; ++kb) {
                    // one k-block per accumulator buffer
                    if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * 128;
                    const uint32_t sa = tiles_base + stage * STAGE_BYTES, sb = sa + 2 * T3_A_BYTES;
                    const uint64_t a_hi = make_smem_desc(sa, 16, 1024), a_lo = make_smem_desc(sa + T3_A_BYTES, 16, 1024);
                    const uint64_t b_hi = make_smem_desc(sb, 16, 1024), b_lo = make_smem_desc(sb + B_BYTES, 16, 1024);
                    // 8 fp32 = 32 B further along the row per instruction; the small products go first, while the
                    // accumulator is small
#pragma unroll
                    for (int k = 0; k < T3_BK / 8; ++k) {
                        tc_mma_tf32(d_tmem, a_lo + (uint64_t)(k * 2), b_hi + (uint64_t)(k * 2), idesc, k != 0 ? 1u : 0u);
                        tc_mma_tf32(d_tmem, a_hi + (uint64_t)(k * 2), b_lo + (uint64_t)(k * 2), idesc, 1u);
                    }
#pragma unroll
                    for (int k = 0; k < T3_BK / 8; ++k)
                        tc_mma_tf32(d_tmem, a_hi + (uint64_t)(k * 2), b_hi + (uint64_t)(k * 2), idesc, 1u);
                    tc_commit(bar_empty + 8 * stage);
                    tc_commit(bar_tfull + 8 * acc);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    if (++acc == T3_ACC_BUFS) { acc = 0; acc_phase ^= 1u; }
                }
            }
        }
    } else {
        // ------------------------------------------------ accumulation + epilogue (warps 2..9)
        const int q = warp & 3;                              // tensor-memory lane quarter this warp may read
        const int half = (warp - 2) >> 2;                    // columns half * BN/2 .. of every tile
        constexpr int CPW = BN / 64;                         // 32-column chunks per warp
        int acc = 0; uint32_t acc_phase = 0;
        bool ok = true;
        for (int it = blockIdx.x; it < total_items && ok; it += gridDim.x) {
            const int t = it / ksplit, split = it - t * ksplit;
            const int kb_lo = split * num_kb / ksplit, kb_hi = (split + 1) * num_kb / ksplit;
            int g, m0, n0; coords(t, g, m0, n0);
            const int m = m0 + q * 32 + lane;                // accumulator row of this thread
            const bool m_ok = m < p.M;
            float sum[CPW][32];
#pragma unroll
            for (int cc = 0; cc < CPW; ++cc)
#pragma unroll
                for (int j = 0; j < 32; ++j) sum[cc][j] = 0.f;
            for (int kb = kb_lo; kb < kb_hi; ++kb) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag));
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int cc = 0; cc < CPW; ++cc) {
                    uint32_t r[32];
                    tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * 128 + (half * CPW + cc) * 32), r);
#pragma unroll
                    for (int j = 0; j < 32; ++j) sum[cc][j] += __uint_as_float(r[j]);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
                if (++acc == T3_ACC_BUFS) { acc = 0; acc_phase ^= 1u; }
            }
            if (!ok) break;
#pragma unroll
            for (int cc = 0; cc < CPW; ++cc) {
                const int nb = n0 + (half * CPW + cc) * 32;
                if (nb >= p.N) break;                        // warp-uniform
                const float (&r)[32] = sum[cc];
                float bias_lane = 0.f;
                if (EPI == T3_FWD_HIDDEN || EPI == T3_FWD_LAST)
                    bias_lane = (nb + lane < p.N && ksplit == 1) ? __ldg(p.bias + (long long)g * p.bias_gs + nb + lane) : 0.f;
                if (EPI == T3_FWD_HIDDEN || EPI == T3_DGRAD) {
                    float *th = p.outT_hi + (long long)g * p.outT_gs + (long long)nb * p.outT_ld + m;
                    float *tl = p.outT_lo + (long long)g * p.outT_gs + (long long)nb * p.outT_ld + m;
                    float mk[32];                                        // ReLU mask source: all 32 loads in flight at once
                    if (EPI == T3_DGRAD) {
                        const float *mh = p.mask_hi + (long long)g * p.mask_gs + (long long)nb * p.mask_ld + m;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            mk[j] = (m_ok && nb + j < p.N) ? __ldg(mh + (long long)j * p.mask_ld) : 0.f;
                    }
                    float hi[32], lo[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        float v = r[j];
                        if (EPI == T3_FWD_HIDDEN) v = fmaxf(v + __shfl_sync(0xffffffffu, bias_lane, j), 0.f);
                        hi[j] = 0.f; lo[j] = 0.f;
                        if (m_ok && nb + j < p.N) {
                            if (EPI == T3_DGRAD && !(mk[j] > 0.f)) v = 0.f;
                            split_tf32(v, hi[j], lo[j]);
                            th[(long long)j * p.outT_ld] = hi[j];         // lanes = consecutive batch rows: coalesced
                            tl[(long long)j * p.outT_ld] = lo[j];
                        }
                    }
                    if (m_ok) {                                          // row-major: 32 consecutive floats of this thread's row
                        float *oh = p.out_hi + (long long)g * p.out_gs + (long long)m * p.out_ld + nb;
                        float *ol = p.out_lo + (long long)g * p.out_gs + (long long)m * p.out_ld + nb;
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            if (nb + j < p.out_ld) {                     // out_ld % 4 == 0; columns in [N, out_ld) get zeros
                                *reinterpret_cast<float4 *>(oh + j) = make_float4(hi[j], hi[j + 1], hi[j + 2], hi[j + 3]);
                                *reinterpret_cast<float4 *>(ol + j) = make_float4(lo[j], lo[j + 1], lo[j + 2], lo[j + 3]);
                            }
                        }
                    }
                }
                if (EPI == T3_FWD_LAST) {
                    float *o = p.outf + (long long)split * p.part_ss + (long long)g * p.outf_gs + (long long)m * p.outf_ld + nb;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float v = r[j] + __shfl_sync(0xffffffffu, bias_lane, j);
                        if (m_ok && nb + j < p.N) o[j] = v;
                    }
                }
                if (EPI == T3_WGRAD) {
                    if (m_ok) {
                        float *o = p.outf + (long long)g * p.outf_gs + (long long)nb * p.outf_ld + m;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (nb + j < p.N) o[(long long)j * p.outf_ld] = r[j];
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) p.status[SLOT_WAIT_LIMIT] = 1;
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---------------------------------------------------------------- helpers of the path
// src fp32 -> hi, lo (same indexing), 16-byte accesses.
__global__ void __launch_bounds__(256)
split_tf32_kernel(const float4 *__restrict__ src, float4 *__restrict__ hi, float4 *__restrict__ lo, size_t n4) {
    const size_t step = (size_t)gridDim.x * 256;
    for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < n4; i += step) {
        const float4 v = src[i];
        float4 h, l;
        split_tf32(v.x, h.x, l.x); split_tf32(v.y, h.y, l.y); split_tf32(v.z, h.z, l.z); split_tf32(v.w, h.w, l.w);
        hi[i] = h; lo[i] = l;
    }
}

// Minibatch inputs fp32 [n, B, d] -> hi/lo pairs in both layouts: [n, B, d] and transposed [n, d, B];
// 32 x 32 tiles through shared memory.
__global__ void __launch_bounds__(256)
input_split_kernel(const float *__restrict__ X, float *__restrict__ Xhi, float *__restrict__ Xlo,
                   float *__restrict__ Thi, float *__restrict__ Tlo, int B, int d) {
    __shared__ float tile[32][33];
    const int g = blockIdx.z;
    const int i0 = blockIdx.y * 32, j0 = blockIdx.x * 32;
    const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;            // 8 rows per pass
#pragma unroll
    for (int r = ty; r < 32; r += 8) {
        const int i = i0 + r, j = j0 + tx;
        float v = 0.f;
        if (i < B && j < d) {
            v = __ldcs(X + ((size_t)g * B + i) * d + j);
            float h, l;
            split_tf32(v, h, l);
            Xhi[((size_t)g * B + i) * d + j] = h;
            Xlo[((size_t)g * B + i) * d + j] = l;
        }
        tile[r][tx] = v;
    }
    __syncthreads();
#pragma unroll
    for (int r = ty; r < 32; r += 8) {
        const int j = j0 + r, i = i0 + tx;
        if (j < d && i < B) {
            float h, l;
            split_tf32(tile[tx][r], h, l);
            Thi[((size_t)g * d + j) * B + i] = h;
            Tlo[((size_t)g * d + j) * B + i] = l;
        }
    }
}

// Transposed hi/lo copy of the weights of the layers that have a data-gradient product (l >= 1):
// W_l [d_out, d_in] fp32 inside a replica's vector -> W_l^T [d_in, ld] (ld = d_out rounded up to 4), 64 x 64 tiles, 16-byte accesses.
struct TransposePlan {
    int n_layers;                                   // entries used (layers 1 .. of the network)
    long long w_off[PARLE_MAX_LAYERS], t_off[PARLE_MAX_LAYERS];
    int d_in[PARLE_MAX_LAYERS], d_out[PARLE_MAX_LAYERS], ld[PARLE_MAX_LAYERS];
    int tiles_in[PARLE_MAX_LAYERS], first_tile[PARLE_MAX_LAYERS + 1];
};

__global__ void __launch_bounds__(256)
split_transpose_kernel(const TransposePlan tp, const float *__restrict__ src, long long stride,
                       float *__restrict__ Thi, float *__restrict__ Tlo, long long t_stride) {
    __shared__ float tile[64][65];
    const int g = blockIdx.y;
    int l = 0;
    while (l + 1 < tp.n_layers && (int)blockIdx.x >= tp.first_tile[l + 1]) ++l;
    const int t = blockIdx.x - tp.first_tile[l];
    const int r0 = (t / tp.tiles_in[l]) * 64, c0 = (t % tp.tiles_in[l]) * 64;      // rows = d_out, columns = d_in
    const int d_in = tp.d_in[l], d_out = tp.d_out[l], ld = tp.ld[l];
    const float *W = src + (long long)g * stride + tp.w_off[l];
    const int q4 = (threadIdx.x % 16) * 4, rr = threadIdx.x / 16;                  // 16 threads x 4 floats = one 64-float row
#pragma unroll
    for (int r = rr; r < 64; r += 16) {
        const int row = r0 + r, col = c0 + q4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row < d_out && col < d_in) v = *reinterpret_cast<const float4 *>(W + (long long)row * d_in + col);   // d_in % 4 == 0
        tile[r][q4] = v.x; tile[r][q4 + 1] = v.y; tile[r][q4 + 2] = v.z; tile[r][q4 + 3] = v.w;
    }
    __syncthreads();
    float *oh = Thi + (long long)g * t_stride + tp.t_off[l], *ol = Tlo + (long long)g * t_stride + tp.t_off[l];
#pragma unroll
    for (int r = rr; r < 64; r += 16) {
        const int col = c0 + r, row = r0 + q4;                // W column (row of W^T), first of four W rows
        if (col < d_in && row < ld) {                         // ld % 4 == 0: the four are inside the padded row; rows >= d_out hold 0
            float4 h, lo;
            split_tf32(tile[q4][r], h.x, lo.x); split_tf32(tile[q4 + 1][r], h.y, lo.y);
            split_tf32(tile[q4 + 2][r], h.z, lo.z); split_tf32(tile[q4 + 3][r], h.w, lo.w);
            *reinterpret_cast<float4 *>(oh + (long long)col * ld + row) = h;
            *reinterpret_cast<float4 *>(ol + (long long)col * ld + row) = lo;
        }
    }
}

// db_l[g, j] = sum_i dH_l^T[g, j, i] from the hi/lo pairs [n, d_l, B] of all layers in one launch (blockIdx.z = layer):
// one warp per row, fixed-order tree.
struct BiasGradPlan {
    const float *hi[PARLE_MAX_LAYERS], *lo[PARLE_MAX_LAYERS];
    long long b_off[PARLE_MAX_LAYERS];              // offset of the layer's biases inside a replica's gradient
    int d[PARLE_MAX_LAYERS];
};
__global__ void __launch_bounds__(256)
bias_grad_split_kernel(const __grid_constant__ BiasGradPlan bp, float *__restrict__ grad, long long grad_gs, int B) {
    const int l = blockIdx.z, d = bp.d[l];
    const int j = blockIdx.x * 8 + threadIdx.x / 32, lane = threadIdx.x % 32;
    const int g = blockIdx.y;
    if (j >= d) return;
    const float *ph = bp.hi[l] + ((size_t)g * d + j) * B, *pl = bp.lo[l] + ((size_t)g * d + j) * B;
    float s = 0.f;
    for (int i = lane; i < B; i += 32) s += ph[i] + pl[i];
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) grad[(long long)g * grad_gs + bp.b_off[l] + j] = s;
}

}  // namespace parle
