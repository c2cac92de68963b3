// Replica-grouped bf16 GEMMs on the sm_100a tensor cores for the MLP
// forward / backward (Section 1.1 / 2.1: the minibatch gradient of f):
//   forward      H_l      = act(H_{l-1} W_l^T + b_l)           A=[B,d_in]   K-major, B=W [d_out,d_in] K-major
//   data grad    dH_{l-1} = (dH_l W_l) * 1[H_{l-1} > 0]        A=[B,d_out]  K-major, B=W [d_out(K), d_in(N)] MN-major
//                (W is read from its bf16 operand copy, which is stored in 128-row x 64-column blocks of 16 KiB
//                 so that every TMA box of either product is one contiguous run of memory)
//   weight grad  dW_l^T   = H_{l-1}^T dH_l                     A=H^T [d_in,B] K-major, B=dH^T [d_out,B] K-major
//                (computed transposed: accumulator rows = d_in, the contiguous direction of W in memory,
//                 so the 32 lanes of an epilogue warp touch 32 consecutive floats of one W row)
// One persistent CTA per SM walks (replica, m-tile, n-tile) work items.
// Two producer warps stage 128x64 operand tiles with TMA (128-byte swizzle) through
// two rings of shared-memory buffers (one per operand), warp 1 issues tcgen05.mma (M=128, N=128, K=16,
// fp32 accumulators in tensor memory, two accumulator buffers), warps 2-5 read
// the accumulators back with tcgen05.ld and run the fused epilogue.
// Every wait is bounded: on a time-out the CTA records it in the status block,
// drains and returns (tensor memory is always released).
#pragma once

#include "common.cuh"

namespace parle {

constexpr int UM_BM = 128, UM_BN = 128, UM_BK = 64;
constexpr int UM_A_BYTES = UM_BM * UM_BK * 2;              // 16 KiB
constexpr int UM_B_BYTES = UM_BN * UM_BK * 2;              // 16 KiB
constexpr int UM_STAGE_BYTES = UM_A_BYTES + UM_B_BYTES;    // one k-block of both operands
// The two operands have separate rings.  In the forward and data-gradient products the B operand is the
// replica's weights, which stream from HBM exactly once (about 3 us loaded latency), while the A operand
// (activations) is shared by all n-tiles of a replica and comes from L2: B gets the deep ring.  With
// 8 x 16 KiB of weights in flight on every SM the weight stream is not latency-bound.
constexpr int UM_A_STAGES = 4, UM_B_STAGES = 8;            // B stages of 128 rows; a 256-row tile uses them in pairs
// Tile width BN (accumulator columns): 128, or 256 where the product is compute-bound and has tiles to spare --
// per flop a 128 x 256 tile moves 25 % less through shared memory (the limit of a 128 x 128 tile whose both
// operands stream from shared memory), at the price of all 512 tensor-memory columns for its two accumulators.
// Warps: 0 = B producer, 1 = MMA issuer, 2..9 = epilogue (two per 32-lane quarter of tensor memory, each taking
// two of the four 32-column chunks of a tile), 10 = A producer.
__host__ __device__ constexpr int umma_epi_warps(int) { return 8; }
__host__ __device__ constexpr int umma_threads(int epi) { return 96 + 32 * umma_epi_warps(epi); }
constexpr int UM_TMEM_COLS = 256;                          // two 128-column accumulators
// Per epilogue warp: a 32 x 32 bf16 scratch tile (rows padded to 80 bytes) through which the transposed copy of an
// output chunk is turned into 16-byte stores.
constexpr int UM_EPI_PITCH = 40;                           // bf16 elements per scratch row (32 + 8 padding)
constexpr int UM_EPI_SCRATCH = 32 * UM_EPI_PITCH * 2;      // bytes per warp
constexpr size_t UM_SMEM_BYTES = (size_t)UM_A_STAGES * UM_A_BYTES + (size_t)UM_B_STAGES * UM_B_BYTES +
                                 8 * UM_EPI_SCRATCH + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr unsigned long long UM_WAIT_LIMIT_NS = 2000000000ull;   // 2 s per wait

// How the B operand is fetched.
enum UmmaBKind {
    UB_ROWMAJOR_K = 0,     // plain [rows, K] row-major tensor, K-major operand (3-D map: K, row, replica)
    UB_BLOCKED_K = 1,      // blocked weight copy, K-major operand: box = one whole 128 x 64 block
    UB_BLOCKED_MN = 2      // blocked weight copy, MN-major operand: boxes = 64 k-rows x 64 n-columns (half blocks)
};

enum UmmaEpilogue {
    UEPI_FWD_HIDDEN = 0,   // + bias[n], ReLU, bf16 out [M,ld] and transposed out [N,ldT]
    UEPI_FWD_LAST = 1,     // + bias[n], fp32 out [M,ld]
    UEPI_DGRAD = 2,        // * (mask[m,n] > 0), bf16 out and transposed out
    UEPI_WGRAD = 3,        // fp32 out, transposed: element (m, n) -> outf[n * ld + m]
    UEPI_FWD_LAST_CE = 4   // last layer with the loss in the epilogue (N <= 128): + bias[n], fp32 logits out, then row-wise
                           // softmax cross-entropy: dlogits = (softmax - onehot)/M as bf16 in both layouts, row losses, mean loss
};

struct UmmaParams {
    int M, N, K;                 // per-replica problem: D[M,N] = A[M,K] * B[N,K]^T
    int groups, tiles_m, tiles_n;
    const float *bias; long long bias_gs;
    __nv_bfloat16 *out; long long out_gs; int out_ld;
    __nv_bfloat16 *outT; long long outT_gs; int outT_ld;
    float *outf; long long outf_gs; int outf_ld;
    const __nv_bfloat16 *mask; long long mask_gs; int mask_ld;
    // split-K (UEPI_FWD_LAST only): each tile's k-blocks are divided among ksplit work items, each of which
    // stores its raw partial sums (no bias) at outf + split * part_ss; a later kernel adds them up in fixed order
    int ksplit; long long part_ss;
    // UEPI_FWD_LAST_CE: labels [groups, M]; dlogits bf16 [M, dbf_ld] and transposed [N, M] per replica (out / outT fields);
    // row_loss [groups, M]; loss [groups] or NULL with its row counters (see replica_loss_finish)
    const int32_t *labels; float *row_loss; float *loss; int *rows_done;
    int *status;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false when the limit passed or another role of this
// CTA already gave up (abort_flag, shared memory).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > UM_WAIT_LIMIT_NS) { *abort_flag = 1; return false; }
        }
    }
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tm, uint32_t bar,
                                            int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap *tm, uint32_t bar,
                                            int c0, int c1, int c2, int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                            uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Loads from tensor memory: 32 lanes x N consecutive columns, one column per register.  The load is asynchronous --
// its destination registers hold the data only after tcgen05.wait::ld -- and the compiler does not know that: with the
// wait in a statement of its own, arithmetic on the registers may be scheduled between the two.  So each wrapper issues
// the load AND the wait in one statement; what it returns is ready to use.
__device__ __forceinline__ void tc_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_ld_32x4(uint32_t taddr, uint32_t (&r)[4]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];\n\t"
                 "tcgen05.wait::ld.sync.aligned;"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
}

// Shared-memory matrix descriptor of a 128-byte-swizzled operand tile.
//   K-major tile  : rows of 64 bf16 (128 B), 8-row groups 1024 B apart (SBO).
//   MN-major tile : 64 k-rows of 64 MN-elements (128 B), 8-row groups 1024 B
//                   apart (SBO); the next 64 MN-elements start lbo_bytes later.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;          // descriptor version of this architecture
    d |= (uint64_t)2 << 61;          // 128-byte swizzle
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 128.
__host__ __device__ constexpr uint32_t make_idesc(bool a_mn_major, bool b_mn_major, int bn = UM_BN) {
    return (1u << 4)                       // D format fp32
         | (1u << 7) | (1u << 10)          // A, B format bf16
         | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16)
         | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(UM_BM >> 4) << 24);
}

__device__ __forceinline__ void tile_coords(const UmmaParams &p, int t, int bn, int &g, int &m0, int &n0) {
    const int per_g = p.tiles_m * p.tiles_n;
    g = t / per_g;
    const int r = t - g * per_g;
    m0 = (r % p.tiles_m) * UM_BM;
    n0 = (r / p.tiles_m) * bn;
}

template <int EPI, int BKIND, int BN = UM_BN>
__global__ void __launch_bounds__(umma_threads(EPI), 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const UmmaParams p) {
    static_assert(BN == 128 || BN == 256, "tile width");
    constexpr int B_STAGES = UM_B_STAGES * UM_BN / BN;                 // stages of BN rows in the same ring bytes
    constexpr int B_BYTES = BN * UM_BK * 2;
    constexpr uint32_t TMEM_COLS = 2 * BN;                             // two accumulators
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;                 // 1024-byte aligned (swizzle atom)
    const uint32_t a_base = tiles_base, b_base = tiles_base + UM_A_STAGES * UM_A_BYTES;
    uint8_t *epi_scratch = smem_raw + (tiles_base - raw) + (size_t)UM_A_STAGES * UM_A_BYTES + (size_t)UM_B_STAGES * UM_B_BYTES;
    uint8_t *ctl = epi_scratch + 8 * UM_EPI_SCRATCH;
    uint64_t *bars = reinterpret_cast<uint64_t *>(ctl);   // a_full[SA], a_empty[SA], b_full[SB], b_empty[SB], tfull[2], tempty[2]
    constexpr int NBARS = 2 * UM_A_STAGES + 2 * UM_B_STAGES + 4;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(ctl + 8 * NBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const uint32_t bar_afull = smem_u32(bars), bar_aempty = bar_afull + 8 * UM_A_STAGES;
    const uint32_t bar_bfull = bar_aempty + 8 * UM_A_STAGES, bar_bempty = bar_bfull + 8 * UM_B_STAGES;
    const uint32_t bar_tfull = bar_bempty + 8 * UM_B_STAGES, bar_tempty = bar_tfull + 16;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = p.groups * p.tiles_m * p.tiles_n;
    const int num_kb = (p.K + UM_BK - 1) / UM_BK;
    const int ksplit = (EPI == UEPI_FWD_LAST && p.ksplit > 1) ? p.ksplit : 1;
    const int total_items = total_tiles * ksplit;

    if (threadIdx.x == 0) {
        for (int s = 0; s < UM_A_STAGES; ++s) { mbar_init(bar_afull + 8 * s, 1); mbar_init(bar_aempty + 8 * s, 1); }
        for (int s = 0; s < B_STAGES; ++s) { mbar_init(bar_bfull + 8 * s, 1); mbar_init(bar_bempty + 8 * s, 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar_tfull + 8 * s, 1); mbar_init(bar_tempty + 8 * s, umma_epi_warps(EPI)); }
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

    if (warp == 0) {
        // ------------------------------------------------ TMA producer of the B operand (deep ring)
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            for (int it = blockIdx.x; it < total_items && ok; it += gridDim.x) {
                const int t = it / ksplit, split = it - t * ksplit;
                const int kb_lo = split * num_kb / ksplit, kb_hi = (split + 1) * num_kb / ksplit;
                int g, m0, n0; tile_coords(p, t, BN, g, m0, n0);
                for (int kb = kb_lo; kb < kb_hi; ++kb) {
                    if (!mbar_wait(bar_bempty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t sb = b_base + stage * B_BYTES;
                    const uint32_t fb = bar_bfull + 8 * stage;
                    mbar_expect_tx(fb, B_BYTES);
                    if (BKIND == UB_ROWMAJOR_K) {
#pragma unroll
                        for (int h = 0; h < BN / 128; ++h)
                            tma_load_3d(sb + h * UM_B_BYTES, &tmB, fb, kb * UM_BK, n0 + h * 128, g);
                    } else if (BKIND == UB_BLOCKED_K) {
                        // blocks (row block n0/128 [+1], column block kb) of the blocked weight copy
#pragma unroll
                        for (int h = 0; h < BN / 128; ++h)
                            tma_load_5d(sb + h * UM_B_BYTES, &tmB, fb, 0, 0, kb, n0 / 128 + h, g);
                    } else {
                        // k-rows kb*64 .. +63 = half of row block kb/2; n-columns n0 .. n0+BN-1 = column blocks n0/64 ...
#pragma unroll
                        for (int h = 0; h < BN / 64; ++h)
                            tma_load_5d(sb + h * (UM_B_BYTES / 2), &tmB, fb, 0, (kb & 1) * 64, n0 / 64 + h, kb >> 1, g);
                    }
                    if (++stage == B_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // gave up: let the copies already issued land before the CTA exits
                // (slots below `stage` were armed in this pass of the ring, the others in the previous one)
                for (int s = 0; s < B_STAGES; ++s) {
                    const uint32_t armed_parity = (s < stage) ? phase : (phase ^ 1u);
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_bfull + 8 * s, armed_parity) && global_ns() - t0 < 20000000ull) {}
                }
            }
        }
    } else if (warp == 2 + umma_epi_warps(EPI)) {
        // ------------------------------------------------ TMA producer of the A operand
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            for (int it = blockIdx.x; it < total_items && ok; it += gridDim.x) {
                const int t = it / ksplit, split = it - t * ksplit;
                const int kb_lo = split * num_kb / ksplit, kb_hi = (split + 1) * num_kb / ksplit;
                int g, m0, n0; tile_coords(p, t, BN, g, m0, n0);
                for (int kb = kb_lo; kb < kb_hi; ++kb) {
                    if (!mbar_wait(bar_aempty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t fb = bar_afull + 8 * stage;
                    mbar_expect_tx(fb, UM_A_BYTES);
                    tma_load_3d(a_base + stage * UM_A_BYTES, &tmA, fb, kb * UM_BK, m0, g);
                    if (++stage == UM_A_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                for (int s = 0; s < UM_A_STAGES; ++s) {
                    const uint32_t armed_parity = (s < stage) ? phase : (phase ^ 1u);
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_afull + 8 * s, armed_parity) && global_ns() - t0 < 20000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr bool B_MN = (BKIND == UB_BLOCKED_MN);
            constexpr uint32_t idesc = make_idesc(false, B_MN, BN);
            int sa_i = 0, sb_i = 0; uint32_t pa = 0, pb = 0; int acc = 0; uint32_t acc_phase = 0; bool ok = true;
            for (int it = blockIdx.x; it < total_items && ok; it += gridDim.x) {
                const int t = it / ksplit, split = it - t * ksplit;
                const int kb_lo = split * num_kb / ksplit, kb_hi = (split + 1) * num_kb / ksplit;
                if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = kb_lo; kb < kb_hi; ++kb) {
                    if (!mbar_wait(bar_afull + 8 * sa_i, pa, abort_flag)) { ok = false; break; }
                    if (!mbar_wait(bar_bfull + 8 * sb_i, pb, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = a_base + sa_i * UM_A_BYTES, sb = b_base + sb_i * B_BYTES;
                    const uint64_t adesc = make_smem_desc(sa, 16, 1024);
                    const uint64_t bdesc = B_MN ? make_smem_desc(sb, UM_B_BYTES / 2, 1024)
                                                : make_smem_desc(sb, 16, 1024);
#pragma unroll
                    for (int k = 0; k < UM_BK / 16; ++k) {
                        // K-major: 16 bf16 = 32 B further along the row; MN-major: two 8-row groups = 2048 B
                        const uint64_t a_k = adesc + (uint64_t)(k * 2);
                        const uint64_t b_k = bdesc + (uint64_t)(B_MN ? k * 128 : k * 2);
                        tc_mma_bf16(d_tmem, a_k, b_k, idesc, (kb != kb_lo || k != 0) ? 1u : 0u);
                    }
                    tc_commit(bar_aempty + 8 * sa_i);        // both slots are free once these MMAs retire
                    tc_commit(bar_bempty + 8 * sb_i);
                    if (++sa_i == UM_A_STAGES) { sa_i = 0; pa ^= 1u; }
                    if (++sb_i == B_STAGES) { sb_i = 0; pb ^= 1u; }
                }
                if (!ok) break;
                tc_commit(bar_tfull + 8 * acc);              // accumulator complete
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else if (warp < 2 + umma_epi_warps(EPI)) {
        // ------------------------------------------------ epilogue (warps 2..9)
        const int q = warp & 3;                              // TMEM lane quarter this warp may read
        const int half = (warp - 2) >> 2;                    // chunks 2*half, 2*half + 1 of every tile
        int acc = 0; uint32_t acc_phase = 0;
        for (int it = blockIdx.x; it < total_items; it += gridDim.x) {
            const int t = it / ksplit, split = it - t * ksplit;
            int g, m0, n0; tile_coords(p, t, BN, g, m0, n0);
            const int m = m0 + q * 32 + lane;                // output row of this thread
            const bool m_ok = m < p.M;
            // what the epilogue needs besides the accumulator is fetched before the accumulator is awaited
            constexpr int CPW = BN / 64;                     // 32-column chunks per epilogue warp
            constexpr bool MASK_AHEAD = (BN == 128);         // wide tiles: the mask is read chunk by chunk (registers)
            float bias_lane[CPW];                            // bias[nb + lane] of this warp's chunks
            uint4 mk[MASK_AHEAD ? CPW : 1][4];               // ReLU mask source: 32 bf16 of row m per chunk
            if (EPI == UEPI_FWD_HIDDEN || EPI == UEPI_FWD_LAST || EPI == UEPI_FWD_LAST_CE) {
                const float *bias = p.bias + (long long)g * p.bias_gs;
#pragma unroll
                for (int cc = 0; cc < CPW; ++cc) {
                    const int col = n0 + (CPW * half + cc) * 32 + lane;
                    bias_lane[cc] = (col < p.N && ksplit == 1) ? __ldg(bias + col) : 0.f;
                }
            }
            if (EPI == UEPI_DGRAD && MASK_AHEAD) {
#pragma unroll
                for (int cc = 0; cc < CPW; ++cc) {
                    const int nb = n0 + (CPW * half + cc) * 32;
                    const __nv_bfloat16 *mkp = p.mask + (long long)g * p.mask_gs + (long long)m * p.mask_ld + nb;
#pragma unroll
                    for (int j8 = 0; j8 < 4; ++j8) {
                        mk[cc][j8] = make_uint4(0u, 0u, 0u, 0u);
                        if (m_ok && nb + j8 * 8 < p.N) mk[cc][j8] = *reinterpret_cast<const uint4 *>(mkp + j8 * 8);
                    }
                }
            }
            const bool ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag));
            if (!ok) break;
            tc_fence_after();
            if (EPI == UEPI_FWD_LAST_CE) {
                // The whole logit row of a batch entry lies in this tile (N <= 128): this warp holds columns 64*half .. +63
                // of its 32 rows, its partner warp (same lane quarter, other half) the rest.  The two exchange the row
                // maximum, the sum of exponentials and the label's logit through their scratch tiles (named barrier of
                // the 64 threads), then each forms its half of dlogits = (softmax - onehot)/M.
                static_assert(EPI != UEPI_FWD_LAST_CE || BN == 128, "loss epilogue: one 128-wide tile per row");
                float *mine = reinterpret_cast<float *>(epi_scratch + (warp - 2) * UM_EPI_SCRATCH);
                const float *theirs = reinterpret_cast<const float *>(epi_scratch + ((warp - 2) ^ 4) * UM_EPI_SCRATCH);
                auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + q) : "memory"); };
                float v[2][32];
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    uint32_t r[32];
                    tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + (2 * half + cc) * 32), r);
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[cc][j] = __uint_as_float(r[j]) + __shfl_sync(0xffffffffu, bias_lane[cc], j);
                }
                const int c0 = n0 + half * 64;                   // first column of this warp
                const int label = m_ok ? p.labels[(long long)g * p.M + m] : 0;
                const bool label_ok = label >= 0 && label < p.N;
                float mx = -INFINITY, cand = 0.f;
#pragma unroll
                for (int cc = 0; cc < 2; ++cc)
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int col = c0 + cc * 32 + j;
                        if (col < p.N) mx = fmaxf(mx, v[cc][j]);
                        if (col == label) cand = v[cc][j];
                    }
                mine[lane] = mx; mine[64 + lane] = cand;
                pair_sync();
                mx = fmaxf(mx, theirs[lane]);
                const float label_logit = half == 0 ? cand + theirs[64 + lane] : theirs[64 + lane] + cand;
                float se = 0.f;
#pragma unroll
                for (int cc = 0; cc < 2; ++cc)
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (c0 + cc * 32 + j < p.N) se += __expf(v[cc][j] - mx);
                mine[32 + lane] = se;
                pair_sync();
                const float s_all = half == 0 ? se + theirs[32 + lane] : theirs[32 + lane] + se;     // same sum in both warps
                const float inv_s = 1.f / s_all, inv_M = 1.f / (float)p.M;
                if (m_ok) {                                      // fp32 logits, as the plain last-layer epilogue stores them
                    float *o = p.outf + (long long)g * p.outf_gs + (long long)m * p.outf_ld + c0;
                    const bool vec = (p.outf_ld & 3) == 0;       // rows start 16-byte aligned: four columns per store
#pragma unroll
                    for (int cc = 0; cc < 2; ++cc)
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const int col = c0 + cc * 32 + j;
                            if (vec && col + 3 < p.N) {
                                *reinterpret_cast<float4 *>(o + cc * 32 + j) = make_float4(v[cc][j], v[cc][j + 1], v[cc][j + 2], v[cc][j + 3]);
                            } else {
#pragma unroll
                                for (int k = 0; k < 4; ++k)
                                    if (col + k < p.N) o[cc * 32 + j + k] = v[cc][j + k];
                            }
                        }
                }
#pragma unroll
                for (int cc = 0; cc < 2; ++cc)
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int col = c0 + cc * 32 + j;
                        float d = __expf(v[cc][j] - mx) * inv_s;
                        if (col == label) d -= 1.f;
                        v[cc][j] = col < p.N ? d * inv_M : 0.f;
                    }
                if (half == 0) {
                    if (m_ok) {
                        p.row_loss[(long long)g * p.M + m] = label_ok ? (mx + __logf(s_all) - label_logit) : 0.f;
                        if (!label_ok) p.status[SLOT_BAD_LABEL] = 1;
                    }
                    __syncwarp();
                    if (p.loss) {
                        int cnt = p.M - (m0 + q * 32);
                        cnt = cnt < 0 ? 0 : (cnt > 32 ? 32 : cnt);
                        replica_loss_finish(p.row_loss, p.loss, p.rows_done, g, p.M, cnt, lane);
                    }
                }
                pair_sync();                                     // the partner has read this warp's scratch: it is free for the transposition
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    const int nb = c0 + cc * 32;
                    if (nb >= p.out_ld) break;                   // warp-uniform (out_ld = N rounded up to 8)
                    if (m_ok) {                                  // [M, out_ld]: 32 consecutive columns of the thread's row
                        __nv_bfloat16 *o = p.out + (long long)g * p.out_gs + (long long)m * p.out_ld + nb;
#pragma unroll
                        for (int j8 = 0; j8 < 32; j8 += 8) {
                            if (nb + j8 < p.out_ld) {
                                uint4 pk;
                                __nv_bfloat162 t0 = __floats2bfloat162_rn(v[cc][j8 + 0], v[cc][j8 + 1]);
                                __nv_bfloat162 t1 = __floats2bfloat162_rn(v[cc][j8 + 2], v[cc][j8 + 3]);
                                __nv_bfloat162 t2 = __floats2bfloat162_rn(v[cc][j8 + 4], v[cc][j8 + 5]);
                                __nv_bfloat162 t3 = __floats2bfloat162_rn(v[cc][j8 + 6], v[cc][j8 + 7]);
                                pk.x = *reinterpret_cast<uint32_t *>(&t0); pk.y = *reinterpret_cast<uint32_t *>(&t1);
                                pk.z = *reinterpret_cast<uint32_t *>(&t2); pk.w = *reinterpret_cast<uint32_t *>(&t3);
                                *reinterpret_cast<uint4 *>(o + j8) = pk;
                            }
                        }
                    }
                    // [N, M]: through the scratch tile, 8 consecutive batch rows of one class per store
                    __nv_bfloat16 *sT = reinterpret_cast<__nv_bfloat16 *>(mine);
#pragma unroll
                    for (int j = 0; j < 32; ++j) sT[j * UM_EPI_PITCH + lane] = __float2bfloat16_rn(v[cc][j]);
                    __syncwarp();
                    const int seg = lane & 3;
                    const int mrow = m0 + q * 32 + seg * 8;
                    if (mrow < p.M) {
                        __nv_bfloat16 *oT = p.outT + (long long)g * p.outT_gs + mrow;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int f = (lane >> 2) + 8 * i;
                            if (nb + f < p.N)
                                *reinterpret_cast<uint4 *>(oT + (long long)(nb + f) * p.outT_ld) =
                                    *reinterpret_cast<const uint4 *>(sT + f * UM_EPI_PITCH + seg * 8);
                        }
                    }
                    __syncwarp();
                }
            } else {
#pragma unroll
            for (int cc = 0; cc < CPW; ++cc) {
                const int c = CPW * half + cc;
                const int nb = n0 + c * 32;
                if (nb >= p.N) break;                        // warp-uniform
                if (EPI == UEPI_DGRAD && !MASK_AHEAD) {
                    const __nv_bfloat16 *mkp = p.mask + (long long)g * p.mask_gs + (long long)m * p.mask_ld + nb;
#pragma unroll
                    for (int j8 = 0; j8 < 4; ++j8) {
                        mk[0][j8] = make_uint4(0u, 0u, 0u, 0u);
                        if (m_ok && nb + j8 * 8 < p.N) mk[0][j8] = *reinterpret_cast<const uint4 *>(mkp + j8 * 8);
                    }
                }
                uint32_t r[32];
                tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + c * 32), r);
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
                if (EPI == UEPI_FWD_HIDDEN || EPI == UEPI_FWD_LAST) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        v[j] += __shfl_sync(0xffffffffu, bias_lane[cc], j);
                        if (EPI == UEPI_FWD_HIDDEN) v[j] = fmaxf(v[j], 0.f);
                    }
                }
                if (EPI == UEPI_DGRAD) {
#pragma unroll
                    for (int j8 = 0; j8 < 4; ++j8) {
                        const __nv_bfloat16 *h = reinterpret_cast<const __nv_bfloat16 *>(&mk[MASK_AHEAD ? cc : 0][j8]);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            if (!(__bfloat162float(h[j]) > 0.f)) v[j8 * 8 + j] = 0.f;
                    }
                }
                if (EPI == UEPI_FWD_HIDDEN || EPI == UEPI_DGRAD) {
                    // row-major bf16 [M, ld]: each thread owns 32 consecutive columns of its row
                    if (m_ok) {
                        __nv_bfloat16 *o = p.out + (long long)g * p.out_gs + (long long)m * p.out_ld + nb;
#pragma unroll
                        for (int j8 = 0; j8 < 32; j8 += 8) {
                            if (nb + j8 < p.N) {
                                uint4 pk;
                                __nv_bfloat162 t0 = __floats2bfloat162_rn(v[j8 + 0], v[j8 + 1]);
                                __nv_bfloat162 t1 = __floats2bfloat162_rn(v[j8 + 2], v[j8 + 3]);
                                __nv_bfloat162 t2 = __floats2bfloat162_rn(v[j8 + 4], v[j8 + 5]);
                                __nv_bfloat162 t3 = __floats2bfloat162_rn(v[j8 + 6], v[j8 + 7]);
                                pk.x = *reinterpret_cast<uint32_t *>(&t0); pk.y = *reinterpret_cast<uint32_t *>(&t1);
                                pk.z = *reinterpret_cast<uint32_t *>(&t2); pk.w = *reinterpret_cast<uint32_t *>(&t3);
                                *reinterpret_cast<uint4 *>(o + j8) = pk;
                            }
                        }
                    }
                    // transposed bf16 [N, ldT]: through this warp's scratch tile, so that a lane stores 8 consecutive
                    // batch rows of one feature (16 bytes) instead of 32 two-byte pieces
                    {
                        __nv_bfloat16 *sT = reinterpret_cast<__nv_bfloat16 *>(epi_scratch + (warp - 2) * UM_EPI_SCRATCH);
#pragma unroll
                        for (int j = 0; j < 32; ++j) sT[j * UM_EPI_PITCH + lane] = __float2bfloat16_rn(v[j]);
                        __syncwarp();
                        const int seg = lane & 3;                          // 8 batch rows each
                        const int mrow = m0 + q * 32 + seg * 8;
                        if (mrow < p.M) {                                  // M % 8 == 0: the whole group is inside
                            __nv_bfloat16 *oT = p.outT + (long long)g * p.outT_gs + mrow;
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int f = (lane >> 2) + 8 * i;
                                if (nb + f < p.N)
                                    *reinterpret_cast<uint4 *>(oT + (long long)(nb + f) * p.outT_ld) =
                                        *reinterpret_cast<const uint4 *>(sT + f * UM_EPI_PITCH + seg * 8);
                            }
                        }
                        __syncwarp();
                    }
                }
                if (EPI == UEPI_FWD_LAST) {
                    if (m_ok) {
                        float *o = p.outf + (long long)split * p.part_ss + (long long)g * p.outf_gs + (long long)m * p.outf_ld + nb;
                        if ((p.outf_ld & 3) == 0) {          // rows start 16-byte aligned: four columns per store
#pragma unroll
                            for (int j = 0; j < 32; j += 4) {
                                if (nb + j + 3 < p.N) {
                                    *reinterpret_cast<float4 *>(o + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                                } else {
#pragma unroll
                                    for (int k = 0; k < 4; ++k)
                                        if (nb + j + k < p.N) o[j + k] = v[j + k];
                                }
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (nb + j < p.N) o[j] = v[j];
                        }
                    }
                }
                if (EPI == UEPI_WGRAD) {
                    // accumulator row m = column of W, accumulator column = row of W: for each j the
                    // 32 lanes store 32 consecutive floats of W row nb + j
                    if (m_ok) {
                        float *o = p.outf + (long long)g * p.outf_gs + (long long)nb * p.outf_ld + m;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (nb + j < p.N) o[(long long)j * p.outf_ld] = v[j];
                    }
                }
            }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
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

}  // namespace parle
