// Forward and data-gradient products of the hidden layers (Section 1.1 / 2.1: the minibatch gradient of f) on pairs
// of SMs: one tcgen05.mma.cta_group::2 instruction multiplies a 256-row A tile, half of it in each CTA's shared
// memory, with a B tile of which each CTA holds half.
//
// These products are bound by what an SM takes in: every k-block of weights (read from HBM exactly once) needs the
// matching k-block of the replica's activations (from L2) next to it.  The weights are therefore made the A operand
// (M = output features, 128 rows per CTA, each CTA its own rows) and the activations the B operand (N = batch),
// so that the two CTAs of a pair share one activation tile and each fetches only half of it:
//     forward      H_l^T      [d_out, B] = W_l [d_out, d_in]   x H_{l-1} [B, d_in]^T     A K-major,  B K-major
//     data grad    dH_{l-1}^T [d_in,  B] = W_l^T [d_in, d_out] x dH_l [B, d_out]^T        A MN-major, B K-major
// Per k-block a CTA takes in 16 KiB of weights and 8 KiB (batch tile 128) or 16 KiB (batch tile 256) of
// activations, against 16 + 16 or 32 + 16 KiB per 128 x 128 or 128 x 256 tile of the one-SM kernel.
//
// The accumulator is the transposed output: tensor-memory lane = output feature, column = batch row.  The epilogue
// (bias + ReLU, or the ReLU mask of the data gradient) stores both layouts the other kernels read, [d, B] and
// [B, d], each through a per-warp shared-memory tile so that every store instruction fills whole 32-byte sectors.
//
// Synchronisation inside a pair (cluster of two CTAs, rank 0 = leader):
//   * both CTAs load their own halves with TMA (plain loads, no multicast) and signal the LEADER's "full" barrier,
//     on which the leader's producer has announced the bytes of both;
//   * the leader's MMA warp issues the instructions for the pair and commits to the "empty" barrier of both CTAs
//     (tcgen05.commit with a CTA mask), likewise to both CTAs' "accumulator full" barriers;
//   * the epilogue warps of both CTAs arrive on the leader's "accumulator empty" barrier.
// Tensor memory is allocated and freed by warp 1 of both CTAs (cta_group::2).  Every wait is bounded; the two CTAs
// meet at a cluster barrier before tensor memory is released.
//
// Several layers in one launch.  At batch 128 a layer is one tile per pair, so a launch per layer pays its start-up
// (barriers, tensor memory, the first weights' latency) and its epilogue with nothing to overlap them with.  A launch
// therefore takes a chain of products, each reading what the one before it wrote (forward: hidden layers 1, 2, ...;
// backward: the data gradients from the top down).  The tiles of all links form one list, link by link; a pair
// walks its share of the list in order.  Only the activation operand of a tile depends on the link before it (all
// tiles of that link for the same replica), the weights do not: the producer fetches the weights of the first
// k-blocks, then waits until the replica's counter of the previous link has reached its full count, then fetches the
// activations.  So the weight stream of the next layer runs under the epilogue of this one.  The counters live in the
// caller's workspace (an epilogue warp adds 1 per tile after a device-wide fence), are polled with acquire loads and
// a bounded wait, and are zeroed again by the last CTA to leave.

#pragma once

#include "umma_gemm.cuh"

namespace parle {

constexpr int UP_BM = 128;                                  // output features per CTA (256 per pair)
constexpr int UP_A_BYTES = UP_BM * UM_BK * 2;               // 16 KiB of weights per k-block
constexpr int UP_RING_BYTES = 192 * 1024;
constexpr int UP_THREADS = 320;                             // warp 0 producer, 1 MMA, 2..9 epilogue
constexpr int UP_MAX_LINKS = PARLE_MAX_LAYERS;
constexpr int UP_SYNC_INTS = UP_MAX_LINKS * PARLE_MAX_REPLICAS + 1;   // per-(link, replica) counters + the exit counter

template <int BNB> struct UpShape {
    static_assert(BNB == 128 || BNB == 256, "batch tile");
    // 64-wide k-blocks that travel through the ring as one stage.  With the batch tile of 128 the MMAs of a k-block
    // take the issuing thread 130 ns and the commit that frees the stage another 70 ns: two k-blocks share a commit.
    static constexpr int KPS = BNB == 128 ? 2 : 1;
    static constexpr int B_BYTES = (BNB / 2) * UM_BK * 2;   // this CTA's half of the activation k-block
    static constexpr int STAGE_BYTES = KPS * (UP_A_BYTES + B_BYTES);   // [W k-block 0 .. | X k-block 0 ..]
    static constexpr int STAGES = UP_RING_BYTES / STAGE_BYTES;
    static constexpr uint32_t TMEM_COLS = 2 * BNB;          // two accumulators
    static constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 8 * UM_EPI_SCRATCH + 1024 /*alignment*/ + 256 /*barriers*/;
};

enum UmmaPairEpilogue {
    UPE_FWD_HIDDEN = 0,    // + bias[f], ReLU
    UPE_DGRAD = 1          // * (H_{l-1}[b, f] > 0)
};

// One product of a chain: out^T [F, Bt] = W-operand [F, K] x X [Bt, K]^T.
struct UpLink {
    int F, K;                         // output features (rows of the weight operand), reduction length
    int tiles_f;                      // 256-feature tiles per replica
    int tile_begin;                   // index of the link's first tile in the launch's list
    const float *bias; long long bias_gs;
    __nv_bfloat16 *out; long long out_gs; int out_ld;          // [Bt, out_ld]
    __nv_bfloat16 *outT; long long outT_gs; int outT_ld;       // [F, outT_ld]
    const __nv_bfloat16 *maskT; long long maskT_gs; int maskT_ld;   // data gradient: H_{l-1}^T [F, maskT_ld]
};
struct UmmaPairParams {
    int Bt, groups, tiles_b;          // batch rows, replicas, BNB-row tiles per replica
    int n_links, total_tiles;
    UpLink link[UP_MAX_LINKS];        // link k > 0 reads, as its X operand, the `out` of link k - 1
    int *sync;                        // sync[k * groups + g]: epilogue warps that have stored their part of a tile of (link k,
                                      // replica g); sync[UP_MAX_LINKS * PARLE_MAX_REPLICAS]: CTAs that have left.  All zero between launches
    int *status;
};
struct UpMaps { CUtensorMap w[UP_MAX_LINKS], x[UP_MAX_LINKS]; };

// ---------------------------------------------------------------- PTX wrappers (pair forms)
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory location in the CTA of rank `rank` of this cluster.
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Barrier over all threads of both CTAs (the forms that do not ask for converged warps: after the role branches the
// lanes of a warp may arrive one by one).
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
// TMA loads of a CTA of a pair: the destination is this CTA's shared memory, the barrier may be the peer's.
__device__ __forceinline__ void tma_pair_load_3d(uint32_t dst, const CUtensorMap *tm, uint32_t bar_cluster,
                                                 int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tma_pair_load_5d(uint32_t dst, const CUtensorMap *tm, uint32_t bar_cluster,
                                                 int c0, int c1, int c2, int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}
__device__ __forceinline__ void tc_pair_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                                 uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrive, once the pair's MMAs issued so far have retired, on the barrier at this shared-memory offset in every CTA of `mask`.
__device__ __forceinline__ void tc_pair_commit(uint32_t bar, uint16_t mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
// Instruction descriptor of the pair: bf16 x bf16 -> fp32, M = 256 (128 rows per CTA), N = bn.
__host__ __device__ constexpr uint32_t make_pair_idesc(bool a_mn_major, int bn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) |
           ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}
__device__ __forceinline__ int ld_acquire_gpu(const int *p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Bounded wait until *counter >= need (another CTA's epilogue warps count up).  Returns false on a time-out or when
// another role of this CTA gave up.
__device__ __forceinline__ bool wait_counter(const int *counter, int need, volatile int *abort_flag) {
    if (ld_acquire_gpu(counter) >= need) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t it = 0;; ++it) {
        if (ld_acquire_gpu(counter) >= need) return true;
        __nanosleep(64);
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > UM_WAIT_LIMIT_NS) { *abort_flag = 1; return false; }
        }
    }
}

template <int EPI, int BNB>
__global__ void __launch_bounds__(UP_THREADS, 1)
umma_pair_gemm_kernel(const __grid_constant__ UpMaps maps, const __grid_constant__ UmmaPairParams p) {
    using SH = UpShape<BNB>;
    constexpr int STAGES = SH::STAGES, STAGE_BYTES = SH::STAGE_BYTES, B_BYTES = SH::B_BYTES, KPS = SH::KPS;
    constexpr bool A_MN = (EPI == UPE_DGRAD);
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;                          // 1024-byte aligned (swizzle atom)
    uint8_t *epi_scratch = smem_raw + (ring - raw) + (size_t)STAGES * STAGE_BYTES;
    uint8_t *ctl = epi_scratch + 8 * UM_EPI_SCRATCH;
    uint64_t *bars = reinterpret_cast<uint64_t *>(ctl);                    // full[S], empty[S], tfull[2], tempty[2]
    constexpr int NBARS = 2 * STAGES + 4;
    static_assert(8 * NBARS + 16 <= 256, "control block");
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(ctl + 8 * NBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * STAGES, bar_tempty = bar_tfull + 16;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                               // 0 = leader of the pair
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int total_tiles = p.total_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        // an accumulator is handed back by the 8 epilogue warps of both CTAs (the barrier that counts is the leader's)
        for (int s = 0; s < 2; ++s) { mbar_init(bar_tfull + 8 * s, 1); mbar_init(bar_tempty + 8 * s, 16); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(SH::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync_all();                                                    // the peer's barriers exist from here on
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // tile t -> link k, replica g, first feature f0 of the pair, first batch row b0
    auto tile_coords = [&](int t, int &k, int &g, int &f0, int &b0) {
        k = 0;
        while (k + 1 < p.n_links && t >= p.link[k + 1].tile_begin) ++k;
        const int per_g = p.link[k].tiles_f * p.tiles_b;
        t -= p.link[k].tile_begin;
        g = t / per_g;
        const int r = t - g * per_g;
        b0 = (r % p.tiles_b) * BNB;
        f0 = (r / p.tiles_b) * (2 * UP_BM);
    };

    if (warp == 0) {
        // ------------------------------------------------ TMA producer: this CTA's rows of W and its half of the batch tile
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            // stage `st` takes the k-blocks s * KPS .. s * KPS + nb - 1 of a tile
            auto load_w = [&](int k, int s, int nb, int st, int fr, int g) {
                const uint32_t fb = mapa_shared(bar_full + 8 * st, 0);     // both CTAs' copies complete on the leader's barrier
                for (int j = 0; j < nb; ++j) {
                    const int kb = s * KPS + j;
                    const uint32_t sa = ring + st * STAGE_BYTES + j * UP_A_BYTES;
                    if (!A_MN) {
                        // K-major weights: block (row block fr/128, column block kb) of the blocked copy
                        tma_pair_load_5d(sa, &maps.w[k], fb, 0, 0, kb, fr / 128, g);
                    } else {
                        // MN-major weights: k-rows kb*64 .. +63 = half of row block kb/2; features fr .. fr+127 = two column blocks
#pragma unroll
                        for (int h = 0; h < 2; ++h)
                            tma_pair_load_5d(sa + h * (UP_A_BYTES / 2), &maps.w[k], fb, 0, (kb & 1) * 64, fr / 64 + h, kb >> 1, g);
                    }
                }
            };
            auto load_x = [&](int k, int s, int nb, int st, int br, int g) {
                const uint32_t fb = mapa_shared(bar_full + 8 * st, 0);
                for (int j = 0; j < nb; ++j)
                    tma_pair_load_3d(ring + st * STAGE_BYTES + KPS * UP_A_BYTES + j * B_BYTES, &maps.x[k], fb, (s * KPS + j) * UM_BK, br, g);
            };
            auto blocks_in = [&](int s, int num_kb) { return num_kb - s * KPS < KPS ? num_kb - s * KPS : KPS; };
            for (int t = pair; t < total_tiles && ok; t += num_pairs) {
                int k, g, f0, b0; tile_coords(t, k, g, f0, b0);
                const int num_kb = (p.link[k].K + UM_BK - 1) / UM_BK;
                const int num_s = (num_kb + KPS - 1) / KPS;                // stages of this tile
                const int fr = f0 + (int)rank * UP_BM;                     // first feature of this CTA
                const int br = b0 + (int)rank * (BNB / 2);                 // first batch row of this CTA's half
                int s = 0;
                if (k > 0) {
                    // The activations of this tile are what link k - 1 wrote for this replica; its weights depend on
                    // nothing.  Weights of the first stages first, then the wait, then their activations.
                    const int ahead = num_s < STAGES ? num_s : STAGES;
                    int st = stage; uint32_t ph = phase;
                    for (int i = 0; i < ahead; ++i) {
                        if (!mbar_wait(bar_empty + 8 * st, ph ^ 1u, abort_flag)) { ok = false; break; }
                        const int nb = blocks_in(i, num_kb);
                        if (rank == 0) mbar_expect_tx(bar_full + 8 * st, 2 * nb * (UP_A_BYTES + B_BYTES));
                        load_w(k, i, nb, st, fr, g);
                        if (++st == STAGES) { st = 0; ph ^= 1u; }
                    }
                    if (!ok) break;
                    const int need = p.link[k - 1].tiles_f * p.tiles_b * 16;   // 8 epilogue warps of 2 CTAs per tile
                    if (!wait_counter(p.sync + (k - 1) * p.groups + g, need, abort_flag)) { ok = false; break; }
                    asm volatile("fence.proxy.async;" ::: "memory");       // the TMA reads below come after the acquire above
                    for (int i = 0; i < ahead; ++i) {
                        load_x(k, i, blocks_in(i, num_kb), stage, br, g);
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    }
                    s = ahead;
                }
                for (; s < num_s; ++s) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const int nb = blocks_in(s, num_kb);
                    if (rank == 0) mbar_expect_tx(bar_full + 8 * stage, 2 * nb * (UP_A_BYTES + B_BYTES));
                    load_w(k, s, nb, stage, fr, g);
                    load_x(k, s, nb, stage, br, g);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // gave up (after a wait of seconds): copies issued just before may still be on their way into this
                // CTA's shared memory; they take microseconds, the CTA stays for two milliseconds
                const unsigned long long t0 = global_ns();
                while (global_ns() - t0 < 2000000ull) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (leader only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = make_pair_idesc(A_MN, BNB);
            int stage = 0; uint32_t phase = 0; int acc = 0; uint32_t acc_phase = 0; bool ok = true;
            for (int t = pair; t < total_tiles && ok; t += num_pairs) {
                int k, g, f0, b0; tile_coords(t, k, g, f0, b0);
                const int num_kb = (p.link[k].K + UM_BK - 1) / UM_BK;
                if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BNB;
                for (int kb0 = 0; kb0 < num_kb; kb0 += KPS) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int j = 0; j < KPS; ++j) {
                        if (kb0 + j >= num_kb) break;
                        const uint32_t sa = ring + stage * STAGE_BYTES + j * UP_A_BYTES;
                        const uint32_t sb = ring + stage * STAGE_BYTES + KPS * UP_A_BYTES + j * B_BYTES;
                        const uint64_t adesc = A_MN ? make_smem_desc(sa, UP_A_BYTES / 2, 1024) : make_smem_desc(sa, 16, 1024);
                        const uint64_t bdesc = make_smem_desc(sb, 16, 1024);
#pragma unroll
                        for (int kk = 0; kk < UM_BK / 16; ++kk) {
                            // K-major: 16 bf16 = 32 B further along the row; MN-major: two 8-row groups = 2048 B
                            const uint64_t a_k = adesc + (uint64_t)(A_MN ? kk * 128 : kk * 2);
                            const uint64_t b_k = bdesc + (uint64_t)(kk * 2);
                            tc_pair_mma_bf16(d_tmem, a_k, b_k, idesc, (kb0 | j | kk) != 0 ? 1u : 0u);
                        }
                    }
                    tc_pair_commit(bar_empty + 8 * stage, 3);              // the stage is free in both CTAs once these retire
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_pair_commit(bar_tfull + 8 * acc, 3);                    // accumulator complete, in both CTAs
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------ epilogue (warps 2..9 of both CTAs)
        const int q = warp & 3;                              // tensor-memory lane quarter this warp may read
        const int half = (warp - 2) >> 2;                    // chunks CPW*half .. of every tile
        constexpr int CPW = BNB / 64;                        // 32-column chunks per warp
        constexpr bool MASK_AHEAD = (BNB == 128);
        int acc = 0; uint32_t acc_phase = 0;
        const uint32_t tempty_leader = mapa_shared(bar_tempty, 0);
        for (int t = pair; t < total_tiles; t += num_pairs) {
            int k, g, f0, b0; tile_coords(t, k, g, f0, b0);
            const UpLink &L = p.link[k];
            const int fw = f0 + (int)rank * UP_BM + q * 32;  // first feature of this warp
            const int f = fw + lane;                         // feature of this thread (= its tensor-memory lane)
            const bool f_ok = f < L.F;
            float bias_v = 0.f;
            uint4 mk[MASK_AHEAD ? CPW : 1][4];
            if (EPI == UPE_FWD_HIDDEN && f_ok) bias_v = __ldg(L.bias + (long long)g * L.bias_gs + f);
            if (EPI == UPE_DGRAD && MASK_AHEAD) {
#pragma unroll
                for (int cc = 0; cc < CPW; ++cc) {
                    const int bb = b0 + (CPW * half + cc) * 32;
                    const __nv_bfloat16 *mkp = L.maskT + (long long)g * L.maskT_gs + (long long)f * L.maskT_ld + bb;
#pragma unroll
                    for (int j8 = 0; j8 < 4; ++j8) {
                        mk[cc][j8] = make_uint4(0u, 0u, 0u, 0u);
                        if (f_ok && bb + j8 * 8 < p.Bt) mk[cc][j8] = *reinterpret_cast<const uint4 *>(mkp + j8 * 8);
                    }
                }
            }
            const bool ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag));
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int cc = 0; cc < CPW; ++cc) {
                const int c = CPW * half + cc;
                const int bb = b0 + c * 32;                  // first batch row of the chunk
                if (bb >= p.Bt) break;                       // warp-uniform
                if (EPI == UPE_DGRAD && !MASK_AHEAD) {
                    const __nv_bfloat16 *mkp = L.maskT + (long long)g * L.maskT_gs + (long long)f * L.maskT_ld + bb;
#pragma unroll
                    for (int j8 = 0; j8 < 4; ++j8) {
                        mk[0][j8] = make_uint4(0u, 0u, 0u, 0u);
                        if (f_ok && bb + j8 * 8 < p.Bt) mk[0][j8] = *reinterpret_cast<const uint4 *>(mkp + j8 * 8);
                    }
                }
                uint32_t r[32];
                tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BNB + c * 32), r);
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
                if (EPI == UPE_FWD_HIDDEN) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j] + bias_v, 0.f);
                }
                if (EPI == UPE_DGRAD) {
#pragma unroll
                    for (int j8 = 0; j8 < 4; ++j8) {
                        const __nv_bfloat16 *h = reinterpret_cast<const __nv_bfloat16 *>(&mk[MASK_AHEAD ? cc : 0][j8]);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            if (!(__bfloat162float(h[j]) > 0.f)) v[j8 * 8 + j] = 0.f;
                    }
                }
                // [F, ldT]: the thread owns 32 consecutive batch entries of its feature
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    __nv_bfloat162 t2 = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
                    pk[j] = *reinterpret_cast<uint32_t *>(&t2);
                }
                __nv_bfloat16 *sT = reinterpret_cast<__nv_bfloat16 *>(epi_scratch + (warp - 2) * UM_EPI_SCRATCH);
                {
                    // through this warp's scratch tile (row = feature), so that four lanes store the 64 bytes a feature
                    // has in this chunk and an instruction covers eight features: stored straight from the registers,
                    // every lane would touch a line of its own four times over
#pragma unroll
                    for (int j8 = 0; j8 < 4; ++j8)
                        *reinterpret_cast<uint4 *>(sT + lane * UM_EPI_PITCH + j8 * 8) = make_uint4(pk[4 * j8], pk[4 * j8 + 1], pk[4 * j8 + 2], pk[4 * j8 + 3]);
                    __syncwarp();
                    const int seg = lane & 3;                              // 8 batch entries each
                    if (bb + seg * 8 < p.Bt) {                             // Bt % 8 == 0: the whole group is inside
                        __nv_bfloat16 *oT = L.outT + (long long)g * L.outT_gs + bb + seg * 8;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int fj = (lane >> 2) + 8 * i;
                            if (fw + fj < L.F)
                                *reinterpret_cast<uint4 *>(oT + (long long)(fw + fj) * L.outT_ld) =
                                    *reinterpret_cast<const uint4 *>(sT + fj * UM_EPI_PITCH + seg * 8);
                        }
                    }
                    __syncwarp();
                }
                // [Bt, ld]: the same way with row = batch entry, column = feature, so that a lane stores 8 consecutive
                // features of one batch row (16 bytes)
                {
#pragma unroll
                    for (int j = 0; j < 32; ++j) sT[j * UM_EPI_PITCH + lane] = __float2bfloat16_rn(v[j]);
                    __syncwarp();
                    const int seg = lane & 3;                              // 8 features each
                    const int fs = fw + seg * 8;
                    if (fs < L.F) {                                        // F % 8 == 0: the whole group is inside
                        __nv_bfloat16 *o = L.out + (long long)g * L.out_gs + fs;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int bj = (lane >> 2) + 8 * i;
                            if (bb + bj < p.Bt)
                                *reinterpret_cast<uint4 *>(o + (long long)(bb + bj) * L.out_ld) =
                                    *reinterpret_cast<const uint4 *>(sT + bj * UM_EPI_PITCH + seg * 8);
                        }
                    }
                    __syncwarp();
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive_cluster(tempty_leader + 8 * acc);
                if (k + 1 < p.n_links) {                     // the next link reads what this warp has just stored
                    __threadfence();
                    atomicAdd(p.sync + k * p.groups + g, 1);
                }
            }
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    }

    tc_fence_before();
    cluster_sync_all();                                      // nobody touches the peer's shared or tensor memory after this
    if (threadIdx.x == 0 && *abort_flag) p.status[SLOT_WAIT_LIMIT] = 1;
    if (threadIdx.x == 0 && p.n_links > 1) {
        // every wait of this CTA on the counters is over; the last CTA to leave zeroes them for the next launch
        int *leave = p.sync + UP_MAX_LINKS * PARLE_MAX_REPLICAS;
        __threadfence();
        if (atomicAdd(leave, 1) == (int)gridDim.x - 1) {
            __threadfence();
            for (int i = 0; i < (p.n_links - 1) * p.groups; ++i) p.sync[i] = 0;
            *leave = 0;
        }
    }
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"(SH::TMEM_COLS) : "memory");
    }
}

}  // namespace parle
