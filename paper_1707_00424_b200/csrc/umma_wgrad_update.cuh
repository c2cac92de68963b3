// Weight-gradient GEMM with the inner update fused into its epilogue
// (Section 2.1 gradient; Eq. parle_y, parle_z applied in place):
//     G^T  = H_{l-1}^T dH_l                (tcgen05.mma, bf16 operands, fp32 accumulators in tensor memory)
//     y   <- y - eta' (G + (y - x)/gamma)
//     z   <- alpha z + (1 - alpha) y,     operand copy <- bf16(y)
// for the W_l segment of every replica.  The gradient never reaches memory.
//
// The accumulator is the *transposed* gradient: its 128 rows (tensor-memory
// lanes) run along d_in, the contiguous direction of W in memory, so a warp's
// 32 lanes always touch 32 consecutive elements of one W row.
//
// This is a streaming kernel with a small GEMM inside (K = batch): 22 bytes per
// weight go through the epilogue.  To keep enough bytes in flight, x, y and z
// tiles are not loaded through registers: a loader warp brings 32-row x 128-col
// fp32 boxes of x, y, z into a ring of shared-memory stages with TMA, running
// several stages ahead of the epilogue warps, which read them conflict-free
// (consecutive lanes -> consecutive words), combine them with the accumulator
// chunk from tensor memory and store y, z and the bf16 copy straight from
// registers (coalesced 128-byte / 64-byte warp stores).
//
// Roles: warp 0 operand TMA producer, warp 1 MMA issuer, warp 2 state loader,
// warps 3.. epilogue: G groups of 4 warps (the four 32-lane quarters of tensor
// memory).  Every epilogue warp consumes every chunk, in order -- group g takes
// its own slice of the chunk's rows -- so each stage barrier sees all its
// consumers in every phase and no waiter can fall a phase behind.
//
// Tiles are handed out dynamically.  SMs do not get equal shares of a saturated
// memory system (with a fixed tile list per CTA the first CTA of a 2048 x 2048
// layer finished after 85 us and the last after 120 us), so after its first tile
// (blockIdx.x) a CTA claims the next one from a global counter.  The operand
// producer is the scheduler: it publishes every claimed tile index (or -1: no
// tiles left) through a small shared-memory ring with full/empty barriers, and
// the other roles read it from there.  The last CTA to leave resets the counter
// pair, so consecutive launches on one stream can share it.  Which CTA runs a
// tile does not change what is computed for it: results stay bit-identical.
//
// Eq. (parle_z) two steps at a time (ZMODE).  z is only needed by the outer step, and
//     z_{k+2} = alpha z_{k+1} + (1-alpha) y_{k+2} = alpha^2 z_k + (1-alpha) (alpha y_{k+1} + y_{k+2})
// needs, besides z_k, exactly the two y values the kernel of step k+2 holds anyway (the y it reads and the y it
// writes).  So inside a whole round z is read and written every other step only: ZMODE 1 leaves z alone (14 bytes
// per weight instead of 22), ZMODE 2 applies the two-step form, ZMODE 0 the one-step form (single steps, and the last
// step of a round with an even number of steps).  Same recurrence, different fp32 rounding of z (1e-7 relative).
//
// y in two 16-bit planes (YSPLIT).  Inside a whole round nobody but this kernel reads the fp32 y of the weights, and the
// kernel writes a bf16 copy of y for the GEMMs anyway.  That copy is the upper half of (fp32 word + 0x8000): y rounded to
// nearest, ties away from zero.  The lower half of the same sum goes to a second plane (workspace), and
// word = ((upper << 16) | lower) - 0x8000 gives the fp32 y back exactly.  So y is read and written as 2 + 2 bytes and the
// separate 2-byte operand copy comes for free: 12 / 20 bytes per weight and step instead of 14 / 22.  The last step of a
// round also writes the fp32 y, so y is current again when the round returns.
// All waits are bounded.
#pragma once

#include "umma_gemm.cuh"

namespace parle {

constexpr int WU_OP_STAGES = 2;                                // operand ring (K = batch is short)
constexpr int WU_STATE_RING_BYTES = 144 * 1024;                // shared memory given to the x/y/z stages
constexpr int WU_TILE_SLOTS = 4;                               // depth of the tile-index ring
constexpr int WU_CTL_BYTES = 512;                              // barriers, tile ring, tensor-memory slot, abort flag

// Shape of the epilogue: G groups of 4 warps share chunks of CR W-rows (accumulator columns);
// every thread owns CR / G rows of one column.
template <int G, int CR, int NA = 3>
struct WuShape {
    static constexpr int GROUPS = G, CHUNK_ROWS = CR, RPG = CR / G;
    static constexpr int CHUNKS = UM_BN / CR;
    static constexpr int ARRAY_BYTES = CR * UM_BM * 4;          // one fp32 box of x, y, z (or the momentum v)
    static constexpr int MAX_ARRAYS = NA;                       // x | y | z [| v]
    // A stage holds only the arrays its kind of step loads (x alone on the first step of a round, no z on the steps
    // that leave z untouched), so those steps get more, smaller stages out of the same ring: the bytes in flight per
    // SM stay the same, which is what keeps a step with few bytes per weight from becoming latency-bound.
    __host__ __device__ static constexpr int stages(int arrays) { return WU_STATE_RING_BYTES / (arrays * ARRAY_BYTES); }
    static constexpr int MAX_STAGES = stages(1);
    static constexpr int THREADS = 96 + 128 * G;
    static constexpr size_t SMEM_BYTES = (size_t)WU_OP_STAGES * UM_STAGE_BYTES + (size_t)WU_STATE_RING_BYTES +
                                         1024 /*alignment slack*/ + WU_CTL_BYTES;
    static_assert(RPG == 4 || RPG == 8 || RPG == 16, "rows per thread must match a tcgen05.ld shape");
    static_assert(stages(NA) >= 2 && 8 * (2 * WU_OP_STAGES + 4 + 2 * MAX_STAGES + 2 * WU_TILE_SLOTS) + 8 + 4 * WU_TILE_SLOTS <= WU_CTL_BYTES,
                  "stage count");
};
using WuDefault = WuShape<2, 32>;
using WuMomentum = WuShape<4, 16, 4>;                          // with the momentum buffer staged too: 16-row chunks
constexpr int WU_CHUNK_ROWS = WuDefault::CHUNK_ROWS;           // TMA box height of the x/y/z tensor maps
constexpr int WU_CHUNK_ROWS_MOM = WuMomentum::CHUNK_ROWS;      // ... of the maps used by the momentum variant

template <int N> __device__ __forceinline__ void tc_ld_cols(uint32_t taddr, uint32_t (&r)[N]);
template <> __device__ __forceinline__ void tc_ld_cols<4>(uint32_t taddr, uint32_t (&r)[4]) { tc_ld_32x4(taddr, r); }
template <> __device__ __forceinline__ void tc_ld_cols<8>(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n\t"
                 "tcgen05.wait::ld.sync.aligned;"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
}
template <> __device__ __forceinline__ void tc_ld_cols<16>(uint32_t taddr, uint32_t (&r)[16]) { tc_ld_32x16(taddr, r); }

// One launch covers the W segments of all layers: its tile list is layer 0's tiles (replica-major, then
// n-tile, then m-tile), then layer 1's, ...
struct WuLayer {
    int M, N;                    // M = d_in (tile rows), N = d_out (tile columns)
    int tiles_m, tiles_n;
    int tile_begin;              // index of the layer's first tile in the launch's list
    int ld;                      // row pitch of W_l (= d_in)
    int shadow_cb;               // column blocks per row block of the blocked bf16 copy
    long long w_off;             // W_l inside a replica's parameter vector (elements)
    long long shadow_off;        // blocked copy of W_l inside a replica's copy (elements)
};
struct WgradUpdateParams {
    int K;                       // batch
    int groups, n_layers, total_tiles;
    WuLayer layer[PARLE_MAX_LAYERS];
    float *y, *z;                // replica 0; element (replica g, layer l, W row r, W col c) at g*gs + w_off + r*ld + c
    __nv_bfloat16 *shadow;       // blocked bf16 copy of replica 0 (128 x 64 blocks, row-block major)
    long long shadow_gs;         // replica pitch of the copy (elements)
    long long gs;
    float eta_p, inv_gamma, alpha, wd;
    uint16_t *ylo;               // YSPLIT: low halves of the fp32 words of y (same addressing as y); the high halves are `shadow`
    float *v; float mu;          // Nesterov momentum buffer of y (same addressing as y), used by the MOM variant
    int *sched;                  // sched[0]: tiles claimed beyond the first of every CTA, sched[1]: CTAs that have left; both 0 between launches
    int *status;
};
// Tensor maps of every layer: A = H_{l-1}^T, B = dH_l^T (bf16 operands), and the W_l segments of x, y, z (and the
// momentum buffer) as fp32 boxes.
struct WuMaps {
    CUtensorMap a[PARLE_MAX_LAYERS], b[PARLE_MAX_LAYERS];
    CUtensorMap x[PARLE_MAX_LAYERS], y[PARLE_MAX_LAYERS], z[PARLE_MAX_LAYERS], v[PARLE_MAX_LAYERS];
    // YSPLIT: y as its two 16-bit planes -- boxes of 64 columns x chunk rows of the blocked bf16 copy (no swizzle),
    // and boxes of 128 columns x chunk rows of the lo plane
    CUtensorMap yhi[PARLE_MAX_LAYERS], ylo[PARLE_MAX_LAYERS];
};

// MOM: Nesterov momentum on the y step (see inner_update_kernel): v <- mu v + d, y <- y - eta' (d + mu v),
// v = 0 at the start of a round (FIRST: v is only written).
// ZMODE (ignored when FIRST): 0 = z <- alpha z + (1-alpha) y_new; 1 = z untouched; 2 = z <- alpha^2 z + (1-alpha)(alpha y_old + y_new).
constexpr int WU_Z_SINGLE = 0, WU_Z_SKIP = 1, WU_Z_DOUBLE = 2;
// YSPLIT: y is read and written as two 16-bit planes (see the head of this file); YWRITE: such a step also stores the
// fp32 y (the last step of a round).
template <int LD> struct WuPitch { static constexpr int value = LD; };
template <bool FIRST, class SH, bool MOM = false, int ZMODE = WU_Z_SINGLE, bool YSPLIT = false, bool YWRITE = false>
__global__ void __launch_bounds__(SH::THREADS, 1)
umma_wgrad_update_kernel(const __grid_constant__ WuMaps maps, const __grid_constant__ WgradUpdateParams p) {
    constexpr int WU_GROUPS = SH::GROUPS, WU_CHUNKS = SH::CHUNKS, WU_ARRAY_BYTES = SH::ARRAY_BYTES;
    constexpr bool LOADS_Z = !FIRST && ZMODE != WU_Z_SKIP;
    constexpr int WU_ARRAYS = FIRST ? 1 : 2 + (LOADS_Z ? 1 : 0) + (MOM ? 1 : 0);           // arrays a stage of this step holds
    constexpr int WU_Z_SLOT = 2, WU_V_SLOT = LOADS_Z ? 3 : 2;                               // x = 0, y = 1
    constexpr int WU_STATE_BYTES = WU_ARRAYS * WU_ARRAY_BYTES, WU_STATE_STAGES = SH::stages(WU_ARRAYS), RPG = SH::RPG;
    static_assert(WU_ARRAYS <= SH::MAX_ARRAYS, "stage layout");
    constexpr int WU_CHUNK_ROWS = SH::CHUNK_ROWS;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t op_base = (raw + 1023u) & ~1023u;
    const uint32_t st_base = op_base + WU_OP_STAGES * UM_STAGE_BYTES;
    uint8_t *st_ptr = smem_raw + (st_base - raw);
    uint8_t *ctl = st_ptr + (size_t)WU_STATE_RING_BYTES;
    // barriers: op_full[2], op_empty[2], tfull[2], tempty[2], st_full[S], st_empty[S], tile_full[T], tile_empty[T]
    uint64_t *bars = reinterpret_cast<uint64_t *>(ctl);
    constexpr int NBARS = 2 * WU_OP_STAGES + 4 + 2 * WU_STATE_STAGES + 2 * WU_TILE_SLOTS;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(ctl + 8 * NBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    volatile int *tile_ids = reinterpret_cast<volatile int *>(tmem_slot + 2);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * WU_OP_STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * WU_OP_STAGES, bar_tempty = bar_tfull + 16;
    const uint32_t bar_sfull = bar_tempty + 16, bar_sempty = bar_sfull + 8 * WU_STATE_STAGES;
    const uint32_t bar_qfull = bar_sempty + 8 * WU_STATE_STAGES, bar_qempty = bar_qfull + 8 * WU_TILE_SLOTS;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = p.total_tiles;
    const int num_kb = (p.K + UM_BK - 1) / UM_BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < WU_OP_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar_tfull + 8 * s, 1); mbar_init(bar_tempty + 8 * s, 4 * WU_GROUPS); }
        for (int s = 0; s < WU_STATE_STAGES; ++s) { mbar_init(bar_sfull + 8 * s, 1); mbar_init(bar_sempty + 8 * s, 4 * WU_GROUPS); }
        // a tile index is read by the MMA issuer, the state loader and every epilogue warp
        for (int s = 0; s < WU_TILE_SLOTS; ++s) { mbar_init(bar_qfull + 8 * s, 1); mbar_init(bar_qempty + 8 * s, 2 + 4 * WU_GROUPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)UM_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    auto coords = [&](int t, int &l, int &g, int &m0, int &n0) {
        l = 0;
        while (l + 1 < p.n_layers && t >= p.layer[l + 1].tile_begin) ++l;
        const WuLayer &ly = p.layer[l];
        const int per_g = ly.tiles_m * ly.tiles_n;
        t -= ly.tile_begin;
        g = t / per_g;
        const int r = t - g * per_g;
        m0 = (r % ly.tiles_m) * UM_BM;
        n0 = (r / ly.tiles_m) * UM_BN;
    };
    // Consumer side of the tile ring (one lane per role calls it): the next tile of this CTA, -1 when there is
    // none, -2 when a wait gave up.
    auto take_tile = [&](int &slot, uint32_t &ph) -> int {
        if (!mbar_wait(bar_qfull + 8 * slot, ph, abort_flag)) return -2;
        const int t = tile_ids[slot];
        if (t >= -1) mbar_arrive(bar_qempty + 8 * slot);      // always true: the arrive waits for the index to have been read
        if (++slot == WU_TILE_SLOTS) { slot = 0; ph ^= 1u; }
        return t;
    };

    if (warp == 0) {
        // ------------------------------------------------ tile scheduler + operand producer (A = H^T tile, B = dH^T tile)
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            int qslot = 0; uint32_t qphase = 0;
            int t = blockIdx.x;                                               // the first tile needs no claim
            int t_next = (int)gridDim.x + atomicAdd(p.sched, 1);              // claimed one tile ahead: its latency is hidden
            while (ok) {
                if (!mbar_wait(bar_qempty + 8 * qslot, qphase ^ 1u, abort_flag)) { ok = false; break; }
                tile_ids[qslot] = t < total_tiles ? t : -1;
                mbar_arrive(bar_qfull + 8 * qslot);                           // release: the index is visible to the waiters
                if (++qslot == WU_TILE_SLOTS) { qslot = 0; qphase ^= 1u; }
                if (t >= total_tiles) break;
                int l, g, m0, n0; coords(t, l, g, m0, n0);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t sa = op_base + stage * UM_STAGE_BYTES, sb = sa + UM_A_BYTES;
                    const uint32_t fb = bar_full + 8 * stage;
                    mbar_expect_tx(fb, UM_STAGE_BYTES);
                    tma_load_3d(sa, &maps.a[l], fb, kb * UM_BK, m0, g);
                    tma_load_3d(sb, &maps.b[l], fb, kb * UM_BK, n0, g);
                    if (++stage == WU_OP_STAGES) { stage = 0; phase ^= 1u; }
                }
                t = t_next;
                if (t < total_tiles) t_next = (int)gridDim.x + atomicAdd(p.sched, 1);
            }
            if (!ok) {
                for (int s = 0; s < WU_OP_STAGES; ++s) {
                    const uint32_t armed_parity = (s < stage) ? phase : (phase ^ 1u);
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_full + 8 * s, armed_parity) && global_ns() - t0 < 20000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(false, false);
            int stage = 0; uint32_t phase = 0; int acc = 0; uint32_t acc_phase = 0; bool ok = true;
            int qslot = 0; uint32_t qphase = 0;
            while (ok && take_tile(qslot, qphase) >= 0) {
                if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * UM_BN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = op_base + stage * UM_STAGE_BYTES, sb = sa + UM_A_BYTES;
                    const uint64_t adesc = make_smem_desc(sa, 16, 1024), bdesc = make_smem_desc(sb, 16, 1024);
#pragma unroll
                    for (int k = 0; k < UM_BK / 16; ++k)
                        tc_mma_bf16(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
                    tc_commit(bar_empty + 8 * stage);
                    if (++stage == WU_OP_STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit(bar_tfull + 8 * acc);
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------ state loader: x (, y, z) boxes, chunk by chunk
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            int qslot = 0; uint32_t qphase = 0;
            for (int t; ok && (t = take_tile(qslot, qphase)) >= 0;) {
                int l, g, m0, n0; coords(t, l, g, m0, n0);
                const int N = p.layer[l].N;
                for (int c = 0; c < WU_CHUNKS; ++c) {
                    const int nb = n0 + c * WU_CHUNK_ROWS;
                    if (nb >= N) break;
                    if (!mbar_wait(bar_sempty + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t dst = st_base + stage * WU_STATE_BYTES;
                    const uint32_t fb = bar_sfull + 8 * stage;
                    mbar_expect_tx(fb, WU_STATE_BYTES);
                    tma_load_3d(dst, &maps.x[l], fb, m0, nb, g);
                    if (!FIRST) {
                        if (YSPLIT) {
                            // hi plane: rows nb % 128 .. of the two 64-column blocks under this tile; lo plane: one box
                            const uint32_t yd = dst + WU_ARRAY_BYTES;
                            tma_load_5d(yd, &maps.yhi[l], fb, 0, nb & 127, m0 >> 6, nb >> 7, g);
                            tma_load_5d(yd + WU_ARRAY_BYTES / 4, &maps.yhi[l], fb, 0, nb & 127, (m0 >> 6) + 1, nb >> 7, g);
                            tma_load_3d(yd + WU_ARRAY_BYTES / 2, &maps.ylo[l], fb, m0, nb, g);
                        } else {
                            tma_load_3d(dst + WU_ARRAY_BYTES, &maps.y[l], fb, m0, nb, g);
                        }
                        if (LOADS_Z) tma_load_3d(dst + WU_Z_SLOT * WU_ARRAY_BYTES, &maps.z[l], fb, m0, nb, g);
                        if (MOM) tma_load_3d(dst + WU_V_SLOT * WU_ARRAY_BYTES, &maps.v[l], fb, m0, nb, g);
                    }
                    if (++stage == WU_STATE_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                for (int s = 0; s < WU_STATE_STAGES; ++s) {
                    const uint32_t armed_parity = (s < stage) ? phase : (phase ^ 1u);
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_sfull + 8 * s, armed_parity) && global_ns() - t0 < 20000000ull) {}
                }
            }
        }
    } else {
        // ------------------------------------------------ epilogue groups
        const int q = warp & 3;                              // tensor-memory lane quarter of this warp
        const int grp = (warp - 3) >> 2;                     // rows grp*RPG .. of every chunk
        const float one_m_alpha = 1.0f - p.alpha, alpha_sq = p.alpha * p.alpha;
        const float neg_eta_p = -p.eta_p;
        constexpr bool USE_Z = FIRST || ZMODE != WU_Z_SKIP;
        int acc = 0; uint32_t acc_phase = 0;
        int stage = 0; uint32_t sphase = 0;                  // state ring position: every warp walks every chunk
        float chk = 0.f;                                     // 0 * y summed: turns NaN as soon as a y is NaN or Inf
        bool ok = true;
        int qslot = 0; uint32_t qphase = 0;
        while (ok) {
            // every lane waits for the tile index and reads it; lane 0 hands the slot back for the warp
            if (!__all_sync(0xffffffffu, mbar_wait(bar_qfull + 8 * qslot, qphase, abort_flag))) break;
            const int t = tile_ids[qslot];
            // (the vote uses the index every lane has read: no lane's load of it is still on its way at the arrive)
            if (__all_sync(0xffffffffu, t >= -1) && lane == 0) mbar_arrive(bar_qempty + 8 * qslot);
            if (++qslot == WU_TILE_SLOTS) { qslot = 0; qphase ^= 1u; }
            if (t < 0) break;
            int l, g, m0, n0; coords(t, l, g, m0, n0);
            const int N = p.layer[l].N, ld = p.layer[l].ld;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag));
            if (!ok) break;
            tc_fence_after();
            const int col = q * 32 + lane;                   // tile column along d_in
            const int m = m0 + col;
            const bool m_ok = m < p.layer[l].M;
            const long long tile_e0 = (long long)g * p.gs + p.layer[l].w_off + (long long)(n0 + grp * RPG) * ld + m;
            const long long chunk_step = (long long)WU_CHUNK_ROWS * ld;
            float *yp = p.y + tile_e0, *zp = p.z + tile_e0;
            uint16_t *lp = YSPLIT ? p.ylo + tile_e0 : nullptr;
            float *vp = MOM ? p.v + tile_e0 : nullptr;
            // blocked copy: W row r, column m live in block (r/128, m/64) at (r%128)*64 + m%64; n0 % 128 == 0
            __nv_bfloat16 *sp = p.shadow + (long long)g * p.shadow_gs + p.layer[l].shadow_off +
                                ((long long)(n0 / UM_BN) * p.layer[l].shadow_cb + (m >> 6)) * (UM_BN * 64) +
                                (grp * RPG) * 64 + (m & 63);
            // The rows a thread owns inside a chunk are `ld` elements apart.  For the usual widths the pitch is a
            // compile-time constant, so every row's address is the chunk pointer plus an immediate offset and the
            // loop below carries no address arithmetic; other widths take the run-time pitch.
            auto run_chunks = [&](auto ld_tag, auto wd_tag) {
                constexpr int LDC = decltype(ld_tag)::value;
                constexpr bool HAS_WD = decltype(wd_tag)::value != 0;        // without weight decay its term is not computed at all
                const long long ldv = LDC > 0 ? (long long)LDC : (long long)ld;
#pragma unroll 1
                for (int c = 0; c < WU_CHUNKS; ++c, yp += chunk_step, zp += chunk_step, sp += WU_CHUNK_ROWS * 64) {
                    if (MOM && c > 0) vp += chunk_step;
                    if (YSPLIT && c > 0) lp += chunk_step;
                    const int nb0 = n0 + c * WU_CHUNK_ROWS;
                    if (nb0 >= N) break;                         // same rule as the loader
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_sfull + 8 * stage, sphase, abort_flag));
                    if (!ok) break;
                    const int nb = nb0 + grp * RPG;
                    const float *sx = reinterpret_cast<const float *>(st_ptr + (size_t)stage * WU_STATE_BYTES) +
                                      grp * RPG * UM_BM + col;
                    float xv[RPG], yv[RPG], zv[RPG], vv[RPG];
#pragma unroll
                    for (int j = 0; j < RPG; ++j) {
                        xv[j] = sx[j * UM_BM];
                        if (!FIRST) {
                            if (YSPLIT) {
                                const uint16_t *sy = reinterpret_cast<const uint16_t *>(st_ptr + (size_t)stage * WU_STATE_BYTES + WU_ARRAY_BYTES);
                                const int rr = grp * RPG + j;
                                const uint32_t hi = sy[(col >> 6) * (WU_CHUNK_ROWS * 64) + rr * 64 + (col & 63)];
                                const uint32_t lo = sy[WU_CHUNK_ROWS * 128 + rr * UM_BM + col];
                                yv[j] = __uint_as_float(((hi << 16) | lo) - 0x8000u);
                            } else {
                                yv[j] = sx[WU_ARRAY_BYTES / 4 + j * UM_BM];
                            }
                            if (USE_Z) zv[j] = sx[WU_Z_SLOT * (WU_ARRAY_BYTES / 4) + j * UM_BM];
                            if (MOM) vv[j] = sx[WU_V_SLOT * (WU_ARRAY_BYTES / 4) + j * UM_BM];
                        }
                    }
                    uint32_t r[RPG];
                    tc_ld_cols<RPG>(tmem_base + ((uint32_t)(q * 32) << 16) +
                                    (uint32_t)(acc * UM_BN + c * WU_CHUNK_ROWS + grp * RPG), r);
                    // Eq. (parle_y) and (parle_z) for the RPG rows of this thread, in registers.  Rows past the end of
                    // the layer hold whatever the box was filled with; they are computed and never stored.
                    float yn[RPG], zn[RPG];
#pragma unroll
                    for (int j = 0; j < RPG; ++j) {
                        const float yo = FIRST ? xv[j] : yv[j], zo = FIRST ? xv[j] : (USE_Z ? zv[j] : 0.f);
                        float d = fmaf(p.inv_gamma, yo - xv[j], HAS_WD ? fmaf(p.wd, yo, __uint_as_float(r[j])) : __uint_as_float(r[j]));
                        if (MOM) {
                            const float vn = FIRST ? d : fmaf(p.mu, vv[j], d);      // v = 0 before the first step of a round
                            vv[j] = vn;
                            d = fmaf(p.mu, vn, d);
                        }
                        yn[j] = fmaf(neg_eta_p, d, yo);
                        zn[j] = !USE_Z ? 0.f
                              : (!FIRST && ZMODE == WU_Z_DOUBLE) ? fmaf(alpha_sq, zo, one_m_alpha * fmaf(p.alpha, yo, yn[j]))
                                                                 : fmaf(p.alpha, zo, one_m_alpha * yn[j]);
                    }
                    const int rows = m_ok ? (N - nb) : 0;        // rows of this thread that exist
                    auto store_row = [&](int j) {
                        const long long o = (long long)j * ldv;
                        if (MOM) vp[o] = vv[j];
                        if (USE_Z) chk = fmaf(yn[j], 0.f, chk);  // steps that skip z skip the check: the next step sees the same y
                        if (YSPLIT) {
                            const uint32_t w = bf16_split_word(yn[j]);
                            lp[o] = (uint16_t)w;                 // lower half; the upper half is the operand copy below
                            if (YWRITE) yp[o] = yn[j];
                        } else {
                            yp[o] = yn[j];
                        }
                        if (USE_Z) zp[o] = zn[j];
                        sp[j * 64] = bf16_weight(yn[j]);
                    };
                    if (rows >= RPG) {                           // common case: no per-row bounds checks
#pragma unroll
                        for (int j = 0; j < RPG; ++j) store_row(j);
                    } else {
#pragma unroll
                        for (int j = 0; j < RPG; ++j)
                            if (j < rows) store_row(j);
                    }
                    // Only now is the stage handed back to the loader.  A shared-memory load that has merely been issued does
                    // not hold back an arrive, and arithmetic on its result may be scheduled after one: with the arrive placed
                    // right after the loads, and the load/store unit kept busy by another kernel's CTAs on the same SM, the
                    // loader's next copy was seen to land in the stage before such a load had read it.  The stores above use
                    // every value read from the stage and, being memory operations, stay in front of the arrive.
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_sempty + 8 * stage);
                    if (++stage == WU_STATE_STAGES) { stage = 0; sphase ^= 1u; }
                }
            };
            if (MOM || p.wd != 0.f) {
                run_chunks(WuPitch<0>(), WuPitch<1>());
            } else {
                switch (ld) {
                    case 2048: run_chunks(WuPitch<2048>(), WuPitch<0>()); break;
                    case 3072: run_chunks(WuPitch<3072>(), WuPitch<0>()); break;
                    case 4096: run_chunks(WuPitch<4096>(), WuPitch<0>()); break;
                    case 8192: run_chunks(WuPitch<8192>(), WuPitch<0>()); break;
                    default: run_chunks(WuPitch<0>(), WuPitch<0>()); break;
                }
            }
            if (!ok) break;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (chk != 0.f) p.status[SLOT_NONFINITE] = 1;        // NaN != 0 is true
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) p.status[SLOT_WAIT_LIMIT] = 1;
    if (threadIdx.x == 0) {
        // all claims of this CTA are done; the last CTA to leave puts both counters back to zero for the next launch
        __threadfence();
        if (atomicAdd(p.sched + 1, 1) == (int)gridDim.x - 1) {
            __threadfence();
            p.sched[0] = 0;
            p.sched[1] = 0;
        }
    }
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"((uint32_t)UM_TMEM_COLS) : "memory");
    }
}

}  // namespace parle
