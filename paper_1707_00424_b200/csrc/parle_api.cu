// C ABI of the Parle round: context, planning, launches.  See include/parle.h
// for the contract of every entry point.
#include <math.h>
#include <new>
#include <string.h>

#include "common.cuh"
#include "mlp_simt.cuh"
#include "umma_gemm.cuh"
#include "umma_pair_gemm.cuh"
#include "umma_wgrad_update.cuh"
#include "umma_tf32x3.cuh"
#include "update_kernels.cuh"

using namespace parle;

namespace {

constexpr size_t kWsAlign = 1024;
constexpr int kProfCapacity = 65536;       // launches recorded between two parle_profile_read calls
// SM count the split-K factors of the last forward layer are planned for.  They are fixed at parle_init (the size
// of the workspace depends on them) where no device is known yet; the launches themselves use the bound device's
// count.  On a part with another count the split is merely sized for 148.
constexpr int kPlanSmCount = 148;

enum KernelClass {
    KC_INPUT_CVT = 0, KC_FWD_GEMM, KC_SOFTMAX_CE, KC_WGRAD_GEMM, KC_BIAS_GRAD, KC_DGRAD_GEMM,
    KC_INNER_UPDATE, KC_OUTER_MEAN, KC_MEAN, KC_TO_BF16, KC_WGRAD_UPDATE, KC_TAIL_UPDATE, KC_COUNT
};
const char *const kClassNames[KC_COUNT] = {
    "input_to_bf16", "fwd_gemm", "softmax_ce_backward", "wgrad_gemm", "bias_grad", "dgrad_gemm",
    "inner_update", "outer_mean", "mean", "to_bf16", "wgrad_gemm_fused_update", "tail_update"};

struct Workspace {
    // byte offsets into parle_buffers.workspace; index = layer (0-based)
    size_t act[PARLE_MAX_LAYERS];      // fp32 mode: output of layer l  [n,B,d_{l+1}] fp32 (last = logits)
    size_t dact[PARLE_MAX_LAYERS];     // fp32 mode: gradient w.r.t. layer l's output [n,B,d_{l+1}] fp32
    size_t logits;                     // bf16 mode: fp32 logits [n,B,C] (x last_ksplit partial sums when split-K is used)
    size_t shadow;                     // bf16 mode: blocked bf16 copy of the weights [n, sh_stride]
    size_t xb, xbT;                    // bf16 mode: inputs [n,B,d_0] and transposed [n,d_0,B]
    size_t hb[PARLE_MAX_LAYERS], hbT[PARLE_MAX_LAYERS];      // hidden activations, both layouts
    size_t dhb[PARLE_MAX_LAYERS], dhbT[PARLE_MAX_LAYERS];    // their gradients, both layouts
    int dh_ld[PARLE_MAX_LAYERS];       // row pitch of dhb[l] (d_{l+1} rounded up to 8)
    size_t row_loss;                   // [n,B] fp32
    size_t rows_done;                  // [n] ints: rows of a replica the softmax kernel has finished (zero between launches)
    // fp32 mode on the tensor cores (3 x tf32): tf32-exact hi/lo pairs, index [0] = hi, [1] = lo
    size_t t3_logits;                  // fp32 logits [n, B, C] x t3_ksplit partial sums
    size_t w_split[2];                 // parameters [n, stride]
    size_t wT_split[2];                // transposed weights of layers >= 1, [n, t3_t_stride]
    size_t xs[2], xT[2];               // inputs [n, B, d_0] and transposed [n, d_0, B]
    size_t hs[PARLE_MAX_LAYERS][2], hT[PARLE_MAX_LAYERS][2];     // hidden activations [n, B, d_{l+1}] and transposed
    size_t dhs[PARLE_MAX_LAYERS][2], dhT[PARLE_MAX_LAYERS][2];   // their gradients [n, B, ld_l] (ld_l = d_{l+1} rounded up to 4) and transposed [n, d_{l+1}, B]
    size_t ylo;                        // bf16 mode: low 16 bits of the fp32 words of y, [n, stride] uint16 (whole rounds keep y as bf16 copy + this)
    size_t sched;                      // bf16 mode: two ints, the tile counters of the fused weight-gradient kernel (zero between launches)
    size_t pair_sync;                  // bf16 mode: per-(link, replica) progress counters of the chained pair kernel (zero between launches)
    size_t stage_in[2], stage_lab[2], stage_loss[2];   // double-buffered staging for the host-buffer entry points
    size_t total;
};

}  // namespace

namespace {
// Everything a captured round depends on: if any of it changes, the graph is rebuilt.
struct RoundKey {
    int L;
    const void *inputs, *labels, *loss;
    float scal[7];                   // 1/gamma, 1/rho, alpha, eta, eta', weight decay, momentum
    int fused, wide_thr, shadow_is_x, fresh;   // L == 0: a single inner step (fresh = first of its round)
    int pair_gemm, fused_loss;
    int paired_z, z_mode;            // whole rounds: Eq. (parle_z) in pairs or not; single steps: how this step treats z
    int split_y, y_step;             // whole rounds: y in two 16-bit planes or not; single steps: bit 0 = in that mode, bit 1 = stores fp32 y
    const void *ptrs[9];             // x, y, z, grad, xbar, workspace, vy, vx, stream
};
struct RoundGraph {
    RoundKey key;
    cudaGraphExec_t exec;
    long long launches;              // kernels inside the graph
    unsigned long long last_use;
};
constexpr int kRoundGraphs = 8;
}  // namespace

struct parle_ctx {
    int n, n_layers, batch, gemm_dtype;
    int dims[PARLE_MAX_LAYERS + 1];
    float inv_gamma, inv_rho, alpha, eta, eta_prime, weight_decay;
    int last_ksplit;                 // split-K factor of the last forward layer (1 = off)
    int wide_tiles_per_sm;           // 128 x 256 GEMM tiles are used when at least this many of them fall on every SM
    float momentum;                  // Nesterov momentum on the y and x^a steps (0 = off)
    float *vy, *vx;                  // caller-owned momentum buffers [n, stride] (parle_bind_momentum)
    size_t P, stride;
    size_t sh_stride;                // bf16 path: elements of one replica's blocked weight copy
    size_t sh_off[PARLE_MAX_LAYERS]; int sh_cb[PARLE_MAX_LAYERS], sh_rb[PARLE_MAX_LAYERS];   // per layer: offset, column / row blocks
    LayerPlan layers[PARLE_MAX_LAYERS];
    Workspace ws;
    bool bound;
    parle_buffers buf;
    cudaStream_t stream;
    int *status_host, *status_dev;
    bool round_open, fresh, shadow_is_x;
    bool paired_z;                   // whole rounds: Eq. (parle_z) applied two steps at a time
    bool split_y;                    // fused bf16 path, whole rounds: y of the weights kept as bf16 copy + low-half plane
    bool y_split_step, y_write_step; // this step runs in that mode / also stores the fp32 y (set per step by the round drivers)
    int z_mode;                      // how the next fused step treats z (WU_Z_*); set per step by the round drivers
    bool fused_update;               // bf16 path: apply Eq. (parle_y)/(parle_z) inside the weight-gradient GEMM
    bool fused_loss;                 // bf16 path, at most 128 classes: softmax cross-entropy backward inside the last forward GEMM's epilogue
    int steps_in_round;
    long long launches;
    int last_cuda;
    int sm_count;
    CUtensorMap tm_fwd_a[PARLE_MAX_LAYERS], tm_fwd_b[PARLE_MAX_LAYERS];
    CUtensorMap tm_dg_a[PARLE_MAX_LAYERS], tm_dg_b[PARLE_MAX_LAYERS];
    CUtensorMap tm_wg_a[PARLE_MAX_LAYERS], tm_wg_b[PARLE_MAX_LAYERS];
    // forward / data-gradient products on pairs of SMs: the activation operand in boxes of half a batch tile
    CUtensorMap tm_pf_x[PARLE_MAX_LAYERS], tm_pd_x[PARLE_MAX_LAYERS];
    int pair_gemm;                   // pair kernel where the shapes allow: 0 = never, 1 = one launch per layer, 2 = chained where it pays, 3 = always chained
    // fp32 configurations on the tensor cores (three tf32 products per GEMM)
    int t3_mode;                     // 0 = never, 1 = when the layers are wide enough to fill 128-row tiles, 2 = whenever possible
    bool t3_shapes_ok;               // widths and batch are multiples of 4 (16-byte rows for TMA)
    bool t3_ready;                   // tensor maps exist for the bound buffers (needs an sm_100 device)
    size_t t3_t_off[PARLE_MAX_LAYERS], t3_t_stride;   // transposed weight copy: W_l^T [d_in, ld_l] of layers >= 1 inside a replica's copy
    int t3_ksplit;                   // split-K factor of the last forward layer on this path (1 = off)
    int t3_bn_fwd[PARLE_MAX_LAYERS], t3_bn_dg[PARLE_MAX_LAYERS], t3_bn_wg[PARLE_MAX_LAYERS];   // tile widths (64 or 128)
    CUtensorMap t3_fa[PARLE_MAX_LAYERS][2], t3_fb[PARLE_MAX_LAYERS][2];    // forward operands, hi / lo
    CUtensorMap t3_da[PARLE_MAX_LAYERS][2], t3_db[PARLE_MAX_LAYERS][2];    // data gradient
    CUtensorMap t3_wa[PARLE_MAX_LAYERS][2], t3_wb[PARLE_MAX_LAYERS][2];    // weight gradient
    WuMaps wu_maps;                  // fused weight-gradient kernel: operands + fp32 W_l segments of x, y, z (32-row boxes)
    WuMaps wu_maps_mom;              // its momentum variant: same + vy, 16-row boxes
    bool mom_maps;
    // parle_round as a CUDA graph (optional): a small cache of instantiated rounds
    bool graphs_on;
    cudaStream_t capture_stream;     // rounds are captured here (the bound stream may be the default stream, which cannot be)
    RoundGraph graphs[kRoundGraphs];
    int n_graphs;
    unsigned long long graph_clock;
    // host-buffer rounds: a second stream uploads the next minibatch while the current step runs
    cudaStream_t copy_stream;
    cudaEvent_t ev_copied[2], ev_consumed[2];
    bool copy_ready;
    // optional per-launch timing (events, host-side bookkeeping only)
    bool prof_on, prof_open;
    int prof_used, prof_dropped;
    cudaEvent_t *prof_ev;            // 2 * kProfCapacity events
    unsigned char *prof_cls;
};

extern "C" { static void drop_round_graphs(parle_ctx *c); }

namespace {

inline int cuda_fail(parle_ctx *c, cudaError_t e) {
    c->last_cuda = (int)e;
    return PARLE_ECUDA;
}
#define PARLE_CUDA(c, expr) do { cudaError_t e_ = (expr); if (e_ != cudaSuccess) return cuda_fail((c), e_); } while (0)
#define PARLE_LAUNCHED(c) do { (c)->launches++; prof_end(c); cudaError_t e_ = cudaGetLastError(); if (e_ != cudaSuccess) return cuda_fail((c), e_); } while (0)

inline void prof_begin(parle_ctx *c, int cls) {
    if (!c->prof_on) return;
    if (c->prof_used >= kProfCapacity) { c->prof_dropped++; return; }
    cudaEventRecord(c->prof_ev[2 * c->prof_used], c->stream);
    c->prof_cls[c->prof_used] = (unsigned char)cls;
    c->prof_open = true;
}
inline void prof_end(parle_ctx *c) {
    if (!c->prof_open) return;
    cudaEventRecord(c->prof_ev[2 * c->prof_used + 1], c->stream);
    c->prof_used++;
    c->prof_open = false;
}
#define PARLE_TRY(expr) do { int rc_ = (expr); if (rc_ != PARLE_OK) return rc_; } while (0)

inline bool coupling_ok(double v) { return v > 0.0 && !isnan(v); }
inline float inverse_or_zero(double v) { return isinf(v) ? 0.0f : (float)(1.0 / v); }

void plan_workspace(parle_ctx *c) {
    Workspace &w = c->ws;
    memset(&w, 0, sizeof(w));
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = round_up(off + bytes, kWsAlign); return o; };
    const size_t n = c->n, B = c->batch;
    const int nl = c->n_layers;
    if (nl == 0) { w.total = kWsAlign; return; }
    const size_t C = c->dims[nl];
    if (c->gemm_dtype == PARLE_GEMM_FP32) {
        for (int l = 0; l < nl; ++l) w.act[l] = take(n * B * c->dims[l + 1] * sizeof(float));
        for (int l = 0; l < nl; ++l) w.dact[l] = take(n * B * c->dims[l + 1] * sizeof(float));
        if (c->t3_shapes_ok) {
            w.t3_logits = take(n * B * C * sizeof(float) * (size_t)c->t3_ksplit);
            for (int h = 0; h < 2; ++h) {
                w.w_split[h] = take(n * c->stride * sizeof(float));
                w.wT_split[h] = take(n * c->t3_t_stride * sizeof(float));
                w.xs[h] = take(n * B * c->dims[0] * sizeof(float));
                w.xT[h] = take(n * B * c->dims[0] * sizeof(float));
                for (int l = 0; l + 1 < nl; ++l) {
                    w.hs[l][h] = take(n * B * c->dims[l + 1] * sizeof(float));
                    w.hT[l][h] = take(n * B * c->dims[l + 1] * sizeof(float));
                }
                for (int l = 0; l < nl; ++l) {
                    w.dhs[l][h] = take(n * B * round_up(c->dims[l + 1], 4) * sizeof(float));
                    w.dhT[l][h] = take(n * B * c->dims[l + 1] * sizeof(float));
                }
            }
        }
    } else {
        w.shadow = take(n * c->sh_stride * 2);
        w.xb = take(n * B * c->dims[0] * 2);
        w.xbT = take(n * B * c->dims[0] * 2);
        for (int l = 0; l + 1 < nl; ++l) {
            w.hb[l] = take(n * B * c->dims[l + 1] * 2);
            w.hbT[l] = take(n * B * c->dims[l + 1] * 2);
        }
        w.logits = take(n * B * C * sizeof(float) * (size_t)c->last_ksplit);
        for (int l = 0; l < nl; ++l) {
            w.dh_ld[l] = (int)round_up(c->dims[l + 1], 8);
            w.dhb[l] = take(n * B * w.dh_ld[l] * 2);
            w.dhbT[l] = take(n * B * c->dims[l + 1] * 2);
        }
        w.ylo = take(n * c->stride * sizeof(uint16_t));
        w.sched = take(2 * sizeof(int));
        w.pair_sync = take(UP_SYNC_INTS * sizeof(int));
    }
    w.row_loss = take(n * B * sizeof(float));
    w.rows_done = take(n * sizeof(int));
    for (int b = 0; b < 2; ++b) {
        w.stage_in[b] = take(n * B * c->dims[0] * sizeof(float));
        w.stage_lab[b] = take(n * B * sizeof(int32_t));
        w.stage_loss[b] = take(n * sizeof(float));
    }
    w.total = off;
}

template <typename T> inline T *ws_ptr(parle_ctx *c, size_t off) {
    return reinterpret_cast<T *>(static_cast<char *>(c->buf.workspace) + off);
}

// ---------------------------------------------------------------- tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

int get_encoder(parle_ctx *c, EncodeTiledFn *fn) {
    static EncodeTiledFn cached = nullptr;
    if (!cached) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        PARLE_CUDA(c, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q));
        if (!p || q != cudaDriverEntryPointSuccess) return cuda_fail(c, cudaErrorNotSupported);
        cached = reinterpret_cast<EncodeTiledFn>(p);
    }
    *fn = cached;
    return PARLE_OK;
}

// bf16 tensor [groups][rows][cols] (cols contiguous), row pitch and group pitch
// in elements; box = box_cols x box_rows x 1, 128-byte swizzle, zero fill.
int encode_bf16_map(parle_ctx *c, CUtensorMap *tm, const void *base, size_t cols, size_t rows, size_t groups,
                    size_t row_pitch, size_t group_pitch, unsigned box_cols, unsigned box_rows) {
    EncodeTiledFn enc;
    PARLE_TRY(get_encoder(c, &enc));
    cuuint64_t dims[3] = {cols, rows, groups};
    cuuint64_t strides[2] = {row_pitch * 2, (group_pitch ? group_pitch : row_pitch * rows) * 2};
    cuuint32_t box[3] = {box_cols, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { c->last_cuda = (int)r; return PARLE_ECUDA; }
    return PARLE_OK;
}

// fp32 tensor [groups][rows][cols], no swizzle (boxes are read back word by word, lane = column).
int encode_f32_map(parle_ctx *c, CUtensorMap *tm, const void *base, size_t cols, size_t rows, size_t groups,
                   size_t row_pitch, size_t group_pitch, unsigned box_cols, unsigned box_rows) {
    EncodeTiledFn enc;
    PARLE_TRY(get_encoder(c, &enc));
    cuuint64_t dims[3] = {cols, rows, groups};
    cuuint64_t strides[2] = {row_pitch * 4, group_pitch * 4};
    cuuint32_t box[3] = {box_cols, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { c->last_cuda = (int)r; return PARLE_ECUDA; }
    return PARLE_OK;
}

// Blocked bf16 weight copy of one layer as a 5-D tensor (column in block, row in block, column block,
// row block, replica); box = box_rows x 64 columns of one block, 128-byte swizzle, zero fill outside.
int encode_blocked_map(parle_ctx *c, CUtensorMap *tm, const void *base, int cb, int rb, size_t groups,
                       size_t group_pitch, unsigned box_rows) {
    EncodeTiledFn enc;
    PARLE_TRY(get_encoder(c, &enc));
    cuuint64_t dims[5] = {64, 128, (cuuint64_t)cb, (cuuint64_t)rb, groups};
    cuuint64_t strides[4] = {128, 16384, (cuuint64_t)cb * 16384, group_pitch * 2};
    cuuint32_t box[5] = {64, box_rows, 1, 1, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { c->last_cuda = (int)r; return PARLE_ECUDA; }
    return PARLE_OK;
}

// fp32 tensor [groups][rows][cols] as a tf32 operand: boxes of 32 columns (128 bytes) x box_rows, 128-byte swizzle.
int encode_tf32_map(parle_ctx *c, CUtensorMap *tm, const void *base, size_t cols, size_t rows, size_t groups,
                    size_t row_pitch, size_t group_pitch, unsigned box_rows) {
    EncodeTiledFn enc;
    PARLE_TRY(get_encoder(c, &enc));
    cuuint64_t dims[3] = {cols, rows, groups};
    cuuint64_t strides[2] = {row_pitch * 4, group_pitch * 4};
    cuuint32_t box[3] = {32, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { c->last_cuda = (int)r; return PARLE_ECUDA; }
    return PARLE_OK;
}

// Tile width of a tf32 product: 128 columns, or 64 when 128-wide tiles would leave a quarter of the SMs idle.
inline int t3_tile_width(const parle_ctx *c, int M, int N) {
    const long long wide = (long long)c->n * ((M + T3_BM - 1) / T3_BM) * ((N + 127) / 128);
    return wide * 4 < (long long)c->sm_count * 3 ? 64 : 128;
}

// The two 16-bit planes of y for the fused kernel: boxes of 64 columns x box_rows of the blocked bf16 copy (5-D, no
// swizzle: they are read back element by element), and boxes of 128 columns x box_rows of the uint16 lo plane.
int encode_yhi_map(parle_ctx *c, CUtensorMap *tm, const void *base, int cb, int rb, size_t groups, size_t group_pitch,
                   unsigned box_rows) {
    EncodeTiledFn enc;
    PARLE_TRY(get_encoder(c, &enc));
    cuuint64_t dims[5] = {64, 128, (cuuint64_t)cb, (cuuint64_t)rb, groups};
    cuuint64_t strides[4] = {128, 16384, (cuuint64_t)cb * 16384, group_pitch * 2};
    cuuint32_t box[5] = {64, box_rows, 1, 1, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { c->last_cuda = (int)r; return PARLE_ECUDA; }
    return PARLE_OK;
}
int encode_ylo_map(parle_ctx *c, CUtensorMap *tm, const void *base, size_t cols, size_t rows, size_t groups,
                   size_t row_pitch, size_t group_pitch, unsigned box_rows) {
    EncodeTiledFn enc;
    PARLE_TRY(get_encoder(c, &enc));
    cuuint64_t dims[3] = {cols, rows, groups};
    cuuint64_t strides[2] = {row_pitch * 2, group_pitch * 2};
    cuuint32_t box[3] = {(cuuint32_t)UM_BM, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { c->last_cuda = (int)r; return PARLE_ECUDA; }
    return PARLE_OK;
}

int build_tf32_maps(parle_ctx *c) {
    const Workspace &w = c->ws;
    const size_t n = c->n, B = c->batch, S = c->stride;
    for (int l = 0; l < c->n_layers; ++l) {
        const size_t din = c->dims[l], dout = c->dims[l + 1], wo = c->layers[l].w_off;
        c->t3_bn_fwd[l] = t3_tile_width(c, (int)B, (int)dout);
        c->t3_bn_dg[l] = t3_tile_width(c, (int)B, (int)din);
        c->t3_bn_wg[l] = t3_tile_width(c, (int)din, (int)dout);
        const size_t ld = round_up(dout, 4);
        for (int h = 0; h < 2; ++h) {
            const float *in = l == 0 ? ws_ptr<float>(c, w.xs[h]) : ws_ptr<float>(c, w.hs[l - 1][h]);
            const float *inT = l == 0 ? ws_ptr<float>(c, w.xT[h]) : ws_ptr<float>(c, w.hT[l - 1][h]);
            const float *W = ws_ptr<float>(c, w.w_split[h]) + wo;
            // forward: A = input [B, d_in], B = W [d_out, d_in] (K = d_in)
            PARLE_TRY(encode_tf32_map(c, &c->t3_fa[l][h], in, din, B, n, din, B * din, T3_BM));
            PARLE_TRY(encode_tf32_map(c, &c->t3_fb[l][h], W, din, dout, n, din, S, c->t3_bn_fwd[l]));
            if (l > 0) {
                // data gradient: A = dH [B, d_out] (pitch ld), B = W^T [d_in, d_out] (pitch ld) (K = d_out)
                const float *WT = ws_ptr<float>(c, w.wT_split[h]) + c->t3_t_off[l];
                PARLE_TRY(encode_tf32_map(c, &c->t3_da[l][h], ws_ptr<float>(c, w.dhs[l][h]), dout, B, n, ld, B * ld, T3_BM));
                PARLE_TRY(encode_tf32_map(c, &c->t3_db[l][h], WT, dout, din, n, ld, c->t3_t_stride, c->t3_bn_dg[l]));
            }
            // weight gradient (transposed): A = input^T [d_in, B], B = dH^T [d_out, B] (K = batch)
            PARLE_TRY(encode_tf32_map(c, &c->t3_wa[l][h], inT, B, din, n, B, din * B, T3_BM));
            PARLE_TRY(encode_tf32_map(c, &c->t3_wb[l][h], ws_ptr<float>(c, w.dhT[l][h]), B, dout, n, B, dout * B, c->t3_bn_wg[l]));
        }
    }
    return PARLE_OK;
}

template <int EPI, int BN>
int launch_t3_bn(parle_ctx *c, int cls, const CUtensorMap *a, const CUtensorMap *b, T3Params p) {
    p.groups = c->n;
    p.tiles_m = (p.M + T3_BM - 1) / T3_BM;
    p.tiles_n = (p.N + BN - 1) / BN;
    p.status = c->status_dev;
    const int tiles = p.groups * p.tiles_m * p.tiles_n * ((EPI == T3_FWD_LAST && p.ksplit > 1) ? p.ksplit : 1);
    const int grid = tiles < c->sm_count ? tiles : c->sm_count;
    prof_begin(c, cls);
    umma_tf32x3_kernel<EPI, BN><<<grid, T3_THREADS, T3Shape<BN>::SMEM_BYTES, c->stream>>>(a[0], a[1], b[0], b[1], p);
    PARLE_LAUNCHED(c);
    return PARLE_OK;
}
template <int EPI>
int launch_t3(parle_ctx *c, int cls, int bn, const CUtensorMap *a, const CUtensorMap *b, const T3Params &p) {
    return bn == 64 ? launch_t3_bn<EPI, 64>(c, cls, a, b, p) : launch_t3_bn<EPI, 128>(c, cls, a, b, p);
}
template <int EPI>
cudaError_t allow_t3_smem() {
    cudaError_t e = cudaFuncSetAttribute(umma_tf32x3_kernel<EPI, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)T3Shape<64>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(umma_tf32x3_kernel<EPI, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)T3Shape<128>::SMEM_BYTES);
}

// fp32 products on the tensor cores?  Automatic mode wants every layer input at least one 128-wide tile.
inline bool use_t3(const parle_ctx *c) {
    if (c->gemm_dtype != PARLE_GEMM_FP32 || !c->t3_ready || c->t3_mode == 0) return false;
    if (c->t3_mode == 2) return true;
    if (c->batch < 32) return false;
    for (int l = 0; l < c->n_layers; ++l)
        if (c->dims[l] < 128) return false;
    return true;
}

// Batch tile of the pair kernel: 128 rows, or 256 when the batch has more than 128.
inline int pair_batch_tile(const parle_ctx *c) { return c->batch > 128 ? 256 : 128; }
// The pair kernel takes a product when its weight operand has at least one full pair tile of output features.
inline bool use_pair_gemm(const parle_ctx *c, int features) { return c->pair_gemm > 0 && features >= 2 * UP_BM; }
// Chain a product with `features` output rows to its predecessor in one launch?  Mode 3: always.  Mode 2: when the
// product gives a pair of SMs at most two tiles -- there the start-up and the epilogue of a launch have nothing to
// hide behind; with many tiles per pair they already overlap with the neighbouring tiles and separate launches do as well.
inline bool chain_pair_gemm(const parle_ctx *c, int features) {
    if (c->pair_gemm >= 3) return true;
    if (c->pair_gemm < 2) return false;
    const int bt = pair_batch_tile(c);
    const long long tiles = (long long)c->n * ((features + 2 * UP_BM - 1) / (2 * UP_BM)) * ((c->batch + bt - 1) / bt);
    return tiles <= 2LL * (c->sm_count / 2);
}

// One launch of the pair kernel over a chain of products: forward, the hidden layers [first, last] in ascending order
// (each reads the activations the one before it wrote); backward, the data gradients of layers first, first - 1, ...,
// last (each reads the gradient the one before it wrote).
template <int EPI, int BNB>
int launch_pair_bn(parle_ctx *c, int cls, int first, int last) {
    const Workspace &w = c->ws;
    const int B = c->batch;
    const long long S = (long long)c->stride;
    const float *params = c->fresh ? c->buf.x : c->buf.y;      // fp32 biases come from the master copy
    UpMaps maps;
    UmmaPairParams p = {};
    p.Bt = B; p.groups = c->n; p.tiles_b = (B + BNB - 1) / BNB;
    int tiles = 0, k = 0;
    const int step = EPI == UPE_FWD_HIDDEN ? 1 : -1;
    for (int l = first; l != last + step; l += step, ++k) {
        const int din = c->dims[l], dout = c->dims[l + 1];
        UpLink &q = p.link[k];
        if (EPI == UPE_FWD_HIDDEN) {                            // H_l^T = W_l H_{l-1}^T
            q.F = dout; q.K = din;
            q.bias = params + c->layers[l].b_off; q.bias_gs = S;
            q.out = ws_ptr<__nv_bfloat16>(c, w.hb[l]); q.out_gs = (long long)B * dout; q.out_ld = dout;
            q.outT = ws_ptr<__nv_bfloat16>(c, w.hbT[l]); q.outT_gs = (long long)B * dout; q.outT_ld = B;
            maps.w[k] = c->tm_fwd_b[l]; maps.x[k] = c->tm_pf_x[l];
        } else {                                                // dH_{l-1}^T = W_l^T dH_l^T, masked by H_{l-1} > 0
            q.F = din; q.K = dout;
            q.out = ws_ptr<__nv_bfloat16>(c, w.dhb[l - 1]); q.out_gs = (long long)B * w.dh_ld[l - 1]; q.out_ld = w.dh_ld[l - 1];
            q.outT = ws_ptr<__nv_bfloat16>(c, w.dhbT[l - 1]); q.outT_gs = (long long)B * din; q.outT_ld = B;
            q.maskT = ws_ptr<__nv_bfloat16>(c, w.hbT[l - 1]); q.maskT_gs = (long long)B * din; q.maskT_ld = B;
            maps.w[k] = c->tm_dg_b[l]; maps.x[k] = c->tm_pd_x[l];
        }
        q.tiles_f = (q.F + 2 * UP_BM - 1) / (2 * UP_BM);
        q.tile_begin = tiles;
        tiles += c->n * q.tiles_f * p.tiles_b;
    }
    p.n_links = k; p.total_tiles = tiles;
    p.sync = ws_ptr<int>(c, w.pair_sync);
    p.status = c->status_dev;
    const int pairs = c->sm_count / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (tiles < pairs ? tiles : pairs));
    cfg.blockDim = dim3(UP_THREADS);
    cfg.dynamicSmemBytes = UpShape<BNB>::SMEM_BYTES;
    cfg.stream = c->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    prof_begin(c, cls);
    const cudaError_t e = cudaLaunchKernelEx(&cfg, umma_pair_gemm_kernel<EPI, BNB>, maps, p);
    if (e != cudaSuccess) { prof_end(c); return cuda_fail(c, e); }
    PARLE_LAUNCHED(c);
    return PARLE_OK;
}
template <int EPI>
int launch_pair(parle_ctx *c, int cls, int first, int last) {
    return pair_batch_tile(c) == 256 ? launch_pair_bn<EPI, 256>(c, cls, first, last) : launch_pair_bn<EPI, 128>(c, cls, first, last);
}
template <int EPI>
cudaError_t allow_pair_smem() {
    cudaError_t e = cudaFuncSetAttribute(umma_pair_gemm_kernel<EPI, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpShape<128>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(umma_pair_gemm_kernel<EPI, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpShape<256>::SMEM_BYTES);
}

int build_tensor_maps(parle_ctx *c) {
    const Workspace &w = c->ws;
    const size_t n = c->n, B = c->batch;
    const __nv_bfloat16 *shadow = ws_ptr<__nv_bfloat16>(c, w.shadow);
    for (int l = 0; l < c->n_layers; ++l) {
        const size_t din = c->dims[l], dout = c->dims[l + 1];
        const __nv_bfloat16 *a_in = l == 0 ? ws_ptr<__nv_bfloat16>(c, w.xb) : ws_ptr<__nv_bfloat16>(c, w.hb[l - 1]);
        const __nv_bfloat16 *a_inT = l == 0 ? ws_ptr<__nv_bfloat16>(c, w.xbT) : ws_ptr<__nv_bfloat16>(c, w.hbT[l - 1]);
        const __nv_bfloat16 *W = shadow + c->sh_off[l];
        // forward: A = layer input [B, din], B = W [dout, din], both K-major (K = din)
        PARLE_TRY(encode_bf16_map(c, &c->tm_fwd_a[l], a_in, din, B, n, din, B * din, UM_BK, UM_BM));
        // the same input as the shared operand of a pair of CTAs: boxes of half a batch tile
        PARLE_TRY(encode_bf16_map(c, &c->tm_pf_x[l], a_in, din, B, n, din, B * din, UM_BK, pair_batch_tile(c) / 2));
        PARLE_TRY(encode_blocked_map(c, &c->tm_fwd_b[l], W, c->sh_cb[l], c->sh_rb[l], n, c->sh_stride, 128));
        // weight gradient, computed transposed (dW^T = input^T dH): A = input^T [din, B], B = dH^T [dout, B],
        // both K-major (K = batch)
        PARLE_TRY(encode_bf16_map(c, &c->tm_wg_a[l], a_inT, B, din, n, B, din * B, UM_BK, UM_BM));
        PARLE_TRY(encode_bf16_map(c, &c->tm_wg_b[l], ws_ptr<__nv_bfloat16>(c, w.dhbT[l]), B, dout, n, B, dout * B, UM_BK, UM_BN));
        // fused update: the W_l segments of x, y, z as [n][dout][din] fp32, fetched in 16-row x 128-column boxes
        const size_t wo = c->layers[l].w_off;
        PARLE_TRY(encode_f32_map(c, &c->wu_maps.x[l], c->buf.x + wo, din, dout, n, din, c->stride, UM_BM, WU_CHUNK_ROWS));
        PARLE_TRY(encode_f32_map(c, &c->wu_maps.y[l], c->buf.y + wo, din, dout, n, din, c->stride, UM_BM, WU_CHUNK_ROWS));
        PARLE_TRY(encode_f32_map(c, &c->wu_maps.z[l], c->buf.z + wo, din, dout, n, din, c->stride, UM_BM, WU_CHUNK_ROWS));
        c->wu_maps.v[l] = c->wu_maps.z[l];                                   // not read without momentum
        c->wu_maps.a[l] = c->tm_wg_a[l]; c->wu_maps.b[l] = c->tm_wg_b[l];
        PARLE_TRY(encode_yhi_map(c, &c->wu_maps.yhi[l], W, c->sh_cb[l], c->sh_rb[l], n, c->sh_stride, WU_CHUNK_ROWS));
        PARLE_TRY(encode_ylo_map(c, &c->wu_maps.ylo[l], ws_ptr<uint16_t>(c, w.ylo) + wo, din, dout, n, din, c->stride, WU_CHUNK_ROWS));
        if (l > 0) {
            // data gradient: A = dH [B, dout] K-major (K = dout); B = W [dout (K), din (N)] MN-major,
            // fetched as 64 k-rows x 64 n-columns boxes
            PARLE_TRY(encode_bf16_map(c, &c->tm_dg_a[l], ws_ptr<__nv_bfloat16>(c, w.dhb[l]), dout, B, n,
                                      w.dh_ld[l], B * (size_t)w.dh_ld[l], UM_BK, UM_BM));
            PARLE_TRY(encode_blocked_map(c, &c->tm_dg_b[l], W, c->sh_cb[l], c->sh_rb[l], n, c->sh_stride, 64));
            PARLE_TRY(encode_bf16_map(c, &c->tm_pd_x[l], ws_ptr<__nv_bfloat16>(c, w.dhb[l]), dout, B, n,
                                      w.dh_ld[l], B * (size_t)w.dh_ld[l], UM_BK, pair_batch_tile(c) / 2));
        }
    }
    return PARLE_OK;
}

template <int EPI, int BKIND, int BN>
int launch_umma_bn(parle_ctx *c, int cls, const CUtensorMap &a, const CUtensorMap &b, UmmaParams p) {
    p.groups = c->n;
    p.tiles_m = (p.M + UM_BM - 1) / UM_BM;
    p.tiles_n = (p.N + BN - 1) / BN;
    p.status = c->status_dev;
    const int tiles = p.groups * p.tiles_m * p.tiles_n * ((EPI == UEPI_FWD_LAST && p.ksplit > 1) ? p.ksplit : 1);
    const int grid = tiles < c->sm_count ? tiles : c->sm_count;
    prof_begin(c, cls);
    umma_gemm_kernel<EPI, BKIND, BN><<<grid, umma_threads(EPI), UM_SMEM_BYTES, c->stream>>>(a, b, p);
    PARLE_LAUNCHED(c);
    return PARLE_OK;
}

// 256-wide tiles where the product is compute-bound and still leaves every SM several tiles
// (batch of at least 256 rows and four 128 x 256 tiles per SM), or where they turn two passes over the SMs into
// one (more 128-wide tiles than SMs, at most one 256-wide tile per SM: a tile then moves 48 instead of 64 KiB into
// shared memory per 128 x 256 x 64 block of the product); 128-wide tiles otherwise.
template <int EPI, int BKIND>
int launch_umma(parle_ctx *c, int cls, const CUtensorMap &a, const CUtensorMap &b, const UmmaParams &p) {
    if (BKIND != UB_ROWMAJOR_K && p.M >= 256) {
        const long long per_n = (long long)c->n * ((p.M + UM_BM - 1) / UM_BM);
        const long long wide_tiles = per_n * ((p.N + 255) / 256), narrow_tiles = per_n * ((p.N + 127) / 128);
        if (wide_tiles >= (long long)c->wide_tiles_per_sm * c->sm_count ||
            (c->wide_tiles_per_sm <= 1024 && narrow_tiles > c->sm_count && wide_tiles <= c->sm_count && 4 * wide_tiles >= 3 * c->sm_count))
            return launch_umma_bn<EPI, BKIND, 256>(c, cls, a, b, p);
    }
    return launch_umma_bn<EPI, BKIND, 128>(c, cls, a, b, p);
}

template <int EPI, int BKIND>
cudaError_t allow_big_smem() {
    cudaError_t e = cudaFuncSetAttribute(umma_gemm_kernel<EPI, BKIND, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)UM_SMEM_BYTES);
    if (e != cudaSuccess || BKIND == UB_ROWMAJOR_K) return e;
    return cudaFuncSetAttribute(umma_gemm_kernel<EPI, BKIND, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)UM_SMEM_BYTES);
}

// fp32 product: the largest register tile (8 x 8 outputs per thread) that still gives (nearly) every SM a
// CTA; small problems get 64 x 64 tiles with 4 x 4 outputs per thread (more warps per output).
template <int EPI>
int launch_simt(parle_ctx *c, int cls, const SimtGemmArgs &a) {
    auto ctas = [&](int bm, int bn) { return (long long)((a.M + bm - 1) / bm) * ((a.N + bn - 1) / bn) * c->n; };
    const long long want = (long long)c->sm_count * 85 / 100;
    prof_begin(c, cls);
    if (ctas(128, 128) >= want) {
        dim3 grid((a.N + 127) / 128, (a.M + 127) / 128, c->n);
        simt_gemm_tiled_kernel<EPI, 128, 128><<<grid, 256, 0, c->stream>>>(a);
    } else if (ctas(128, 64) >= want) {
        dim3 grid((a.N + 63) / 64, (a.M + 127) / 128, c->n);
        simt_gemm_tiled_kernel<EPI, 128, 64><<<grid, 128, 0, c->stream>>>(a);
    } else {
        dim3 grid((a.N + SG_BN - 1) / SG_BN, (a.M + SG_BM - 1) / SG_BM, c->n);
        simt_gemm_kernel<EPI><<<grid, SG_THREADS, 0, c->stream>>>(a);
    }
    PARLE_LAUNCHED(c);
    return PARLE_OK;
}

inline int stream_grid(const parle_ctx *c, size_t items, int per_thread) {
    size_t blocks = (items + (size_t)kUpdThreads * per_thread - 1) / ((size_t)kUpdThreads * per_thread);
    size_t cap = (size_t)c->sm_count * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

// ---------------------------------------------------------------- the steps
// Refresh the blocked bf16 weight copy from an fp32 vector (x at the start of a round; y after a
// separate update step).
int run_blocked_copy(parle_ctx *c, const float *src) {
    BlockedPlan bp = {};
    bp.n_layers = c->n_layers;
    int blocks = 0;
    for (int l = 0; l < c->n_layers; ++l) {
        bp.w_off[l] = (long long)c->layers[l].w_off; bp.sh_off[l] = (long long)c->sh_off[l];
        bp.d_in[l] = c->dims[l]; bp.d_out[l] = c->dims[l + 1]; bp.cb[l] = c->sh_cb[l];
        bp.first_block[l] = blocks;
        blocks += c->sh_rb[l] * c->sh_cb[l];
    }
    bp.first_block[c->n_layers] = blocks;
    prof_begin(c, KC_TO_BF16);
    blocked_bf16_kernel<<<dim3(blocks, c->n), 256, 0, c->stream>>>(
        bp, src, (long long)c->stride, ws_ptr<__nv_bfloat16>(c, c->ws.shadow), (long long)c->sh_stride);
    PARLE_LAUNCHED(c);
    return PARLE_OK;
}

int run_split_transpose(parle_ctx *c, const float *src);

template <bool FIRST, bool MOM, bool SPLIT, int ZMODE>
void launch_inner_update(parle_ctx *c, int grid, const float4 *g, float4 *y, const float4 *x, float4 *z, size_t n4, float wd) {
    constexpr int U = FIRST ? 4 : 2;          // the first step of a round reads two arrays instead of four: more of them in flight per thread
    inner_update_kernel<FIRST, U, MOM, SPLIT, ZMODE><<<grid, kUpdThreads, 0, c->stream>>>(
        g, y, x, z, n4, c->eta_prime, c->inv_gamma, c->alpha, wd, c->status_dev,
        MOM ? reinterpret_cast<float4 *>(c->vy) : nullptr, c->momentum,
        SPLIT ? ws_ptr<float4>(c, c->ws.w_split[0]) : nullptr, SPLIT ? ws_ptr<float4>(c, c->ws.w_split[1]) : nullptr);
}
template <bool MOM, bool SPLIT>
void launch_inner_update_z(parle_ctx *c, int zm, int grid, const float4 *g, float4 *y, const float4 *x, float4 *z, size_t n4, float wd) {
    if (c->fresh) launch_inner_update<true, MOM, SPLIT, UPD_Z_SINGLE>(c, grid, g, y, x, z, n4, wd);
    else if (zm == UPD_Z_SKIP) launch_inner_update<false, MOM, SPLIT, UPD_Z_SKIP>(c, grid, g, y, x, z, n4, wd);
    else if (zm == UPD_Z_DOUBLE) launch_inner_update<false, MOM, SPLIT, UPD_Z_DOUBLE>(c, grid, g, y, x, z, n4, wd);
    else launch_inner_update<false, MOM, SPLIT, UPD_Z_SINGLE>(c, grid, g, y, x, z, n4, wd);
}

// split: also refresh the tf32 hi/lo copy of the parameters from the new y (fp32 products on the tensor cores)
// zm: how this step treats z (UPD_Z_*; the round drivers pair the steps, single calls use the one-step form)
int run_inner_update(parle_ctx *c, const float *grad, float wd, bool split = false, int zm = UPD_Z_SINGLE) {
    const size_t n4 = (size_t)c->n * c->stride / 4;
    const int grid = stream_grid(c, n4, 2);
    const float4 *g = reinterpret_cast<const float4 *>(grad);
    float4 *y = reinterpret_cast<float4 *>(c->buf.y), *z = reinterpret_cast<float4 *>(c->buf.z);
    const float4 *x = reinterpret_cast<const float4 *>(c->buf.x);
    prof_begin(c, KC_INNER_UPDATE);
    const bool mom = c->momentum > 0.f;
    if (mom && split) launch_inner_update_z<true, true>(c, zm, grid, g, y, x, z, n4, wd);
    else if (mom) launch_inner_update_z<true, false>(c, zm, grid, g, y, x, z, n4, wd);
    else if (split) launch_inner_update_z<false, true>(c, zm, grid, g, y, x, z, n4, wd);
    else launch_inner_update_z<false, false>(c, zm, grid, g, y, x, z, n4, wd);
    PARLE_LAUNCHED(c);
    c->fresh = false;
    c->shadow_is_x = false;
    c->steps_in_round++;
    if (c->gemm_dtype == PARLE_GEMM_BF16 && c->n_layers > 0) PARLE_TRY(run_blocked_copy(c, c->buf.y));
    if (split) PARLE_TRY(run_split_transpose(c, c->buf.y));
    return PARLE_OK;
}

// Transposed tf32 hi/lo copy of the weights of layers >= 1 (the B operand of the data-gradient products).
int run_split_transpose(parle_ctx *c, const float *src) {
    if (c->n_layers < 2) return PARLE_OK;
    TransposePlan tp = {};
    int tiles = 0;
    for (int l = 1; l < c->n_layers; ++l) {
        const int k = l - 1;
        tp.w_off[k] = (long long)c->layers[l].w_off; tp.t_off[k] = (long long)c->t3_t_off[l];
        tp.d_in[k] = c->dims[l]; tp.d_out[k] = c->dims[l + 1]; tp.ld[k] = (int)round_up(c->dims[l + 1], 4);
        tp.tiles_in[k] = (c->dims[l] + 63) / 64;
        tp.first_tile[k] = tiles;
        tiles += tp.tiles_in[k] * ((c->dims[l + 1] + 63) / 64);
    }
    tp.n_layers = c->n_layers - 1;
    tp.first_tile[tp.n_layers] = tiles;
    prof_begin(c, KC_TO_BF16);
    split_transpose_kernel<<<dim3(tiles, c->n), 256, 0, c->stream>>>(
        tp, src, (long long)c->stride, ws_ptr<float>(c, c->ws.wT_split[0]), ws_ptr<float>(c, c->ws.wT_split[1]), (long long)c->t3_t_stride);
    PARLE_LAUNCHED(c);
    return PARLE_OK;
}

// tf32 hi/lo copies of the parameters from an fp32 vector (x at the start of a round).
int run_split_copy(parle_ctx *c, const float *src) {
    const size_t n4 = (size_t)c->n * c->stride / 4;
    prof_begin(c, KC_TO_BF16);
    split_tf32_kernel<<<stream_grid(c, n4, 1), 256, 0, c->stream>>>(
        reinterpret_cast<const float4 *>(src), ws_ptr<float4>(c, c->ws.w_split[0]), ws_ptr<float4>(c, c->ws.w_split[1]), n4);
    PARLE_LAUNCHED(c);
    return run_split_transpose(c, src);
}

// fp32 configuration on the tensor cores: every product as three tf32 products of hi/lo operand pairs.
int forward_backward_tf32(parle_ctx *c, const float *inputs, const int32_t *labels, float *loss_out) {
    const Workspace &w = c->ws;
    const int nl = c->n_layers, n = c->n, B = c->batch;
    const float *params = c->fresh ? c->buf.x : c->buf.y;      // biases come from the fp32 master copy
    const long long S = (long long)c->stride;
    {
        const int d0 = c->dims[0];
        prof_begin(c, KC_INPUT_CVT);
        input_split_kernel<<<dim3((d0 + 31) / 32, (B + 31) / 32, n), 256, 0, c->stream>>>(
            inputs, ws_ptr<float>(c, w.xs[0]), ws_ptr<float>(c, w.xs[1]), ws_ptr<float>(c, w.xT[0]), ws_ptr<float>(c, w.xT[1]), B, d0);
        PARLE_LAUNCHED(c);
    }
    for (int l = 0; l < nl; ++l) {
        const int din = c->dims[l], dout = c->dims[l + 1];
        T3Params p = {};
        p.M = B; p.N = dout; p.K = din;
        p.bias = params + c->layers[l].b_off; p.bias_gs = S;
        if (l + 1 < nl) {
            p.out_hi = ws_ptr<float>(c, w.hs[l][0]); p.out_lo = ws_ptr<float>(c, w.hs[l][1]);
            p.out_gs = (long long)B * dout; p.out_ld = dout;
            p.outT_hi = ws_ptr<float>(c, w.hT[l][0]); p.outT_lo = ws_ptr<float>(c, w.hT[l][1]);
            p.outT_gs = (long long)B * dout; p.outT_ld = B;
            PARLE_TRY(launch_t3<T3_FWD_HIDDEN>(c, KC_FWD_GEMM, c->t3_bn_fwd[l], c->t3_fa[l], c->t3_fb[l], p));
        } else {
            p.outf = ws_ptr<float>(c, w.t3_logits); p.outf_gs = (long long)B * dout; p.outf_ld = dout;
            p.ksplit = c->t3_ksplit; p.part_ss = (long long)n * B * dout;
            PARLE_TRY(launch_t3<T3_FWD_LAST>(c, KC_FWD_GEMM, c->t3_bn_fwd[l], c->t3_fa[l], c->t3_fb[l], p));
        }
    }
    const int C = c->dims[nl], rows = n * B;
    prof_begin(c, KC_SOFTMAX_CE);
    softmax_ce_backward_kernel<0><<<(rows + 7) / 8, 256, 0, c->stream>>>(
        ws_ptr<float>(c, w.t3_logits), labels, nullptr, nullptr, nullptr, ws_ptr<float>(c, w.row_loss), rows, B, C, 0,
        c->status_dev, c->t3_ksplit, (long long)n * B * C, params + c->layers[nl - 1].b_off, S,
        ws_ptr<float>(c, w.dhT[nl - 1][0]), ws_ptr<float>(c, w.dhT[nl - 1][1]),
        ws_ptr<float>(c, w.dhs[nl - 1][0]), ws_ptr<float>(c, w.dhs[nl - 1][1]), (int)round_up(C, 4),
        loss_out, ws_ptr<int>(c, w.rows_done));
    PARLE_LAUNCHED(c);
    for (int l = nl - 1; l >= 0; --l) {
        const int din = c->dims[l], dout = c->dims[l + 1];
        T3Params p = {};                                        // dW_l^T = H_{l-1}^T dH_l
        p.M = din; p.N = dout; p.K = B;
        p.outf = c->buf.grad + c->layers[l].w_off; p.outf_gs = S; p.outf_ld = din;
        PARLE_TRY(launch_t3<T3_WGRAD>(c, KC_WGRAD_GEMM, c->t3_bn_wg[l], c->t3_wa[l], c->t3_wb[l], p));
        if (l > 0) {                                            // dH_{l-1} = (dH_l W_l) * 1[H_{l-1} > 0]
            T3Params d = {};
            d.M = B; d.N = din; d.K = dout;
            d.out_hi = ws_ptr<float>(c, w.dhs[l - 1][0]); d.out_lo = ws_ptr<float>(c, w.dhs[l - 1][1]);
            d.out_gs = (long long)B * din; d.out_ld = din;      // d_in % 4 == 0: no padding
            d.outT_hi = ws_ptr<float>(c, w.dhT[l - 1][0]); d.outT_lo = ws_ptr<float>(c, w.dhT[l - 1][1]);
            d.outT_gs = (long long)B * din; d.outT_ld = B;
            d.mask_hi = ws_ptr<float>(c, w.hT[l - 1][0]);
            d.mask_gs = (long long)B * din; d.mask_ld = B;
            PARLE_TRY(launch_t3<T3_DGRAD>(c, KC_DGRAD_GEMM, c->t3_bn_dg[l], c->t3_da[l], c->t3_db[l], d));
        }
    }
    {                                                           // bias gradients of all layers: one launch
        BiasGradPlan bp = {};
        int dmax = 0;
        for (int l = 0; l < nl; ++l) {
            bp.hi[l] = ws_ptr<float>(c, w.dhT[l][0]); bp.lo[l] = ws_ptr<float>(c, w.dhT[l][1]);
            bp.b_off[l] = (long long)c->layers[l].b_off; bp.d[l] = c->dims[l + 1];
            if (c->dims[l + 1] > dmax) dmax = c->dims[l + 1];
        }
        prof_begin(c, KC_BIAS_GRAD);
        bias_grad_split_kernel<<<dim3((dmax + 7) / 8, n, nl), 256, 0, c->stream>>>(bp, c->buf.grad, S, B);
        PARLE_LAUNCHED(c);
    }
    return PARLE_OK;
}

int forward_backward_fp32(parle_ctx *c, const float *inputs, const int32_t *labels, float *loss_out) {
    const Workspace &w = c->ws;
    const int nl = c->n_layers, n = c->n, B = c->batch;
    const float *params = c->fresh ? c->buf.x : c->buf.y;      // folded reset: y == x on the first step
    const long long S = (long long)c->stride;
    for (int l = 0; l < nl; ++l) {
        const int din = c->dims[l], dout = c->dims[l + 1];
        SimtGemmArgs a = {};
        a.A = l == 0 ? inputs : ws_ptr<float>(c, w.act[l - 1]);
        a.a_gs = (long long)B * din; a.a_ms = din; a.a_ks = 1;
        a.B = params + c->layers[l].w_off; a.b_gs = S; a.b_ks = 1; a.b_ns = din;
        a.C = ws_ptr<float>(c, w.act[l]); a.c_gs = (long long)B * dout; a.ldc = dout;
        a.M = B; a.N = dout; a.K = din;
        a.bias = params + c->layers[l].b_off; a.bias_gs = S;
        if (l + 1 < nl) PARLE_TRY(launch_simt<EPI_BIAS_RELU>(c, KC_FWD_GEMM, a)); else PARLE_TRY(launch_simt<EPI_BIAS>(c, KC_FWD_GEMM, a));
    }
    const int C = c->dims[nl], rows = n * B;
    prof_begin(c, KC_SOFTMAX_CE);
    softmax_ce_backward_kernel<0><<<(rows + 7) / 8, 256, 0, c->stream>>>(
        ws_ptr<float>(c, w.act[nl - 1]), labels, ws_ptr<float>(c, w.dact[nl - 1]), nullptr, nullptr,
        ws_ptr<float>(c, w.row_loss), rows, B, C, 0, c->status_dev, 1, 0, nullptr, 0, nullptr, nullptr, nullptr, nullptr, 0,
        loss_out, ws_ptr<int>(c, w.rows_done));
    PARLE_LAUNCHED(c);
    for (int l = nl - 1; l >= 0; --l) {
        const int din = c->dims[l], dout = c->dims[l + 1];
        const float *act_in = l == 0 ? inputs : ws_ptr<float>(c, w.act[l - 1]);
        SimtGemmArgs a = {};                                    // dW_l = dH_l^T * H_{l-1}
        a.A = ws_ptr<float>(c, w.dact[l]); a.a_gs = (long long)B * dout; a.a_ms = 1; a.a_ks = dout;
        a.B = act_in; a.b_gs = (long long)B * din; a.b_ks = din; a.b_ns = 1;
        a.C = c->buf.grad + c->layers[l].w_off; a.c_gs = S; a.ldc = din;
        a.M = dout; a.N = din; a.K = B;
        PARLE_TRY(launch_simt<EPI_PLAIN>(c, KC_WGRAD_GEMM, a));
        prof_begin(c, KC_BIAS_GRAD);
        bias_grad_f32_kernel<<<dim3((dout + 255) / 256, n), 256, 0, c->stream>>>(
            ws_ptr<float>(c, w.dact[l]), c->buf.grad + c->layers[l].b_off, S, B, dout);
        PARLE_LAUNCHED(c);
        if (l > 0) {                                            // dH_{l-1} = (dH_l W_l) * 1[H_{l-1} > 0]
            SimtGemmArgs d = {};
            d.A = ws_ptr<float>(c, w.dact[l]); d.a_gs = (long long)B * dout; d.a_ms = dout; d.a_ks = 1;
            d.B = params + c->layers[l].w_off; d.b_gs = S; d.b_ks = din; d.b_ns = 1;
            d.C = ws_ptr<float>(c, w.dact[l - 1]); d.c_gs = (long long)B * din; d.ldc = din;
            d.M = B; d.N = din; d.K = dout;
            d.mask = ws_ptr<float>(c, w.act[l - 1]); d.mask_gs = (long long)B * din; d.ldmask = din;
            PARLE_TRY(launch_simt<EPI_MASK>(c, KC_DGRAD_GEMM, d));
        }
    }
    return PARLE_OK;
}

int forward_backward_bf16(parle_ctx *c, const float *inputs, const int32_t *labels, float *loss_out) {
    const Workspace &w = c->ws;
    const int nl = c->n_layers, n = c->n, B = c->batch;
    const long long S = (long long)c->stride;
    const float *params = c->fresh ? c->buf.x : c->buf.y;      // fp32 biases come from the master copy
    const bool loss_in_epilogue = c->fused_loss && c->dims[nl] <= 128;
    {
        const int d0 = c->dims[0];
        prof_begin(c, KC_INPUT_CVT);
        input_to_bf16_kernel<<<dim3((d0 + 63) / 64, (B + 63) / 64, n), 256, 0, c->stream>>>(
            inputs, ws_ptr<__nv_bfloat16>(c, w.xb), ws_ptr<__nv_bfloat16>(c, w.xbT), B, d0);
        PARLE_LAUNCHED(c);
    }
    for (int l = 0; l < nl; ++l) {
        const int din = c->dims[l], dout = c->dims[l + 1];
        if (l + 1 < nl && use_pair_gemm(c, dout)) {
            int e = l;                                          // hidden layers l .. e on pairs of SMs, chained in one launch
            while (e + 2 < nl && use_pair_gemm(c, c->dims[e + 2]) && chain_pair_gemm(c, c->dims[e + 2])) ++e;
            PARLE_TRY(launch_pair<UPE_FWD_HIDDEN>(c, KC_FWD_GEMM, l, e));
            l = e;
            continue;
        }
        UmmaParams p = {};
        p.M = B; p.N = dout; p.K = din;
        p.bias = params + c->layers[l].b_off; p.bias_gs = S;
        if (l + 1 < nl) {
            p.out = ws_ptr<__nv_bfloat16>(c, w.hb[l]); p.out_gs = (long long)B * dout; p.out_ld = dout;
            p.outT = ws_ptr<__nv_bfloat16>(c, w.hbT[l]); p.outT_gs = (long long)B * dout; p.outT_ld = B;
            PARLE_TRY((launch_umma<UEPI_FWD_HIDDEN, UB_BLOCKED_K>(c, KC_FWD_GEMM, c->tm_fwd_a[l], c->tm_fwd_b[l], p)));
        } else if (loss_in_epilogue) {
            // the last layer with the loss: logits, dlogits (both layouts), row losses and the mean loss from one kernel
            p.outf = ws_ptr<float>(c, w.logits); p.outf_gs = (long long)B * dout; p.outf_ld = dout;
            p.out = ws_ptr<__nv_bfloat16>(c, w.dhb[l]); p.out_gs = (long long)B * w.dh_ld[l]; p.out_ld = w.dh_ld[l];
            p.outT = ws_ptr<__nv_bfloat16>(c, w.dhbT[l]); p.outT_gs = (long long)B * dout; p.outT_ld = B;
            p.labels = labels; p.row_loss = ws_ptr<float>(c, w.row_loss);
            p.loss = loss_out; p.rows_done = ws_ptr<int>(c, w.rows_done);
            p.ksplit = 1;
            PARLE_TRY((launch_umma_bn<UEPI_FWD_LAST_CE, UB_BLOCKED_K, 128>(c, KC_FWD_GEMM, c->tm_fwd_a[l], c->tm_fwd_b[l], p)));
        } else {
            p.outf = ws_ptr<float>(c, w.logits); p.outf_gs = (long long)B * dout; p.outf_ld = dout;
            p.ksplit = c->last_ksplit; p.part_ss = (long long)n * B * dout;
            PARLE_TRY((launch_umma<UEPI_FWD_LAST, UB_BLOCKED_K>(c, KC_FWD_GEMM, c->tm_fwd_a[l], c->tm_fwd_b[l], p)));
        }
    }
    if (!loss_in_epilogue) {
        const int C = c->dims[nl], rows = n * B;
        prof_begin(c, KC_SOFTMAX_CE);
        // batches of a multiple of 16 rows (and rows that fit 48 KB of shared memory 16 at a time): the transposed copy
        // goes out in whole 32-byte sectors
        const bool tiled = B % 16 == 0 && (size_t)16 * C * sizeof(__nv_bfloat16) <= 48 * 1024;
        auto *kern = tiled ? softmax_ce_backward_kernel<16> : softmax_ce_backward_kernel<0>;
        kern<<<tiled ? rows / 16 : (rows + 7) / 8, 256, tiled ? (size_t)16 * C * sizeof(__nv_bfloat16) : 0, c->stream>>>(
            ws_ptr<float>(c, w.logits), labels, nullptr, ws_ptr<__nv_bfloat16>(c, w.dhb[nl - 1]),
            ws_ptr<__nv_bfloat16>(c, w.dhbT[nl - 1]), ws_ptr<float>(c, w.row_loss), rows, B, C, w.dh_ld[nl - 1],
            c->status_dev, c->last_ksplit, (long long)n * B * C, params + c->layers[nl - 1].b_off, S,
            nullptr, nullptr, nullptr, nullptr, 0, loss_out, ws_ptr<int>(c, w.rows_done));
        PARLE_LAUNCHED(c);
    }
    auto dgrad = [&](int l) -> int {                            // dH_{l-1} = (dH_l W_l) * 1[H_{l-1} > 0]
        const int din = c->dims[l], dout = c->dims[l + 1];
        if (use_pair_gemm(c, din)) return launch_pair<UPE_DGRAD>(c, KC_DGRAD_GEMM, l, l);
        UmmaParams d = {};
        d.M = B; d.N = din; d.K = dout;
        d.out = ws_ptr<__nv_bfloat16>(c, w.dhb[l - 1]); d.out_gs = (long long)B * w.dh_ld[l - 1]; d.out_ld = w.dh_ld[l - 1];
        d.outT = ws_ptr<__nv_bfloat16>(c, w.dhbT[l - 1]); d.outT_gs = (long long)B * din; d.outT_ld = B;
        d.mask = ws_ptr<__nv_bfloat16>(c, w.hb[l - 1]); d.mask_gs = (long long)B * din; d.mask_ld = din;
        return launch_umma<UEPI_DGRAD, UB_BLOCKED_MN>(c, KC_DGRAD_GEMM, c->tm_dg_a[l], c->tm_dg_b[l], d);
    };
    const bool mom = c->momentum > 0.f;
    if (!c->fused_update) {
        for (int l = nl - 1; l >= 0; --l) {
            const int din = c->dims[l], dout = c->dims[l + 1];
            UmmaParams p = {};                                  // dW_l^T = H_{l-1}^T * dH_l
            p.M = din; p.N = dout; p.K = B;
            p.outf = c->buf.grad + c->layers[l].w_off; p.outf_gs = S; p.outf_ld = din;
            PARLE_TRY((launch_umma<UEPI_WGRAD, UB_ROWMAJOR_K>(c, KC_WGRAD_GEMM, c->tm_wg_a[l], c->tm_wg_b[l], p)));
            prof_begin(c, KC_BIAS_GRAD);
            bias_grad_bf16_kernel<<<dim3((dout + 127) / 128, n), 128, 0, c->stream>>>(
                ws_ptr<__nv_bfloat16>(c, w.dhbT[l]), c->buf.grad + c->layers[l].b_off, S, B, dout);
            PARLE_LAUNCHED(c);
            if (l > 0) PARLE_TRY(dgrad(l));
        }
        return PARLE_OK;
    }
    // Fused: the weight gradient never reaches memory.  All data-gradient products go first (they read the bf16
    // weight copies that the fused kernel overwrites); then ONE launch of the fused kernel walks the W tiles of
    // every layer, so the stream of x, y, z through the SMs starts up and drains once per step, not once per layer.
    for (int l = nl - 1; l > 0; --l) {
        if (use_pair_gemm(c, c->dims[l])) {
            int e = l;                                          // data gradients of layers l, l - 1, ..., e chained in one launch
            while (e - 1 > 0 && use_pair_gemm(c, c->dims[e - 1]) && chain_pair_gemm(c, c->dims[e - 1])) --e;
            PARLE_TRY(launch_pair<UPE_DGRAD>(c, KC_DGRAD_GEMM, l, e));
            l = e;
            continue;
        }
        PARLE_TRY(dgrad(l));
    }
    WgradUpdateParams p = {};
    p.K = B; p.groups = n; p.n_layers = nl;
    int tiles = 0;
    for (int l = 0; l < nl; ++l) {
        WuLayer &ly = p.layer[l];
        ly.M = c->dims[l]; ly.N = c->dims[l + 1];
        ly.tiles_m = (ly.M + UM_BM - 1) / UM_BM; ly.tiles_n = (ly.N + UM_BN - 1) / UM_BN;
        ly.tile_begin = tiles;
        tiles += n * ly.tiles_m * ly.tiles_n;
        ly.ld = ly.M; ly.shadow_cb = c->sh_cb[l];
        ly.w_off = (long long)c->layers[l].w_off; ly.shadow_off = (long long)c->sh_off[l];
    }
    p.total_tiles = tiles;
    p.y = c->buf.y; p.z = c->buf.z;
    p.shadow = ws_ptr<__nv_bfloat16>(c, w.shadow); p.shadow_gs = (long long)c->sh_stride;
    p.gs = S;
    p.eta_p = c->eta_prime; p.inv_gamma = c->inv_gamma; p.alpha = c->alpha; p.wd = c->weight_decay;
    p.status = c->status_dev;
    p.sched = ws_ptr<int>(c, w.sched);
    const int grid = tiles < c->sm_count ? tiles : c->sm_count;
    prof_begin(c, KC_WGRAD_UPDATE);
    const int zm = c->fresh ? WU_Z_SINGLE : c->z_mode;
    if (mom) { p.v = c->vy; p.mu = c->momentum; }
    const WuMaps &maps = mom ? c->wu_maps_mom : c->wu_maps;
#define PARLE_WU_LAUNCH(FIRST, SH, MOM, ZM) do { \
        if (ys && yw) umma_wgrad_update_kernel<FIRST, SH, MOM, ZM, true, true><<<grid, SH::THREADS, SH::SMEM_BYTES, c->stream>>>(maps, p); \
        else if (ys) umma_wgrad_update_kernel<FIRST, SH, MOM, ZM, true, false><<<grid, SH::THREADS, SH::SMEM_BYTES, c->stream>>>(maps, p); \
        else umma_wgrad_update_kernel<FIRST, SH, MOM, ZM, false, false><<<grid, SH::THREADS, SH::SMEM_BYTES, c->stream>>>(maps, p); } while (0)
    const bool ys = c->y_split_step, yw = c->y_write_step;
    p.ylo = ws_ptr<uint16_t>(c, w.ylo);
    if (mom) {
        if (c->fresh) PARLE_WU_LAUNCH(true, WuMomentum, true, WU_Z_SINGLE);
        else if (zm == WU_Z_SKIP) PARLE_WU_LAUNCH(false, WuMomentum, true, WU_Z_SKIP);
        else if (zm == WU_Z_DOUBLE) PARLE_WU_LAUNCH(false, WuMomentum, true, WU_Z_DOUBLE);
        else PARLE_WU_LAUNCH(false, WuMomentum, true, WU_Z_SINGLE);
    } else {
        if (c->fresh) PARLE_WU_LAUNCH(true, WuDefault, false, WU_Z_SINGLE);
        else if (zm == WU_Z_SKIP) PARLE_WU_LAUNCH(false, WuDefault, false, WU_Z_SKIP);
        else if (zm == WU_Z_DOUBLE) PARLE_WU_LAUNCH(false, WuDefault, false, WU_Z_DOUBLE);
        else PARLE_WU_LAUNCH(false, WuDefault, false, WU_Z_SINGLE);
    }
#undef PARLE_WU_LAUNCH
    PARLE_LAUNCHED(c);
    TailPlan tp = {};
    tp.n_layers = nl; tp.batch = B;
    long long longest = 0;
    for (int l = 0; l < nl; ++l) {
        tp.begin[l] = (long long)c->layers[l].w_off + (long long)c->dims[l] * c->dims[l + 1];
        tp.b_off[l] = (long long)c->layers[l].b_off;
        tp.end[l] = l + 1 < nl ? (long long)c->layers[l + 1].w_off : (long long)c->stride;
        tp.d_out[l] = c->dims[l + 1];
        tp.dHT[l] = ws_ptr<__nv_bfloat16>(c, w.dhbT[l]);
        if (tp.end[l] - tp.begin[l] > longest) longest = tp.end[l] - tp.begin[l];
    }
    const dim3 tgrid((unsigned)((longest + 127) / 128), nl, n);
    prof_begin(c, KC_TAIL_UPDATE);
    if (mom && c->fresh)
        tail_update_kernel<true, true><<<tgrid, 128, 0, c->stream>>>(tp, c->buf.y, c->buf.z, c->buf.x, S, c->eta_prime, c->inv_gamma,
                                                                     c->alpha, c->weight_decay, c->status_dev, c->vy, c->momentum);
    else if (mom)
        tail_update_kernel<false, true><<<tgrid, 128, 0, c->stream>>>(tp, c->buf.y, c->buf.z, c->buf.x, S, c->eta_prime, c->inv_gamma,
                                                                      c->alpha, c->weight_decay, c->status_dev, c->vy, c->momentum);
    else if (c->fresh)
        tail_update_kernel<true><<<tgrid, 128, 0, c->stream>>>(tp, c->buf.y, c->buf.z, c->buf.x, S,
                                                               c->eta_prime, c->inv_gamma, c->alpha, c->weight_decay, c->status_dev);
    else
        tail_update_kernel<false><<<tgrid, 128, 0, c->stream>>>(tp, c->buf.y, c->buf.z, c->buf.x, S,
                                                                c->eta_prime, c->inv_gamma, c->alpha, c->weight_decay, c->status_dev);
    PARLE_LAUNCHED(c);
    return PARLE_OK;
}

int check_bound(const parle_ctx *c) {
    if (!c) return PARLE_EINVAL;
    if (!c->bound) return PARLE_ENOTBOUND;
    return PARLE_OK;
}

}  // namespace

// =========================================================================== C ABI
extern "C" {

int parle_init(parle_ctx **out, int n, const parle_model *model, double gamma, double rho, double alpha,
               double eta, double eta_prime) {
    if (!out) return PARLE_EINVAL;
    *out = nullptr;
    if (!model || !model->dims) return PARLE_EINVAL;
    if (n < 1 || n > PARLE_MAX_REPLICAS) return PARLE_EINVAL;
    if (model->n_layers < 0 || model->n_layers > PARLE_MAX_LAYERS) return PARLE_EINVAL;
    if (model->gemm_dtype != PARLE_GEMM_FP32 && model->gemm_dtype != PARLE_GEMM_BF16) return PARLE_EINVAL;
    if (!coupling_ok(gamma) || !coupling_ok(rho)) return PARLE_EINVAL;
    if (!(alpha >= 0.0 && alpha < 1.0)) return PARLE_EINVAL;
    if (!(eta > 0.0) || !(eta_prime > 0.0) || isinf(eta) || isinf(eta_prime)) return PARLE_EINVAL;
    for (int l = 0; l <= model->n_layers; ++l)
        if (model->dims[l] < 1) return PARLE_EINVAL;
    if (model->n_layers > 0 && model->batch < 1) return PARLE_EINVAL;
    if (model->n_layers > 0 && model->gemm_dtype == PARLE_GEMM_BF16) {
        if (model->batch % 8) return PARLE_EUNSUPPORTED;
        for (int l = 0; l < model->n_layers; ++l)
            if (model->dims[l] % 8) return PARLE_EUNSUPPORTED;
    }
    parle_ctx *c = new (std::nothrow) parle_ctx;
    if (!c) return PARLE_EINVAL;
    memset(c, 0, sizeof(*c));
    c->n = n; c->n_layers = model->n_layers; c->batch = model->n_layers ? model->batch : 0;
    c->gemm_dtype = model->gemm_dtype;
    for (int l = 0; l <= model->n_layers; ++l) c->dims[l] = model->dims[l];
    c->inv_gamma = inverse_or_zero(gamma); c->inv_rho = inverse_or_zero(rho);
    c->alpha = (float)alpha; c->eta = (float)eta; c->eta_prime = (float)eta_prime;
    size_t off = 0, P = 0;
    if (c->n_layers == 0) {
        P = (size_t)c->dims[0];
        off = round_up(P, 32);
    } else {
        for (int l = 0; l < c->n_layers; ++l) {
            LayerPlan &lp = c->layers[l];
            lp.d_in = c->dims[l]; lp.d_out = c->dims[l + 1];
            lp.w_off = off; off = round_up(off + (size_t)lp.d_in * lp.d_out, 32);
            lp.b_off = off; off = round_up(off + (size_t)lp.d_out, 32);
            P += (size_t)lp.d_in * lp.d_out + lp.d_out;
        }
    }
    c->P = P; c->stride = off;
    for (int l = 0; l < c->n_layers; ++l) {      // blocked bf16 weight copy: 128 x 64 blocks, row-block major
        c->sh_off[l] = c->sh_stride;
        c->sh_rb[l] = (c->dims[l + 1] + 127) / 128;
        c->sh_cb[l] = (c->dims[l] + 63) / 64;
        c->sh_stride += (size_t)c->sh_rb[l] * c->sh_cb[l] * 8192;
    }
    c->t3_mode = 1;
    c->t3_shapes_ok = (c->gemm_dtype == PARLE_GEMM_FP32 && c->n_layers > 0 && c->batch % 4 == 0);
    for (int l = 0; l < c->n_layers; ++l)
        if (c->dims[l] % 4) c->t3_shapes_ok = false;
    for (int l = 1; l < c->n_layers; ++l) {
        c->t3_t_off[l] = c->t3_t_stride;
        c->t3_t_stride = round_up(c->t3_t_stride + (size_t)c->dims[l] * round_up(c->dims[l + 1], 4), 32);
    }
    if (c->t3_t_stride == 0) c->t3_t_stride = 32;
    c->t3_ksplit = 1;
    if (c->t3_shapes_ok) {
        // the last forward layer usually has one tile per replica: split its k-blocks over several CTAs (partial sums,
        // added up with the bias by the softmax kernel in fixed order)
        const int nl = c->n_layers;
        const int tiles = c->n * ((c->batch + 127) / 128) * ((c->dims[nl] + 63) / 64);
        const int num_kb = (c->dims[nl - 1] + 31) / 32;
        int s = kPlanSmCount / (tiles > 0 ? tiles : 1);
        if (s > 8) s = 8;
        if (s > num_kb / 2) s = num_kb / 2;
        if (s >= 2) c->t3_ksplit = s;
    }
    c->fused_update = (c->gemm_dtype == PARLE_GEMM_BF16 && c->n_layers > 0);
    c->paired_z = true;
    c->split_y = true;
    c->wide_tiles_per_sm = 4;
    c->pair_gemm = 2;
    c->last_ksplit = 1;
    if (c->fused_update) {
        // the last forward layer often has one tile per replica: when its tiles would leave most SMs idle, its k-blocks are
        // split over several CTAs (partial sums, added up with the bias by the softmax kernel in fixed order)
        const int nl = c->n_layers;
        const int tiles = c->n * ((c->batch + 127) / 128) * ((c->dims[nl] + 127) / 128);
        const int num_kb = (c->dims[nl - 1] + 63) / 64;
        int s = kPlanSmCount / (tiles > 0 ? tiles : 1);
        if (s > 8) s = 8;
        if (s > num_kb / 2) s = num_kb / 2;
        if (s >= 2) c->last_ksplit = s;
    }
    // The loss goes into the last layer's epilogue by default only where that layer has tiles enough not to be split
    // along K: with a handful of tiles (C3: 8) one CTA per tile streaming the whole K is slower than the split GEMM plus
    // the loss kernel (measured: +25 us per inner step).
    c->fused_loss = c->fused_update && c->last_ksplit == 1 && c->dims[c->n_layers] <= 128;
    plan_workspace(c);
    *out = c;
    return PARLE_OK;
}

void parle_destroy(parle_ctx *c) {
    if (!c) return;
    if (c->status_host) cudaFreeHost(c->status_host);
    drop_round_graphs(c);
    if (c->capture_stream) cudaStreamDestroy(c->capture_stream);
    if (c->copy_ready) {
        cudaStreamDestroy(c->copy_stream);
        for (int b = 0; b < 2; ++b) { cudaEventDestroy(c->ev_copied[b]); cudaEventDestroy(c->ev_consumed[b]); }
    }
    if (c->prof_ev) {
        for (int i = 0; i < 2 * kProfCapacity; ++i) cudaEventDestroy(c->prof_ev[i]);
        delete[] c->prof_ev;
        delete[] c->prof_cls;
    }
    delete c;
}

size_t parle_param_count(const parle_ctx *c) { return c ? c->P : 0; }
size_t parle_stride(const parle_ctx *c) { return c ? c->stride : 0; }
size_t parle_workspace_bytes(const parle_ctx *c) { return c ? c->ws.total : 0; }

int parle_layer_offset(const parle_ctx *c, int layer, size_t *w_off, size_t *b_off) {
    if (!c || !w_off || !b_off || layer < 0 || layer >= c->n_layers) return PARLE_EINVAL;
    *w_off = c->layers[layer].w_off;
    *b_off = c->layers[layer].b_off;
    return PARLE_OK;
}

int parle_bind(parle_ctx *c, const parle_buffers *b, void *cuda_stream) {
    if (!c || !b) return PARLE_EINVAL;
    if (!b->x || !b->y || !b->z || !b->grad || !b->xbar || !b->workspace) return PARLE_EINVAL;
    const void *ptrs[6] = {b->x, b->y, b->z, b->grad, b->xbar, b->workspace};
    for (const void *p : ptrs)
        if (reinterpret_cast<uintptr_t>(p) % 128) return PARLE_EALIGN;
    if (b->workspace_bytes < c->ws.total) return PARLE_EWORKSPACE;
    c->bound = false;
    drop_round_graphs(c);
    int dev = 0;
    PARLE_CUDA(c, cudaGetDevice(&dev));
    PARLE_CUDA(c, cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev));
    if (!c->status_host) {
        // host memory (pinned, mapped): the one allocation the library makes
        PARLE_CUDA(c, cudaHostAlloc(reinterpret_cast<void **>(&c->status_host), SLOT_COUNT * sizeof(int), cudaHostAllocMapped));
        memset(c->status_host, 0, SLOT_COUNT * sizeof(int));
        PARLE_CUDA(c, cudaHostGetDevicePointer(reinterpret_cast<void **>(&c->status_dev), c->status_host, 0));
    }
    c->buf = *b;
    c->stream = static_cast<cudaStream_t>(cuda_stream);
    // the momentum buffers (and the tensor maps over them) belonged to the previous binding: momentum is off until
    // parle_bind_momentum and parle_set_momentum are called again
    c->momentum = 0.f; c->vy = nullptr; c->vx = nullptr; c->mom_maps = false;
    if (c->n_layers > 0 && c->gemm_dtype == PARLE_GEMM_BF16) {
        int major = 0;
        PARLE_CUDA(c, cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        if (major != 10) return PARLE_EUNSUPPORTED;             // tcgen05 kernels need sm_100
        PARLE_CUDA(c, (allow_big_smem<UEPI_FWD_HIDDEN, UB_BLOCKED_K>()));
        PARLE_CUDA(c, (allow_big_smem<UEPI_FWD_LAST, UB_BLOCKED_K>()));
        PARLE_CUDA(c, cudaFuncSetAttribute(umma_gemm_kernel<UEPI_FWD_LAST_CE, UB_BLOCKED_K, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UM_SMEM_BYTES));
        PARLE_CUDA(c, (allow_big_smem<UEPI_WGRAD, UB_ROWMAJOR_K>()));
#define PARLE_WU_SMEM(FIRST, SH, MOM, ZM) \
        PARLE_CUDA(c, cudaFuncSetAttribute(umma_wgrad_update_kernel<FIRST, SH, MOM, ZM, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SH::SMEM_BYTES)); \
        PARLE_CUDA(c, cudaFuncSetAttribute(umma_wgrad_update_kernel<FIRST, SH, MOM, ZM, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SH::SMEM_BYTES)); \
        PARLE_CUDA(c, cudaFuncSetAttribute(umma_wgrad_update_kernel<FIRST, SH, MOM, ZM, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SH::SMEM_BYTES))
        PARLE_WU_SMEM(true, WuDefault, false, WU_Z_SINGLE); PARLE_WU_SMEM(false, WuDefault, false, WU_Z_SINGLE);
        PARLE_WU_SMEM(false, WuDefault, false, WU_Z_SKIP); PARLE_WU_SMEM(false, WuDefault, false, WU_Z_DOUBLE);
        PARLE_WU_SMEM(true, WuMomentum, true, WU_Z_SINGLE); PARLE_WU_SMEM(false, WuMomentum, true, WU_Z_SINGLE);
        PARLE_WU_SMEM(false, WuMomentum, true, WU_Z_SKIP); PARLE_WU_SMEM(false, WuMomentum, true, WU_Z_DOUBLE);
#undef PARLE_WU_SMEM
        c->mom_maps = false;
        PARLE_CUDA(c, (allow_big_smem<UEPI_DGRAD, UB_BLOCKED_MN>()));
        PARLE_CUDA(c, allow_pair_smem<UPE_FWD_HIDDEN>());
        PARLE_CUDA(c, allow_pair_smem<UPE_DGRAD>());
        PARLE_TRY(build_tensor_maps(c));
        // rows / columns of the blocked weight copy beyond the matrices are never written: they must read as zero
        PARLE_CUDA(c, cudaMemsetAsync(ws_ptr<char>(c, c->ws.shadow), 0, (size_t)c->n * c->sh_stride * 2, c->stream));
        // tile counters of the fused weight-gradient kernel: every launch leaves them at zero again
        PARLE_CUDA(c, cudaMemsetAsync(ws_ptr<char>(c, c->ws.sched), 0, 2 * sizeof(int), c->stream));
        PARLE_CUDA(c, cudaMemsetAsync(ws_ptr<char>(c, c->ws.pair_sync), 0, UP_SYNC_INTS * sizeof(int), c->stream));
    }
    if (c->n_layers > 0)            // row counters of the loss kernel: every launch leaves them at zero again
        PARLE_CUDA(c, cudaMemsetAsync(ws_ptr<char>(c, c->ws.rows_done), 0, (size_t)c->n * sizeof(int), c->stream));
    c->t3_ready = false;
    if (c->t3_shapes_ok) {
        int major = 0;
        PARLE_CUDA(c, cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        if (major == 10) {                                      // other devices keep the FMA-pipe products
            PARLE_CUDA(c, allow_t3_smem<T3_FWD_HIDDEN>());
            PARLE_CUDA(c, allow_t3_smem<T3_FWD_LAST>());
            PARLE_CUDA(c, allow_t3_smem<T3_DGRAD>());
            PARLE_CUDA(c, allow_t3_smem<T3_WGRAD>());
            PARLE_TRY(build_tf32_maps(c));
            c->t3_ready = true;
        }
    }
    c->bound = true;
    c->round_open = false; c->fresh = false; c->shadow_is_x = false; c->steps_in_round = 0;
    return PARLE_OK;
}

int parle_round_begin(parle_ctx *c) {
    PARLE_TRY(check_bound(c));
    if (c->n_layers > 0 && c->gemm_dtype == PARLE_GEMM_BF16 && !c->shadow_is_x) {
        PARLE_TRY(run_blocked_copy(c, c->buf.x));
        c->shadow_is_x = true;
    }
    if (use_t3(c) && !c->shadow_is_x) {
        PARLE_TRY(run_split_copy(c, c->buf.x));
        c->shadow_is_x = true;
    }
    c->round_open = true; c->fresh = true; c->steps_in_round = 0;
    return PARLE_OK;
}

int parle_inner_step(parle_ctx *c, const float *inputs, const int32_t *labels, float *loss_out) {
    PARLE_TRY(check_bound(c));
    if (c->n_layers == 0 || !inputs || !labels) return PARLE_EINVAL;
    if (!c->round_open) return PARLE_ESTATE;
    if (c->gemm_dtype == PARLE_GEMM_BF16) {
        PARLE_TRY(forward_backward_bf16(c, inputs, labels, loss_out));
        if (c->fused_update) {            // y, z and the operand copy were updated by the backward kernels
            c->fresh = false; c->shadow_is_x = false; c->steps_in_round++;
            return PARLE_OK;
        }
    } else if (use_t3(c)) {
        PARLE_TRY(forward_backward_tf32(c, inputs, labels, loss_out));
        return run_inner_update(c, c->buf.grad, c->weight_decay, true, c->z_mode);
    } else {
        PARLE_TRY(forward_backward_fp32(c, inputs, labels, loss_out));
    }
    return run_inner_update(c, c->buf.grad, c->weight_decay, false, c->z_mode);
}

int parle_inner_step_host(parle_ctx *c, const float *inputs_host, const int32_t *labels_host, float *loss_out_host) {
    PARLE_TRY(check_bound(c));
    if (c->n_layers == 0 || !inputs_host || !labels_host) return PARLE_EINVAL;
    if (!c->round_open) return PARLE_ESTATE;
    const size_t nb = (size_t)c->n * c->batch;
    float *din = ws_ptr<float>(c, c->ws.stage_in[0]);
    int32_t *dlab = ws_ptr<int32_t>(c, c->ws.stage_lab[0]);
    float *dloss = ws_ptr<float>(c, c->ws.stage_loss[0]);
    if (c->copy_ready)      // the pipelined entry point may still own the staging buffer
        PARLE_CUDA(c, cudaStreamWaitEvent(c->stream, c->ev_consumed[0], 0));
    PARLE_CUDA(c, cudaMemcpyAsync(din, inputs_host, nb * c->dims[0] * sizeof(float), cudaMemcpyHostToDevice, c->stream));
    PARLE_CUDA(c, cudaMemcpyAsync(dlab, labels_host, nb * sizeof(int32_t), cudaMemcpyHostToDevice, c->stream));
    PARLE_TRY(parle_inner_step(c, din, dlab, loss_out_host ? dloss : nullptr));
    if (loss_out_host)
        PARLE_CUDA(c, cudaMemcpyAsync(loss_out_host, dloss, c->n * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
    return PARLE_OK;
}

int parle_inner_update(parle_ctx *c, const float *grad) {
    PARLE_TRY(check_bound(c));
    if (!grad) return PARLE_EINVAL;
    if (reinterpret_cast<uintptr_t>(grad) % 16) return PARLE_EALIGN;
    if (!c->round_open) return PARLE_ESTATE;
    // the operand copies of the active GEMM path follow y: a later parle_inner_step of the same round reads them
    return run_inner_update(c, grad, 0.f, use_t3(c));
}

int parle_outer_step(parle_ctx *c) {
    PARLE_TRY(check_bound(c));
    if (!c->round_open || c->steps_in_round == 0) return PARLE_ESTATE;
    const size_t s4 = c->stride / 4;
    const int grid = stream_grid(c, s4, 1);
    float4 *x = reinterpret_cast<float4 *>(c->buf.x), *xbar = reinterpret_cast<float4 *>(c->buf.xbar);
    const float4 *z = reinterpret_cast<const float4 *>(c->buf.z);
    prof_begin(c, KC_OUTER_MEAN);
    if (c->momentum > 0.f)
        outer_mean_kernel<4, true><<<grid, kUpdThreads, 0, c->stream>>>(
            x, z, xbar, s4, c->n, c->eta, c->eta * c->inv_rho, (float)c->n, c->status_dev,
            reinterpret_cast<float4 *>(c->vx), c->momentum, c->inv_rho);
    else
        outer_mean_kernel<4><<<grid, kUpdThreads, 0, c->stream>>>(
            x, z, xbar, s4, c->n, c->eta, c->eta * c->inv_rho, (float)c->n, c->status_dev);
    PARLE_LAUNCHED(c);
    c->shadow_is_x = false;
    c->round_open = false; c->fresh = false; c->steps_in_round = 0;
    return PARLE_OK;
}

int parle_mean(parle_ctx *c) {
    PARLE_TRY(check_bound(c));
    const size_t s4 = c->stride / 4;
    prof_begin(c, KC_MEAN);
    mean_kernel<4><<<stream_grid(c, s4, 1), kUpdThreads, 0, c->stream>>>(
        reinterpret_cast<const float4 *>(c->buf.x), reinterpret_cast<float4 *>(c->buf.xbar), s4, c->n, (float)c->n);
    PARLE_LAUNCHED(c);
    return PARLE_OK;
}

static int round_direct(parle_ctx *c, int L, const float *inputs, const int32_t *labels, float *loss_out);

static RoundKey make_round_key(const parle_ctx *c, int L, const void *in, const void *lab, const void *loss) {
    RoundKey k;
    memset(&k, 0, sizeof(k));
    k.L = L; k.inputs = in; k.labels = lab; k.loss = loss;
    const float sc[7] = {c->inv_gamma, c->inv_rho, c->alpha, c->eta, c->eta_prime, c->weight_decay, c->momentum};
    memcpy(k.scal, sc, sizeof(sc));
    k.fused = c->fused_update; k.wide_thr = c->wide_tiles_per_sm; k.shadow_is_x = c->shadow_is_x; k.fresh = c->fresh;
    k.pair_gemm = c->pair_gemm; k.fused_loss = c->fused_loss;
    k.paired_z = c->paired_z; k.z_mode = c->z_mode;
    k.split_y = c->split_y; k.y_step = (c->y_split_step ? 1 : 0) | (c->y_write_step ? 2 : 0);
    const void *pt[9] = {c->buf.x, c->buf.y, c->buf.z, c->buf.grad, c->buf.xbar, c->buf.workspace, c->vy, c->vx, c->stream};
    memcpy(k.ptrs, pt, sizeof(pt));
    return k;
}

static void restore_before(parle_ctx *c, const RoundKey &key, int L, int steps_before) {
    c->shadow_is_x = key.shadow_is_x != 0;
    c->fresh = key.fresh != 0;
    c->steps_in_round = steps_before;
    c->round_open = (L == 0);        // a round call starts with no round open, a step call inside an open round
}

static void drop_round_graphs(parle_ctx *c) {
    for (int i = 0; i < c->n_graphs; ++i) cudaGraphExecDestroy(c->graphs[i].exec);
    c->n_graphs = 0;
}

// The whole round replayed from an instantiated CUDA graph: the kernels are the same and run in the same
// order, only the per-launch host and scheduling cost goes away (one graph launch instead of ~14 L launches).
static int round_graphed(parle_ctx *c, int L, const float *inputs, const int32_t *labels, float *loss_out) {
    const RoundKey key = make_round_key(c, L, inputs, labels, loss_out);
    RoundGraph *g = nullptr;
    for (int i = 0; i < c->n_graphs; ++i)
        if (memcmp(&c->graphs[i].key, &key, sizeof(key)) == 0) g = &c->graphs[i];
    if (!g) {
        cudaGraph_t graph = nullptr;
        const long long before = c->launches;
        if (!c->capture_stream && cudaStreamCreateWithFlags(&c->capture_stream, cudaStreamNonBlocking) != cudaSuccess) {
            cudaGetLastError();
            c->capture_stream = nullptr; c->graphs_on = false;
            return L > 0 ? round_direct(c, L, inputs, labels, loss_out) : parle_inner_step(c, inputs, labels, loss_out);
        }
        if (cudaStreamBeginCapture(c->capture_stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
            cudaGetLastError();
            c->graphs_on = false;                       // capture is not possible here: plain launches from now on
            return L > 0 ? round_direct(c, L, inputs, labels, loss_out) : parle_inner_step(c, inputs, labels, loss_out);
        }
        cudaStream_t bound = c->stream;
        c->stream = c->capture_stream;                  // the launches of this one round are recorded, not run
        const int steps_before = c->steps_in_round;
        const int rc = L > 0 ? round_direct(c, L, inputs, labels, loss_out)
                             : parle_inner_step(c, inputs, labels, loss_out);
        c->stream = bound;
        const cudaError_t e = cudaStreamEndCapture(c->capture_stream, &graph);
        const long long inside = c->launches - before;
        c->launches = before;
        if (rc != PARLE_OK || e != cudaSuccess || !graph) {
            if (graph) cudaGraphDestroy(graph);
            cudaGetLastError();
            c->graphs_on = false;
            // nothing ran during the failed capture: restore the host state of before and run it plainly
            restore_before(c, key, L, steps_before);
            if (rc != PARLE_OK) return rc;
            return L > 0 ? round_direct(c, L, inputs, labels, loss_out) : parle_inner_step(c, inputs, labels, loss_out);
        }
        cudaGraphExec_t exec = nullptr;
        const cudaError_t ei = cudaGraphInstantiate(&exec, graph, 0);
        cudaGraphDestroy(graph);
        if (ei != cudaSuccess) {
            cudaGetLastError();
            c->graphs_on = false;
            restore_before(c, key, L, steps_before);
            return L > 0 ? round_direct(c, L, inputs, labels, loss_out) : parle_inner_step(c, inputs, labels, loss_out);
        }
        // the captured call advanced the host state as if it had run; rewind, the launch below replays it
        restore_before(c, key, L, steps_before);
        int slot = c->n_graphs;
        if (slot == kRoundGraphs) {                     // evict the least recently used
            slot = 0;
            for (int i = 1; i < kRoundGraphs; ++i)
                if (c->graphs[i].last_use < c->graphs[slot].last_use) slot = i;
            cudaGraphExecDestroy(c->graphs[slot].exec);
        } else {
            c->n_graphs++;
        }
        g = &c->graphs[slot];
        g->key = key; g->exec = exec; g->launches = inside;
    }
    g->last_use = ++c->graph_clock;
    PARLE_CUDA(c, cudaGraphLaunch(g->exec, c->stream));
    c->launches += g->launches;
    if (L > 0) {      // host-side state after a round (what round_direct leaves behind)
        c->round_open = false; c->fresh = false; c->steps_in_round = 0; c->shadow_is_x = false;
    } else {          // ... after one inner step
        c->fresh = false; c->shadow_is_x = false; c->steps_in_round++;
    }
    return PARLE_OK;
}

int parle_round(parle_ctx *c, int L, const float *inputs, const int32_t *labels, float *loss_out) {
    PARLE_TRY(check_bound(c));
    if (L < 1 || c->n_layers == 0 || !inputs || !labels) return PARLE_EINVAL;
    if (c->graphs_on && !c->prof_on) return round_graphed(c, L, inputs, labels, loss_out);
    return round_direct(c, L, inputs, labels, loss_out);
}

int parle_round_graph_count(const parle_ctx *c) { return c ? (c->graphs_on ? c->n_graphs : -1) : 0; }

int parle_set_round_graphs(parle_ctx *c, int on) {
    if (!c) return PARLE_EINVAL;
    c->graphs_on = on != 0;
    if (!on) drop_round_graphs(c);
    return PARLE_OK;
}

// How step l (0-based) of an L-step round treats z when Eq. (parle_z) is applied two steps at a time: the first
// step forms z from x; the remaining L - 1 steps go in (skip, two-step) pairs, with a one-step update at the end
// when L - 1 is odd.  (WU_Z_* and UPD_Z_* have the same values.)
static_assert(WU_Z_SINGLE == UPD_Z_SINGLE && WU_Z_SKIP == UPD_Z_SKIP && WU_Z_DOUBLE == UPD_Z_DOUBLE, "z modes");
static int paired_z_mode(const parle_ctx *c, int l, int L) {
    if (!c->paired_z || l == 0) return WU_Z_SINGLE;
    const int rest = L - 1, idx = l - 1;
    if ((rest & 1) && idx == rest - 1) return WU_Z_SINGLE;
    return (idx & 1) ? WU_Z_DOUBLE : WU_Z_SKIP;
}

// Whole rounds on the fused bf16 path keep the y of the weights as bf16 copy + low-half plane (the last step also
// stores the fp32 y).
static bool split_y_round(const parle_ctx *c) {
    return c->split_y && c->fused_update && c->gemm_dtype == PARLE_GEMM_BF16;
}

static int round_direct(parle_ctx *c, int L, const float *inputs, const int32_t *labels, float *loss_out) {
    PARLE_TRY(parle_round_begin(c));
    const size_t nb = (size_t)c->n * c->batch;
    for (int l = 0; l < L; ++l) {
        c->z_mode = paired_z_mode(c, l, L);
        c->y_split_step = split_y_round(c); c->y_write_step = (l == L - 1);
        const int rc = parle_inner_step(c, inputs + (size_t)l * nb * c->dims[0], labels + (size_t)l * nb,
                                        loss_out ? loss_out + (size_t)l * c->n : nullptr);
        c->z_mode = WU_Z_SINGLE; c->y_split_step = false; c->y_write_step = false;
        PARLE_TRY(rc);
    }
    return parle_outer_step(c);
}

int parle_round_host(parle_ctx *c, int L, const float *inputs_host, const int32_t *labels_host, float *loss_out_host) {
    PARLE_TRY(check_bound(c));
    if (L < 1 || c->n_layers == 0 || !inputs_host || !labels_host) return PARLE_EINVAL;
    if (!c->copy_ready) {
        PARLE_CUDA(c, cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
        for (int b = 0; b < 2; ++b) {
            PARLE_CUDA(c, cudaEventCreateWithFlags(&c->ev_copied[b], cudaEventDisableTiming));
            PARLE_CUDA(c, cudaEventCreateWithFlags(&c->ev_consumed[b], cudaEventDisableTiming));
        }
        c->copy_ready = true;
    }
    const size_t nb = (size_t)c->n * c->batch, in_elems = nb * c->dims[0];
    auto upload = [&](int l) -> int {       // minibatch l -> staging buffer l % 2, on the copy stream
        const int b = l & 1;
        PARLE_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->ev_consumed[b], 0));   // its previous user is done
        PARLE_CUDA(c, cudaMemcpyAsync(ws_ptr<float>(c, c->ws.stage_in[b]), inputs_host + (size_t)l * in_elems,
                                      in_elems * sizeof(float), cudaMemcpyHostToDevice, c->copy_stream));
        PARLE_CUDA(c, cudaMemcpyAsync(ws_ptr<int32_t>(c, c->ws.stage_lab[b]), labels_host + (size_t)l * nb,
                                      nb * sizeof(int32_t), cudaMemcpyHostToDevice, c->copy_stream));
        PARLE_CUDA(c, cudaEventRecord(c->ev_copied[b], c->copy_stream));
        return PARLE_OK;
    };
    // everything enqueued on the bound stream so far (earlier users of the staging buffers) comes first
    PARLE_CUDA(c, cudaEventRecord(c->ev_consumed[0], c->stream));
    PARLE_CUDA(c, cudaEventRecord(c->ev_consumed[1], c->stream));
    PARLE_TRY(parle_round_begin(c));
    PARLE_TRY(upload(0));
    for (int l = 0; l < L; ++l) {
        const int b = l & 1;
        if (l + 1 < L) PARLE_TRY(upload(l + 1));
        PARLE_CUDA(c, cudaStreamWaitEvent(c->stream, c->ev_copied[b], 0));
        float *dloss = ws_ptr<float>(c, c->ws.stage_loss[b]);
        c->z_mode = paired_z_mode(c, l, L);
        c->y_split_step = split_y_round(c); c->y_write_step = (l == L - 1);
        int rc;
        if (c->graphs_on && !c->prof_on)       // the step's kernels as one cached graph (staging buffers have fixed addresses)
            rc = round_graphed(c, 0, ws_ptr<float>(c, c->ws.stage_in[b]), ws_ptr<int32_t>(c, c->ws.stage_lab[b]),
                               loss_out_host ? dloss : nullptr);
        else
            rc = parle_inner_step(c, ws_ptr<float>(c, c->ws.stage_in[b]), ws_ptr<int32_t>(c, c->ws.stage_lab[b]),
                                  loss_out_host ? dloss : nullptr);
        c->z_mode = WU_Z_SINGLE; c->y_split_step = false; c->y_write_step = false;
        PARLE_TRY(rc);
        if (loss_out_host)
            PARLE_CUDA(c, cudaMemcpyAsync(loss_out_host + (size_t)l * c->n, dloss, c->n * sizeof(float),
                                          cudaMemcpyDeviceToHost, c->stream));
        PARLE_CUDA(c, cudaEventRecord(c->ev_consumed[b], c->stream));
    }
    return parle_outer_step(c);
}

int parle_set_coupling(parle_ctx *c, double gamma, double rho) {
    if (!c || !coupling_ok(gamma) || !coupling_ok(rho)) return PARLE_EINVAL;
    c->inv_gamma = inverse_or_zero(gamma); c->inv_rho = inverse_or_zero(rho);
    return PARLE_OK;
}

int parle_set_fused_update(parle_ctx *c, int on) {
    if (!c) return PARLE_EINVAL;
    if (on && !(c->gemm_dtype == PARLE_GEMM_BF16 && c->n_layers > 0)) return PARLE_EUNSUPPORTED;
    if (c->round_open && c->steps_in_round > 0) return PARLE_ESTATE;
    c->fused_update = on != 0;
    return PARLE_OK;
}

int parle_set_split_y(parle_ctx *c, int on) {
    if (!c) return PARLE_EINVAL;
    if (c->round_open) return PARLE_ESTATE;
    c->split_y = on != 0;
    return PARLE_OK;
}

int parle_set_paired_z_update(parle_ctx *c, int on) {
    if (!c) return PARLE_EINVAL;
    if (c->round_open) return PARLE_ESTATE;
    c->paired_z = on != 0;
    return PARLE_OK;
}

int parle_set_fp32_tensor_cores(parle_ctx *c, int mode) {
    if (!c || mode < 0 || mode > 2) return PARLE_EINVAL;
    if (c->gemm_dtype != PARLE_GEMM_FP32) return PARLE_EINVAL;
    if (c->round_open) return PARLE_ESTATE;       // the operand copies of a round belong to one path
    if (mode != c->t3_mode) {
        c->t3_mode = mode;
        c->shadow_is_x = false;
        drop_round_graphs(c);
    }
    return PARLE_OK;
}
int parle_fp32_tensor_cores_active(const parle_ctx *c) { return c ? (use_t3(c) ? 1 : 0) : 0; }

int parle_set_wide_tile_threshold(parle_ctx *c, int tiles_per_sm) {
    if (!c || tiles_per_sm < 0) return PARLE_EINVAL;
    c->wide_tiles_per_sm = tiles_per_sm;
    return PARLE_OK;
}

int parle_set_fused_loss(parle_ctx *c, int on) {
    if (!c) return PARLE_EINVAL;
    if (c->gemm_dtype != PARLE_GEMM_BF16 || c->n_layers == 0) return on ? PARLE_EUNSUPPORTED : PARLE_OK;
    c->fused_loss = on != 0;
    return PARLE_OK;
}

int parle_set_pair_gemm(parle_ctx *c, int mode) {
    if (!c || mode < 0 || mode > 3) return PARLE_EINVAL;
    if (c->gemm_dtype != PARLE_GEMM_BF16) return PARLE_EUNSUPPORTED;
    c->pair_gemm = mode;
    return PARLE_OK;
}

int parle_bind_momentum(parle_ctx *c, float *vy, float *vx) {
    if (!c || !vy || !vx) return PARLE_EINVAL;
    if (reinterpret_cast<uintptr_t>(vy) % 128 || reinterpret_cast<uintptr_t>(vx) % 128) return PARLE_EALIGN;
    c->vy = vy; c->vx = vx;
    c->mom_maps = false;
    if (c->bound && c->n_layers > 0 && c->gemm_dtype == PARLE_GEMM_BF16) {
        // tensor maps of the fused weight-gradient kernel's momentum variant (16-row boxes of x, y, z, vy)
        for (int l = 0; l < c->n_layers; ++l) {
            const size_t din = c->dims[l], dout = c->dims[l + 1], wo = c->layers[l].w_off;
            float *base[4] = {c->buf.x + wo, c->buf.y + wo, c->buf.z + wo, vy + wo};
            CUtensorMap *tm[4] = {&c->wu_maps_mom.x[l], &c->wu_maps_mom.y[l], &c->wu_maps_mom.z[l], &c->wu_maps_mom.v[l]};
            for (int k = 0; k < 4; ++k)
                PARLE_TRY(encode_f32_map(c, tm[k], base[k], din, dout, c->n, din, c->stride, UM_BM, WU_CHUNK_ROWS_MOM));
            c->wu_maps_mom.a[l] = c->tm_wg_a[l]; c->wu_maps_mom.b[l] = c->tm_wg_b[l];
            PARLE_TRY(encode_yhi_map(c, &c->wu_maps_mom.yhi[l], ws_ptr<__nv_bfloat16>(c, c->ws.shadow) + c->sh_off[l], c->sh_cb[l],
                                     c->sh_rb[l], c->n, c->sh_stride, WU_CHUNK_ROWS_MOM));
            PARLE_TRY(encode_ylo_map(c, &c->wu_maps_mom.ylo[l], ws_ptr<uint16_t>(c, c->ws.ylo) + wo, din, dout, c->n, din, c->stride,
                                     WU_CHUNK_ROWS_MOM));
        }
        c->mom_maps = true;
    }
    return PARLE_OK;
}

int parle_set_momentum(parle_ctx *c, double mu) {
    if (!c || !(mu >= 0.0 && mu < 1.0)) return PARLE_EINVAL;
    if (mu > 0.0 && (!c->vy || !c->vx)) return PARLE_ENOTBOUND;
    if (mu > 0.0 && c->n_layers > 0 && c->gemm_dtype == PARLE_GEMM_BF16 && !c->mom_maps)
        return PARLE_ENOTBOUND;      // momentum buffers were attached before parle_bind (or parle_bind was called again)
    if (c->round_open && c->steps_in_round > 0) return PARLE_ESTATE;
    c->momentum = (float)mu;
    return PARLE_OK;
}

int parle_scoping(double gamma0, double rho0, long long minibatches_per_epoch, long long round,
                  double gamma_floor, double rho_floor, double *gamma, double *rho) {
    if (!gamma || !rho || !(gamma0 > 0.0) || !(rho0 > 0.0) || minibatches_per_epoch < 1 || round < 0 ||
        !(gamma_floor > 0.0) || !(rho_floor > 0.0))
        return PARLE_EINVAL;
    const double f = pow(1.0 - 1.0 / (2.0 * (double)minibatches_per_epoch), (double)round);
    const double g = gamma0 * f, r = rho0 * f;
    *gamma = g < gamma_floor ? gamma_floor : g;
    *rho = r < rho_floor ? rho_floor : r;
    return PARLE_OK;
}

int parle_set_weight_decay(parle_ctx *c, double lambda) {
    if (!c || !(lambda >= 0.0) || isinf(lambda)) return PARLE_EINVAL;
    c->weight_decay = (float)lambda;
    return PARLE_OK;
}

int parle_set_lr(parle_ctx *c, double eta, double eta_prime) {
    if (!c || !(eta > 0.0) || !(eta_prime > 0.0) || isinf(eta) || isinf(eta_prime)) return PARLE_EINVAL;
    c->eta = (float)eta; c->eta_prime = (float)eta_prime;
    return PARLE_OK;
}

int parle_status(parle_ctx *c, int *device_flags) {
    if (!c || !device_flags) return PARLE_EINVAL;
    int f = 0;
    if (c->status_host) {
        volatile int *s = c->status_host;
        if (s[SLOT_NONFINITE]) f |= PARLE_FLAG_NONFINITE;
        if (s[SLOT_WAIT_LIMIT]) f |= PARLE_FLAG_WAIT_LIMIT;
        if (s[SLOT_BAD_LABEL]) f |= PARLE_FLAG_BAD_LABEL;
    }
    *device_flags = f;
    return PARLE_OK;
}

int parle_clear_status(parle_ctx *c) {
    if (!c) return PARLE_EINVAL;
    if (c->status_host) memset(c->status_host, 0, SLOT_COUNT * sizeof(int));
    return PARLE_OK;
}

int parle_profile_enable(parle_ctx *c, int on) {
    PARLE_TRY(check_bound(c));
    if (on && !c->prof_ev) {
        c->prof_ev = new (std::nothrow) cudaEvent_t[2 * kProfCapacity];
        c->prof_cls = new (std::nothrow) unsigned char[kProfCapacity];
        if (!c->prof_ev || !c->prof_cls) return PARLE_EINVAL;
        for (int i = 0; i < 2 * kProfCapacity; ++i) PARLE_CUDA(c, cudaEventCreate(&c->prof_ev[i]));
    }
    c->prof_on = on != 0;
    c->prof_open = false;
    c->prof_used = 0; c->prof_dropped = 0;
    return PARLE_OK;
}

int parle_profile_read(parle_ctx *c, int n_classes, double *ms, long long *launches, long long *dropped) {
    PARLE_TRY(check_bound(c));
    if (!ms || !launches || n_classes < 1) return PARLE_EINVAL;
    for (int k = 0; k < n_classes; ++k) { ms[k] = 0.0; launches[k] = 0; }
    PARLE_CUDA(c, cudaStreamSynchronize(c->stream));
    for (int i = 0; i < c->prof_used; ++i) {
        float t = 0.f;
        PARLE_CUDA(c, cudaEventElapsedTime(&t, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]));
        const int k = c->prof_cls[i];
        if (k < n_classes) { ms[k] += t; launches[k]++; }
    }
    if (dropped) *dropped = c->prof_dropped;
    c->prof_used = 0; c->prof_dropped = 0;
    return PARLE_OK;
}

int parle_debug_buffer(const parle_ctx *c, int kind, int layer, size_t *byte_offset, size_t *bytes) {
    if (!c || !byte_offset || !bytes || c->n_layers == 0) return PARLE_EINVAL;
    const Workspace &w = c->ws;
    const int nl = c->n_layers;
    const size_t nB = (size_t)c->n * c->batch;
    const bool bf = c->gemm_dtype == PARLE_GEMM_BF16;
    const size_t es = bf ? 2 : 4;
    if (kind == PARLE_DBG_LOGITS) {
        *byte_offset = bf ? w.logits : (use_t3(c) ? w.t3_logits : w.act[nl - 1]);
        *bytes = nB * c->dims[nl] * 4;
        return PARLE_OK;
    }
    if (kind == PARLE_DBG_OPERAND_COPY) {
        if (!bf) return PARLE_EINVAL;
        *byte_offset = w.shadow; *bytes = (size_t)c->n * c->sh_stride * 2;
        return PARLE_OK;
    }
    if (kind >= PARLE_DBG_T3_PARAMS && kind <= PARLE_DBG_T3_DACT_T + 1) {
        if (!c->t3_shapes_ok) return PARLE_EINVAL;
        const int h = (kind - PARLE_DBG_T3_PARAMS) & 1;            // 0 = hi, 1 = lo
        switch (kind - h) {
            case PARLE_DBG_T3_PARAMS: *byte_offset = w.w_split[h]; *bytes = (size_t)c->n * c->stride * 4; return PARLE_OK;
            case PARLE_DBG_T3_INPUT_T: *byte_offset = w.xT[h]; *bytes = nB * c->dims[0] * 4; return PARLE_OK;
            case PARLE_DBG_T3_ACT_T:
                if (layer < 0 || layer >= nl - 1) return PARLE_EINVAL;
                *byte_offset = w.hT[layer][h]; *bytes = nB * c->dims[layer + 1] * 4; return PARLE_OK;
            default:
                if (layer < 0 || layer >= nl) return PARLE_EINVAL;
                *byte_offset = w.dhT[layer][h]; *bytes = nB * c->dims[layer + 1] * 4; return PARLE_OK;
        }
    }
    if (layer < 0 || layer >= nl) return PARLE_EINVAL;
    const size_t d = c->dims[layer + 1];
    switch (kind) {
        case PARLE_DBG_ACT:
            if (layer == nl - 1) return PARLE_EINVAL;
            *byte_offset = bf ? w.hb[layer] : w.act[layer]; *bytes = nB * d * es; return PARLE_OK;
        case PARLE_DBG_ACT_T:
            if (!bf || layer == nl - 1) return PARLE_EINVAL;
            *byte_offset = w.hbT[layer]; *bytes = nB * d * 2; return PARLE_OK;
        case PARLE_DBG_DACT:
            *byte_offset = bf ? w.dhb[layer] : w.dact[layer];
            *bytes = bf ? nB * (size_t)w.dh_ld[layer] * 2 : nB * d * 4; return PARLE_OK;
        case PARLE_DBG_DACT_T:
            if (!bf) return PARLE_EINVAL;
            *byte_offset = w.dhbT[layer]; *bytes = nB * d * 2; return PARLE_OK;
        default: return PARLE_EINVAL;
    }
}

int parle_profile_class_count(void) { return KC_COUNT; }
const char *parle_profile_class_name(int k) { return (k >= 0 && k < KC_COUNT) ? kClassNames[k] : ""; }

long long parle_launch_count(const parle_ctx *c) { return c ? c->launches : 0; }
int parle_last_cuda_error(const parle_ctx *c) { return c ? c->last_cuda : 0; }

const char *parle_strerror(int code) {
    switch (code) {
        case PARLE_OK: return "ok";
        case PARLE_EINVAL: return "invalid argument";
        case PARLE_ENOTBOUND: return "buffers not bound";
        case PARLE_EALIGN: return "buffer not 128-byte aligned";
        case PARLE_ECUDA: return "CUDA error";
        case PARLE_ESTATE: return "call out of order";
        case PARLE_EWORKSPACE: return "workspace too small";
        case PARLE_EUNSUPPORTED: return "shape or device not supported by this GEMM path";
        case PARLE_ETOOBIG: return "size exceeds the fixed capacity of this allocation-free entry point";
        default: return "unknown error";
    }
}

}  // extern "C"
