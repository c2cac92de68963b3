/*
 * parle.h -- C ABI of the single-GPU Parle round (arXiv 1707.00424, Section 3).
 *
 * One Parle round over n replicas of an MLP:
 *     reset   y^a <- x^a, z^a <- x^a                                  (Section 3, text after Eq. parle)
 *     L times y^a <- y^a - eta' [ grad f(y^a) + (y^a - x^a)/gamma ]   (Eq. parle_y)
 *             z^a <- alpha z^a + (1 - alpha) y^a                      (Eq. parle_z)
 *     once    x^a <- x^a - eta (x^a - z^a) - (eta/rho)(x^a - xbar)    (Eq. parle_xa)
 *             xbar <- (1/n) sum_a x^a                                  (Eq. parle_x with eta'' = rho/n, Section 3.1)
 * grad f is the minibatch gradient of the mean softmax cross-entropy of a
 * ReLU MLP (Section 1.1 / 2.1).
 *
 * General rules
 *   - Every function returns PARLE_OK (0) or a negative PARLE_E* code; nothing
 *     throws, aborts or synchronises the host.  All device work is enqueued on
 *     the stream given to parle_bind(); results are valid once the caller has
 *     synchronised that stream.
 *   - The library allocates no device memory.  All state and scratch buffers
 *     are device pointers owned by the caller (parle_buffers).  The context
 *     itself is host memory owned by the library (freed by parle_destroy).
 *   - Pointers marked "dev" are device pointers, "host" are host pointers.
 *   - Parameter vectors are fp32, laid out [n, stride]: replica a starts at
 *     element a*stride.  Inside one replica the packing is
 *         [ W_1 | b_1 | W_2 | b_2 | ... ],   W_l row-major [d_l, d_{l-1}],
 *     each segment starting at a multiple of 32 elements (128 bytes); the
 *     padding elements must be zero in x and stay zero.  parle_layer_offset()
 *     reports the offsets.  With n_layers == 0 the vector has no structure
 *     (dims[0] elements): only the update entry points can be used.
 */
#ifndef PARLE_H
#define PARLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PARLE_OK            0
#define PARLE_EINVAL       -1   /* bad argument (n, dims, batch, alpha not in [0,1), gamma/rho/eta <= 0, NULL) */
#define PARLE_ENOTBOUND    -2   /* parle_bind() has not been called */
#define PARLE_EALIGN       -3   /* a buffer is not 128-byte aligned */
#define PARLE_ECUDA        -4   /* a CUDA call failed; parle_last_cuda_error() has the code */
#define PARLE_ESTATE       -5   /* call out of order (e.g. inner step before parle_round_begin) */
#define PARLE_EWORKSPACE   -6   /* workspace smaller than parle_workspace_bytes() */
#define PARLE_EUNSUPPORTED -7   /* shape not supported by the requested GEMM path */
#define PARLE_ETOOBIG      -8   /* size beyond the fixed capacity of an allocation-free entry point */

/* bits of the device status word, see parle_status() */
#define PARLE_FLAG_NONFINITE   1   /* an update kernel produced a NaN or Inf */
#define PARLE_FLAG_WAIT_LIMIT  2   /* a bounded wait inside a GEMM pipeline gave up */
#define PARLE_FLAG_BAD_LABEL   4   /* a label outside [0, d_last) was seen (treated as no target) */

#define PARLE_GEMM_FP32 0   /* fp32 operands, fp32 FMA accumulation */
#define PARLE_GEMM_BF16 1   /* bf16 operands on the tcgen05 tensor cores, fp32 accumulation;
                               needs batch % 8 == 0 and every d_l % 8 == 0 except the last.
                               Weights are rounded to bf16 to nearest with ties away from zero,
                               activations and their gradients to nearest with ties to even */

#define PARLE_MAX_LAYERS 16
#define PARLE_MAX_REPLICAS 64

typedef struct parle_ctx parle_ctx;      /* opaque; host memory owned by the library */

typedef struct {
    int n_layers;        /* number of affine layers (0: flat vector mode)                 */
    const int *dims;     /* host, n_layers+1 entries d_0 ... d_last (copied by parle_init) */
    int batch;           /* minibatch size B per replica (ignored when n_layers == 0)      */
    int gemm_dtype;      /* PARLE_GEMM_FP32 or PARLE_GEMM_BF16                             */
} parle_model;

typedef struct {
    float *x;            /* dev [n, stride]  replicas x^a (in/out)                    */
    float *y;            /* dev [n, stride]  inner iterates y^a                       */
    float *z;            /* dev [n, stride]  exponential averages z^a                 */
    float *grad;         /* dev [n, stride]  minibatch gradient, same packing         */
    float *xbar;         /* dev [stride]     reference variable (in/out)              */
    void  *workspace;    /* dev, >= parle_workspace_bytes(); contents are scratch     */
    size_t workspace_bytes;
} parle_buffers;

/* Create a context for n replicas (Section 3: a <= n) of `model`, with the
 * scalars of Eq. (parle).  gamma and rho may be +INFINITY, which switches the
 * corresponding coupling off (1/gamma = 0 or 1/rho = 0 exactly).
 * EINVAL: out == NULL, n outside [1, PARLE_MAX_REPLICAS], bad dims/batch,
 * alpha outside [0,1), gamma <= 0, rho <= 0, eta <= 0, eta_prime <= 0.
 * EUNSUPPORTED: PARLE_GEMM_BF16 with shapes it cannot take. */
int parle_init(parle_ctx **out, int n, const parle_model *model,
               double gamma, double rho, double alpha, double eta, double eta_prime);

/* Free the context (host memory only; caller buffers are untouched). NULL ok. */
void parle_destroy(parle_ctx *ctx);

/* Number of real parameters P of one replica, and the padded length `stride`
 * (>= P, multiple of 32) of one replica's vector.  0 if ctx is NULL. */
size_t parle_param_count(const parle_ctx *ctx);
size_t parle_stride(const parle_ctx *ctx);

/* Bytes of scratch the caller must provide in parle_buffers.workspace. */
size_t parle_workspace_bytes(const parle_ctx *ctx);

/* Element offsets of W_layer and b_layer inside one replica's vector
 * (layer in [0, n_layers)).  EINVAL for a bad layer or NULL output. */
int parle_layer_offset(const parle_ctx *ctx, int layer, size_t *w_off, size_t *b_off);

/* Attach the caller's device buffers and CUDA stream (a cudaStream_t passed as
 * void*, NULL = default stream).  The context keeps the pointers, not copies.
 * Must be called with the buffers' device current.  EALIGN if a pointer is not
 * 128-byte aligned, EWORKSPACE if the workspace is too small, EINVAL on NULL.
 * After binding, x and xbar hold the caller's initial state; x must not be
 * modified behind the library's back without binding again. */
int parle_bind(parle_ctx *ctx, const parle_buffers *buffers, void *cuda_stream);

/* Start a round: y^a <- x^a and z^a <- x^a (text after Eq. parle).  The copy is
 * folded into the first inner step of the round, which reads x^a in place of
 * y^a and z^a; y and z hold the round's values from that step on. */
int parle_round_begin(parle_ctx *ctx);

/* One inner step for all replicas: forward/backward of the MLP on each
 * replica's own minibatch at y^a (Section 2.1), then Eq. (parle_y), (parle_z).
 *   inputs  dev [n, B, d_0] fp32, labels dev [n, B] int32 in [0, d_last)
 *   loss_out dev [n] fp32 or NULL: mean cross-entropy of each replica's batch
 * ESTATE if no round is open; EINVAL in flat vector mode. */
int parle_inner_step(parle_ctx *ctx, const float *inputs, const int32_t *labels,
                     float *loss_out);

/* Same step with host buffers: inputs/labels are copied to the device and the
 * losses copied back on the bound stream (asynchronously if the host memory is
 * pinned).  loss_out_host may be NULL. */
int parle_inner_step_host(parle_ctx *ctx, const float *inputs_host,
                          const int32_t *labels_host, float *loss_out_host);

/* Eq. (parle_y), (parle_z) only, from a caller-supplied gradient
 * grad dev [n, stride] (may be the bound grad buffer).  Reads grad, y, x, z
 * once and writes y, z once. */
int parle_inner_update(parle_ctx *ctx, const float *grad);

/* Eq. (parle_xa) for every replica, using the xbar left by the previous mean,
 * and -- fused in the same pass -- the new replica mean written to xbar
 * (Eq. parle_x with eta'' = rho/n).  Closes the round.  ESTATE if the round
 * had no inner step. */
int parle_outer_step(parle_ctx *ctx);

/* xbar <- (1/n) sum_a x^a (Eq. parle_x, Section 3.1).  After parle_outer_step
 * this recomputes the same values; use it after writing x directly. */
int parle_mean(parle_ctx *ctx);

/* A whole round in one call: parle_round_begin, L inner steps on
 * inputs dev [L, n, B, d_0] / labels dev [L, n, B], parle_outer_step.
 * loss_out dev [L, n] or NULL. */
int parle_round(parle_ctx *ctx, int L, const float *inputs, const int32_t *labels,
                float *loss_out);

/* on: parle_round replays the round from a CUDA graph.  The first call with a given (L, inputs, labels, loss_out)
 * and unchanged settings records the round's launches on a stream of the library's own (created at that
 * moment) and instantiates them; later calls with the same arguments launch the graph on the bound stream: same kernels, same order, same results, without the per-launch cost.  Up to eight graphs are cached
 * (least recently used is dropped); changing a setting, the buffers or the stream makes a new graph.  Off by
 * default.  parle_round_host then replays each inner step from a graph of its own (its staging buffers have
 * fixed addresses).  Ignored while per-kernel timing is enabled.  If the stream cannot be captured the library falls
 * back to plain launches by itself. */
int parle_set_round_graphs(parle_ctx *ctx, int on);
/* Number of round graphs currently cached; -1 when graph replay is off (never switched on, or given up). */
int parle_round_graph_count(const parle_ctx *ctx);

/* A whole round from host buffers: inputs host [L, n, B, d_0], labels host
 * [L, n, B], loss_out host [L, n] or NULL.  The minibatch of step l+1 is uploaded
 * on a second stream into a second staging buffer while step l computes, so with
 * pinned host memory the copies hide behind the kernels.  The first call creates
 * that stream and four events (no device memory).  Results (and loss_out) are
 * valid once the bound stream has been synchronised; the host buffers must stay
 * untouched until then. */
int parle_round_host(parle_ctx *ctx, int L, const float *inputs_host, const int32_t *labels_host,
                     float *loss_out_host);

/* bf16 path only.  on (the default): Eq. (parle_y), (parle_z) are applied
 * inside the weight-gradient GEMM's epilogue, so the weight gradient is never
 * written and `grad` is left untouched by parle_inner_step.  off: the gradient is
 * written to `grad` and a separate update kernel follows (same results up to
 * fp32 rounding).  EUNSUPPORTED on the fp32 path, ESTATE in the middle of a round. */
int parle_set_fused_update(parle_ctx *ctx, int on);

/* Whole rounds only (parle_round, parle_round_host).  on (the default): z^a, which
 * only the outer step reads, is updated every other inner step, with Eq. (parle_z) applied twice at once,
 *     z_{k+2} = alpha^2 z_k + (1 - alpha) (alpha y_{k+1} + y_{k+2}),
 * from the two y values the step's kernel holds anyway; the first step of a round and, when L is even, the last
 * one use the one-step form.  The same recurrence, so z and x^a agree with the step-by-step form to fp32 rounding
 * (not bit for bit); y^a is unchanged.  It saves the read and the write of z on half of the steps (8 of the 22 bytes
 * per weight of the fused bf16 kernel, 8 of the 24 of the separate update kernel).  parle_inner_step and
 * parle_inner_update always apply the one-step form: z is current after every call.
 * off: every step of a round updates z.  ESTATE inside a round. */
int parle_set_paired_z_update(parle_ctx *ctx, int on);

/* bf16 path with the fused update, whole rounds only (parle_round, parle_round_host).  on (the default): between the
 * first and the last inner step of a round the y^a of the weights is not kept as fp32 words but as two 16-bit planes:
 * the upper and the lower half of (fp32 word + 0x8000).  The upper half is the bf16 operand copy the GEMMs read (y
 * rounded to nearest, ties away from zero -- the rounding every weight copy of this library uses), the lower half lives
 * in the workspace; ((upper << 16) | lower) - 0x8000 is the fp32 word again, exactly.  So y moves as 2 + 2 bytes with no
 * separate operand copy to write (12 / 20 instead of 14 / 22 bytes per weight and step), and every result is bit for bit
 * what the fp32 form gives.  The last step of the round stores the fp32 y^a again, so y is current when the call
 * returns.  Biases are not affected.  off: y^a is read and written as fp32 at every step.  ESTATE inside a round. */
int parle_set_split_y(parle_ctx *ctx, int on);

/* fp32 configurations only: where the forward / backward products run (Section 1.1 / 2.1, the minibatch
 * gradient).  On an sm_100 device, when the batch and every layer's input width are multiples of 4, they can
 * run on the tensor cores at fp32 accuracy: every fp32 operand is kept as a pair of tf32-exact arrays
 * (hi = the value rounded to tf32, lo = the remainder rounded to tf32) in the workspace and every product is the
 * sum of three tf32 products (lo x hi, hi x lo, hi x hi) with fp32 accumulation; the dropped lo x lo term is
 * 2^-22 relative.  mode 0: always the FMA pipes; 1 (default): tensor cores when the batch has at least 32 rows
 * and every layer's input is at least 128 wide; 2: tensor cores whenever the shapes allow.  The two paths
 * agree to fp32 rounding, not bit for bit.  EINVAL on a bf16 context, ESTATE inside a round.
 * parle_fp32_tensor_cores_active: 1 if the bound context currently uses the tensor-core path. */
int parle_set_fp32_tensor_cores(parle_ctx *ctx, int mode);
int parle_fp32_tensor_cores_active(const parle_ctx *ctx);

/* Change gamma, rho (Eq. scoping changes them between rounds) or the step
 * sizes eta, eta' between calls.  +INFINITY allowed for gamma and rho. */
int parle_set_coupling(parle_ctx *ctx, double gamma, double rho);
int parle_set_lr(parle_ctx *ctx, double eta, double eta_prime);

/* Tuning knob of the bf16 forward / data-gradient GEMMs: tiles of 128 x 256 instead of 128 x 128 are used
 * when the batch has at least 256 rows and at least `tiles_per_sm` wide tiles fall on every SM (default 4;
 * 0 = whenever the batch allows), and also where the 128-wide tiling needs more than one pass over the SMs
 * while the wide one fits in a single, mostly full pass (this second rule is off for values above 1024, which
 * therefore keep every product on 128-wide tiles).  Results do not depend on it beyond fp32 summation order
 * inside a tile (none: the k order is the same). */
int parle_set_wide_tile_threshold(parle_ctx *ctx, int tiles_per_sm);

/* bf16 path, networks with at most 128 classes.  on (the default where the last layer has enough tiles to run without a
 * split along K; with a few tiles only, as in an 8-replica batch-128 workload, the split GEMM followed by the loss kernel
 * is faster and stays the default): the softmax cross-entropy backward of Section 1.1's
 * loss runs in the epilogue of the last forward layer's GEMM (a logit row lies in one tile: the two warps that hold its
 * halves exchange maximum, sum and label logit), which also writes the row losses and the replicas' mean losses; the
 * layer is then not split along K.  off, or more classes: a kernel of its own after the GEMM.  The two agree to fp32
 * rounding (different summation order of the exponentials).  EUNSUPPORTED on an fp32 context. */
int parle_set_fused_loss(parle_ctx *ctx, int on);

/* bf16 path: forward and data-gradient products of the hidden layers (Section 1.1 / 2.1) whose weight matrix has at
 * least 256 output rows run on pairs of SMs (one two-CTA tensor-core instruction per 256 x batch-tile block, the two CTAs
 * sharing the activation tile).  Consecutive such layers can go into ONE launch, whose tiles wait, per replica, for the
 * layer before them (progress counters in the workspace; the weights of a tile are fetched while it waits).  mode 3:
 * always chained; 2 (the default): chained where a layer gives a pair of SMs at most two tiles (the case in which a
 * launch per layer leaves its start-up and epilogue exposed); 1: one launch per layer; 0: the one-SM kernel for every
 * product.  Same products, same reduction order: the
 * results do not depend on the mode.  EINVAL for another mode, EUNSUPPORTED on an fp32 context.  A chained launch whose
 * wait ran out (PARLE_FLAG_WAIT_LIMIT) may leave its counters non-zero: bind again before the next step. */
int parle_set_pair_gemm(parle_ctx *ctx, int mode);

/* Nesterov momentum on the y^a and x^a steps (Remark in Section 3.1; none on xbar).  The paper does not
 * print the form; the one taken is that of SGD with Nesterov momentum: for a step with direction d and
 * step size s,  v <- mu v + d,  p <- p - s (d + mu v), with
 *   y^a: d = grad f(y) + (y - x^a)/gamma, s = eta', v = vy, which restarts from 0 in every round with y;
 *   x^a: d = (x^a - z^a) + (x^a - xbar)/rho, s = eta, v = vx, which carries over between rounds.
 * parle_bind_momentum attaches the two caller-owned buffers, dev [n, stride] fp32, 128-byte aligned;
 * vx must be zero before the first round (vy needs no initialisation).  parle_set_momentum(mu), mu in
 * [0, 1): 0 switches momentum off; ENOTBOUND if mu > 0 without buffers, ESTATE in the middle of a round.
 * Call parle_bind_momentum after parle_bind.  A later parle_bind detaches the momentum buffers and sets mu back to 0:
 * call parle_bind_momentum and parle_set_momentum again after it.  On the bf16 path the
 * fused weight-gradient kernel has a momentum variant (vy is staged with x, y, z: 30 bytes per weight and step). */
int parle_bind_momentum(parle_ctx *ctx, float *vy, float *vx);
int parle_set_momentum(parle_ctx *ctx, double mu);

/* Scoping (Eq. scoping, Section 3.1): gamma and rho of round number `round` = floor(k / L),
 *   gamma = gamma0 (1 - 1/(2B))^round,  rho = rho0 (1 - 1/(2B))^round,   B = minibatches in the dataset,
 * clipped from below at gamma_floor and rho_floor (the paper: gamma0 = 100, rho0 = 1, floors 1 and 0.1).
 * Pure host arithmetic; feed the result to parle_set_coupling before the round.  gamma, rho: host pointers. */
int parle_scoping(double gamma0, double rho0, long long minibatches_per_epoch, long long round,
                  double gamma_floor, double rho_floor, double *gamma, double *rho);

/* Weight-decay regulariser of f (Section 1.1 allows f a regularisation term and names weight decay):
 * parle_inner_step uses grad f(y) + lambda * y in Eq. (parle_y), for every parameter.  Default 0.
 * loss_out stays the data term alone.  parle_inner_update applies its gradient argument as given. */
int parle_set_weight_decay(parle_ctx *ctx, double lambda);

/* Non-blocking read of the device status word (PARLE_FLAG_* bits) set by the
 * kernels launched so far; clears nothing.  parle_clear_status resets it. */
int parle_status(parle_ctx *ctx, int *device_flags);
int parle_clear_status(parle_ctx *ctx);

/* Per-kernel-class device timing.  While enabled, every kernel launch is
 * bracketed by a pair of CUDA events on the bound stream (at most 65536
 * launches between two reads; later ones are counted in *dropped).
 * parle_profile_read is the one call that synchronises the stream: it then
 * sums the elapsed times per class into ms[k] / launches[k] for
 * k < n_classes (arrays in host memory) and restarts the recording.
 * Class names: parle_profile_class_name(k), k < parle_profile_class_count(). */
int parle_profile_enable(parle_ctx *ctx, int on);
int parle_profile_read(parle_ctx *ctx, int n_classes, double *ms, long long *launches, long long *dropped);
int parle_profile_class_count(void);
const char *parle_profile_class_name(int k);

/* Diagnostics: where, inside the caller's workspace, the last inner step left
 * its intermediates (valid until the next call that launches work).
 *   PARLE_DBG_ACT     output of hidden layer `layer`   [n, B, d]   fp32 (fp32 path) or bf16 (bf16 path)
 *   PARLE_DBG_ACT_T   its transposed copy (bf16 path)  [n, d, B]   bf16
 *   PARLE_DBG_DACT    gradient w.r.t. layer's output   [n, B, ld]  fp32 (ld = d) or bf16 (ld = d rounded up to 8)
 *   PARLE_DBG_DACT_T  its transposed copy (bf16 path)  [n, d, B]   bf16
 *   PARLE_DBG_LOGITS  logits                            [n, B, d_last] fp32   (layer ignored)
 *   PARLE_DBG_OPERAND_COPY  bf16 copy of the weights the GEMMs read, stored per layer in 128-row x 64-column
 *                           blocks (row-block major), [n, bytes/(2n)] (bf16 path; layer ignored)
 * fp32 configurations whose shapes allow the tensor-core path hold tf32-exact hi/lo pairs (kind = hi, kind + 1 = lo):
 *   PARLE_DBG_T3_PARAMS   the parameters the products read     [n, stride] fp32   (layer ignored)
 *   PARLE_DBG_T3_INPUT_T  the minibatch, transposed            [n, d_0, B] fp32   (layer ignored)
 *   PARLE_DBG_T3_ACT_T    output of `layer`, transposed        [n, d, B]   fp32   (not for the last layer)
 *   PARLE_DBG_T3_DACT_T   gradient w.r.t. it, transposed       [n, d, B]   fp32
 * EINVAL if that buffer does not exist in this configuration. */
#define PARLE_DBG_T3_PARAMS 6
#define PARLE_DBG_T3_INPUT_T 8
#define PARLE_DBG_T3_ACT_T 10
#define PARLE_DBG_T3_DACT_T 12
#define PARLE_DBG_ACT 0
#define PARLE_DBG_ACT_T 1
#define PARLE_DBG_DACT 2
#define PARLE_DBG_DACT_T 3
#define PARLE_DBG_LOGITS 4
#define PARLE_DBG_OPERAND_COPY 5
int parle_debug_buffer(const parle_ctx *ctx, int kind, int layer, size_t *byte_offset, size_t *bytes);

/* Allocation-free loss step (the paper has no counterpart: this is a packaging
 * variant of the loss part of parle_inner_step, not a step of the method).
 *
 * Who it is for: callers that can neither allocate device memory nor hand the
 * library a workspace -- a plug-in running inside another framework's fixed
 * memory pool, a component whose device memory budget was fully assigned at
 * start-up, code on a path where calling the device allocator is forbidden
 * (it may synchronise or fail).  Such a caller still owns its inputs and outputs.
 *
 * What it does: for n replicas with B rows each, row-wise softmax cross-entropy
 *   dlogits[r, :] = (softmax(logits[r, :]) - onehot(labels[r])) / B,   loss[a] = mean over replica a's rows,
 * exactly the kernels parle_inner_step runs after the last layer.
 *   logits  dev [n*B, C] fp32 (in)     labels dev [n*B] int32 (in)
 *   dlogits dev [n*B, C] fp32 (out)    loss   dev [n] fp32 (out)
 *   flags   dev [1] int32 (out) or NULL: non-zero if a label was outside [0, C)
 * The per-row losses, which parle_inner_step keeps in the caller's workspace,
 * live here in a fixed array inside the library image: PARLE_STATIC_LOSS_MAX_ROWS
 * floats + 256 bytes (about 256 KiB), present on every GPU that loads the library
 * until the process exits.  n*B beyond that limit returns PARLE_ETOOBIG.
 * The function calls no device allocator of any kind.
 *
 * The first call on each device looks up the array's device address (with that
 * device current) and keeps it; make that first call before starting any stream
 * capture.  All calls on a device share the one array: it keeps the previous
 * call's contents (the flag slots are cleared at the start of every call), and
 * two calls whose work overlaps on the GPU (different streams, no ordering) race.
 * Work is enqueued on cuda_stream (cudaStream_t as void*, NULL = default). */
#define PARLE_STATIC_LOSS_MAX_ROWS 65536
int parle_softmax_ce_static(const float *logits, const int32_t *labels, int n, int B, int C,
                            float *dlogits, float *loss, int32_t *flags, void *cuda_stream);

/* Kernels launched by this context since creation (for accounting). */
long long parle_launch_count(const parle_ctx *ctx);

/* Last CUDA error code recorded by a call that returned PARLE_ECUDA. */
int parle_last_cuda_error(const parle_ctx *ctx);

/* Static string for a PARLE_* code. */
const char *parle_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* PARLE_H */
