// fp32 path of the replica-batched MLP forward/backward (Section 1.1 / 2.1:
// minibatch gradient of the mean cross-entropy): a strided, replica-grouped
// SGEMM on the FMA pipes with fused bias / ReLU / ReLU-mask epilogues, the
// softmax cross-entropy backward, and the bias gradient (column sums).
#pragma once

#include "common.cuh"

namespace parle {

enum SimtEpilogue { EPI_PLAIN = 0, EPI_BIAS = 1, EPI_BIAS_RELU = 2, EPI_MASK = 3 };

struct SimtGemmArgs {
    const float *A, *B;
    float *C;
    long long a_gs, b_gs, c_gs;        // per-replica strides (elements)
    int M, N, K;
    long long a_ms, a_ks;              // A(m,k) = A[m*a_ms + k*a_ks]
    long long b_ks, b_ns;              // B(k,n) = B[k*b_ks + n*b_ns]
    int ldc;
    const float *bias; long long bias_gs;          // EPI_BIAS*: bias[n]
    const float *mask; long long mask_gs; int ldmask;   // EPI_MASK: C *= (mask[m,n] > 0)
};

constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 16, SG_THREADS = 256;

// C[g] = A[g] * B[g] for every replica g = blockIdx.z; 64x64 tile per CTA, 4x4 per thread.
template <int EPI>
__global__ void __launch_bounds__(SG_THREADS) simt_gemm_kernel(SimtGemmArgs p) {
    __shared__ float As[SG_BK][SG_BM + 4];
    __shared__ float Bs[SG_BK][SG_BN + 4];
    const int g = blockIdx.z;
    const float *A = p.A + (long long)g * p.a_gs;
    const float *B = p.B + (long long)g * p.b_gs;
    float *C = p.C + (long long)g * p.c_gs;
    const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
    const int t = threadIdx.x, tx = t % 16, ty = t / 16;
    const bool a_kfast = (p.a_ks == 1), b_kfast = (p.b_ks == 1);
    float acc[4][4] = {};
    for (int k0 = 0; k0 < p.K; k0 += SG_BK) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = t + i * SG_THREADS;
            int mm, kk;
            if (a_kfast) { kk = e % SG_BK; mm = e / SG_BK; } else { mm = e % SG_BM; kk = e / SG_BM; }
            const int m = m0 + mm, k = k0 + kk;
            As[kk][mm] = (m < p.M && k < p.K) ? A[(long long)m * p.a_ms + (long long)k * p.a_ks] : 0.f;
            int nn, kb;
            if (b_kfast) { kb = e % SG_BK; nn = e / SG_BK; } else { nn = e % SG_BN; kb = e / SG_BN; }
            const int n = n0 + nn, k2 = k0 + kb;
            Bs[kb][nn] = (n < p.N && k2 < p.K) ? B[(long long)k2 * p.b_ks + (long long)n * p.b_ns] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < SG_BK; ++kk) {
            const float4 a = *reinterpret_cast<const float4 *>(&As[kk][ty * 4]);
            const float4 b = *reinterpret_cast<const float4 *>(&Bs[kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
    const float *bias = (EPI == EPI_BIAS || EPI == EPI_BIAS_RELU) ? p.bias + (long long)g * p.bias_gs : nullptr;
    const float *mask = (EPI == EPI_MASK) ? p.mask + (long long)g * p.mask_gs : nullptr;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= p.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= p.N) continue;
            float v = acc[i][j];
            if (EPI == EPI_BIAS || EPI == EPI_BIAS_RELU) v += bias[n];
            if (EPI == EPI_BIAS_RELU) v = fmaxf(v, 0.f);
            if (EPI == EPI_MASK) v = (mask[(long long)m * p.ldmask + n] > 0.f) ? v : 0.f;
            C[(long long)m * p.ldc + n] = v;
        }
    }
}

// ---------------------------------------------------------------- register-tiled SGEMM (larger problems)
// Same product, same epilogues and the same summation order (every output sums its K products in
// ascending k with one fused multiply-add each, so results are bit-identical to simt_gemm_kernel),
// but 8 x 8 outputs per thread, 16-byte shared-memory reads that a half-warp makes from one
// contiguous run, 16-byte global loads where the operand's layout allows, and the next k-block
// fetched into registers while the current one is multiplied (two shared-memory buffers, one
// barrier per k-block).  The FMA pipes are the bound: 64 FMAs per 4 shared-memory reads.
constexpr int ST_BK = 16;

// One operand tile X(r, k) = X[r * rs + k * ks], rows r0 .. r0 + ROWS - 1, k-block k0 .. k0 + 15,
// as ROWS * 16 / 4 four-element units dealt round-robin to the threads.  A unit runs along k when
// ks == 1 ("k-fast": activations, W in the forward product) and along r otherwise.
template <int ROWS, int THREADS>
struct OperandTile {
    static constexpr int UNITS = ROWS * ST_BK / 4, PER_THREAD = UNITS / THREADS;
    static_assert(UNITS % THREADS == 0, "units per thread");
    const float *X; long long rs, ks; int R, K, r0; bool kfast, vec;

    __device__ __forceinline__ void init(const float *X_, long long rs_, long long ks_, int R_, int K_, int r0_) {
        X = X_; rs = rs_; ks = ks_; R = R_; K = K_; r0 = r0_;
        kfast = (ks == 1);
        // 16-byte loads need the unit's first element 16-byte aligned for every (r, k) it can start at
        const long long slow = kfast ? rs : ks;
        vec = (kfast || rs == 1) && (slow % 4 == 0) && (reinterpret_cast<uintptr_t>(X) % 16 == 0);
    }
    __device__ __forceinline__ void fetch(int k0, float4 (&reg)[PER_THREAD]) const {
#pragma unroll
        for (int i = 0; i < PER_THREAD; ++i) {
            const int u = threadIdx.x + i * THREADS;
            int rr, kk;                                   // first element of the unit inside the tile
            if (kfast) { rr = u / (ST_BK / 4); kk = (u % (ST_BK / 4)) * 4; }
            else       { kk = u / (ROWS / 4);  rr = (u % (ROWS / 4)) * 4; }
            const int r = r0 + rr, k = k0 + kk;
            const int last_r = kfast ? r : r + 3, last_k = kfast ? k + 3 : k;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (vec && last_r < R && last_k < K) {
                v = *reinterpret_cast<const float4 *>(X + (long long)r * rs + (long long)k * ks);
            } else {
                float e[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int rj = kfast ? r : r + j, kj = kfast ? k + j : k;
                    e[j] = (rj < R && kj < K) ? X[(long long)rj * rs + (long long)kj * ks] : 0.f;
                }
                v = make_float4(e[0], e[1], e[2], e[3]);
            }
            reg[i] = v;
        }
    }
    // shared-memory tile: Xs[k][r], row pitch ROWS + 4 floats
    __device__ __forceinline__ void stash(float (*Xs)[ROWS + 4], const float4 (&reg)[PER_THREAD]) const {
#pragma unroll
        for (int i = 0; i < PER_THREAD; ++i) {
            const int u = threadIdx.x + i * THREADS;
            if (kfast) {
                const int rr = u / (ST_BK / 4), kk = (u % (ST_BK / 4)) * 4;
                Xs[kk + 0][rr] = reg[i].x; Xs[kk + 1][rr] = reg[i].y; Xs[kk + 2][rr] = reg[i].z; Xs[kk + 3][rr] = reg[i].w;
            } else {
                const int kk = u / (ROWS / 4), rr = (u % (ROWS / 4)) * 4;
                *reinterpret_cast<float4 *>(&Xs[kk][rr]) = reg[i];
            }
        }
    }
};

// C[g] = A[g] * B[g], tile BM x BN per CTA, (BM/8) x (BN/8) threads.  A thread owns rows
// ty*4 .. +3 and BM/2 + ty*4 .. +3, columns tx*4 .. +3 and BN/2 + tx*4 .. +3 of the tile.
template <int EPI, int BM, int BN>
__global__ void __launch_bounds__((BM / 8) * (BN / 8)) simt_gemm_tiled_kernel(SimtGemmArgs p) {
    constexpr int TX = BN / 8, THREADS = (BM / 8) * (BN / 8);
    __shared__ __align__(16) float As[2][ST_BK][BM + 4];
    __shared__ __align__(16) float Bs[2][ST_BK][BN + 4];
    const int g = blockIdx.z;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int tx = threadIdx.x % TX, ty = threadIdx.x / TX;
    OperandTile<BM, THREADS> ta;
    OperandTile<BN, THREADS> tb;
    ta.init(p.A + (long long)g * p.a_gs, p.a_ms, p.a_ks, p.M, p.K, m0);
    tb.init(p.B + (long long)g * p.b_gs, p.b_ns, p.b_ks, p.N, p.K, n0);
    float4 ra[OperandTile<BM, THREADS>::PER_THREAD], rb[OperandTile<BN, THREADS>::PER_THREAD];
    float acc[8][8] = {};

    ta.fetch(0, ra); tb.fetch(0, rb);
    ta.stash(As[0], ra); tb.stash(Bs[0], rb);
    __syncthreads();
    int cur = 0;
    for (int k0 = 0; k0 < p.K; k0 += ST_BK) {
        const bool more = k0 + ST_BK < p.K;
        if (more) { ta.fetch(k0 + ST_BK, ra); tb.fetch(k0 + ST_BK, rb); }
#pragma unroll
        for (int kk = 0; kk < ST_BK; ++kk) {
            const float4 a0 = *reinterpret_cast<const float4 *>(&As[cur][kk][ty * 4]);
            const float4 a1 = *reinterpret_cast<const float4 *>(&As[cur][kk][BM / 2 + ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4 *>(&Bs[cur][kk][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4 *>(&Bs[cur][kk][BN / 2 + tx * 4]);
            const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        if (more) {
            // the other buffer was last read in the previous iteration, which ended with a barrier
            ta.stash(As[cur ^ 1], ra); tb.stash(Bs[cur ^ 1], rb);
            __syncthreads();
            cur ^= 1;
        }
    }

    float *C = p.C + (long long)g * p.c_gs;
    const float *bias = (EPI == EPI_BIAS || EPI == EPI_BIAS_RELU) ? p.bias + (long long)g * p.bias_gs : nullptr;
    const float *mask = (EPI == EPI_MASK) ? p.mask + (long long)g * p.mask_gs : nullptr;
    const bool c_vec = (p.ldc % 4 == 0) && (reinterpret_cast<uintptr_t>(C) % 16 == 0);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int m = m0 + (i < 4 ? ty * 4 + i : BM / 2 + ty * 4 + i - 4);
        if (m >= p.M) continue;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int n = n0 + (h ? BN / 2 : 0) + tx * 4;
            if (n >= p.N) continue;
            float v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                v[j] = acc[i][h * 4 + j];
                if (n + j < p.N) {
                    if (EPI == EPI_BIAS || EPI == EPI_BIAS_RELU) v[j] += bias[n + j];
                    if (EPI == EPI_BIAS_RELU) v[j] = fmaxf(v[j], 0.f);
                    if (EPI == EPI_MASK) v[j] = (mask[(long long)m * p.ldmask + n + j] > 0.f) ? v[j] : 0.f;
                }
            }
            float *o = C + (long long)m * p.ldc + n;
            if (c_vec && n + 3 < p.N) {
                *reinterpret_cast<float4 *>(o) = make_float4(v[0], v[1], v[2], v[3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (n + j < p.N) o[j] = v[j];
            }
        }
    }
}

// Softmax cross-entropy backward, one warp per batch row:
//   p = softmax(logits) (row max subtracted), dlogits = (p - onehot)/B,
//   row_loss = logsumexp - logits[label].
// Writes fp32 dlogits [rows, C] (d32 != NULL) and/or bf16 copies in both
// layouts: dbf [B, ld_b] per replica and dbfT [C, B] per replica, and/or the
// fp32 copy as a tf32-exact hi/lo pair in both layouts (dhi, dlo: [rows, ld_split]; dThi, dTlo: [C, B] per replica).
// With parts > 1 the logits arrive as split-K partial sums: logits = bias + sum_s part_s (s in fixed order),
// formed here first and written back over part 0 (= the logits buffer).
// With loss != NULL the mean loss of every replica is formed here too: rows_done[g] (zero between launches) counts the
// finished rows of replica g, and the warp that finishes the last one adds up the replica's row losses -- in the
// same fixed order whoever does it (256 strided partial sums, then a binary tree), so the result does not depend on which
// warp that is -- and puts the counter back to zero.
// TR = 16 (bf16 copies only; B % 16 == 0; dynamic shared memory of 16 * C bf16): a block takes 16 consecutive rows, two per
// warp, keeps their bf16 dlogits in shared memory and writes the transposed copy dbfT from there, 32 bytes (16 rows of one
// class) per store instead of one 2-byte element per lane.  Same arithmetic, same values.
template <int TR = 0>
__global__ void __launch_bounds__(256)
softmax_ce_backward_kernel(float *__restrict__ logits, const int32_t *__restrict__ labels,
                           float *__restrict__ d32, __nv_bfloat16 *__restrict__ dbf,
                           __nv_bfloat16 *__restrict__ dbfT, float *__restrict__ row_loss,
                           int rows, int B, int C, int ld_b, int *status,
                           int parts = 1, long long part_stride = 0, const float *__restrict__ bias = nullptr,
                           long long bias_gs = 0, float *__restrict__ dThi = nullptr, float *__restrict__ dTlo = nullptr,
                           float *__restrict__ dhi = nullptr, float *__restrict__ dlo = nullptr, int ld_split = 0,
                           float *__restrict__ loss = nullptr, int *__restrict__ rows_done = nullptr) {
    extern __shared__ __align__(16) unsigned char sce_tile_raw[];
    __nv_bfloat16 *tile = reinterpret_cast<__nv_bfloat16 *>(sce_tile_raw);      // TR > 0: [TR][C]
    const int lane = threadIdx.x % 32;
    for (int rr = 0; rr < (TR > 0 ? TR / 8 : 1); ++rr) {
        const int lr = rr * 8 + threadIdx.x / 32;                                   // row inside the block's tile
        const int row = TR > 0 ? blockIdx.x * TR + lr : blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
        if (row >= rows) { if (TR > 0) continue; else return; }
        float *lg = logits + (size_t)row * C;
        const int label = labels[row];
        const bool label_ok = (label >= 0 && label < C);
        const float inv_B = 1.f / (float)B;
        const int g = row / B, i = row % B;
        const float *bg = parts > 1 ? bias + (long long)g * bias_gs : nullptr;
        // logit j of this row: with split-K partial sums, bias + sum_s part_s in fixed order (all loads in flight first)
        auto logit = [&](int j) -> float {
            if (parts <= 1) return lg[j];
            float pv[8];
    #pragma unroll
            for (int q = 0; q < 8; ++q) pv[q] = (q < parts) ? lg[(long long)q * part_stride + j] : 0.f;
            float s = pv[0];
    #pragma unroll
            for (int q = 1; q < 8; ++q) s += pv[q];
            return s + bg[j];
        };
        auto emit = [&](int j, float d) {                // d = dlogits[row, j]
            if (d32) d32[(size_t)row * C + j] = d;
            if (dbf) {
                const __nv_bfloat16 h = __float2bfloat16_rn(d);
                dbf[((size_t)g * B + i) * ld_b + j] = h;
                if (TR > 0) tile[lr * C + j] = h; else dbfT[((size_t)g * C + j) * B + i] = h;
            }
            if (dThi) {                                  // tf32-exact hi/lo pair, [B, ld_split] and transposed [C, B] per replica
                float hi, lo;
                split_tf32(d, hi, lo);
                dThi[((size_t)g * C + j) * B + i] = hi;
                dTlo[((size_t)g * C + j) * B + i] = lo;
                dhi[(size_t)row * ld_split + j] = hi;
                dlo[(size_t)row * ld_split + j] = lo;
            }
        };
        constexpr int VR = 4;                            // up to 128 classes: the row stays in registers (one pass over memory)
        float mx = -INFINITY, s = 0.f, label_logit = 0.f;
        if (C <= 32 * VR) {
            float v[VR];
    #pragma unroll
            for (int k = 0; k < VR; ++k) {
                const int j = lane + 32 * k;
                v[k] = j < C ? logit(j) : -INFINITY;
                if (parts > 1 && j < C) lg[j] = v[k];    // the logits buffer then holds the complete logits
                mx = fmaxf(mx, v[k]);
            }
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    #pragma unroll
            for (int k = 0; k < VR; ++k)
                if (lane + 32 * k < C) s += __expf(v[k] - mx);
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            const float inv_s = 1.f / s;
            float cand = 0.f;
    #pragma unroll
            for (int k = 0; k < VR; ++k) {
                const int j = lane + 32 * k;
                if (k == (label >> 5)) cand = v[k];
                if (j < C) {
                    float d = __expf(v[k] - mx) * inv_s;
                    if (j == label) d -= 1.f;
                    emit(j, d * inv_B);
                }
            }
            label_logit = __shfl_sync(0xffffffffu, cand, label & 31);
        } else {
            if (parts > 1)
                for (int j = lane; j < C; j += 32) lg[j] = logit(j);      // read back below by the same lane
            for (int j = lane; j < C; j += 32) mx = fmaxf(mx, lg[j]);
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            for (int j = lane; j < C; j += 32) s += __expf(lg[j] - mx);
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            const float inv_s = 1.f / s;
            for (int j = lane; j < C; j += 32) {
                float d = __expf(lg[j] - mx) * inv_s;
                if (j == label) d -= 1.f;
                emit(j, d * inv_B);
            }
            if (lane == 0 && label_ok) label_logit = lg[label];
        }
        if (lane == 0) {
            row_loss[row] = label_ok ? (mx + __logf(s) - label_logit) : 0.f;
            if (!label_ok) status[SLOT_BAD_LABEL] = 1;
        }
        if (loss) replica_loss_finish(row_loss, loss, rows_done, g, B, 1, lane);
    }
    if (TR > 0) {
        __syncthreads();
        const long long r0 = (long long)blockIdx.x * TR;                        // first row of the tile: same replica throughout
        const int g0 = (int)(r0 / B), i0 = (int)(r0 % B);
        for (int j = threadIdx.x; j < C; j += blockDim.x) {
            uint4 v[TR > 0 ? TR / 8 : 1];
            __nv_bfloat16 *e = reinterpret_cast<__nv_bfloat16 *>(v);
#pragma unroll
            for (int r = 0; r < TR; ++r) e[r] = tile[r * C + j];
            uint4 *dst = reinterpret_cast<uint4 *>(dbfT + ((size_t)g0 * C + j) * B + i0);
#pragma unroll
            for (int q = 0; q < TR / 8; ++q) dst[q] = v[q];
        }
    }
}

// db[g, j] = sum_i dH[g, i, j] from fp32 dH [n, B, d] (thread per column).
__global__ void __launch_bounds__(256)
bias_grad_f32_kernel(const float *__restrict__ dH, float *__restrict__ grad, long long grad_gs,
                     int B, int d) {
    const int j = blockIdx.x * 256 + threadIdx.x;
    const int g = blockIdx.y;
    if (j >= d) return;
    const float *p = dH + (size_t)g * B * d + j;
    float s = 0.f;
    for (int i = 0; i < B; ++i) s += p[(size_t)i * d];
    grad[(long long)g * grad_gs + j] = s;
}

// sum_i row[i] over one row of the bf16 transposed copy dH^T (batch % 8 == 0), fp32, in batch order.
__device__ __forceinline__ float bias_grad_row(const __nv_bfloat16 *row, int batch) {
    const uint4 *p = reinterpret_cast<const uint4 *>(row);
    float s = 0.f;
    for (int i = 0; i < batch / 8; ++i) {
        const uint4 v = __ldg(p + i);
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
        for (int k = 0; k < 4; ++k) { const float2 f = __bfloat1622float2(h[k]); s += f.x; s += f.y; }
    }
    return s;
}

// db[g, j] = sum_i dH^T[g, j, i] from the bf16 transposed copy [n, d, B] (thread per row).
__global__ void __launch_bounds__(128)
bias_grad_bf16_kernel(const __nv_bfloat16 *__restrict__ dHT, float *__restrict__ grad,
                      long long grad_gs, int B, int d) {
    const int j = blockIdx.x * 128 + threadIdx.x;
    const int g = blockIdx.y;
    if (j >= d) return;
    grad[(long long)g * grad_gs + j] = bias_grad_row(dHT + ((size_t)g * d + j) * B, B);
}

// Everything of a replica's vector that the weight tiles do not cover -- the
// bias segments and the alignment padding after each segment -- gets its inner
// update (Eq. parle_y, parle_z) here when the update of the weights is fused into
// the weight-gradient GEMM.  One thread per element: for a bias element the thread
// first forms db_j = sum_i dH^T[j, i] (bf16 transposed copy, fp32 sum in batch order);
// padding has gradient 0 and stays 0.
struct TailPlan {
    int n_layers, batch;
    long long begin[PARLE_MAX_LAYERS], b_off[PARLE_MAX_LAYERS], end[PARLE_MAX_LAYERS];   // element ranges in a replica
    int d_out[PARLE_MAX_LAYERS];
    const __nv_bfloat16 *dHT[PARLE_MAX_LAYERS];      // [n, d_out, B]
};

template <bool FIRST, bool MOM = false>
__global__ void __launch_bounds__(128)
tail_update_kernel(const TailPlan tp, float *__restrict__ y, float *__restrict__ z, const float *__restrict__ x,
                   long long stride, float eta_p, float inv_gamma, float alpha, float wd, int *status,
                   float *__restrict__ v = nullptr, float mu = 0.f) {
    const int l = blockIdx.y, g = blockIdx.z;
    const long long e = tp.begin[l] + (long long)blockIdx.x * 128 + threadIdx.x;     // one thread per element
    if (e >= tp.end[l]) return;
    float grad = 0.f;
    const long long j = e - tp.b_off[l];
    if (j >= 0 && j < tp.d_out[l]) {
        grad = bias_grad_row(tp.dHT[l] + ((long long)g * tp.d_out[l] + j) * tp.batch, tp.batch);
    }
    const long long i = (long long)g * stride + e;
    const float xv = x[i];
    const float yo = FIRST ? xv : y[i], zo = FIRST ? xv : z[i];
    float d = fmaf(inv_gamma, yo - xv, fmaf(wd, yo, grad));
    if (MOM) {                                    // Nesterov momentum, v = 0 at the start of a round
        const float vn = FIRST ? d : fmaf(mu, v[i], d);
        v[i] = vn;
        d = fmaf(mu, vn, d);
    }
    const float yn = yo - eta_p * d;
    const float zn = fmaf(alpha, zo, (1.0f - alpha) * yn);
    y[i] = yn;
    z[i] = zn;
    if (!(fabsf(yn) <= 3.402823466e+38f)) status[SLOT_NONFINITE] = 1;
}

// bf16 operand copy of the weights in blocked layout: W_l [d_out, d_in] row-major fp32 ->
// blocks of 128 rows x 64 columns (16 KiB of bf16 each), row-block major; element (r, c) of layer l at
//   sh_off[l] + ((r/128) * cb[l] + c/64) * 8192 + (r%128) * 64 + c%64.
// One CTA per block; rows and columns beyond the matrix are never written (they stay zero).
struct BlockedPlan {
    int n_layers;
    long long w_off[PARLE_MAX_LAYERS], sh_off[PARLE_MAX_LAYERS];
    int d_in[PARLE_MAX_LAYERS], d_out[PARLE_MAX_LAYERS], cb[PARLE_MAX_LAYERS], first_block[PARLE_MAX_LAYERS + 1];
};

__global__ void __launch_bounds__(256)
blocked_bf16_kernel(const BlockedPlan bp, const float *__restrict__ src, long long stride,
                    __nv_bfloat16 *__restrict__ dst, long long sh_stride) {
    const int g = blockIdx.y;
    int l = 0;
    while (l + 1 < bp.n_layers && (int)blockIdx.x >= bp.first_block[l + 1]) ++l;
    const int blk = blockIdx.x - bp.first_block[l];
    const int rb = blk / bp.cb[l], cb = blk % bp.cb[l];
    const float *W = src + (long long)g * stride + bp.w_off[l];
    __nv_bfloat16 *out = dst + (long long)g * sh_stride + bp.sh_off[l] + (long long)blk * 8192;
    const int c4 = (threadIdx.x % 16) * 4;                   // 16 threads x 4 columns = one 64-column row of the block
    const int col = cb * 64 + c4;
    for (int r = threadIdx.x / 16; r < 128; r += 16) {
        const int row = rb * 128 + r;
        if (row < bp.d_out[l] && col < bp.d_in[l]) {          // d_in % 8 == 0: the 4 columns are all inside
            const float4 v = *reinterpret_cast<const float4 *>(W + (long long)row * bp.d_in[l] + col);
            uint2 pk;                                         // weights: nearest, ties away from zero (bf16_weight)
            pk.x = (bf16_split_word(v.x) >> 16) | (bf16_split_word(v.y) & 0xFFFF0000u);
            pk.y = (bf16_split_word(v.z) >> 16) | (bf16_split_word(v.w) & 0xFFFF0000u);
            *reinterpret_cast<uint2 *>(out + r * 64 + c4) = pk;
        }
    }
}

// Minibatch inputs fp32 [n, B, d] -> bf16 [n, B, d] and its transpose [n, d, B]
// (the K-major operand of the first layer's weight-gradient product).
// 64 x 64 tiles; 16-byte reads, 8-byte row-major writes, 16-byte transposed writes (needs d % 8 == 0, B % 8 == 0).
__global__ void __launch_bounds__(256)
input_to_bf16_kernel(const float *__restrict__ X, __nv_bfloat16 *__restrict__ Xb,
                     __nv_bfloat16 *__restrict__ XbT, int B, int d) {
    __shared__ __nv_bfloat16 tile[64][64 + 8];
    const int g = blockIdx.z;
    const int i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
    const int c4 = (threadIdx.x % 16) * 4, r0 = threadIdx.x / 16;          // 16 threads x 4 features per batch row
#pragma unroll
    for (int r = r0; r < 64; r += 16) {
        const int i = i0 + r, j = j0 + c4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < B && j < d) {
            v = __ldcs(reinterpret_cast<const float4 *>(X + ((size_t)g * B + i) * d + j));
            __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t *>(&lo); pk.y = *reinterpret_cast<uint32_t *>(&hi);
            *reinterpret_cast<uint2 *>(Xb + ((size_t)g * B + i) * d + j) = pk;
        }
        tile[r][c4 + 0] = __float2bfloat16_rn(v.x); tile[r][c4 + 1] = __float2bfloat16_rn(v.y);
        tile[r][c4 + 2] = __float2bfloat16_rn(v.z); tile[r][c4 + 3] = __float2bfloat16_rn(v.w);
    }
    __syncthreads();
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        const int item = threadIdx.x + it * 256;          // 64 features x 8 groups of 8 batch rows
        const int jj = item / 8, i8 = (item % 8) * 8;
        const int j = j0 + jj, i = i0 + i8;
        if (j < d && i < B) {
            __align__(16) __nv_bfloat16 o[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) o[k] = tile[i8 + k][jj];
            *reinterpret_cast<uint4 *>(XbT + ((size_t)g * d + j) * B + i) = *reinterpret_cast<const uint4 *>(o);
        }
    }
}

}  // namespace parle
