// Streaming kernels of the Parle round: the fused inner update
// (Eq. parle_y + Eq. parle_z), the fused outer update + replica mean
// (Eq. parle_xa + Eq. parle_x with eta'' = rho/n) and the stand-alone mean.  All are HBM-bound: every vector is touched once,
// with 16-byte accesses, consecutive threads on consecutive addresses.
#pragma once

#include "common.cuh"

namespace parle {

constexpr int kUpdThreads = 256;

__device__ __forceinline__ bool finite4(const float4 &v) {
    // NaN and Inf both fail "|v| <= FLT_MAX"
    return (fabsf(v.x) <= 3.402823466e+38f) & (fabsf(v.y) <= 3.402823466e+38f) &
           (fabsf(v.z) <= 3.402823466e+38f) & (fabsf(v.w) <= 3.402823466e+38f);
}

// Eq. (parle_y): y <- y - eta' (g + (y - x)/gamma), Eq. (parle_z): z <- alpha z + (1-alpha) y_new.
// wd: optional weight-decay regulariser of f (Section 1.1), g <- g + wd * y.
// FIRST: first inner step of a round, where y = z = x (the reset is folded in:
// x is read in place of y and z, which are only written).
// MOM: Nesterov momentum (Remark, Section 3.1): with d = g + (y - x)/gamma,
//      v <- mu v + d, y <- y - eta' (d + mu v); v starts from 0 in every round (FIRST: v is only written).
// SPLIT: also store the new y as a tf32-exact pair (hi = y rounded to tf32, lo = y - hi rounded to tf32):
//      the operands of the fp32-accurate tensor-core products of the next step.
// ZMODE (ignored when FIRST): Eq. (parle_z) may be applied two steps at a time inside a round, since
//      z_{k+2} = alpha^2 z_k + (1-alpha)(alpha y_{k+1} + y_{k+2}) needs only the y this step reads and the y it writes:
//      0 = one-step form, 1 = z untouched (neither read nor written), 2 = two-step form.
constexpr int UPD_Z_SINGLE = 0, UPD_Z_SKIP = 1, UPD_Z_DOUBLE = 2;
template <bool FIRST, int UNROLL, bool MOM = false, bool SPLIT = false, int ZMODE = UPD_Z_SINGLE>
__global__ void __launch_bounds__(kUpdThreads)
inner_update_kernel(const float4 *__restrict__ g, float4 *__restrict__ y, const float4 *__restrict__ x,
                    float4 *__restrict__ z, size_t n4,
                    float eta_p, float inv_gamma, float alpha, float wd, int *status,
                    float4 *__restrict__ v = nullptr, float mu = 0.f,
                    float4 *__restrict__ y_hi = nullptr, float4 *__restrict__ y_lo = nullptr) {
    const size_t tid = (size_t)blockIdx.x * kUpdThreads + threadIdx.x;
    const size_t nthreads = (size_t)gridDim.x * kUpdThreads;
    const float one_m_alpha = 1.0f - alpha, alpha_sq = alpha * alpha;
    constexpr bool USE_Z = FIRST || ZMODE != UPD_Z_SKIP;
    constexpr bool DOUBLE_Z = !FIRST && ZMODE == UPD_Z_DOUBLE;
    bool ok = true;
    for (size_t base = tid; base < n4; base += nthreads * UNROLL) {
        float4 gv[UNROLL], yv[UNROLL], xv[UNROLL], zv[UNROLL], vv[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const size_t i = base + (size_t)u * nthreads;
            if (i < n4) {
                gv[u] = __ldcs(g + i);
                xv[u] = __ldg(x + i);
                if (!FIRST) {
                    yv[u] = y[i];
                    if (USE_Z) zv[u] = z[i];
                    if (MOM) vv[u] = v[i];
                }
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const size_t i = base + (size_t)u * nthreads;
            if (i < n4) {
                float4 yo = FIRST ? xv[u] : yv[u];
                float4 zo = FIRST ? xv[u] : (USE_Z ? zv[u] : make_float4(0.f, 0.f, 0.f, 0.f));
                float4 yn, zn, d;
                d.x = fmaf(inv_gamma, yo.x - xv[u].x, fmaf(wd, yo.x, gv[u].x));
                d.y = fmaf(inv_gamma, yo.y - xv[u].y, fmaf(wd, yo.y, gv[u].y));
                d.z = fmaf(inv_gamma, yo.z - xv[u].z, fmaf(wd, yo.z, gv[u].z));
                d.w = fmaf(inv_gamma, yo.w - xv[u].w, fmaf(wd, yo.w, gv[u].w));
                if (MOM) {
                    float4 vn = d;                                   // FIRST: v = 0 before this step
                    if (!FIRST) {
                        vn.x = fmaf(mu, vv[u].x, d.x); vn.y = fmaf(mu, vv[u].y, d.y);
                        vn.z = fmaf(mu, vv[u].z, d.z); vn.w = fmaf(mu, vv[u].w, d.w);
                    }
                    v[i] = vn;
                    d.x = fmaf(mu, vn.x, d.x); d.y = fmaf(mu, vn.y, d.y);
                    d.z = fmaf(mu, vn.z, d.z); d.w = fmaf(mu, vn.w, d.w);
                }
                yn.x = yo.x - eta_p * d.x;
                yn.y = yo.y - eta_p * d.y;
                yn.z = yo.z - eta_p * d.z;
                yn.w = yo.w - eta_p * d.w;
                if (DOUBLE_Z) {
                    zn.x = fmaf(alpha_sq, zo.x, one_m_alpha * fmaf(alpha, yo.x, yn.x));
                    zn.y = fmaf(alpha_sq, zo.y, one_m_alpha * fmaf(alpha, yo.y, yn.y));
                    zn.z = fmaf(alpha_sq, zo.z, one_m_alpha * fmaf(alpha, yo.z, yn.z));
                    zn.w = fmaf(alpha_sq, zo.w, one_m_alpha * fmaf(alpha, yo.w, yn.w));
                } else {
                    zn.x = fmaf(alpha, zo.x, one_m_alpha * yn.x);
                    zn.y = fmaf(alpha, zo.y, one_m_alpha * yn.y);
                    zn.z = fmaf(alpha, zo.z, one_m_alpha * yn.z);
                    zn.w = fmaf(alpha, zo.w, one_m_alpha * yn.w);
                }
                ok &= finite4(yn);
                y[i] = yn;
                if (USE_Z) z[i] = zn;
                if (SPLIT) {
                    float4 h, l;
                    split_tf32(yn.x, h.x, l.x); split_tf32(yn.y, h.y, l.y);
                    split_tf32(yn.z, h.z, l.z); split_tf32(yn.w, h.w, l.w);
                    y_hi[i] = h;
                    y_lo[i] = l;
                }
            }
        }
    }
    if (!ok) status[SLOT_NONFINITE] = 1;
}

// Eq. (parle_xa) for all replicas of a coordinate, then Eq. (parle_x): each
// thread owns four consecutive coordinates, walks the replica axis in a fixed
// order (deterministic sum, no atomics) and writes the new mean.
// MOM: Nesterov momentum on the x^a step: d = (x - z) + (x - xbar)/rho, vx <- mu vx + d, x <- x - eta (d + mu vx);
//      vx persists across rounds.
template <int RCHUNK, bool MOM = false>
__global__ void __launch_bounds__(kUpdThreads)
outer_mean_kernel(float4 *__restrict__ x, const float4 *__restrict__ z, float4 *__restrict__ xbar,
                  size_t stride4, int n, float eta, float eta_over_rho,
                  float n_as_float, int *status,
                  float4 *__restrict__ vx = nullptr, float mu = 0.f, float inv_rho = 0.f) {
    const size_t nthreads = (size_t)gridDim.x * kUpdThreads;
    bool ok = true;
    for (size_t j = (size_t)blockIdx.x * kUpdThreads + threadIdx.x; j < stride4; j += nthreads) {
        const float4 xb = xbar[j];
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int a0 = 0; a0 < n; a0 += RCHUNK) {
            float4 xv[RCHUNK], zv[RCHUNK], vv[RCHUNK];
#pragma unroll
            for (int r = 0; r < RCHUNK; ++r) {
                if (a0 + r < n) {
                    const size_t i = (size_t)(a0 + r) * stride4 + j;
                    xv[r] = x[i];
                    zv[r] = __ldcs(z + i);
                    if (MOM) vv[r] = vx[i];
                }
            }
#pragma unroll
            for (int r = 0; r < RCHUNK; ++r) {
                if (a0 + r < n) {
                    const size_t i = (size_t)(a0 + r) * stride4 + j;
                    float4 xn;
                    if (MOM) {
                        float4 d, vn;
                        d.x = fmaf(inv_rho, xv[r].x - xb.x, xv[r].x - zv[r].x);
                        d.y = fmaf(inv_rho, xv[r].y - xb.y, xv[r].y - zv[r].y);
                        d.z = fmaf(inv_rho, xv[r].z - xb.z, xv[r].z - zv[r].z);
                        d.w = fmaf(inv_rho, xv[r].w - xb.w, xv[r].w - zv[r].w);
                        vn.x = fmaf(mu, vv[r].x, d.x); vn.y = fmaf(mu, vv[r].y, d.y);
                        vn.z = fmaf(mu, vv[r].z, d.z); vn.w = fmaf(mu, vv[r].w, d.w);
                        vx[i] = vn;
                        xn.x = xv[r].x - eta * fmaf(mu, vn.x, d.x);
                        xn.y = xv[r].y - eta * fmaf(mu, vn.y, d.y);
                        xn.z = xv[r].z - eta * fmaf(mu, vn.z, d.z);
                        xn.w = xv[r].w - eta * fmaf(mu, vn.w, d.w);
                    } else {
                    xn.x = xv[r].x - eta * (xv[r].x - zv[r].x) - eta_over_rho * (xv[r].x - xb.x);
                    xn.y = xv[r].y - eta * (xv[r].y - zv[r].y) - eta_over_rho * (xv[r].y - xb.y);
                    xn.z = xv[r].z - eta * (xv[r].z - zv[r].z) - eta_over_rho * (xv[r].z - xb.z);
                    xn.w = xv[r].w - eta * (xv[r].w - zv[r].w) - eta_over_rho * (xv[r].w - xb.w);
                    }
                    ok &= finite4(xn);
                    x[i] = xn;
                    acc.x += xn.x; acc.y += xn.y; acc.z += xn.z; acc.w += xn.w;
                }
            }
        }
        xbar[j] = make_float4(acc.x / n_as_float, acc.y / n_as_float, acc.z / n_as_float, acc.w / n_as_float);
    }
    if (!ok) status[SLOT_NONFINITE] = 1;
}

// Eq. (parle_x) with eta'' = rho/n alone: xbar <- (1/n) sum_a x^a.
template <int RCHUNK>
__global__ void __launch_bounds__(kUpdThreads)
mean_kernel(const float4 *__restrict__ x, float4 *__restrict__ xbar, size_t stride4, int n, float n_as_float) {
    const size_t nthreads = (size_t)gridDim.x * kUpdThreads;
    for (size_t j = (size_t)blockIdx.x * kUpdThreads + threadIdx.x; j < stride4; j += nthreads) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int a0 = 0; a0 < n; a0 += RCHUNK) {
            float4 xv[RCHUNK];
#pragma unroll
            for (int r = 0; r < RCHUNK; ++r)
                if (a0 + r < n) xv[r] = __ldcs(x + (size_t)(a0 + r) * stride4 + j);
#pragma unroll
            for (int r = 0; r < RCHUNK; ++r)
                if (a0 + r < n) { acc.x += xv[r].x; acc.y += xv[r].y; acc.z += xv[r].z; acc.w += xv[r].w; }
        }
        xbar[j] = make_float4(acc.x / n_as_float, acc.y / n_as_float, acc.z / n_as_float, acc.w / n_as_float);
    }
}

}  // namespace parle
