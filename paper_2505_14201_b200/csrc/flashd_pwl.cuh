// Per-key FLASH-D forward with piece-wise linear sigmoid and ln (Sec. IV-B).
//
// Same walk as perkey_kernel (one warp per query row, the paper's state
// (s_{i-1}, ln w_{i-1}, o_{i-1})), but the two non-linear functions are read
// from caller-supplied tables of a continuous PWL function (nodes x_0<...<x_n
// with values y_0..y_n, end values outside), and the sigmoid argument
// x = s_i - s_{i-1} + ln w_{i-1} is confined to [lo, hi]:
//   range_mode 0: x is clamped to [lo, hi];
//   range_mode 1: x < lo bypasses the key (no update, state unchanged);
//                 x > hi replaces the output by v_i (w = 1, ln w = 0).
// n = 0 for a table selects the exact function.  Scores and x are fp64 as in
// perkey_kernel; the table look-up, the interpolation and the blend are fp32.
#pragma once

#include "flashd_common.cuh"

namespace flashd {

struct PwlTables {
    int sig_n, ln_n;
    float sig_x[FLASHD_PWL_MAX_SEGMENTS + 1], sig_y[FLASHD_PWL_MAX_SEGMENTS + 1];
    float ln_x[FLASHD_PWL_MAX_SEGMENTS + 1], ln_y[FLASHD_PWL_MAX_SEGMENTS + 1];
};

__device__ __forceinline__ float pwl_eval(const float* xs, const float* ys, int n, float x) {
    if (x <= xs[0]) return ys[0];
    if (x >= xs[n]) return ys[n];
    int m = 0;
    while (m + 1 < n && x >= xs[m + 1]) ++m;
    return fmaf(x - xs[m], (ys[m + 1] - ys[m]) / (xs[m + 1] - xs[m]), ys[m]);
}

template <typename TIn, typename TOut, int E>
__global__ void __launch_bounds__(128)
perkey_pwl_kernel(const TIn* __restrict__ q, const TIn* __restrict__ k, const TIn* __restrict__ v,
                  TOut* __restrict__ o, unsigned long long* __restrict__ counts, long long rows, int Nq, int Nk,
                  float scale, int causal, const __grid_constant__ PwlTables tab, float lo, float hi,
                  int range_mode, int D) {
    // D = row length: 32*E, or 16 with E = 1 (lanes 16..31 then hold no column)
    __shared__ float sx[FLASHD_PWL_MAX_SEGMENTS + 1], sy[FLASHD_PWL_MAX_SEGMENTS + 1];
    __shared__ float lx[FLASHD_PWL_MAX_SEGMENTS + 1], ly[FLASHD_PWL_MAX_SEGMENTS + 1];
    for (int t = threadIdx.x; t <= FLASHD_PWL_MAX_SEGMENTS; t += blockDim.x) {
        sx[t] = tab.sig_x[t]; sy[t] = tab.sig_y[t]; lx[t] = tab.ln_x[t]; ly[t] = tab.ln_y[t];
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const long long bh = row / Nq;
    const int i = (int)(row - bh * Nq);
    const int nv = causal ? min(i + 1, Nk) : Nk;

    const bool active = lane * E < D;
    double qd[E];
    float of[E];
    const TIn* qrow = q + row * D + lane * E;
#pragma unroll
    for (int e = 0; e < E; ++e) { qd[e] = active ? (double)to_f32<TIn>(qrow[e]) : 0.0; of[e] = 0.f; }
    const TIn* kb = k + bh * (long long)Nk * D + lane * E;
    const TIn* vb = v + bh * (long long)Nk * D + lane * E;
    const double scale_d = (double)scale;
    double s_prev = 0.0, lnw = 0.0;
    unsigned int n_skip = 0, n_repl = 0;

    for (int j = 0; j < nv; ++j) {
        float kf[E], vf[E];
#pragma unroll
        for (int e = 0; e < E; ++e) {
            kf[e] = active ? to_f32<TIn>(kb[(long long)j * D + e]) : 0.f;
            vf[e] = active ? to_f32<TIn>(vb[(long long)j * D + e]) : 0.f;
        }
        double part = 0.0;
#pragma unroll
        for (int e = 0; e < E; ++e) part = fma(qd[e], (double)kf[e], part);
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) part += __shfl_xor_sync(0xffffffffu, part, m);
        const double s = scale_d * part;
        float w;
        if (j == 0) {
            w = 1.f;
            lnw = 0.0;
        } else {
            double xd = s - s_prev + lnw;
            if (range_mode == 1 && xd < (double)lo) { ++n_skip; continue; }      // uniform in the warp
            if (range_mode == 1 && xd > (double)hi) {
                ++n_repl;
                w = 1.f;
                lnw = 0.0;
            } else {
                xd = fmin(fmax(xd, (double)lo), (double)hi);
                const float x = (float)xd;
                if (tab.sig_n > 0) {
                    w = pwl_eval(sx, sy, tab.sig_n, x);
                } else if (x >= 0.f) {
                    w = 1.f / (1.f + expf(-x));
                } else {
                    const float ex = expf(x);
                    w = ex / (1.f + ex);
                }
                if (tab.ln_n > 0) lnw = (double)pwl_eval(lx, ly, tab.ln_n, w);
                else if (tab.sig_n > 0) lnw = (double)logf(w);
                else lnw = x >= 0.f ? -(double)log1pf(expf(-x)) : xd - (double)log1pf(expf(x));
            }
        }
#pragma unroll
        for (int e = 0; e < E; ++e) of[e] = fmaf(vf[e] - of[e], w, of[e]);
        s_prev = s;
    }

    TOut* orow = o + row * D + lane * E;
#pragma unroll
    for (int e = 0; e < E; ++e)
        if (active) orow[e] = from_f32<TOut>(of[e]);
    if (counts != nullptr && lane == 0) {
        if (n_skip) atomicAdd(&counts[0], (unsigned long long)n_skip);
        if (n_repl) atomicAdd(&counts[1], (unsigned long long)n_repl);
    }
}

}  // namespace flashd
