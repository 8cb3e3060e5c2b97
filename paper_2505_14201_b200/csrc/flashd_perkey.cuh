// Per-key FLASH-D forward: Algorithm 3 one key at a time.
//
// One warp owns one query row; lane l holds elements [l*E, l*E+E) of q and of
// the running output o (d = 32*E).  For every visible key, in index order:
//   s_i = scale * dot(q, k_i)                        (Sec. II-A)
//   i = 1:  w_1 = 1, o_1 = v_1                        (Alg. 3, else branch)
//   i > 1:  w_i = sigma(s_i - s_{i-1} + ln w_{i-1})   (Eq. w-last)
//           o_i = o_{i-1} + (v_i - o_{i-1}) w_i       (Sec. IV-A form of Eq. out-final)
// The carried state is exactly the paper's (s_{i-1}, ln w_{i-1}, o_{i-1}).
// ln w_i is obtained as ln sigma(x) from the same exponential that gives
// sigma(x), so it stays finite when w_i underflows, and sigma is evaluated over
// the whole real line (no clamp to a range, no skipped update).
//
// Precision: scores and the carried ln w are fp64 (their difference cancels
// when logits are in the hundreds), sigma / log1p / blend are fp32.
#pragma once

#include "flashd_common.cuh"

namespace flashd {

template <typename TIn, typename TOut, int E>
__global__ void __launch_bounds__(128)
perkey_kernel(const TIn* __restrict__ q, const TIn* __restrict__ k, const TIn* __restrict__ v,
              TOut* __restrict__ o, float* __restrict__ lse, long long rows, int Nq, int Nk,
              float scale, int causal, int D) {
    // D = row length: 32*E, or 16 with E = 1 (lanes 16..31 then hold no column)
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
            const double xd = s - s_prev + lnw;      // argument of Eq. (w-last)
            const float x = (float)xd;
            if (x >= 0.f) {
                const float ex = expf(-x);
                w = 1.f / (1.f + ex);
                lnw = -(double)log1pf(ex);
            } else {
                const float ex = expf(x);
                w = ex / (1.f + ex);
                lnw = xd - (double)log1pf(ex);
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
    if (lse != nullptr && lane == 0) lse[row] = (float)(s_prev - lnw);
}

}  // namespace flashd
