// Bypassable-update statistic of Sec. III-C / Sec. V-B on the GPU.
//
// One warp walks one query row over its visible keys exactly like the per-key
// forward (scores in fp64, state (s_{i-1}, ln w_{i-1}) of Algorithm 3) but keeps
// no output; it counts the steps whose score difference s_i - s_{i-1} leaves
// [lo, hi] (the paper's static criterion, [-6, 11]) and the steps whose sigmoid
// argument x_i = s_i - s_{i-1} + ln w_{i-1} (Eq. w-last) leaves [alo, ahi] (a
// reading of the adaptive criterion the paper announces as future work).
// counts[0] steps, [1] diff <= lo, [2] diff >= hi, [3] x <= alo, [4] x >= ahi.
#pragma once

#include "flashd_common.cuh"

namespace flashd {

template <typename TIn, int E>
__global__ void __launch_bounds__(128)
skipstats_kernel(const TIn* __restrict__ q, const TIn* __restrict__ k, unsigned long long* __restrict__ counts,
                 long long rows, int Nq, int Nk, float scale, int causal, float lo, float hi, float alo, float ahi) {
    constexpr int D = 32 * E;
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const long long bh = row / Nq;
    const int i = (int)(row - bh * Nq);
    const int nv = causal ? min(i + 1, Nk) : Nk;

    double qd[E];
    const TIn* qrow = q + row * D + lane * E;
#pragma unroll
    for (int e = 0; e < E; ++e) qd[e] = (double)to_f32<TIn>(qrow[e]);
    const TIn* kb = k + bh * (long long)Nk * D + lane * E;
    const double scale_d = (double)scale;
    double s_prev = 0.0, lnw = 0.0;
    unsigned int below = 0, above = 0, abelow = 0, aabove = 0;

    for (int j = 0; j < nv; ++j) {
        double part = 0.0;
#pragma unroll
        for (int e = 0; e < E; ++e) part = fma(qd[e], (double)to_f32<TIn>(kb[(long long)j * D + e]), part);
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) part += __shfl_xor_sync(0xffffffffu, part, m);
        const double s = scale_d * part;
        if (j > 0) {
            const double diff = s - s_prev;
            const double xd = diff + lnw;            // argument of Eq. (w-last)
            below += diff <= (double)lo;
            above += diff >= (double)hi;
            abelow += xd <= (double)alo;
            aabove += xd >= (double)ahi;
            const float x = (float)xd;
            if (x >= 0.f) lnw = -(double)log1pf(expf(-x));
            else lnw = xd - (double)log1pf(expf(x));
        } else {
            lnw = 0.0;
        }
        s_prev = s;
    }
    if (lane == 0) {
        if (nv > 1) atomicAdd(&counts[0], (unsigned long long)(nv - 1));
        if (below) atomicAdd(&counts[1], (unsigned long long)below);
        if (above) atomicAdd(&counts[2], (unsigned long long)above);
        if (abelow) atomicAdd(&counts[3], (unsigned long long)abelow);
        if (aabove) atomicAdd(&counts[4], (unsigned long long)aabove);
    }
}

}  // namespace flashd
