// Split-K FLASH-D forward for long key sequences (decode) and its combine.
//
// Partial kernel: one work item = (query row, split).  A producer warp streams
// the split's K and V rows from HBM into a shared-memory ring with bulk async
// copies; eight consumer warps fold them into G independent running states
// (L, o) - one per group of lanes that covers a key row - using the group form
// of Algorithm 3: for a group of keys with scores s_j and log-sum-exp L_T,
//     W = sigma(L_T - L_old)                       Eq. (w-last) on the super-key
//     L_new = L_T - ln W,  P_j = exp(s_j - L_new),  alpha = exp(L_old - L_new)
//     o <- alpha o + sum_j P_j v_j                  Eq. (out-final) for the group
// so o is normalised after every group and nothing is divided at the end.  The
// G states of the CTA are then merged, and later the splits are merged, by the
// same super-key step in the one-multiplier form of Sec. IV-A:
//     o <- o + (o_p - o) W,  L <- L_p - ln W.
// L is kept in log2 units inside the kernels and written in natural log.
//
// Paged variant (PAGED = true): K and V live in a pool of fixed-size pages
// [num_pages, H, page_size, D]; sequence b owns the pages block_table[b][0..] in order and
// has its own length seq_lens[b].  The split ranges are then cut per sequence, in multiples
// of a ring stage, so that a stage never straddles two pages.  The function computed per
// sequence is the one of the contiguous kernel.
//
// K and V are stored either as bf16 (KVB = 2 bytes per element) or as FP8-E4M3
// (KVB = 1; the second number format of Sec. V-A).  E4M3 rows are half as long, so
// the same bytes per ring stage hold twice the keys; every element is widened
// exactly (e4m3 -> f16 -> f32) and all arithmetic stays in fp32, as for bf16.
#pragma once

#include <cuda_fp16.h>

#include "flashd_common.cuh"

namespace flashd {

template <int D, int KVB = 2>
struct DecodeCfg {
    static constexpr int kChunk = 16384 / (D * KVB);         // keys per ring stage (16 KB of K, 16 KB of V)
    static constexpr int kStages = 5;
    static constexpr int kConsumerWarps = 8;
    static constexpr int kThreads = (kConsumerWarps + 1) * 32;
    static constexpr int kElems = 16 / KVB;                  // elements of a 16-byte slice
    static constexpr int kLanesPerRow = D / kElems;          // 16-byte slices per key row
    static constexpr int kRowsPerWarp = 32 / kLanesPerRow;
    static constexpr int kGroups = kConsumerWarps * kRowsPerWarp;
    static constexpr int kKeysPerGroup = kChunk / kGroups;   // = 4
    static constexpr int kTileBytes = kChunk * D * KVB;
    static constexpr int kStageBytes = 2 * kTileBytes;
    static constexpr int kMergeFloats = kGroups * (D + 1);
    static constexpr int kSmemBytes = kStages * kStageBytes + kMergeFloats * 4 + 256;
};

// Page pool description of the paged variant (all pointers are device pointers).
struct PagedKV {
    const int* block_table;   // [B, max_pages] page index of the p-th page of sequence b
    const int* seq_lens;      // [B] keys of sequence b
    int max_pages;            // row length of block_table
    int page_size;            // keys per page, a multiple of DecodeCfg::kChunk
    int num_pages;            // pages in the pool
    int H;                    // heads (pool layout [num_pages, H, page_size, D])
};
// detail code stored in the status word when a sequence length or page index is out of range
enum { kBadPageTable = 0x1f0 };

// which-wait codes reported on timeout
enum { kWaitDecFull = 0x100, kWaitDecEmpty = 0x101, kWaitDecMergeReady = 0x102, kWaitDecMergeFree = 0x103 };

// One super-key step on (L_acc, W): returns W for merging a state with
// log-sum-exp Lp (log2 units) into L_acc and updates L_acc.  sigma and
// ln sigma are evaluated in their overflow-free branch form.
__device__ __forceinline__ float superkey_weight(float& L_acc, float Lp) {
    if (Lp == -INFINITY) return 0.f;                 // empty group: nothing to blend
    if (L_acc == -INFINITY) { L_acc = Lp; return 1.f; }   // first group: W = 1 (Alg. 3, i = 1)
    float W;
    if (Lp >= L_acc) {
        const float e = ex2(L_acc - Lp);
        W = rcp(1.f + e);
        L_acc = Lp + lg2(1.f + e);
    } else {
        const float e = ex2(Lp - L_acc);
        W = e * rcp(1.f + e);
        L_acc = L_acc + lg2(1.f + e);
    }
    return W;
}

// One 16-byte slice of a K or V row widened to fp32: 8 bf16 or 16 e4m3 elements.
template <int KVB> __device__ __forceinline__ void widen_slice(const uint4& raw, float (&f)[16 / KVB]);
template <> __device__ __forceinline__ void widen_slice<2>(const uint4& raw, float (&f)[8]) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) { f[2 * e] = bf16_lo(w[e]); f[2 * e + 1] = bf16_hi(w[e]); }
}
template <> __device__ __forceinline__ void widen_slice<1>(const uint4& raw, float (&f)[16]) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        uint32_t h01, h23;      // two f16x2 pairs: bytes 0,1 and bytes 2,3 of the word
        asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\t"
            "cvt.rn.f16x2.e4m3x2 %0, lo;\n\tcvt.rn.f16x2.e4m3x2 %1, hi;\n\t}"
            : "=r"(h01), "=r"(h23) : "r"(w[e]));
        const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&h01));
        const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&h23));
        f[4 * e] = a.x; f[4 * e + 1] = a.y; f[4 * e + 2] = b.x; f[4 * e + 3] = b.y;
    }
}

// keys [k0, k1) of split `split` of a sequence of Nk keys.  Contiguous K/V: ceil(Nk/S) keys per
// split (per_split precomputed).  Paged: the same, rounded up to whole ring stages.
template <int CHUNK, bool PAGED>
__device__ __forceinline__ void split_range(int Nk, int num_splits, int per_split, int split, int& k0, int& k1) {
    if (PAGED) {
        const int ps = (Nk + num_splits - 1) / num_splits;
        per_split = (ps + CHUNK - 1) / CHUNK * CHUNK;
    }
    k0 = min(split * per_split, Nk);
    k1 = min(k0 + per_split, Nk);
}

template <int D, int KVB, bool PAGED = false>
__global__ void __launch_bounds__(DecodeCfg<D, KVB>::kThreads, 1)
splitk_partial_kernel(const __nv_bfloat16* __restrict__ q, const unsigned char* __restrict__ k,
                      const unsigned char* __restrict__ v, float* __restrict__ workspace,
                      long long rows, int Nq, int Nk, float scale_log2e, int num_splits, const PagedKV pg) {
    using C = DecodeCfg<D, KVB>;
    constexpr int EL = C::kElems;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* ring = smem_raw;
    float* merge = reinterpret_cast<float*>(smem_raw + C::kStages * C::kStageBytes);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw + C::kStages * C::kStageBytes + C::kMergeFloats * 4);
    uint64_t* full = bars;                   // [kStages]
    uint64_t* empty = bars + C::kStages;     // [kStages]
    uint64_t* merge_ready = bars + 2 * C::kStages;
    uint64_t* merge_free = merge_ready + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], C::kConsumerWarps); }
        mbar_init(merge_ready, C::kConsumerWarps);
        mbar_init(merge_free, C::kConsumerWarps);
        mbar_init_fence();
    }
    __syncthreads();

    const long long n_items = rows * num_splits;
    const int per_split = (Nk + num_splits - 1) / num_splits;

    if (warp == C::kConsumerWarps) {
        // ------------------------------------------------------ producer
        if (lane != 0) return;
        uint32_t it = 0;
        for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
            const long long row = item / num_splits;
            const int split = (int)(item - row * num_splits);
            const long long bh = row / Nq;
            int seq_nk = Nk;
            const int* pages = nullptr;
            int head = 0;
            if (PAGED) {
                const int b = (int)(bh / pg.H);
                head = (int)(bh - (long long)b * pg.H);
                seq_nk = pg.seq_lens[b];
                pages = pg.block_table + (long long)b * pg.max_pages;
                if (seq_nk < 0 || seq_nk > pg.max_pages * pg.page_size) {
                    // a length the table cannot hold: flag it and treat the sequence as empty
                    if (atomicCAS(&g_status[0], 0u, (unsigned int)FLASHD_ERR_SHAPE) == 0u) {
                        g_status[1] = blockIdx.x; g_status[2] = kBadPageTable; g_status[3] = (unsigned int)b;
                    }
                    seq_nk = 0;
                }
            }
            int k0, k1;
            split_range<C::kChunk, PAGED>(seq_nk, num_splits, per_split, split, k0, k1);
            const unsigned char* kb = k + (bh * Nk) * (long long)(D * KVB);
            const unsigned char* vb = v + (bh * Nk) * (long long)(D * KVB);
            for (int c0 = k0; c0 < k1; c0 += C::kChunk, ++it) {
                const int stage = it % C::kStages;
                const uint32_t round = it / C::kStages;
                if (round > 0 && !mbar_wait(&empty[stage], (round - 1) & 1, kWaitDecEmpty)) return;
                const int nk = min(C::kChunk, k1 - c0);
                const uint32_t bytes = (uint32_t)nk * D * KVB;
                unsigned char* dst = ring + stage * C::kStageBytes;
                long long src = (long long)c0 * (D * KVB);
                if (PAGED) {
                    int page = pages[c0 / pg.page_size];
                    if ((unsigned int)page >= (unsigned int)pg.num_pages) {
                        // a page outside the pool: flag it and read page 0 so that the pipeline completes
                        if (atomicCAS(&g_status[0], 0u, (unsigned int)FLASHD_ERR_SHAPE) == 0u) {
                            g_status[1] = blockIdx.x; g_status[2] = kBadPageTable; g_status[3] = (unsigned int)page;
                        }
                        page = 0;
                    }
                    src = (((long long)page * pg.H + head) * pg.page_size + c0 % pg.page_size) * (long long)(D * KVB);
                    kb = k;
                    vb = v;
                }
                mbar_arrive_expect_tx(&full[stage], 2 * bytes);
                bulk_load(dst, kb + src, bytes, &full[stage]);
                bulk_load(dst + C::kTileBytes, vb + src, bytes, &full[stage]);
            }
        }
        return;
    }

    // ---------------------------------------------------------- consumers
    const int sl = lane % C::kLanesPerRow;                      // 16-byte slice of the row
    const int g = warp * C::kRowsPerWarp + lane / C::kLanesPerRow;   // this lane's group
    uint32_t it = 0;
    uint32_t item_idx = 0;
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x, ++item_idx) {
        const long long row = item / num_splits;
        const int split = (int)(item - row * num_splits);
        int seq_nk = Nk;
        if (PAGED) {
            seq_nk = pg.seq_lens[(row / Nq) / pg.H];
            if (seq_nk < 0 || seq_nk > pg.max_pages * pg.page_size) seq_nk = 0;
        }
        int k0, k1;
        split_range<C::kChunk, PAGED>(seq_nk, num_splits, per_split, split, k0, k1);

        float qf[EL];
#pragma unroll
        for (int h = 0; h < EL / 8; ++h) {
            const uint4 qw = *reinterpret_cast<const uint4*>(q + row * D + sl * EL + h * 8);
            const uint32_t w[4] = {qw.x, qw.y, qw.z, qw.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                qf[8 * h + 2 * e] = bf16_lo(w[e]) * scale_log2e;
                qf[8 * h + 2 * e + 1] = bf16_hi(w[e]) * scale_log2e;
            }
        }
        float of[EL];
#pragma unroll
        for (int e = 0; e < EL; ++e) of[e] = 0.f;
        float L = -INFINITY;

        for (int c0 = k0; c0 < k1; c0 += C::kChunk, ++it) {
            const int stage = it % C::kStages;
            const uint32_t round = it / C::kStages;
            if (!mbar_wait(&full[stage], round & 1, kWaitDecFull)) return;
            const int nk = min(C::kChunk, k1 - c0);
            const unsigned char* ks = ring + stage * C::kStageBytes;
            const unsigned char* vs = ks + C::kTileBytes;

            float s[C::kKeysPerGroup];
            bool valid[C::kKeysPerGroup];
#pragma unroll
            for (int m = 0; m < C::kKeysPerGroup; ++m) {
                const int r = g + C::kGroups * m;
                valid[m] = r < nk;
                const uint4 kw = *reinterpret_cast<const uint4*>(ks + r * (D * KVB) + sl * 16);
                float kf[EL];
                widen_slice<KVB>(kw, kf);
                float acc = 0.f;
#pragma unroll
                for (int e = 0; e < EL; ++e) acc = fmaf(qf[e], kf[e], acc);
                s[m] = acc;
            }
#pragma unroll
            for (int sh = C::kLanesPerRow / 2; sh >= 1; sh >>= 1) {
#pragma unroll
                for (int m = 0; m < C::kKeysPerGroup; ++m) s[m] += __shfl_xor_sync(0xffffffffu, s[m], sh);
            }
            float ref = L;
#pragma unroll
            for (int m = 0; m < C::kKeysPerGroup; ++m) {
                s[m] = valid[m] ? s[m] : -INFINITY;
                ref = fmaxf(ref, s[m]);
            }
            if (ref != -INFINITY) {      // uniform within the group
                // log-sum-exp of {L_old, s_j} relative to a group-local reference
                const float e_old = ex2(L - ref);
                float p[C::kKeysPerGroup];
                float l = e_old;
#pragma unroll
                for (int m = 0; m < C::kKeysPerGroup; ++m) { p[m] = ex2(s[m] - ref); l += p[m]; }
                const float inv = rcp(l);
                const float alpha = e_old * inv;          // = 1 - W = exp(L_old - L_new)
                L = ref + lg2(l);                          // L_new
#pragma unroll
                for (int e = 0; e < EL; ++e) of[e] *= alpha;
#pragma unroll
                for (int m = 0; m < C::kKeysPerGroup; ++m) {
                    const int r = g + C::kGroups * m;
                    const float P = p[m] * inv;            // = exp(s_j - L_new)
                    uint4 vw = *reinterpret_cast<const uint4*>(vs + r * (D * KVB) + sl * 16);
                    if (!valid[m]) vw = make_uint4(0u, 0u, 0u, 0u);
                    float vf[EL];
                    widen_slice<KVB>(vw, vf);
#pragma unroll
                    for (int e = 0; e < EL; ++e) of[e] = fmaf(P, vf[e], of[e]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[stage]);
        }

        // ---- merge the CTA's group states, in group order, as super-keys
        if (item_idx > 0 && !mbar_wait(merge_free, (item_idx - 1) & 1, kWaitDecMergeFree)) return;
        {
            float* mine = merge + g * (D + 1);
#pragma unroll
            for (int e = 0; e < EL; ++e) mine[sl * EL + e] = of[e];
            if (sl == 0) mine[D] = L;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(merge_ready);
        if (!mbar_wait(merge_ready, item_idx & 1, kWaitDecMergeReady)) return;
        if (threadIdx.x < D) {
            const int c = threadIdx.x;
            float L_acc = -INFINITY, o_acc = 0.f;
            for (int gg = 0; gg < C::kGroups; ++gg) {
                const float W = superkey_weight(L_acc, merge[gg * (D + 1) + D]);
                o_acc = fmaf(merge[gg * (D + 1) + c] - o_acc, W, o_acc);
            }
            float* wp = workspace + (row * num_splits + split) * (long long)(D + 1);
            wp[c] = o_acc;
            if (c == 0) wp[D] = L_acc * kLn2;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(merge_free);
    }
}

// Combine: one CTA of D threads per query row; thread c owns output column c.
template <int D, typename TOut>
__global__ void __launch_bounds__(D)
splitk_combine_kernel(const float* __restrict__ workspace, TOut* __restrict__ o,
                      float* __restrict__ lse, int num_splits) {
    const long long row = blockIdx.x;
    const int c = threadIdx.x;
    const float* wp = workspace + row * num_splits * (long long)(D + 1);
    float L_acc = -INFINITY, o_acc = 0.f;
    for (int s = 0; s < num_splits; ++s) {
        const float W = superkey_weight(L_acc, wp[s * (D + 1) + D] * kLog2e);
        o_acc = fmaf(wp[s * (D + 1) + c] - o_acc, W, o_acc);
    }
    o[row * D + c] = from_f32<TOut>(o_acc);
    if (lse != nullptr && c == 0) lse[row] = L_acc * kLn2;
}

}  // namespace flashd
