// Grouped-query split-K FLASH-D decode: G query heads share one K/V head, and
// each may carry a few query positions (the last Nq positions of the sequence,
// causal among themselves): R = G*Nq <= 8 query rows per K/V head.
//
// One work item = (batch, K/V head, split).  The split's K and V rows cross HBM
// once and serve all G queries of the group, so the kernel is bound by the same
// K/V stream as the single-query split-K kernel while doing G times the
// arithmetic; that arithmetic is moved to the tensor cores (warp-level
// m16n8k16 products, the G <= 8 queries padded to the 16-row operand) so that
// the ALUs do not become the limit.
//
// A producer thread streams 128-key chunks of K and V into a shared-memory ring
// with tiled TMA loads (128-byte swizzle, so the matrix loads below are free of
// bank conflicts; rows past the end of the sequence read as zero).  Consumer
// warp w owns keys [16w, 16w+16) of every chunk and folds them into its own
// running state (L, o) per query with the group form of Algorithm 3 - the same
// step as the single-query kernel:
//     ref = max(L_old, max_j s_j), l = 2^(L_old-ref) + sum_j 2^(s_j-ref)
//     L_new = ref + log2 l,  P_j = 2^(s_j-ref)/l = exp(s_j - L_new)
//     o <- (2^(L_old-ref)/l) o + sum_j P_j v_j            Eq. (out-final) for the group
// so o stays normalised after every group of 16 keys and nothing is divided at
// the end.  The eight warp states are then merged as super-keys (Eq. (w-last),
// one-multiplier blend of Sec. IV-A) and written as one partial state per
// (query, split) in the workspace layout of the single-query kernel, so the
// same combine kernel finishes the job.
#pragma once

#include "flashd_decode.cuh"
#include "flashd_prefill.cuh"

namespace flashd {

template <int D>
struct GqaCfg {
    static constexpr int kChunk = 128;                           // keys per ring stage
    static constexpr int kPanels = D / 64;                       // 64-column (128-byte) swizzle panels
    static constexpr int kPanelBytes = kChunk * 128;
    static constexpr int kTileBytes = kPanels * kPanelBytes;     // K or V of one chunk
    static constexpr int kStageBytes = 2 * kTileBytes;
    static constexpr int kStages = (D == 128) ? 3 : 5;
    static constexpr int kConsumerWarps = kChunk / 16;           // 8
    static constexpr int kThreads = (kConsumerWarps + 1) * 32;
    static constexpr int kMaxG = 8;
    static constexpr int kMergeFloats = kConsumerWarps * kMaxG * (D + 1);
    static constexpr int kSmemBytes = kStages * kStageBytes + kMergeFloats * 4 + 256 + 1024;
};

enum { kWaitGqaFull = 0x300, kWaitGqaEmpty = 0x301, kWaitGqaMergeReady = 0x302, kWaitGqaMergeFree = 0x303 };

// Four 8x8 b16 matrices from shared memory; lane l supplies the address of row
// l%8 of matrix l/8.  Plain form: thread t receives elements (row t/4, columns
// 2(t%4), 2(t%4)+1) of each matrix; transposed form: (rows 2(t%4), 2(t%4)+1, column t/4).
__device__ __forceinline__ void ldsm_x4(uint32_t saddr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(saddr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t saddr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(saddr));
}

// D(16x8) += A(16x16, rows 8..15 zero) B(16x8), bf16 operands, fp32 accumulate.
// Only rows 0..7 of A are populated (a1 = a3 = 0), so only d0, d1 carry results;
// the accumulators of rows 8..15 are fed zeros and dropped.
__device__ __forceinline__ void mma_rows8(float& d0, float& d1, uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    [[maybe_unused]] float x2, x3;
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %10, %10};"
        : "+f"(d0), "+f"(d1), "=f"(x2), "=f"(x3)
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1), "f"(0.f));
}

// PAGED = true: K and V live in a page pool [num_pages, Hkv, page_size, D] (the tensor maps then
// cover (D, page_size, num_pages * Hkv)), sequence b owns the pages block_table[b][..] and has
// seq_lens[b] keys; split ranges are whole 128-key chunks, so a chunk never straddles two pages.
// Rows of a page past the sequence's end hold whatever the pool held: their weights are exactly
// zero, and their V entries are cleared in registers so that 0 x NaN cannot reach the output.
template <int D, bool PAGED = false>
__global__ void __launch_bounds__(GqaCfg<D>::kThreads, 1)
gqa_partial_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                   const __nv_bfloat16* __restrict__ q, float* __restrict__ workspace, int BHkv, int R, int Nq,
                   int causal, int Nk, float scale_log2e, int num_splits, const PagedKV pg) {
    using C = GqaCfg<D>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // swizzle atoms: 1 KB
    float* merge = reinterpret_cast<float*>(ring + C::kStages * C::kStageBytes);
    uint64_t* bars = reinterpret_cast<uint64_t*>(ring + C::kStages * C::kStageBytes + C::kMergeFloats * 4);
    uint64_t* full = bars;
    uint64_t* empty = bars + C::kStages;
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

    const long long n_items = (long long)BHkv * num_splits;
    const int per_split = (Nk + num_splits - 1) / num_splits;

    if (warp == C::kConsumerWarps) {
        // ------------------------------------------------------ producer
        if (lane != 0) return;
        uint32_t it = 0;
        for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
            const int bh = (int)(item / num_splits);
            const int split = (int)(item - (long long)bh * num_splits);
            int seq_nk = Nk, head = 0;
            const int* pages = nullptr;
            if (PAGED) {
                const int b = bh / pg.H;
                head = bh - b * pg.H;
                seq_nk = pg.seq_lens[b];
                pages = pg.block_table + (long long)b * pg.max_pages;
                if (seq_nk < 0 || seq_nk > pg.max_pages * pg.page_size) {
                    if (atomicCAS(&g_status[0], 0u, (unsigned int)FLASHD_ERR_SHAPE) == 0u) {
                        g_status[1] = blockIdx.x; g_status[2] = kBadPageTable; g_status[3] = (unsigned int)b;
                    }
                    seq_nk = 0;
                }
            }
            int k0, k1;
            split_range<C::kChunk, PAGED>(seq_nk, num_splits, per_split, split, k0, k1);
            for (int c0 = k0; c0 < k1; c0 += C::kChunk, ++it) {
                const int stage = it % C::kStages;
                const uint32_t round = it / C::kStages;
                if (round > 0 && !mbar_wait(&empty[stage], (round - 1) & 1, kWaitGqaEmpty)) return;
                unsigned char* dst = ring + stage * C::kStageBytes;
                int row0 = c0, slab = bh;
                if (PAGED) {
                    int page = pages[c0 / pg.page_size];
                    if ((unsigned int)page >= (unsigned int)pg.num_pages) {
                        if (atomicCAS(&g_status[0], 0u, (unsigned int)FLASHD_ERR_SHAPE) == 0u) {
                            g_status[1] = blockIdx.x; g_status[2] = kBadPageTable; g_status[3] = (unsigned int)page;
                        }
                        page = 0;
                    }
                    row0 = c0 % pg.page_size;
                    slab = page * pg.H + head;
                }
                mbar_arrive_expect_tx(&full[stage], C::kStageBytes);
#pragma unroll
                for (int p = 0; p < C::kPanels; ++p) {
                    tma_load_3d(dst + p * C::kPanelBytes, &map_k, p * 64, row0, slab, &full[stage]);
                    tma_load_3d(dst + C::kTileBytes + p * C::kPanelBytes, &map_v, p * 64, row0, slab, &full[stage]);
                }
            }
        }
        return;
    }

    // ---------------------------------------------------------- consumers
    const int grow = lane >> 2;            // query row (head g, position iq: grow = g*Nq + iq) of this lane's accumulators
    // keys [0, row_lim) are visible to the row: all of them, or, causal, up to the row's own
    // position Nk - Nq + iq (the queries are the last Nq positions of the sequence)
    int row_lim = causal ? Nk - Nq + (grow % Nq) + 1 : Nk;
    const int quad = lane & 3;
    constexpr int KS = D / 16;             // k-steps of the score product = pairs of output column tiles
    // shared-memory offsets of this lane's matrix rows (within a K or V tile)
    const int msel = lane >> 3;
    const int k_row = warp * 16 + (msel >> 1) * 8 + (lane & 7);      // K: matrices {keys lo, keys lo, keys hi, keys hi}
    const int k_csel = msel & 1;                                      //    16-byte column chunk {0, 1, 0, 1}
    const int v_row = warp * 16 + (msel & 1) * 8 + (lane & 7);       // V: matrices {keys lo, keys hi, keys lo, keys hi}
    const int v_csel = msel >> 1;                                     //    16-byte column chunk {0, 0, 1, 1}

    uint32_t it = 0;
    uint32_t item_idx = 0;
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x, ++item_idx) {
        const int bh = (int)(item / num_splits);
        const int split = (int)(item - (long long)bh * num_splits);
        int seq_nk = Nk;
        if (PAGED) {
            seq_nk = pg.seq_lens[bh / pg.H];
            if (seq_nk < 0 || seq_nk > pg.max_pages * pg.page_size) seq_nk = 0;
            row_lim = causal ? seq_nk - Nq + (grow % Nq) + 1 : seq_nk;
        }
        int k0, k1;
        split_range<C::kChunk, PAGED>(seq_nk, num_splits, per_split, split, k0, k1);

        // Q fragments of the group: row grow, columns 16 ks + 2 quad (+8)
        uint32_t qa0[KS], qa2[KS];
        {
            const __nv_bfloat16* qrow = q + ((long long)bh * R + grow) * D;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                qa0[ks] = 0u;
                qa2[ks] = 0u;
                if (grow < R) {
                    qa0[ks] = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * quad);
                    qa2[ks] = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + 2 * quad);
                }
            }
        }
        float oacc[2 * KS][2];
#pragma unroll
        for (int n = 0; n < 2 * KS; ++n) { oacc[n][0] = 0.f; oacc[n][1] = 0.f; }
        float L = -INFINITY;

        for (int c0 = k0; c0 < k1; c0 += C::kChunk, ++it) {
            const int stage = it % C::kStages;
            const uint32_t round = it / C::kStages;
            if (!mbar_wait(&full[stage], round & 1, kWaitGqaFull)) return;
            const uint32_t ks_base = smem_u32(ring + stage * C::kStageBytes);
            const uint32_t vs_base = ks_base + C::kTileBytes;

            if (c0 + warp * 16 < k1) {       // this warp's 16 keys hold at least one key of the split
                // ---- scores of 8 queries x 16 keys
                float s[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const int chunk = 2 * ks + k_csel;
                    uint32_t b[4];
                    ldsm_x4(ks_base + (chunk >> 3) * C::kPanelBytes + k_row * 128 + (((chunk & 7) ^ (k_row & 7)) << 4), b);
                    mma_rows8(s[0][0], s[0][1], qa0[ks], qa2[ks], b[0], b[1]);
                    mma_rows8(s[1][0], s[1][1], qa0[ks], qa2[ks], b[2], b[3]);
                }
                // ---- group step of Algorithm 3 on row grow (the four lanes of a quad share it)
                float mx = -INFINITY;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int key = c0 + warp * 16 + nt * 8 + 2 * quad + e;
                        s[nt][e] = key < min(k1, row_lim) ? s[nt][e] * scale_log2e : -INFINITY;
                        mx = fmaxf(mx, s[nt][e]);
                    }
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                // -inf only while the row has seen no visible key yet (causal rows at the end of
                // the sequence): the step then leaves the empty state as it is
                const float ref_raw = fmaxf(L, mx);
                const float ref = ref_raw == -INFINITY ? 0.f : ref_raw;
                const float e_old = ex2(L - ref);
                float p[2][2];
                float sum = 0.f;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) { p[nt][e] = ex2(s[nt][e] - ref); sum += p[nt][e]; }
                sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                const float l = e_old + sum;
                const float inv = l > 0.f ? rcp(l) : 0.f;
                const float alpha = e_old * inv;         // = exp(L_old - L_new)
                L = l > 0.f ? ref + lg2(l) : -INFINITY;
                const uint32_t pa0 = pack_bf16x2(p[0][0] * inv, p[0][1] * inv);   // keys 2 quad, +1
                const uint32_t pa2 = pack_bf16x2(p[1][0] * inv, p[1][1] * inv);   // keys 8 + 2 quad, +1
#pragma unroll
                for (int n = 0; n < 2 * KS; ++n) { oacc[n][0] *= alpha; oacc[n][1] *= alpha; }
                // V entries of keys past the sequence's end (this lane holds key rows 2 quad, 2 quad + 1
                // of the warp's lower and upper eight keys, packed as bf16 pairs)
                uint32_t vmask_lo = 0xffffffffu, vmask_hi = 0xffffffffu;
                if (PAGED) {
                    const int kb = c0 + warp * 16 + 2 * quad;
                    vmask_lo = (kb < seq_nk ? 0x0000ffffu : 0u) | (kb + 1 < seq_nk ? 0xffff0000u : 0u);
                    vmask_hi = (kb + 8 < seq_nk ? 0x0000ffffu : 0u) | (kb + 9 < seq_nk ? 0xffff0000u : 0u);
                }
                // ---- o += P V : output column tiles 2j, 2j+1 per matrix load
#pragma unroll
                for (int j = 0; j < KS; ++j) {
                    const int chunk = 2 * j + v_csel;
                    uint32_t b[4];
                    ldsm_x4_trans(vs_base + (chunk >> 3) * C::kPanelBytes + v_row * 128 + (((chunk & 7) ^ (v_row & 7)) << 4), b);
                    if (PAGED) { b[0] &= vmask_lo; b[1] &= vmask_hi; b[2] &= vmask_lo; b[3] &= vmask_hi; }
                    mma_rows8(oacc[2 * j][0], oacc[2 * j][1], pa0, pa2, b[0], b[1]);
                    mma_rows8(oacc[2 * j + 1][0], oacc[2 * j + 1][1], pa0, pa2, b[2], b[3]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[stage]);
        }

        // ---- merge the eight warp states per query, in warp order, as super-keys
        if (item_idx > 0 && !mbar_wait(merge_free, (item_idx - 1) & 1, kWaitGqaMergeFree)) return;
        {
            float* mine = merge + (warp * C::kMaxG + grow) * (D + 1);
#pragma unroll
            for (int n = 0; n < 2 * KS; ++n) {
                mine[n * 8 + 2 * quad] = oacc[n][0];
                mine[n * 8 + 2 * quad + 1] = oacc[n][1];
            }
            if (quad == 0) mine[D] = L;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(merge_ready);
        if (!mbar_wait(merge_ready, item_idx & 1, kWaitGqaMergeReady)) return;
        for (int idx = threadIdx.x; idx < R * D; idx += C::kConsumerWarps * 32) {
            const int gq = idx / D;
            const int c = idx - gq * D;
            float L_acc = -INFINITY, o_acc = 0.f;
#pragma unroll
            for (int w = 0; w < C::kConsumerWarps; ++w) {
                const float* st = merge + (w * C::kMaxG + gq) * (D + 1);
                const float W = superkey_weight(L_acc, st[D]);
                o_acc = fmaf(st[c] - o_acc, W, o_acc);
            }
            float* wp = workspace + (((long long)bh * R + gq) * num_splits + split) * (long long)(D + 1);
            wp[c] = o_acc;
            if (c == 0) wp[D] = L_acc * kLn2;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(merge_free);
    }
}

}  // namespace flashd
