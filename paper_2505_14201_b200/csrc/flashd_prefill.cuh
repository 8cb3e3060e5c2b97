// Tiled FLASH-D forward on the 5th-generation tensor cores (sm_100a).
//
// One CTA owns a pair of 128-row query tiles of one head and walks the key
// sequence in tiles of 128 keys.  The per-key step of Algorithm 3 with the
// division written out is, for x = s_i - L_{i-1} and L = s - ln w the carried state,
//     w_i = sigma(x) = e^x / (1 + e^x)             Eq. (w-last)
//     o_i = (o_{i-1} + e^x v_i) / (1 + e^x)        Eq. (out-final)
// Applied to a tile of keys as one group this becomes, per query row,
//     O_t = (O_{t-1} + sum_j e^{x_j} v_j) / (1 + sum_j e^{x_j}),   x_j = s_j - L_{t-1}
//     L_t = L_{t-1} + ln(1 + sum_j e^{x_j})
// and that is what the kernel evaluates (log2 units, c = scale*log2(e)):
//   S = Q K^T                      tcgen05.mma, operands in shared memory (TMA),
//                                  accumulator in tensor memory
//   per row (one thread per row):
//       ref   = max(L_{t-1}, max_j c*s_j)          tile-local reference, not carried;
//                                                  equals L_{t-1} unless a new key dominates
//       e_old = 2^(L_{t-1} - ref)                  (= 1 in the common case)
//       pt_j  = 2^(c*s_j - ref)                    (= e^{x_j} in the common case)
//       l_t   = e_old + sum_j pt_j ,  L_t = ref + log2 l_t
//   O~_t = beta_t O~_{t-1} + Pt V    beta_t = e_old / l_{t-1}: the division that closes
//                                    step t-1 is applied, as a reciprocal-multiply by the
//                                    correction warps, when step t opens; so the
//                                    accumulator holds the normalised output O_{t-1} (times
//                                    e_old) while the new keys are added, and the last
//                                    reciprocal 1/l_T is applied in the epilogue.
// There is no running maximum and no separate softmax denominator: the state per row
// is L alone (l_t is L_t - ref_t in the linear domain), one reciprocal per row and
// tile plays the part of the sigmoid's division.
//
// D = 256 runs a single query tile per CTA (warps 4-7 idle): the accumulator of one tile takes
// 256 tensor-memory columns and one Q tile 64 KB.  The scores then alternate between the two S
// regions, so that S(t+1) is computed under the weights of step t and P V(t) under those of t+1.
// Warp roles (16 warps): 0-3 weights of query tile 0, 4-7 weights of query tile 1,
// 8-11 correction + epilogue, 12 MMA issue (whole warp in uniform control flow, one elected
// lane issues), 13 TMA loads (one lane), 14-15 idle.
// Tensor memory (512 columns), D = 128: S0 | S1 | O0 | O1, P_i overlays the first 64
// columns of S_i as packed bf16 pairs and is handed to the P V product in two halves of 64
// keys; D = 64: S0 | S1 | P0 | P1 | O0 | O1.
// Operands: bf16 (tcgen05.mma kind::f16) or FP8-E4M3 (kind::f8f6f4, D = 128 or 256; the weights are then
// stored as E4M3 with a per-row power-of-two scale, see the weights warps).
// Every mbarrier wait is bounded; a wait that runs out records itself in the
// device status word, raises the CTA's abort flag and the CTA drains and exits.
#pragma once

#include <cuda.h>

#include "flashd_common.cuh"

namespace flashd {

// EB = bytes per element of Q, K, V and P: 2 (bf16, tcgen05.mma kind::f16) or 1 (FP8-E4M3,
// kind::f8f6f4; D = 128 or 256).  A product instruction covers 32 bytes of the contraction
// dimension: 16 bf16 or 32 E4M3 elements.
template <int D, int EB = 2>
struct PrefillCfg {
    static_assert(EB == 2 || (EB == 1 && (D == 128 || D == 256)), "E4M3 operands: D = 128 or 256");
    // D = 256: one query tile per CTA (its accumulator alone takes 256 of the 512 tensor-memory
    // columns, and one Q tile 64 KB of shared memory); D = 64, 128: two.
    static constexpr int kQTiles = (D == 256) ? 1 : 2;
    static constexpr int kItemRows = 128 * kQTiles;              // query rows of a work item
    // With one query tile the second S region is free: the scores alternate between the two
    // S regions step by step (P overlaying the region its scores came from), S(t+1) is computed
    // under the weights of step t and P V(t) under those of step t+1.  Everything indexed by
    // query tile in the two-tile schedule (S/P regions, s_full, p_half, p_full, alpha_full and
    // the slots of the per-row factors) is then indexed by the parity of the step.
    static constexpr bool kAltS = (kQTiles == 1);
    static constexpr int kBlockM = 128;
    static constexpr int kBlockN = 128;
    static constexpr int kPanels = D * EB / 128;                 // 128-byte swizzle panels (64 bf16 / 128 E4M3 columns)
    static constexpr int kPanelCols = 128 / EB;
    static constexpr int kStepsS = D * EB / 32;                  // product instructions of S = Q K^T
    static constexpr int kStepsPV = 128 * EB / 32;               // product instructions of O += P V (128 keys)
    static constexpr int kVStepBytes = (32 / EB) * 128;          // V rows (keys) of one instruction x 128 bytes
    static constexpr int kPCols = 128 * EB / 4;                  // tensor-memory columns of P (packed)
    static constexpr int kPanelBytes = 128 * 128;                // 128 rows x 128 bytes
    static constexpr int kTileBytes = kPanels * kPanelBytes;     // one Q / K / V tile
    static constexpr int kStages = (D * EB == 512) ? 2 : (D == 64) ? 6 : 4;   // K/V ring (tiles of 16 KB x panels)
    static constexpr int kThreads = 512;
    static constexpr int kBarriers = 22 + 2 * kStages;
    static constexpr int kSmemBytes = kQTiles * kTileBytes + kStages * kTileBytes + 3 * 2 * 128 * 4 + kBarriers * 8 + 64 + 1024;
    static constexpr uint32_t kTmemCols = 512;
    // At D = 64 tensor memory has room for P next to S (S0 S1 P0 P1 O0 O1 = 512 columns), so
    // the score product of step t+1 can run while the weights of step t are computed
    // (lookahead 2).  At D = 128 P has to overlay S and S(t+1) follows P V(t) (lookahead 1).
    static constexpr int kLookahead = (D == 64) ? 2 : 1;
    static constexpr uint32_t kColS0 = 0, kColS1 = 128;
    static constexpr uint32_t kColP0 = (D == 64) ? 256 : kColS0, kColP1 = (D == 64) ? 320 : kColS1;
    static constexpr uint32_t kColO0 = (D == 64) ? 384 : 256, kColO1 = kColO0 + D;
};

enum {
    kWaitQFull = 0x200, kWaitQEmpty, kWaitKVFull, kWaitKVEmpty, kWaitSFull, kWaitPFull,
    kWaitAlphaFull, kWaitPVDone, kWaitOReady, kWaitSFree
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* map, int c0, int c1, int c2,
                                            uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
// D[tmem] (+)= A * B with A in shared memory (mma_ss64) or tensor memory (mma_ts64), B in shared
// memory; 64-bit descriptors: one instruction per product, nothing to compute at issue time
template <int EB = 2>
__device__ __forceinline__ void mma_ss64(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
    if constexpr (EB == 2) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
    }
}
template <int EB = 2>
__device__ __forceinline__ void mma_ts64(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
    if constexpr (EB == 2) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], %2, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
    }
}
// 16 consecutive 32-bit columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(taddr)
        : "memory");
}
// four fp32 -> four E4M3 codes (round to nearest even, saturating at +-448), first argument in the low byte
__device__ __forceinline__ uint32_t pack_e4m3x4(float a, float b, float c, float d) {
    uint32_t r;
    asm("{\n\t.reg .b16 lo, hi;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
        "mov.b32 %0, {lo, hi};\n\t}"
        : "=r"(r) : "f"(a), "f"(b), "f"(c), "f"(d));
    return r;
}
__device__ __forceinline__ uint64_t desc64(uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | lo; }
// 32 consecutive 32-bit columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
          "r"(taddr)
        : "memory");
}
// setmaxnreg is a warpgroup instruction: the four warps of a warpgroup (0-3, 4-7, 8-11, 12-15)
// must all execute it with the same value, or they wait for each other forever.
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

// Shared-memory matrix descriptor, 128-byte swizzle, split in two 32-bit words.
// Low word: start address >> 4 (bits 0-13) and leading-dimension byte offset >> 4
// (bits 16-29).  High word: stride-dimension byte offset >> 4 (bits 0-13),
// descriptor version 1 (bit 14), swizzle mode 2 = 128 bytes (bits 29-31).  Moving
// the start address inside a tile only changes the low word.
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t saddr, uint32_t lbo) {
    return ((saddr & 0x3FFFFu) >> 4) | ((lbo >> 4) << 16);
}
__host__ __device__ constexpr uint32_t smem_desc_hi(uint32_t sbo) {
    return (sbo >> 4) | (1u << 14) | (2u << 29);
}
// Instruction descriptor: bf16 x bf16 -> fp32 (operand format code 1 of kind::f16) or
// E4M3 x E4M3 -> fp32 (format code 0 of kind::f8f6f4); A K-major, B K-major (b_mn = 0) or
// MN-major (1).  Bits: 4-5 accumulator format (1 = fp32), 7-9 A format, 10-12 B format,
// 16 B major, 17-22 N / 8, 24-28 M / 16.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, int b_mn, int eb = 2) {
    return (1u << 4) | ((eb == 2 ? 1u : 0u) << 7) | ((eb == 2 ? 1u : 0u) << 10) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

struct PrefillParams {
    void* o;            // [B*H, Nq, D] bf16 or fp32
    float* lse;         // nullable, [B*H, Nq]
    int BH, Nq, Nk;
    float scale_log2e;  // scale * log2(e)
    int causal;
    int out_f32;
    int n_qpairs;       // ceil(Nq / rows of a work item)
    int n_work;         // BH * n_qpairs
};


// Wait bounded to about two seconds; also leaves when another thread of the CTA
// has raised the abort flag.
__device__ __forceinline__ bool pf_wait(uint64_t* bar, uint32_t parity, unsigned int which,
                                        volatile uint32_t* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_ns() - t0 > kWaitLimitNs) break;
    }
    report_timeout(which, parity);
    *abort_flag = 1;
    return false;
}

// Non-blocking look at a barrier phase (a later pf_wait covers a miss).
__device__ __forceinline__ uint32_t mbar_test(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok;
}
// One lane of a converged warp
__device__ __forceinline__ uint32_t elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
    return pred;
}

template <int D, int EB = 2>
__global__ void __launch_bounds__(512, 1)
prefill_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const PrefillParams prm) {
    using C = PrefillCfg<D, EB>;
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment for the swizzled tiles
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* sQ = smem;                               // 2 tiles
    unsigned char* sKV = smem + C::kQTiles * C::kTileBytes; // kStages tiles
    // Per-row factors handed from the weights warps to the correction warps, [slot][tile][row].
    // Two slots used alternately: message n of a tile is written only after the product that
    // needed message n-1 has been issued, and that product waits for the correction warps to
    // have consumed message n-1, so message n-2 (same slot) is never overwritten unread.
    // The reciprocal that closes the last step of a work item travels on a channel of its own
    // (sFinal / final_full): it is posted without waiting for anything, so on the shared channel
    // it could complete a second barrier phase before the first one was observed.
    float* sAlpha = reinterpret_cast<float*>(sKV + C::kStages * C::kTileBytes);   // [2][2][128]
    float* sFinal = sAlpha + 512;                                                  // [2][128]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sFinal + 256);
    uint64_t* q_full = bars;            // [2]
    uint64_t* q_empty = bars + 2;       // [2]
    uint64_t* s_full = bars + 4;        // [2]
    uint64_t* p_full = bars + 6;        // [2]
    uint64_t* alpha_full = bars + 8;    // [2]
    uint64_t* pv_done = bars + 12;      // [2]
    uint64_t* o_ready = bars + 14;      // [2]
    uint64_t* final_full = bars + 16;   // [2]
    uint64_t* s_free = bars + 18;       // [2]  S has been read into registers (lookahead 2 only)
    uint64_t* p_half = bars + 20;       // [2]  first 64 keys of P stored (lookahead 1 only)
    uint64_t* kv_full = bars + 22;                 // [kStages]
    uint64_t* kv_empty = bars + 22 + C::kStages;   // [kStages]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C::kBarriers);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&q_full[i], 1);
            mbar_init(&q_empty[i], 1);
            mbar_init(&s_full[i], 1);
            mbar_init(&p_full[i], 128);
            mbar_init(&alpha_full[i], 128);
            mbar_init(&final_full[i], 128);
            mbar_init(&s_free[i], 128);
            mbar_init(&p_half[i], 128);
            mbar_init(&pv_done[i], 1);
            mbar_init(&o_ready[i], 128);
        }
        for (int s = 0; s < C::kStages; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1); }
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 0) {
        tmem_alloc(tmem_slot, C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: the set-up above may run while the previous kernel of the
    // stream drains; nothing of global memory is touched before that kernel has completed and its
    // writes are visible.  The next kernel of the stream is released in the same way when every
    // CTA of this grid has begun its last work item (it waits for this grid to complete before
    // it touches memory).
    asm volatile("griddepcontrol.wait;" ::: "memory");

    const int Nq = prm.Nq, Nk = prm.Nk;
    const int n_kt_all = (Nk + 127) >> 7;
    // Work items are ordered heaviest first (late query tiles when causal) and dealt to the
    // CTAs in snake order: round n goes 0..G-1 when n is even and G-1..0 when n is odd, which
    // evens out the per-CTA totals of a descending cost sequence without a dynamic scheduler.
    auto work_index = [&](int n) -> int {
        const int g = (int)gridDim.x, k = (int)blockIdx.x;
        return n * g + ((n & 1) ? g - 1 - k : k);
    };
    // key tiles needed by query tile i (rows q0 .. q0+127) of a work item; 0 if the tile is empty
    auto n_tiles = [&](int q0) -> int {
        if (q0 >= Nq) return 0;
        if (!prm.causal) return n_kt_all;
        const int lim = min(Nk, q0 + 128);
        return (lim + 127) >> 7;
    };

    if (warp == 13) {
        // ================================================================ TMA loader
        reg_dec<96>();
        if (lane == 0) {
            uint32_t kv_it = 0;
            uint32_t n_q[2] = {0, 0};     // uses of each Q buffer so far
            for (int nw = 0, w = work_index(0); w < prm.n_work; w = work_index(++nw)) {
                if (work_index(nw + 1) >= prm.n_work) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
                const int qpair = prm.n_qpairs - 1 - w / prm.BH;
                const int bh = w % prm.BH;
                const int q0 = qpair * C::kItemRows;
                const int T0 = n_tiles(q0), T1 = (C::kQTiles == 2) ? n_tiles(q0 + 128) : 0;
                const int T = max(T0, T1);
                for (int i = 0; i < 2; ++i) {
                    if ((i == 0 ? T0 : T1) == 0) continue;
                    if (n_q[i] > 0 && !pf_wait(&q_empty[i], (n_q[i] - 1) & 1, kWaitQEmpty, abort_flag)) goto done;
                    ++n_q[i];
                    mbar_arrive_expect_tx(&q_full[i], C::kTileBytes);
                    for (int p = 0; p < C::kPanels; ++p)
                        tma_load_3d(sQ + i * C::kTileBytes + p * C::kPanelBytes, &map_q, p * C::kPanelCols, q0 + i * 128, bh,
                                    &q_full[i]);
                }
                // ring order = order of use: K0 V0 K1 V1 ... (two tiles), K0 K1 V0 K2 V1 ... (alternating S)
                for (int n = 0; n < 2 * T; ++n, ++kv_it) {
                    int kv = n & 1, t = n >> 1;
                    if (C::kAltS) {
                        if (n < 2 && n < T) { kv = 0; t = n; }                       // K0, K1
                        else {
                            const int m = n - min(T, 2);                             // V0 K2 V1 K3 ... then the last V's
                            const int pairs = max(T - 2, 0);                         // (V, K) pairs
                            if (m < 2 * pairs) { kv = (m & 1) ? 0 : 1; t = (m & 1) ? (m >> 1) + 2 : (m >> 1); }
                            else { kv = 1; t = pairs + (m - 2 * pairs); }
                        }
                    }
                    const int stage = kv_it % C::kStages;
                    const uint32_t round = kv_it / C::kStages;
                    if (round > 0 && !pf_wait(&kv_empty[stage], (round - 1) & 1, kWaitKVEmpty, abort_flag)) goto done;
                    mbar_arrive_expect_tx(&kv_full[stage], C::kTileBytes);
                    for (int p = 0; p < C::kPanels; ++p)
                        tma_load_3d(sKV + stage * C::kTileBytes + p * C::kPanelBytes, kv == 0 ? &map_k : &map_v,
                                    p * C::kPanelCols, t * 128, bh, &kv_full[stage]);
                }
            }
        }
    } else if (warp == 12) {
        // ================================================================ MMA issue
        // The whole warp runs the loop (uniform control flow, waits by all lanes); one elected
        // lane issues the products and the commits.  The barriers the next batch of products
        // will need are looked at between the products of the current batch, while the tensor
        // pipe still has work queued, so that in the common case no wait sits between batches.
        reg_dec<96>();
        {
            const uint32_t leader = elect_one();
            constexpr uint32_t idesc_s = make_idesc(128, 128, 0, EB);
            constexpr uint32_t idesc_o = make_idesc(128, D, 1, EB);
            const uint32_t tS[2] = {tmem_base + C::kColS0, tmem_base + C::kColS1};
            const uint32_t tO[2] = {tmem_base + C::kColO0, tmem_base + C::kColO1};
            const uint32_t tP[2] = {tmem_base + C::kColP0, tmem_base + C::kColP1};
            uint32_t kv_it = 0;
            uint32_t n_ph0 = 0, n_ph1 = 0;
            uint32_t n_p0 = 0, n_p1 = 0, n_or0 = 0, n_or1 = 0, n_qf0 = 0, n_qf1 = 0, n_sf0 = 0, n_sf1 = 0;
            constexpr uint32_t desc_hi = smem_desc_hi(1024);
            const uint32_t q_lo[2] = {smem_desc_lo(smem_u32(sQ), 16), smem_desc_lo(smem_u32(sQ + C::kTileBytes), 16)};
            const uint32_t k_lo0 = smem_desc_lo(smem_u32(sKV), 16);
            const uint32_t v_lo0 = smem_desc_lo(smem_u32(sKV), C::kPanelBytes);
            constexpr int KS = C::kStepsS;
            constexpr int KP = C::kStepsPV;
            constexpr int LA = C::kLookahead;
            auto koff = [](int ks) -> uint32_t { return (uint32_t)(((ks >> 2) * C::kPanelBytes + (ks & 3) * 32) >> 4); };
            // products of one batch; mid(ks) runs on all lanes after product ks
            auto fire_S = [&](int i, int stage, auto&& mid) {
                const uint32_t ka = k_lo0 + stage * (C::kTileBytes >> 4);
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    if (leader) mma_ss64<EB>(tS[i], desc64(q_lo[C::kAltS ? 0 : i] + koff(ks), desc_hi), desc64(ka + koff(ks), desc_hi), idesc_s, ks > 0);
                    __syncwarp();
                    mid(ks * (8 / KS));
                }
            };
            auto fire_PV_part = [&](int i, int stage, bool first, int part) {      // keys 64*part .. 64*part+63
                const uint32_t va = v_lo0 + stage * (C::kTileBytes >> 4);
#pragma unroll
                for (int kk = 0; kk < KP / 2; ++kk) {
                    const int ks = part * (KP / 2) + kk;
                    if (leader) mma_ts64<EB>(tO[C::kAltS ? 0 : i], tP[i] + ks * 8, desc64(va + ks * (C::kVStepBytes >> 4), desc_hi), idesc_o, (!first) || ks > 0);
                    __syncwarp();
                }
            };
            auto fire_PV = [&](int i, int stage, bool first, auto&& mid) {
                const uint32_t va = v_lo0 + stage * (C::kTileBytes >> 4);
#pragma unroll
                for (int ks = 0; ks < KP; ++ks) {
                    if (leader) mma_ts64<EB>(tO[i], tP[i] + ks * 8, desc64(va + ks * (C::kVStepBytes >> 4), desc_hi), idesc_o, (!first) || ks > 0);
                    __syncwarp();
                    mid(ks * (8 / KP));
                }
            };
            auto commit = [&](uint64_t* bar) {
                if (leader) tc_commit(bar);
                __syncwarp();
            };
            bool early0 = false;        // S_0(0) of the work item about to start has been issued already
            uint32_t gstep = 0;         // steps so far on this CTA (alternating S: region of a step = its parity)
            uint32_t n_sb[2] = {0, 0};  // alternating S: uses of p_half / p_full of each region
            for (int nw = 0, w = work_index(0); w < prm.n_work; w = work_index(++nw)) {
                const int qpair = prm.n_qpairs - 1 - w / prm.BH;
                const int q0 = qpair * C::kItemRows;
                const int T0 = n_tiles(q0), T1 = (C::kQTiles == 2) ? n_tiles(q0 + 128) : 0;
                const int T = max(T0, T1);
                auto stage_of = [&](uint32_t it) { return (int)(it % C::kStages); };
                auto parity_of = [&](uint32_t it) { return (it / C::kStages) & 1u; };
                if constexpr (C::kAltS) {
                    // ---- one query tile, scores alternating between the two S regions.
                    // Order on the tensor pipe: S(0) S(1) | P V(0) S(2) | P V(1) S(3) | ...; S(t+2) goes
                    // into the region P V(t) has just read P from (same issuing thread: in order).
                    auto none1 = [](int) {};
                    uint32_t r = kv_it;                      // ring position, in order of use
                    for (int u = 0; u < 2 && u < T; ++u, ++r) {
                        const int b = (int)((gstep + u) & 1);
                        if (!pf_wait(&kv_full[stage_of(r)], parity_of(r), kWaitKVFull, abort_flag)) goto done;
                        if (u == 0) { if (!pf_wait(&q_full[0], n_qf0 & 1, kWaitQFull, abort_flag)) goto done; ++n_qf0; }
                        tc_fence_after();
                        fire_S(b, stage_of(r), none1);
                        commit(&s_full[b]);
                        if (u + 1 == T) commit(&q_empty[0]);
                        commit(&kv_empty[stage_of(r)]);
                    }
                    for (int t = 0; t < T; ++t) {
                        const int b = (int)((gstep + t) & 1);
                        if (!pf_wait(&kv_full[stage_of(r)], parity_of(r), kWaitKVFull, abort_flag)) goto done;
                        if (!pf_wait(&o_ready[0], n_or0 & 1, kWaitOReady, abort_flag)) goto done;
                        ++n_or0;
                        if (!pf_wait(&p_half[b], n_sb[b] & 1, kWaitPFull, abort_flag)) goto done;
                        tc_fence_after();
                        fire_PV_part(b, stage_of(r), t == 0, 0);
                        if (!pf_wait(&p_full[b], n_sb[b] & 1, kWaitPFull, abort_flag)) goto done;
                        ++n_sb[b];
                        tc_fence_after();
                        fire_PV_part(b, stage_of(r), false, 1);
                        commit(&pv_done[0]);
                        commit(&kv_empty[stage_of(r)]);
                        ++r;
                        if (t + 2 < T) {
                            if (!pf_wait(&kv_full[stage_of(r)], parity_of(r), kWaitKVFull, abort_flag)) goto done;
                            tc_fence_after();
                            fire_S(b, stage_of(r), none1);
                            commit(&s_full[b]);
                            if (t + 3 == T) commit(&q_empty[0]);
                            commit(&kv_empty[stage_of(r)]);
                            ++r;
                        }
                    }
                    kv_it += 2 * T;
                    gstep += T;
                    continue;
                }
                // "known complete" flags of the next unconsumed phase of each barrier
                uint32_t e_sf0 = 0, e_sf1 = 0, e_pf0 = 0, e_pf1 = 0, e_or0 = 0, e_or1 = 0, e_kvv = 0, e_kvk = 0;
                auto none = [](int) {};
                // prologue: S_i(0) .. S_i(LA-1)
                for (int u = 0; u < LA && u < T; ++u) {
                    const uint32_t it_k = kv_it + 2 * u;
                    if (!pf_wait(&kv_full[stage_of(it_k)], parity_of(it_k), kWaitKVFull, abort_flag)) goto done;
                    if (u == 0 && early0) {
                        early0 = false;
                    } else if (u < T0) {
                        if (u == 0) { if (!pf_wait(&q_full[0], n_qf0 & 1, kWaitQFull, abort_flag)) goto done; ++n_qf0; }
                        else { if (!pf_wait(&s_free[0], n_sf0 & 1, kWaitSFree, abort_flag)) goto done; ++n_sf0; }
                        tc_fence_after();
                        fire_S(0, stage_of(it_k), none);
                        commit(&s_full[0]);
                        if (u + 1 == T0) commit(&q_empty[0]);
                    }
                    if (u < T1) {
                        if (u == 0) { if (!pf_wait(&q_full[1], n_qf1 & 1, kWaitQFull, abort_flag)) goto done; ++n_qf1; }
                        else { if (!pf_wait(&s_free[1], n_sf1 & 1, kWaitSFree, abort_flag)) goto done; ++n_sf1; }
                        tc_fence_after();
                        fire_S(1, stage_of(it_k), none);
                        commit(&s_full[1]);
                        if (u + 1 == T1) commit(&q_empty[1]);
                    }
                    commit(&kv_empty[stage_of(it_k)]);
                }
                for (int t = 0; t < T; ++t) {
                    const uint32_t it_v = kv_it + 2 * t + 1;
                    const uint32_t it_kn = kv_it + 2 * (t + LA);
                    const int st_v = stage_of(it_v), st_k = stage_of(it_kn);
                    const bool pv0 = t < T0, pv1 = t < T1, s0 = t + LA < T0, s1 = t + LA < T1;
                    const bool nxt0 = t + 1 < T0;      // PV_0(t+1) exists
                    if (!e_kvv && !pf_wait(&kv_full[st_v], parity_of(it_v), kWaitKVFull, abort_flag)) goto done;
                    e_kvv = 0;
                    if (pv0 && LA == 1) {
                        // P overlays S, so S_0(t+1) has to follow P V_0(t) and the chain per tile is
                        // weights -> P V -> S -> weights: the first four products (keys 0-63) are
                        // issued under the second half of the weights step
                        if (!e_or0 && !pf_wait(&o_ready[0], n_or0 & 1, kWaitOReady, abort_flag)) goto done;
                        if (!pf_wait(&p_half[0], n_ph0 & 1, kWaitPFull, abort_flag)) goto done;
                        e_or0 = 0; ++n_or0; ++n_ph0;
                        tc_fence_after();
                        fire_PV_part(0, st_v, t == 0, 0);
                        if (s0 || s1) e_kvk = mbar_test(&kv_full[st_k], parity_of(it_kn));
                        if (!pf_wait(&p_full[0], n_p0 & 1, kWaitPFull, abort_flag)) goto done;
                        e_pf0 = 0; ++n_p0;
                        tc_fence_after();
                        fire_PV_part(0, st_v, false, 1);
                        commit(&pv_done[0]);
                    } else if (pv0) {
                        if (!e_pf0 && !pf_wait(&p_full[0], n_p0 & 1, kWaitPFull, abort_flag)) goto done;
                        if (!e_or0 && !pf_wait(&o_ready[0], n_or0 & 1, kWaitOReady, abort_flag)) goto done;
                        e_pf0 = 0; e_or0 = 0; ++n_p0; ++n_or0;
                        tc_fence_after();
                        fire_PV(0, st_v, t == 0, [&](int ks) {
                            if (ks == 2 && (s0 || s1)) e_kvk = mbar_test(&kv_full[st_k], parity_of(it_kn));
                            if (ks == 4 && s0 && LA > 1) e_sf0 = mbar_test(&s_free[0], n_sf0 & 1);
                            if (ks == 4 && !s0 && pv1) e_pf1 = mbar_test(&p_full[1], n_p1 & 1);
                            if (ks == 5 && !s0 && pv1) e_or1 = mbar_test(&o_ready[1], n_or1 & 1);
                        });
                        commit(&pv_done[0]);
                    }
                    if (s0) {
                        if (!e_kvk && !pf_wait(&kv_full[st_k], parity_of(it_kn), kWaitKVFull, abort_flag)) goto done;
                        e_kvk = 1;      // stays known for S_1 of this step
                        if (LA > 1) {
                            if (!e_sf0 && !pf_wait(&s_free[0], n_sf0 & 1, kWaitSFree, abort_flag)) goto done;
                            e_sf0 = 0; ++n_sf0;
                        }
                        tc_fence_after();
                        fire_S(0, st_k, [&](int ks) {
                            if (ks == 2 && pv1) e_pf1 = mbar_test(&p_full[1], n_p1 & 1);
                            if (ks == 4 && pv1) e_or1 = mbar_test(&o_ready[1], n_or1 & 1);
                        });
                        commit(&s_full[0]);
                        if (t + LA + 1 == T0) commit(&q_empty[0]);
                    }
                    if (LA > 1 && t == T0 - 1) {
                        // Tile 0 has had its last products of this work item.  Its first score product
                        // of the NEXT work item does not have to wait for tile 1 to finish: S_0 is free
                        // (its weights warps are past their last step), so if the next Q_0 and K(0)
                        // have arrived it is issued here, and tile 0's weights start the next item
                        // while tile 1 still closes this one (c1: +1.7 %).  Not at lookahead 1: there
                        // it pulls the two tiles into phase, which costs more than it saves (c3: -2.5 %).
                        const int wn = work_index(nw + 1);
                        if (wn < prm.n_work) {
                            const int T0n = n_tiles((prm.n_qpairs - 1 - wn / prm.BH) * C::kItemRows);
                            const uint32_t it_k0 = kv_it + 2 * T;
                            if (T0n > 0 && mbar_test(&q_full[0], n_qf0 & 1) &&
                                mbar_test(&kv_full[stage_of(it_k0)], parity_of(it_k0))) {
                                ++n_qf0;
                                tc_fence_after();
                                fire_S(0, stage_of(it_k0), none);
                                commit(&s_full[0]);
                                if (T0n == 1) commit(&q_empty[0]);
                                early0 = true;
                            }
                        }
                    }
                    if (pv1 && LA == 1) {
                        if (!e_or1 && !pf_wait(&o_ready[1], n_or1 & 1, kWaitOReady, abort_flag)) goto done;
                        if (!pf_wait(&p_half[1], n_ph1 & 1, kWaitPFull, abort_flag)) goto done;
                        e_or1 = 0; ++n_or1; ++n_ph1;
                        tc_fence_after();
                        fire_PV_part(1, st_v, t == 0, 0);
                        if (s1 && !e_kvk) e_kvk = mbar_test(&kv_full[st_k], parity_of(it_kn));
                        if (!pf_wait(&p_full[1], n_p1 & 1, kWaitPFull, abort_flag)) goto done;
                        e_pf1 = 0; ++n_p1;
                        tc_fence_after();
                        fire_PV_part(1, st_v, false, 1);
                        commit(&pv_done[1]);
                    } else if (pv1) {
                        if (!e_pf1 && !pf_wait(&p_full[1], n_p1 & 1, kWaitPFull, abort_flag)) goto done;
                        if (!e_or1 && !pf_wait(&o_ready[1], n_or1 & 1, kWaitOReady, abort_flag)) goto done;
                        e_pf1 = 0; e_or1 = 0; ++n_p1; ++n_or1;
                        tc_fence_after();
                        fire_PV(1, st_v, t == 0, [&](int ks) {
                            if (ks == 2 && s1 && !e_kvk) e_kvk = mbar_test(&kv_full[st_k], parity_of(it_kn));
                            if (ks == 4 && s1 && LA > 1) e_sf1 = mbar_test(&s_free[1], n_sf1 & 1);
                            if (ks == 4 && !s1 && t + 1 < T) e_kvv = mbar_test(&kv_full[stage_of(it_v + 2)], parity_of(it_v + 2));
                            if (ks == 5 && !s1 && nxt0) e_pf0 = mbar_test(&p_full[0], n_p0 & 1);
                            if (ks == 6 && !s1 && nxt0) e_or0 = mbar_test(&o_ready[0], n_or0 & 1);
                        });
                        commit(&pv_done[1]);
                    }
                    if (s1) {
                        if (!e_kvk && !pf_wait(&kv_full[st_k], parity_of(it_kn), kWaitKVFull, abort_flag)) goto done;
                        if (LA > 1) {
                            if (!e_sf1 && !pf_wait(&s_free[1], n_sf1 & 1, kWaitSFree, abort_flag)) goto done;
                            e_sf1 = 0; ++n_sf1;
                        }
                        tc_fence_after();
                        fire_S(1, st_k, [&](int ks) {
                            if (ks == 0 && t + 1 < T) e_kvv = mbar_test(&kv_full[stage_of(it_v + 2)], parity_of(it_v + 2));
                            if (ks == 2 && nxt0) e_pf0 = mbar_test(&p_full[0], n_p0 & 1);
                            if (ks == 4 && nxt0) e_or0 = mbar_test(&o_ready[0], n_or0 & 1);
                        });
                        commit(&s_full[1]);
                        if (t + LA + 1 == T1) commit(&q_empty[1]);
                    }
                    e_kvk = 0;
                    commit(&kv_empty[st_v]);
                    if (t + LA < T) commit(&kv_empty[st_k]);
                }
                kv_it += 2 * T;
            }
        }
    } else if (warp < 8) {
        // ================================================================ softmax (weight recurrence)
        reg_inc<168>();
        const int i = warp >> 2;                       // query tile of this warpgroup
        const int row = threadIdx.x & 127;             // row within the tile = tensor-memory lane
        const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
        const float c = prm.scale_log2e;
        uint32_t n_s[2] = {0, 0}, n_ae = 0, n_pk = 0;
        uint32_t gstep = 0;                            // steps so far (alternating S: region of a step = its parity)
        for (int nw = 0, w = work_index(0); w < prm.n_work; w = work_index(++nw)) {
            const int qpair = prm.n_qpairs - 1 - w / prm.BH;
            const int bh = w % prm.BH;
            const int q0 = qpair * C::kItemRows + i * 128;
            const int Ti = (i < C::kQTiles) ? n_tiles(q0) : 0;
            const int gi = q0 + row;                   // global query index of this thread's row
            const int limit = prm.causal ? min(Nk, gi + 1) : Nk;   // keys [0, limit) are visible
            float L = -INFINITY;                       // log2-domain state: L = (s_i - ln w_i) * log2(e)
            float inv_l = 1.f;                         // 1 / l of the previous tile
            float K_prev = 0.f;                        // exponent offset of the stored weights (E4M3 only)
            for (int t = 0; t < Ti; ++t) {
                // region of this step's scores and weights, and index of its barriers: the query
                // tile, or, with one tile and alternating S regions, the parity of the step
                const int bi = C::kAltS ? (int)((gstep + t) & 1) : i;
                const uint32_t tS = tmem_base + (bi == 0 ? C::kColS0 : C::kColS1) + lane_sel;
                const uint32_t tP = tmem_base + (bi == 0 ? C::kColP0 : C::kColP1) + lane_sel;
                if (!pf_wait(&s_full[bi], n_s[bi] & 1, kWaitSFull, abort_flag)) goto done;
                ++n_s[bi];
                tc_fence_after();
                float s[128];
#pragma unroll
                for (int cb = 0; cb < 4; ++cb) tmem_ld32(tS + cb * 32, reinterpret_cast<uint32_t*>(s) + cb * 32);
                tc_wait_ld();
                if (C::kLookahead > 1 && t + 1 < Ti) {
                    // S is in registers: the score product of the next step may overwrite it
                    tc_fence_before();
                    mbar_arrive(&s_free[i]);
                }
                const int n0 = t * 128;
                if (n0 + 128 > Nk || (prm.causal && n0 + 127 > q0)) {
#pragma unroll
                    for (int j = 0; j < 128; ++j) s[j] = (n0 + j < limit) ? s[j] : (c >= 0.f ? -INFINITY : INFINITY);
                }
                // tile-local reference: max over {L_{t-1}, c*s_j}
                float m0 = s[0], m1 = s[1], m2 = s[2], m3 = s[3];     // four chains: short dependent latency
                if (c >= 0.f) {
#pragma unroll
                    for (int j = 4; j < 124; j += 8) {
                        m0 = max3(m0, s[j], s[j + 1]); m1 = max3(m1, s[j + 2], s[j + 3]);
                        m2 = max3(m2, s[j + 4], s[j + 5]); m3 = max3(m3, s[j + 6], s[j + 7]);
                    }
                    m0 = max3(m0, s[124], s[125]); m1 = max3(m1, s[126], s[127]);
                    m0 = fmaxf(max3(m0, m1, m2), m3);
                } else {
#pragma unroll
                    for (int j = 4; j < 124; j += 8) {
                        m0 = min3(m0, s[j], s[j + 1]); m1 = min3(m1, s[j + 2], s[j + 3]);
                        m2 = min3(m2, s[j + 4], s[j + 5]); m3 = min3(m3, s[j + 6], s[j + 7]);
                    }
                    m0 = min3(m0, s[124], s[125]); m1 = min3(m1, s[126], s[127]);
                    m0 = fminf(min3(m0, m1, m2), m3);
                }
                const float ref = fmaxf(L, m0 * c);
                const float e_old = ex2(L - ref);            // 0 for the first tile (L = -inf), else usually 1
                // beta = e_old / l_{t-1}: closes step t-1 (its division) and opens step t.
                // The hand-off has no back-pressure barrier, so message n+1 may only be posted
                // once message n is known to be consumed.  With lookahead 1 that follows from
                // the order of the products (S(t) is issued after P V(t-1), which needed the
                // correction of step t-1).  With lookahead 2 S(t) runs ahead, so the message is
                // posted below, after the wait for P V(t-1) that the P store needs anyway.
                float beta = e_old * inv_l;
                // E4M3 weights: in this form the weights of a late tile are small against the mass
                // already accumulated (x_j = s_j - L_{t-1} is far below zero on long rows), below
                // E4M3's normal range (2^-6).  They are therefore stored times 2^K, K chosen per row
                // and tile so that the tile's largest weight lands in [2^7, 2^8): an exact power of
                // two that rides in the exponent of the exponential, is taken out of the row sum
                // again, and reaches the accumulator through the factor beta (2^(K_t - K_{t-1})) and
                // the final reciprocal (2^-K_T).  K is capped at 64: a tile whose largest weight is
                // below 2^-57 of the accumulated mass is lost in fp32 anyway.
                float Kf = 0.f;
                if constexpr (EB == 1) {
                    Kf = fminf(floorf(ref - m0 * c) + 7.f, 64.f);
                    beta *= ex2(Kf - K_prev);
                    K_prev = Kf;
                }
                if (C::kLookahead == 1 && t > 0) {
                    if (C::kAltS) {
                        sAlpha[bi * 256 + row] = beta;       // slot and barrier of this step's parity
                        mbar_arrive(&alpha_full[bi]);
                    } else {
                        sAlpha[(n_ae & 1) * 256 + i * 128 + row] = beta;
                        ++n_ae;
                        mbar_arrive(&alpha_full[i]);
                    }
                }
                const uint64_t c2 = pack2(c, c), nref2 = pack2(Kf - ref, Kf - ref);
                uint64_t acc0 = pack2(0.f, 0.f), acc1 = acc0;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t pk[C::kPCols / 2];     // the weights of 64 keys, packed
#pragma unroll
                    for (int j = 0; j < 64; j += 4) {
                        if (C::kLookahead == 1 && h == 1 && j == 32) {
                            // the first 64 weights are in tensor memory: their product may start
                            tc_wait_st();
                            tc_fence_before();
                            mbar_arrive(&p_half[bi]);
                        }
                        float x0, x1, x2, x3;
                        unpack2(fma2(pack2(s[64 * h + j], s[64 * h + j + 1]), c2, nref2), x0, x1);
                        unpack2(fma2(pack2(s[64 * h + j + 2], s[64 * h + j + 3]), c2, nref2), x2, x3);
                        const float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);
                        acc0 = add2(acc0, pack2(p0, p1));
                        acc1 = add2(acc1, pack2(p2, p3));
                        if constexpr (EB == 2) {
                            pk[j / 2] = pack_bf16x2(p0, p1);
                            pk[j / 2 + 1] = pack_bf16x2(p2, p3);
                        } else {
                            pk[j / 4] = pack_e4m3x4(p0, p1, p2, p3);
                        }
                    }
                    if (C::kLookahead > 1 && h == 0 && n_pk > 0) {
                        // P has a region of its own: the previous P V must have read it
                        if (!pf_wait(&pv_done[i], (n_pk - 1) & 1, kWaitPVDone, abort_flag)) goto done;
                        tc_fence_after();
                        if (t > 0) {
                            sAlpha[(n_ae & 1) * 256 + i * 128 + row] = beta;
                            ++n_ae;
                            mbar_arrive(&alpha_full[i]);
                        }
                    }
                    if constexpr (EB == 2) tmem_st32(tP + 32 * h, pk);
                    else tmem_st16(tP + 16 * h, pk);
                }
                ++n_pk;
                float a0, a1, a2, a3;
                unpack2(acc0, a0, a1);
                unpack2(acc1, a2, a3);
                float rowsum = (a0 + a1) + (a2 + a3);
                if constexpr (EB == 1) rowsum *= ex2(-Kf);
                const float l = e_old + rowsum;
                inv_l = rcp(l);                              // the hidden division: one reciprocal per row and tile
                L = ref + lg2(l);
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(&p_full[bi]);
            }
            gstep += Ti;
            if (Ti > 0) {
                // the reciprocal that closes the last step goes to the epilogue.  The previous
                // work item's message must have been consumed: for items of two or more tiles
                // that follows from the product order; a one-tile item waits for its own P V,
                // which is issued only after the previous epilogue has released O.
                if (Ti == 1 && !pf_wait(&pv_done[i], (n_pk - 1) & 1, kWaitPVDone, abort_flag)) goto done;
                sFinal[i * 128 + row] = (EB == 1) ? inv_l * ex2(-K_prev) : inv_l;
                mbar_arrive(&final_full[i]);
            }
            if (prm.lse != nullptr && Ti > 0 && gi < Nq) prm.lse[(long long)bh * Nq + gi] = L * kLn2;
        }
    } else if (warp < 12) {
        // ================================================================ correction + epilogue
        reg_dec<80>();
        const int row = threadIdx.x & 127;
        const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tO[2] = {tmem_base + C::kColO0 + lane_sel, tmem_base + C::kColO1 + lane_sel};
        uint32_t n_af[2] = {0, 0}, n_pv[2] = {0, 0}, n_fin[2] = {0, 0};
        uint32_t gstep_run = 0;                        // steps so far (alternating S: parity selects the factor's slot)
        for (int nw = 0, w = work_index(0); w < prm.n_work; w = work_index(++nw)) {
            const int qpair = prm.n_qpairs - 1 - w / prm.BH;
            const int bh = w % prm.BH;
            const int q0 = qpair * C::kItemRows;
            const int Ti[2] = {n_tiles(q0), (C::kQTiles == 2) ? n_tiles(q0 + 128) : 0};
            const int T = max(Ti[0], Ti[1]);
            // the O accumulators are free (the previous epilogue has read them)
            for (int i = 0; i < 2; ++i)
                if (Ti[i] > 0) { tc_fence_before(); mbar_arrive(&o_ready[i]); }
            const uint32_t gstep = gstep_run;
            gstep_run += (uint32_t)T;
            for (int t = 1; t < T; ++t) {
                for (int i = 0; i < 2; ++i) {
                    if (t >= Ti[i]) continue;
                    // per-row factor of this step: slot and barrier of the query tile or, with
                    // alternating S regions, of the step's parity
                    const int ai = C::kAltS ? (int)((gstep + t) & 1) : i;
                    if (!pf_wait(&alpha_full[ai], n_af[ai] & 1, kWaitAlphaFull, abort_flag)) goto done;
                    const float beta = C::kAltS ? sAlpha[ai * 256 + row] : sAlpha[(n_af[i] & 1) * 256 + i * 128 + row];
                    ++n_af[ai];
                    if (!pf_wait(&pv_done[i], n_pv[i] & 1, kWaitPVDone, abort_flag)) goto done;
                    ++n_pv[i];
                    tc_fence_after();
                    // O~ <- beta O~
#pragma unroll
                    for (int cb = 0; cb < D / 32; ++cb) {
                        float ov[32];
                        tmem_ld32(tO[i] + cb * 32, reinterpret_cast<uint32_t*>(ov));
                        tc_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j) ov[j] *= beta;
                        tmem_st32(tO[i] + cb * 32, reinterpret_cast<const uint32_t*>(ov));
                    }
                    tc_wait_st();
                    tc_fence_before();
                    mbar_arrive(&o_ready[i]);
                }
            }
            // epilogue: apply the reciprocal of the last step, convert and store
            for (int i = 0; i < 2; ++i) {
                if (Ti[i] == 0) continue;
                if (!pf_wait(&final_full[i], n_fin[i] & 1, kWaitAlphaFull, abort_flag)) goto done;
                const float inv_l = sFinal[i * 128 + row];
                ++n_fin[i];
                if (!pf_wait(&pv_done[i], n_pv[i] & 1, kWaitPVDone, abort_flag)) goto done;
                ++n_pv[i];
                tc_fence_after();
                const int gi = q0 + i * 128 + row;
                const long long orow = ((long long)bh * Nq + gi) * D;
#pragma unroll
                for (int cb = 0; cb < D / 32; ++cb) {
                    float ov[32];
                    tmem_ld32(tO[i] + cb * 32, reinterpret_cast<uint32_t*>(ov));
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) ov[j] *= inv_l;
                    if (gi < Nq) {
                        if (prm.out_f32) {
                            float4* dst = reinterpret_cast<float4*>(static_cast<float*>(prm.o) + orow + cb * 32);
#pragma unroll
                            for (int j = 0; j < 8; ++j) dst[j] = make_float4(ov[4 * j], ov[4 * j + 1], ov[4 * j + 2], ov[4 * j + 3]);
                        } else {
                            uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(prm.o) + orow + cb * 32);
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                dst[j] = make_uint4(pack_bf16x2(ov[8 * j], ov[8 * j + 1]), pack_bf16x2(ov[8 * j + 2], ov[8 * j + 3]),
                                                    pack_bf16x2(ov[8 * j + 4], ov[8 * j + 5]), pack_bf16x2(ov[8 * j + 6], ov[8 * j + 7]));
                        }
                    }
                }
            }
        }
    } else {
        reg_dec<96>();
    }

done:
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

}  // namespace flashd
