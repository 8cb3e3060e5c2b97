/*
 * flashd.h - C ABI of the FLASH-D attention forward library for NVIDIA B200
 * (sm_100a).
 *
 * The library computes  O = softmax(scale * Q K^T) V  in the form of the
 * paper "FLASH-D: FlashAttention with Hidden Softmax Division": the running
 * output is a convex blend  o_i = o_{i-1} (1 - w_i) + v_i w_i  (Eq. out-final)
 * whose weight  w_i = sigma(s_i - s_{i-1} + ln w_{i-1})  (Eq. w-last) absorbs
 * the softmax division, so the output is normalised after every step, no
 * running maximum is carried and no final division is made (Algorithm 3).
 *
 * Conventions shared by every entry point
 *   - Tensors are contiguous [B, H, N, d] arrays, d innermost; q and o have
 *     N = Nq, k and v have N = Nk.  The paper treats one head (Sec. II); B*H
 *     independent heads are processed here.
 *   - Unless an argument is documented as a HOST pointer, tensor pointers are
 *     DEVICE pointers owned by the caller, 16-byte aligned.  The library keeps
 *     no reference to them after the work queued on `stream` has finished.
 *   - s = scale * dot(q, k).  The paper's score has no scale factor (Sec. II-A);
 *     pass scale = 1 for the paper's definition, 1/sqrt(d) for transformers.
 *   - causal != 0: key j is visible to query i iff j <= i (0-based indices).
 *     Keys that a query cannot see are removed from its key sequence.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls enqueue work and return without synchronising, except where
 *     stated.
 *   - Every function returns a flashd_status (0 = success).  Arguments are
 *     validated on the host before anything is launched; nothing is launched
 *     when validation fails.  The library never aborts and never throws.
 *   - There is no CPU fallback: without a CUDA device the calls return
 *     FLASHD_ERR_CUDA.
 */
#ifndef FLASHD_H
#define FLASHD_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FLASHD_OK = 0,
    FLASHD_ERR_NULL = 1,        /* a required pointer is NULL                          */
    FLASHD_ERR_SHAPE = 2,       /* a size is <= 0, or scale is not finite              */
    FLASHD_ERR_UNSUPPORTED = 3, /* head size / dtype / mode not built                  */
    FLASHD_ERR_ALIGN = 4,       /* a tensor pointer is not 16-byte aligned             */
    FLASHD_ERR_WORKSPACE = 5,   /* workspace too small or split count out of range     */
    FLASHD_ERR_CUDA = 6,        /* a CUDA runtime / driver call failed                 */
    FLASHD_ERR_TIMEOUT = 7      /* a bounded wait inside a kernel ran out              */
} flashd_status;

typedef enum { FLASHD_BF16 = 0, FLASHD_F32 = 1 } flashd_dtype;

/* Upper bound on num_splits accepted by the split-K entry points. */
#define FLASHD_MAX_SPLITS 64

/* ------------------------------------------------------------------------
 * Tiled tensor-core forward (bf16 in, fp32 accumulate, bf16 out).
 *
 * Computes Algorithm 3 with keys grouped in tiles of 128.  With x_j = s_j - L_old
 * and L = s - ln w the carried state, the per-key step of Eq. (w-last) and
 * Eq. (out-final) with its division written out, o = (o_old + e^x v)/(1 + e^x),
 * becomes for a tile
 *     O_new = (O_old + sum_j e^{x_j} v_j) / (1 + sum_j e^{x_j}),
 *     L_new = L_old + ln(1 + sum_j e^{x_j}),
 * evaluated relative to a tile-local reference max(L_old, max_j s_j) so that no
 * exponent is positive.  The reciprocal that closes a tile step is applied when
 * the next step opens (the last one when the result is stored); no running
 * maximum and no separate softmax denominator are carried.  S = Q K^T and P V
 * run on the 5th generation tensor cores (tcgen05.mma, accumulators in tensor
 * memory).
 *
 * q, o: [B,H,Nq,d] bf16; k, v: [B,H,Nk,d] bf16.  d must be 64, 128 or 256
 * (the hidden sizes of Sec. V-A that a 128-row tensor-core tile can take).
 * o must not overlap q, k or v.  Returns after the launch.               */
int flashd_attn_fwd(const void* q, const void* k, const void* v, void* o,
                    int B, int H, int Nq, int Nk, int d, float scale, int causal,
                    void* stream);

/* Same computation with options.  in_dtype must be FLASHD_BF16.  out_dtype
 * selects the type of o (FLASHD_BF16 or FLASHD_F32).  lse_out (nullable,
 * [B,H,Nq] fp32) receives the final state L_N = s_N - ln w_N = ln sum_j e^{s_j}
 * (natural log; Eq. w-basic solved for the running sum).                  */
int flashd_attn_fwd_ex(const void* q, const void* k, const void* v, void* o, float* lse_out,
                       int in_dtype, int out_dtype,
                       int B, int H, int Nq, int Nk, int d, float scale, int causal,
                       void* stream);

/* ------------------------------------------------------------------------
 * Per-key forward: Algorithm 3 exactly as stated, one key at a time, state
 * (s_{i-1}, ln w_{i-1}, o_{i-1}) per query, w_1 = 1, weight by Eq. (w-last)
 * with sigma evaluated over the full range (no clamp, no skip), blend in the
 * one-multiplier form of Sec. IV-A, o + (v - o) w.  Scores and the carried
 * ln w are kept in fp64, sigma / ln sigma / blend in fp32.
 *
 * flashd_attn_fwd_f32: fp32 in, fp32 out.
 * flashd_attn_fwd_perkey: in_dtype / out_dtype in {FLASHD_BF16, FLASHD_F32}.
 * d must be 16, 32, 64, 128 or 256 (the hidden sizes of the paper's evaluation,
 * Sec. V-A).  lse_out nullable.                        */
int flashd_attn_fwd_f32(const void* q, const void* k, const void* v, void* o,
                        int B, int H, int Nq, int Nk, int d, float scale, int causal,
                        void* stream);
int flashd_attn_fwd_perkey(const void* q, const void* k, const void* v, void* o, float* lse_out,
                           int in_dtype, int out_dtype,
                           int B, int H, int Nq, int Nk, int d, float scale, int causal,
                           void* stream);

/* ------------------------------------------------------------------------
 * Algorithm 3 with piece-wise linear sigmoid and ln (Sec. IV-B): the numerical
 * model of the paper's datapath, for accuracy studies.  One key at a time like
 * flashd_attn_fwd_perkey; not a throughput path.
 *
 * A table describes a continuous piece-wise linear function by n + 1 nodes:
 * x[0] < ... < x[n] with values y[0..n]; linear in between, y[0] / y[n]
 * outside.  sig_* replaces the sigmoid of Eq. (w-last), ln_* replaces the
 * natural logarithm that yields ln w_i from w_i.  n = 0 (pointers may be NULL)
 * selects the exact function.  1 <= n <= FLASHD_PWL_MAX_SEGMENTS otherwise.
 * The tables are HOST arrays of n + 1 floats, read during the call (the caller
 * may free them on return).  The paper uses n = 8 for both and does not print
 * its coefficients.
 *
 * The sigmoid argument x = s_i - s_(i-1) + ln w_(i-1) is confined to [lo, hi]
 * (the paper: [-6, 11]; -INFINITY / +INFINITY lift a bound):
 *   range_mode 0: x is clamped to the range;
 *   range_mode 1: x < lo bypasses the key - no output update, carried state
 *                 unchanged (Sec. III-C); x > hi replaces the output by v_i
 *                 (w_i = 1).
 * counts: nullable DEVICE pointer to two 64-bit counters, incremented by the
 * number of bypassed keys and of replacements (the caller zeroes them).
 * in_dtype / out_dtype, d, layout and errors as flashd_attn_fwd_perkey;
 * a malformed table or range returns FLASHD_ERR_SHAPE.                       */
#define FLASHD_PWL_MAX_SEGMENTS 64
int flashd_attn_fwd_pwl(const void* q, const void* k, const void* v, void* o,
                        unsigned long long* counts, int in_dtype, int out_dtype,
                        int B, int H, int Nq, int Nk, int d, float scale, int causal,
                        int sig_n, const float* sig_x, const float* sig_y,
                        int ln_n, const float* ln_x, const float* ln_y,
                        float lo, float hi, int range_mode, void* stream);

/* ------------------------------------------------------------------------
 * Tiled tensor-core forward with FP8-E4M3 operands (the second number format
 * of the paper's evaluation, Sec. V-A): q, k, v hold one-byte E4M3 values
 * (4 exponent bits, bias 7, 3 mantissa bits, no infinities), [B,H,N,d]
 * contiguous, 16-byte aligned; d = 128 or 256.  Same kernel and same steps as
 * flashd_attn_fwd (tile form of Algorithm 3, state L per row in fp32): both
 * products run as E4M3 x E4M3 -> fp32 on the tensor cores, the scores, the
 * weights' exponentials and row sums and the accumulator stay fp32, and the
 * per-tile weights e^{x_j} (in [0, 1] relative to the tile's reference) are
 * rounded to E4M3 (round to nearest even) for the P V product, as they are
 * rounded to bf16 in the bf16 kernel.  That rounding is the only
 * approximation beyond the bf16 kernel's: a relative error of at most 2^-4
 * per weight (absolute 2^-10 below 2^-6, where E4M3 is subnormal or flushes
 * to zero), so every output element is within
 * 2^-4 * sum_j f_j |v_j| (+ 2^-6) of the exact result on the stored values.
 * o: bf16 or fp32 (out_dtype); lse_out nullable, [B,H,Nq] fp32, = L_N.
 * Dequantisation scales: one of Q and K folds into `scale`; one of V
 * multiplies the output and is the caller's.  Errors as flashd_attn_fwd_ex;
 * any other d returns FLASHD_ERR_UNSUPPORTED.                             */
int flashd_attn_fwd_fp8(const void* q, const void* k, const void* v, void* o,
                        float* lse_out, int out_dtype,
                        int B, int H, int Nq, int Nk, int d, float scale, int causal,
                        void* stream);

/* ------------------------------------------------------------------------
 * Split-K forward for long key sequences and few queries (decode).
 * Non-causal, bf16 in, d = 128 or 64.
 *
 * The Nk keys are cut into num_splits contiguous ranges of
 * ceil(Nk / num_splits) keys.  flashd_splitk_partial runs the tile form of
 * Algorithm 3 over each range from an empty state and writes, per
 * (b, h, query, split), the range's own attention output o_p (d floats)
 * followed by its state L_p (1 float; -inf for an empty range) to
 * `workspace`, laid out [B,H,Nq,num_splits,d+1] fp32.
 * flashd_splitk_combine folds the partials in split order as super-keys
 * (score L_p, value o_p) with Eq. (w-last) and the Sec. IV-A blend:
 *     W = sigma(L_p - L_acc); o_acc += (o_p - o_acc) W; L_acc = L_p - ln W,
 * the first non-empty split taking W = 1.  No division is made anywhere.
 *
 * workspace: device memory of at least flashd_splitk_workspace_bytes(...)
 * bytes, 16-byte aligned, owned by the caller; contents need not be
 * initialised.  num_splits in [1, FLASHD_MAX_SPLITS] and <= Nk.
 * flashd_splitk_num_splits returns the split count the library would pick.
 * flashd_attn_fwd_splitk queues partial + combine on `stream`
 * (num_splits <= 0: library's choice; the workspace must then be sized for
 * flashd_splitk_num_splits(...)).                                          */
size_t flashd_splitk_workspace_bytes(int B, int H, int Nq, int d, int num_splits);
int flashd_splitk_num_splits(int B, int H, int Nq, int Nk, int d);
int flashd_splitk_partial(const void* q, const void* k, const void* v,
                          void* workspace, size_t workspace_bytes,
                          int B, int H, int Nq, int Nk, int d, float scale,
                          int num_splits, void* stream);
int flashd_splitk_combine(const void* workspace, void* o, float* lse_out,
                          int B, int H, int Nq, int d, int num_splits, int out_dtype,
                          void* stream);
int flashd_attn_fwd_splitk(const void* q, const void* k, const void* v, void* o,
                           void* workspace, size_t workspace_bytes,
                           int B, int H, int Nq, int Nk, int d, float scale,
                           int num_splits, void* stream);

/* ------------------------------------------------------------------------
 * Split-K forward over a PAGED K/V cache with one length per sequence
 * (decode in a serving loop).  The function is the one of
 * flashd_attn_fwd_splitk, sequence by sequence (the paper treats one query
 * over one key sequence, Sec. II-A; where the keys are stored and that
 * sequences differ in length is outside it); only the addressing differs.
 *
 * k_pages, v_pages : [num_pages, H, page_size, d] bf16, contiguous, 16-byte
 *                    aligned: the pool.  page_size must be a multiple of the
 *                    kernel's ring stage (64 keys at d = 128, 128 at d = 64).
 * block_table      : [B, max_pages] int32, DEVICE memory; entry (b, p) is the
 *                    pool index of the page holding keys p*page_size ...
 *                    (p+1)*page_size - 1 of sequence b.  Entries beyond the
 *                    sequence's last page are not read.
 * seq_lens         : [B] int32, DEVICE memory; keys of sequence b, in
 *                    [0, max_pages*page_size].  A sequence of length 0 gives
 *                    o = 0.
 * q, o             : [B,H,Nq,d] bf16; every query row of sequence b sees all
 *                    seq_lens[b] keys (non-causal).
 * Each sequence's keys are cut into num_splits ranges of
 * ceil(seq_lens[b] / num_splits) keys rounded up to whole ring stages (so
 * short sequences leave late ranges empty); workspace and combine as for
 * flashd_splitk_partial (flashd_splitk_workspace_bytes(B, H, Nq, d,
 * num_splits)).  num_splits <= 0 in flashd_attn_fwd_splitk_paged selects
 * flashd_splitk_num_splits(B, H, Nq, max_pages*page_size, d).
 * The table and the lengths live on the device, so the host cannot check
 * them: a length outside its range, or a page index outside
 * [0, num_pages), is caught by the kernel, which then records
 * FLASHD_ERR_SHAPE in the device status word (flashd_last_device_status),
 * treats that sequence as empty or reads page 0 instead, and finishes;
 * the output of that sequence is then meaningless.  No out-of-pool read is
 * made.  Other errors as flashd_splitk_partial.                            */
int flashd_splitk_partial_paged(const void* q, const void* k_pages, const void* v_pages,
                                const int* block_table, const int* seq_lens,
                                void* workspace, size_t workspace_bytes,
                                int B, int H, int Nq, int max_pages, int page_size, int num_pages,
                                int d, float scale, int num_splits, void* stream);
int flashd_attn_fwd_splitk_paged(const void* q, const void* k_pages, const void* v_pages, void* o,
                                 const int* block_table, const int* seq_lens,
                                 void* workspace, size_t workspace_bytes,
                                 int B, int H, int Nq, int max_pages, int page_size, int num_pages,
                                 int d, float scale, int num_splits, void* stream);
/* The same over a pool of FP8-E4M3 pages (one byte per element, widened exactly
 * as in flashd_splitk_partial_fp8kv; q and o stay bf16).  A ring stage then
 * holds twice the keys: page_size must be a multiple of 128 keys at d = 128
 * and of 256 at d = 64.                                                     */
int flashd_splitk_partial_paged_fp8kv(const void* q, const void* k_pages, const void* v_pages,
                                      const int* block_table, const int* seq_lens,
                                      void* workspace, size_t workspace_bytes,
                                      int B, int H, int Nq, int max_pages, int page_size, int num_pages,
                                      int d, float scale, int num_splits, void* stream);
int flashd_attn_fwd_splitk_paged_fp8kv(const void* q, const void* k_pages, const void* v_pages, void* o,
                                       const int* block_table, const int* seq_lens,
                                       void* workspace, size_t workspace_bytes,
                                       int B, int H, int Nq, int max_pages, int page_size, int num_pages,
                                       int d, float scale, int num_splits, void* stream);

/* ------------------------------------------------------------------------
 * Split-K forward with K and V stored as FP8-E4M3 (the second number format of
 * the paper's evaluation, Sec. V-A).  q and o stay bf16; k, v : [B,H,Nk,d] of
 * one-byte E4M3 values (4 exponent bits, bias 7, 3 mantissa bits, no
 * infinities: the "fn" variant), contiguous, 16-byte aligned.  Every element
 * is widened exactly and the arithmetic is the fp32 arithmetic of
 * flashd_splitk_partial: same function, same workspace layout, same combine,
 * half the bytes per key.  A dequantisation scale of K folds into `scale`; one
 * of V multiplies the output and is the caller's.  Other arguments, split
 * rules and errors as flashd_splitk_partial / flashd_attn_fwd_splitk.       */
int flashd_splitk_partial_fp8kv(const void* q, const void* k, const void* v,
                                void* workspace, size_t workspace_bytes,
                                int B, int H, int Nq, int Nk, int d, float scale,
                                int num_splits, void* stream);
int flashd_attn_fwd_splitk_fp8kv(const void* q, const void* k, const void* v, void* o,
                                 void* workspace, size_t workspace_bytes,
                                 int B, int H, int Nq, int Nk, int d, float scale,
                                 int num_splits, void* stream);

/* ------------------------------------------------------------------------
 * Grouped-query split-K forward (decode with shared K/V heads, one or a few
 * query positions).  bf16 in, d = 128 or 64.
 *
 * G consecutive query heads attend to the same K/V head: query head
 * h = hkv*G + g reads k[b,hkv], v[b,hkv].  The attention function of every
 * query head is unchanged (Eq. (out-final)/(w-last) per head); only the data
 * movement differs: each split's K and V rows are read from device memory
 * once and serve all G queries.
 *   q, o : [B, Hkv*G, Nq, d] contiguous;  k, v : [B, Hkv, Nk, d] contiguous.
 *   G >= 1, Nq >= 1, G*Nq <= FLASHD_MAX_GROUP (larger: FLASHD_ERR_UNSUPPORTED).
 * The Nq query positions are the LAST Nq positions of the Nk-key sequence
 * (a decode step over several tokens: speculative or chunked decoding).
 * causal != 0: query position iq sees keys 0 .. Nk-Nq+iq (needs Nq <= Nk);
 * causal == 0: every query sees all Nk keys.
 * flashd_gqa_partial writes the partial states [B, Hkv*G, Nq, num_splits, d+1]
 * fp32 exactly as flashd_splitk_partial does for a [B, Hkv*G, Nq, d] query
 * tensor (a split with no visible key for a row is written as empty), so
 * flashd_splitk_combine(workspace, o, lse, B, Hkv*G, Nq, d, ...) finishes
 * it; flashd_attn_fwd_gqa queues both (bf16 output).  Workspace size:
 * flashd_splitk_workspace_bytes(B, Hkv*G, Nq, d, num_splits); ownership,
 * alignment, split rules and errors as for the split-K calls above.
 * flashd_gqa_num_splits returns the library's split count (num_splits <= 0
 * in flashd_attn_fwd_gqa selects it).                                      */
#define FLASHD_MAX_GROUP 8
int flashd_gqa_num_splits(int B, int Hkv, int G, int Nk, int d);
int flashd_gqa_partial(const void* q, const void* k, const void* v,
                       void* workspace, size_t workspace_bytes,
                       int B, int Hkv, int G, int Nq, int Nk, int d, float scale, int causal,
                       int num_splits, void* stream);
int flashd_attn_fwd_gqa(const void* q, const void* k, const void* v, void* o,
                        void* workspace, size_t workspace_bytes,
                        int B, int Hkv, int G, int Nq, int Nk, int d, float scale, int causal,
                        int num_splits, void* stream);

/* ------------------------------------------------------------------------
 * Grouped-query decode over a paged K/V pool with one length per sequence:
 * flashd_gqa_partial / flashd_attn_fwd_gqa with the addressing of
 * flashd_splitk_partial_paged.  k_pages, v_pages : [num_pages, Hkv,
 * page_size, d] bf16; page_size a multiple of 128 keys; block_table
 * [B, max_pages] and seq_lens [B] int32 in DEVICE memory; q, o :
 * [B, Hkv*G, Nq, d] bf16.  The Nq positions of sequence b are its last Nq
 * (causal: position iq sees keys 0 .. seq_lens[b] - Nq + iq; a position
 * that would see no key gives o = 0).  Split ranges are whole 128-key
 * chunks of ceil(seq_lens[b] / num_splits) keys; workspace, combine, the
 * handling of a bad table or length (device status word) and the other
 * errors as for the calls they combine.  num_splits <= 0 in
 * flashd_attn_fwd_gqa_paged selects flashd_gqa_num_splits(B, Hkv, G,
 * max_pages*page_size, d).                                                */
int flashd_gqa_partial_paged(const void* q, const void* k_pages, const void* v_pages,
                             const int* block_table, const int* seq_lens,
                             void* workspace, size_t workspace_bytes,
                             int B, int Hkv, int G, int Nq, int max_pages, int page_size, int num_pages,
                             int d, float scale, int causal, int num_splits, void* stream);
int flashd_attn_fwd_gqa_paged(const void* q, const void* k_pages, const void* v_pages, void* o,
                              const int* block_table, const int* seq_lens,
                              void* workspace, size_t workspace_bytes,
                              int B, int Hkv, int G, int Nq, int max_pages, int page_size, int num_pages,
                              int d, float scale, int causal, int num_splits, void* stream);

/* ------------------------------------------------------------------------
 * Split-K forward that allocates nothing.  (The paper has no counterpart: this
 * entry point exists for integration reasons only.)
 *
 * Who needs it: a decode loop inside an inference server usually hands every
 * byte of device memory to its own pool at start-up and runs each token under
 * a fixed memory plan.  Such a caller has nowhere to take the split-K
 * workspace from, and cudaMalloc inside the per-token call would either fail
 * or stall the device while the driver maps memory.  Plugin hosts that forbid
 * allocation inside the hot call are in the same position.
 *
 * Same computation and same kernels as flashd_attn_fwd_splitk, but the
 * partial states live in a fixed array that is part of the library image
 * (FLASHD_STATIC_SCRATCH_BYTES of device memory on every GPU that loads the
 * library, held until the process exits).  The caller passes only inputs and
 * the output.  The call makes no cudaMalloc / cudaFree and uses no allocating
 * library routine.
 *
 * Limit: B*H*Nq*num_splits*(d+1)*4 bytes must not exceed
 * FLASHD_STATIC_SCRATCH_BYTES; a larger problem is rejected with
 * FLASHD_ERR_WORKSPACE and nothing is launched (num_splits <= 0 takes the
 * library's choice first, then the check is made).
 *
 * First call on a device: it looks up the device address of the array (once
 * per device, with that device current) before launching.  Make that first
 * call before starting any stream capture.
 *
 * Sharing: every call on a device uses the same array, and the array keeps
 * whatever the previous call left in it.  Nothing in it needs clearing - the
 * partial kernel rewrites every (row, split) slot it later reads, empty splits
 * included - but two calls whose kernels overlap on the GPU (different
 * streams, or different host threads) race on it and give wrong results.
 * Serialise such calls on one stream.                                      */
#define FLASHD_STATIC_SCRATCH_BYTES (8u << 20)
int flashd_attn_fwd_splitk_static(const void* q, const void* k, const void* v, void* o,
                                  int B, int H, int Nq, int Nk, int d, float scale,
                                  int num_splits, void* stream);

/* ------------------------------------------------------------------------
 * Bypassable-update statistic (Sec. III-C, Sec. V-B, Table I).
 *
 * Walks every query over its visible keys as Algorithm 3 does (state
 * s_{i-1}, ln w_{i-1}; no output is formed) and counts, over all steps i >= 2,
 *   counts[0]  steps examined
 *   counts[1]  s_i - s_{i-1} <= lo   (static criterion: w_i ~ 0, update bypassed)
 *   counts[2]  s_i - s_{i-1} >= hi   (static criterion: w_i ~ 1, output replaced)
 *   counts[3]  x_i <= alo            x_i = s_i - s_{i-1} + ln w_{i-1}, the sigmoid
 *   counts[4]  x_i >= ahi            argument of Eq. (w-last)
 * The paper uses [lo, hi] = [-6, 11]; [alo, ahi] is this library's reading of
 * the adaptive criterion the paper leaves to future work ([-6, 6] suits the
 * unshifted sigmoid).  Scores and the decisions are taken in fp64.
 * counts: DEVICE pointer to 5 unsigned 64-bit integers, 8-byte aligned; the
 * call zeroes them on `stream` before the kernel adds to them.
 * in_dtype FLASHD_BF16 or FLASHD_F32; d in {32, 64, 128, 256}.               */
int flashd_skip_stats(const void* q, const void* k, unsigned long long* counts, int in_dtype,
                      int B, int H, int Nq, int Nk, int d, float scale, int causal,
                      float lo, float hi, float alo, float ahi, void* stream);

/* ------------------------------------------------------------------------
 * End-to-end call on HOST buffers: q, k, v, o are host pointers (pinned
 * memory gives asynchronous copies).  The call allocates device buffers from
 * the stream-ordered pool of the current device, cuts the batch into chunks
 * of whole heads (about 12 MB of input each, at most 8) and pipelines them:
 * chunk c+1 is copied in while chunk c runs the forward selected by `path`
 * and chunk c-1 is copied out, on two helper streams of the library that
 * start after the work already queued on `stream` and are joined back into
 * it.  It frees the buffers and SYNCHRONISES `stream` before returning.
 * Calls on the same device are serialised by a lock (they share the helper
 * streams).  Not for use under stream capture.
 * path 0: flashd_attn_fwd (bf16)   path 1: flashd_attn_fwd_f32
 * path 2: flashd_attn_fwd_splitk (bf16, library's split count per chunk)   */
int flashd_attn_fwd_host(const void* q, const void* k, const void* v, void* o,
                         int path, int B, int H, int Nq, int Nk, int d, float scale,
                         int causal, void* stream);

/* ------------------------------------------------------------------------
 * Utilities.
 * flashd_last_device_status synchronises `stream`, then reads and clears the
 * device-side status word of the current device: FLASHD_OK, or
 * FLASHD_ERR_TIMEOUT if a bounded wait inside a kernel gave up (its output is
 * then undefined).  detail (nullable, HOST int[4]) receives
 * {code, blockIdx.x, which wait, iteration}.                              */
int flashd_last_device_status(void* stream, int* detail);
const char* flashd_status_string(int status);
int flashd_version(void);
/* Number of kernels launched by this library in this process so far. */
long long flashd_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* FLASHD_H */
