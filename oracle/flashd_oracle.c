/*
 * FLASH-D oracle: plain, slow CPU fp64 implementations of attention.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT PRODUCT CODE.  It exists so that the CUDA
 * library can be checked against something written independently from the
 * paper.  It shares no code, header, table or helper with the CUDA path and
 * must never be linked or imported by it.
 *
 * Every function works on host double arrays laid out [B, H, N, d] row-major
 * (d innermost).  Inputs stored as bf16 / fp32 are upcast exactly to double by
 * the caller.  Each formulation cites the passage of the paper
 * (FLASH-D: FlashAttention with Hidden Softmax Division) that it follows.
 *
 * Formulations
 *   oracle_attn_naive   Sec. II-A: the definition, with the safe-softmax
 *                       max subtraction.
 *   oracle_attn_alg1    Algorithm 1 (baseline FlashAttention, divides at
 *                       every step).
 *   oracle_attn_alg2    Algorithm 2 (FlashAttention2, one division at the end).
 *   oracle_attn_flashd  Algorithm 3 (FLASH-D) with the weight of Eq. (w-last)
 *                       and the blend of Eq. (out-final); variants document
 *                       the readings taken where the paper is at odds with
 *                       itself.
 *   oracle_attn_tiled   the same recurrence applied to groups of keys
 *                       ("super-keys"): tile update and split merge, derived
 *                       from Eq. (w-last) / Eq. (out-final).
 *   oracle_flashd_weights  the scalar weight sequence w_1..w_N of Alg. 3 for
 *                       one score vector.
 *   oracle_skip_stats   Sec. III-C / Sec. V-B: how often s_i - s_{i-1} falls
 *                       outside [-6, 11].
 *   oracle_attn_flashd_pwl  Sec. IV-B: Algorithm 3 with piece-wise linear
 *                       sigmoid and ln and a confined sigmoid input range.
 *
 * Masking is not in the paper (it treats one query over N keys).  Reading
 * taken here: a key that a query may not see is removed from that query's key
 * sequence.  Causal means key j is visible to query i iff j <= i (0-based
 * global indices).
 *
 * Parity status: every function here is pinned by tests/test_oracle_*.py
 * (brute force at 50 digits, exact rationals, the paper's two-key worked
 * example, closed forms, invariants).  oracle_skip_stats: parity unpinned
 * against the paper's Table I (needs model weights and datasets that are not
 * available); it is pinned only by brute-force counting on small inputs.
 * oracle_attn_flashd_pwl: parity unpinned against the paper (its PWL
 * coefficients are not printed and it reports no accuracy figure); it is
 * pinned by its limits: exact functions and an unbounded range give
 * oracle_attn_flashd, a bypassed key gives the recurrence without that key,
 * and refined tables converge at second order.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* global index of local query row i (used only for the causal mask) */
static int q_global(const int* q_index, int i) { return q_index ? q_index[i] : i; }

/* number of visible keys for query row with global index gi */
static int n_visible(int gi, int Nk, int causal) {
    if (!causal) return Nk;
    int n = gi + 1;
    if (n > Nk) n = Nk;
    if (n < 0) n = 0;
    return n;
}

static double dot_scaled(const double* q, const double* k, int d, double scale) {
    double acc = 0.0;
    for (int c = 0; c < d; ++c) acc += q[c] * k[c];
    return scale * acc;
}

/* sigma(x) = 1/(1+e^{-x}), evaluated without overflow for any finite x */
static double sigmoid(double x) {
    if (x >= 0.0) return 1.0 / (1.0 + exp(-x));
    double e = exp(x);
    return e / (1.0 + e);
}

/* ln sigma(x), evaluated without overflow and without forming sigma first */
static double log_sigmoid(double x) {
    if (x >= 0.0) return -log1p(exp(-x));
    return x - log1p(exp(x));
}

/* ------------------------------------------------------------------------ */
/* Sec. II-A: s_i = dot(q,k_i); f_i = e^{s_i}/sum_j e^{s_j}; Attn = sum f_i v_i.
 * Safe softmax: subtract the row maximum before exponentiating.
 * lse (nullable) receives ln sum_j e^{s_j}; weights (nullable, [B,H,Nq,Nk])
 * receives f (0 for invisible keys).                                        */
void oracle_attn_naive(const double* q, const double* k, const double* v,
                       double* o, double* lse, double* weights,
                       int B, int H, int Nq, int Nk, int d,
                       double scale, int causal, const int* q_index) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        for (int i = 0; i < Nq; ++i) {
            const double* qi = q + ((size_t)bh * Nq + i) * d;
            const double* kb = k + (size_t)bh * Nk * d;
            const double* vb = v + (size_t)bh * Nk * d;
            double* oi = o + ((size_t)bh * Nq + i) * d;
            int nv = n_visible(q_global(q_index, i), Nk, causal);
            double* s = (double*)malloc(sizeof(double) * (size_t)(nv > 0 ? nv : 1));
            double m = -INFINITY;
            for (int j = 0; j < nv; ++j) {
                s[j] = dot_scaled(qi, kb + (size_t)j * d, d, scale);
                if (s[j] > m) m = s[j];
            }
            double Z = 0.0;
            for (int j = 0; j < nv; ++j) { s[j] = exp(s[j] - m); Z += s[j]; }
            for (int c = 0; c < d; ++c) oi[c] = 0.0;
            for (int j = 0; j < nv; ++j) {
                const double* vj = vb + (size_t)j * d;
                for (int c = 0; c < d; ++c) oi[c] += s[j] * vj[c];
            }
            for (int c = 0; c < d; ++c) oi[c] = (nv > 0) ? oi[c] / Z : NAN;
            if (lse) lse[(size_t)bh * Nq + i] = (nv > 0) ? m + log(Z) : -INFINITY;
            if (weights) {
                double* wi = weights + ((size_t)bh * Nq + i) * Nk;
                for (int j = 0; j < Nk; ++j) wi[j] = (j < nv) ? s[j] / Z : 0.0;
            }
            free(s);
        }
    }
}

/* ------------------------------------------------------------------------ */
/* Algorithm 1 (baseline FlashAttention): state (m, l, o); the output is
 * divided by l at every step.  The paper does not give the initial state;
 * reading: m_0 = -inf, l_0 = 0, o_0 = 0 with e^{-inf} = 0.                  */
void oracle_attn_alg1(const double* q, const double* k, const double* v, double* o,
                      int B, int H, int Nq, int Nk, int d,
                      double scale, int causal, const int* q_index) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        for (int i = 0; i < Nq; ++i) {
            const double* qi = q + ((size_t)bh * Nq + i) * d;
            const double* kb = k + (size_t)bh * Nk * d;
            const double* vb = v + (size_t)bh * Nk * d;
            double* oi = o + ((size_t)bh * Nq + i) * d;
            int nv = n_visible(q_global(q_index, i), Nk, causal);
            double m = -INFINITY, l = 0.0;
            for (int c = 0; c < d; ++c) oi[c] = (nv > 0) ? 0.0 : NAN;
            for (int j = 0; j < nv; ++j) {
                double s = dot_scaled(qi, kb + (size_t)j * d, d, scale);
                double m_new = s > m ? s : m;
                double carry = (l == 0.0) ? 0.0 : l * exp(m - m_new);
                double e = exp(s - m_new);
                double l_new = carry + e;
                const double* vj = vb + (size_t)j * d;
                for (int c = 0; c < d; ++c)
                    oi[c] = oi[c] * (carry / l_new) + vj[c] * (e / l_new);
                m = m_new; l = l_new;
            }
        }
    }
}

/* Algorithm 2 (FlashAttention2, lazy softmax division): same state, the
 * accumulator is left unnormalised and divided by l_N once at the end.      */
void oracle_attn_alg2(const double* q, const double* k, const double* v, double* o,
                      int B, int H, int Nq, int Nk, int d,
                      double scale, int causal, const int* q_index) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        for (int i = 0; i < Nq; ++i) {
            const double* qi = q + ((size_t)bh * Nq + i) * d;
            const double* kb = k + (size_t)bh * Nk * d;
            const double* vb = v + (size_t)bh * Nk * d;
            double* oi = o + ((size_t)bh * Nq + i) * d;
            int nv = n_visible(q_global(q_index, i), Nk, causal);
            double m = -INFINITY, l = 0.0;
            for (int c = 0; c < d; ++c) oi[c] = 0.0;
            for (int j = 0; j < nv; ++j) {
                double s = dot_scaled(qi, kb + (size_t)j * d, d, scale);
                double m_new = s > m ? s : m;
                double r = (l == 0.0) ? 0.0 : exp(m - m_new);
                double e = exp(s - m_new);
                l = l * r + e;
                const double* vj = vb + (size_t)j * d;
                for (int c = 0; c < d; ++c) oi[c] = oi[c] * r + vj[c] * e;
                m = m_new;
            }
            for (int c = 0; c < d; ++c) oi[c] = (nv > 0) ? oi[c] / l : NAN;
        }
    }
}

/* ------------------------------------------------------------------------ */
/* One step of the FLASH-D weight recurrence, Eq. (w-last):
 *     w_i = sigma(s_i - s_{i-1} + ln w_{i-1}).
 * variant 0: the reading used for parity.  The carried quantity is ln w
 *            (Sec. III-B rewrites w_{i-1} as e^{ln w_{i-1}}), obtained as
 *            ln sigma(x) directly, so it never becomes -inf.
 * variant 1: literal data flow of the hardware figure: w is carried as a
 *            number in [0,1] and ln is applied to it.  Once w rounds to 0 the
 *            logarithm is -inf and every later weight is 0.  Kept only to
 *            show why variant 0 carries the logarithm.
 * variant 2: Algorithm 3 exactly as printed, whose sigmoid argument has
 *            "- ln w_{i-1}".  This contradicts Eq. (w-last) and its
 *            derivation; kept only so that a test can show that the printed
 *            sign does not reproduce softmax for N >= 3.
 * On return *w is w_i and *lnw is the value to carry to step i+1.           */
static void flashd_weight_step(int variant, double s, double s_prev, double lnw_prev,
                               double* w, double* lnw) {
    if (variant == 2) {
        double x = s - s_prev - lnw_prev;
        *w = sigmoid(x);
        *lnw = log_sigmoid(x);
    } else if (variant == 1) {
        double x = s - s_prev + lnw_prev;
        *w = (lnw_prev == -INFINITY) ? 0.0 : sigmoid(x);
        *lnw = log(*w);
    } else {
        double x = s - s_prev + lnw_prev;
        *w = sigmoid(x);
        *lnw = log_sigmoid(x);
    }
}

/* Weight sequence of Algorithm 3 for one score vector s[0..N-1]; w_1 = 1.   */
void oracle_flashd_weights(const double* s, int N, double* w, int variant) {
    double lnw = 0.0;
    for (int i = 0; i < N; ++i) {
        if (i == 0) { w[0] = 1.0; lnw = 0.0; continue; }
        flashd_weight_step(variant, s[i], s[i - 1], lnw, &w[i], &lnw);
    }
}

/* Algorithm 3 (FLASH-D).  Per query: loop over its visible keys in index
 * order; first key w = 1 (so o_1 = v_1); afterwards the weight of
 * Eq. (w-last) and the blend of Eq. (out-final), written with one multiplier
 * as in Sec. IV-A:  o_i = o_{i-1} + (v_i - o_{i-1}) w_i.
 * blend_form 0: o + (v - o) w          (Sec. IV-A)
 * blend_form 1: o (1 - w) + v w        (Eq. out-final)
 * lse (nullable) receives s_N - ln w_N, which equals ln sum_j e^{s_j}
 * because w_N = e^{s_N} / sum_j e^{s_j} (Eq. w-basic).                      */
void oracle_attn_flashd(const double* q, const double* k, const double* v,
                        double* o, double* lse,
                        int B, int H, int Nq, int Nk, int d,
                        double scale, int causal, const int* q_index,
                        int variant, int blend_form) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        for (int i = 0; i < Nq; ++i) {
            const double* qi = q + ((size_t)bh * Nq + i) * d;
            const double* kb = k + (size_t)bh * Nk * d;
            const double* vb = v + (size_t)bh * Nk * d;
            double* oi = o + ((size_t)bh * Nq + i) * d;
            int nv = n_visible(q_global(q_index, i), Nk, causal);
            double s_prev = 0.0, lnw = 0.0;
            for (int c = 0; c < d; ++c) oi[c] = (nv > 0) ? 0.0 : NAN;
            for (int j = 0; j < nv; ++j) {
                double s = dot_scaled(qi, kb + (size_t)j * d, d, scale);
                const double* vj = vb + (size_t)j * d;
                double w;
                if (j == 0) { w = 1.0; lnw = 0.0; }
                else flashd_weight_step(variant, s, s_prev, lnw, &w, &lnw);
                if (blend_form == 1) {
                    for (int c = 0; c < d; ++c) oi[c] = oi[c] * (1.0 - w) + vj[c] * w;
                } else {
                    for (int c = 0; c < d; ++c) oi[c] = oi[c] + (vj[c] - oi[c]) * w;
                }
                s_prev = s;
            }
            if (lse) lse[(size_t)bh * Nq + i] = (nv > 0) ? s_prev - lnw : -INFINITY;
        }
    }
}

/* ------------------------------------------------------------------------ */
/* Derived group form.  A group T of keys processed from a fresh state yields
 * its own attention output obar_T and L_T = ln sum_{j in T} e^{s_j}.  Treating
 * the group as one "super-key" with score L_T and value obar_T, one step of
 * Alg. 3 merges it into a running state (L, o) where L = s - ln w of the last
 * step (so the sigmoid argument of Eq. (w-last) is L_T - L):
 *     W = sigma(L_T - L);  o <- o + (obar_T - o) W;  L <- L_T - ln W.
 * Multiplying through gives the fused tile update used inside a split:
 *     L_new = L_T - ln W;  P_j = e^{s_j - L_new};  alpha = e^{L - L_new};
 *     o <- alpha o + sum_j P_j v_j.
 * Keys [0, nv) are cut into num_splits contiguous splits of
 * ceil(Nk/num_splits) keys (the split grid is laid over all Nk keys, visible
 * or not); inside a split, tiles of `tile` keys are folded with the fused
 * update starting from an empty state; the split results are then merged in
 * split order with the super-key step.  Empty splits are skipped.
 * partial_o [B,H,Nq,num_splits,d] and partial_L [B,H,Nq,num_splits]
 * (both nullable) receive the per-split states (L = -inf, o = 0 when empty). */
void oracle_attn_tiled(const double* q, const double* k, const double* v,
                       double* o, double* lse, double* partial_o, double* partial_L,
                       int B, int H, int Nq, int Nk, int d,
                       double scale, int causal, const int* q_index,
                       int tile, int num_splits) {
    if (tile < 1) tile = 1;
    if (num_splits < 1) num_splits = 1;
    int per_split = (Nk + num_splits - 1) / num_splits;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        for (int i = 0; i < Nq; ++i) {
            const double* qi = q + ((size_t)bh * Nq + i) * d;
            const double* kb = k + (size_t)bh * Nk * d;
            const double* vb = v + (size_t)bh * Nk * d;
            double* oi = o + ((size_t)bh * Nq + i) * d;
            int nv = n_visible(q_global(q_index, i), Nk, causal);
            double* sp = (double*)malloc(sizeof(double) * (size_t)tile);
            double* os = (double*)malloc(sizeof(double) * (size_t)d);
            double L_acc = -INFINITY;
            for (int c = 0; c < d; ++c) oi[c] = (nv > 0) ? 0.0 : NAN;
            for (int sidx = 0; sidx < num_splits; ++sidx) {
                int j0 = sidx * per_split;
                int j1 = j0 + per_split; if (j1 > nv) j1 = nv;
                double Ls = -INFINITY;
                for (int c = 0; c < d; ++c) os[c] = 0.0;
                for (int t0 = j0; t0 < j1; t0 += tile) {
                    int t1 = t0 + tile; if (t1 > j1) t1 = j1;
                    /* L_T of this tile via a tile-local reference */
                    double ref = -INFINITY;
                    for (int j = t0; j < t1; ++j) {
                        sp[j - t0] = dot_scaled(qi, kb + (size_t)j * d, d, scale);
                        if (sp[j - t0] > ref) ref = sp[j - t0];
                    }
                    double z = 0.0;
                    for (int j = t0; j < t1; ++j) z += exp(sp[j - t0] - ref);
                    double L_T = ref + log(z);
                    /* super-key step on the logarithms */
                    double lnW = (Ls == -INFINITY) ? 0.0 : log_sigmoid(L_T - Ls);
                    double L_new = L_T - lnW;
                    double alpha = (Ls == -INFINITY) ? 0.0 : exp(Ls - L_new);
                    for (int c = 0; c < d; ++c) os[c] *= alpha;
                    for (int j = t0; j < t1; ++j) {
                        double P = exp(sp[j - t0] - L_new);
                        const double* vj = vb + (size_t)j * d;
                        for (int c = 0; c < d; ++c) os[c] += P * vj[c];
                    }
                    Ls = L_new;
                }
                if (partial_L) partial_L[((size_t)bh * Nq + i) * num_splits + sidx] = Ls;
                if (partial_o) {
                    double* po = partial_o + (((size_t)bh * Nq + i) * num_splits + sidx) * d;
                    for (int c = 0; c < d; ++c) po[c] = os[c];
                }
                if (Ls == -INFINITY) continue;           /* empty split */
                if (L_acc == -INFINITY) {                /* first super-key: W = 1 */
                    for (int c = 0; c < d; ++c) oi[c] = os[c];
                    L_acc = Ls;
                } else {
                    double W = sigmoid(Ls - L_acc);
                    double lnW = log_sigmoid(Ls - L_acc);
                    for (int c = 0; c < d; ++c) oi[c] = oi[c] + (os[c] - oi[c]) * W;
                    L_acc = Ls - lnW;
                }
            }
            if (lse) lse[(size_t)bh * Nq + i] = L_acc;
            free(sp); free(os);
        }
    }
}

/* Merge per-split states in split order with the super-key step alone.
 * partial_o [rows, num_splits, d], partial_L [rows, num_splits] -> o [rows,d],
 * lse [rows] (nullable).  Splits with L = -inf are skipped.                 */
void oracle_split_merge(const double* partial_o, const double* partial_L,
                        double* o, double* lse, int rows, int num_splits, int d) {
    for (int r = 0; r < rows; ++r) {
        double* oi = o + (size_t)r * d;
        double L_acc = -INFINITY;
        for (int c = 0; c < d; ++c) oi[c] = NAN;
        for (int sidx = 0; sidx < num_splits; ++sidx) {
            double Ls = partial_L[(size_t)r * num_splits + sidx];
            const double* os = partial_o + ((size_t)r * num_splits + sidx) * d;
            if (Ls == -INFINITY) continue;
            if (L_acc == -INFINITY) {
                for (int c = 0; c < d; ++c) oi[c] = os[c];
                L_acc = Ls;
            } else {
                double W = sigmoid(Ls - L_acc);
                double lnW = log_sigmoid(Ls - L_acc);
                for (int c = 0; c < d; ++c) oi[c] = oi[c] + (os[c] - oi[c]) * W;
                L_acc = Ls - lnW;
            }
        }
        if (lse) lse[r] = L_acc;
    }
}

/* ------------------------------------------------------------------------ */
/* Sec. III-C / Sec. V-B: how often an output update could be bypassed.
 * Static criterion (the paper's): for every query and every visible key after
 * the first, the step is counted when the score difference s_i - s_{i-1} is
 * <= lo (w_i ~ 0, output kept) or >= hi (w_i ~ 1, output replaced); the paper
 * uses [lo, hi] = [-6, 11].
 * Adaptive criterion: Sec. V-B only announces "an adaptive criterion that
 * includes both the range of attention score differences and the value of the
 * previous weight".  Reading taken here: the same test applied to the actual
 * sigmoid argument of Eq. (w-last), x_i = s_i - s_{i-1} + ln w_{i-1}, with its
 * own thresholds [alo, ahi] (for the unshifted sigmoid the paper's figure
 * suggests [-6, 6]).
 * counts[0] steps examined, [1] differences <= lo, [2] differences >= hi,
 * [3] x <= alo, [4] x >= ahi, [5] steps within `near` of any of the four
 * thresholds (so that a comparison with another implementation can tell a
 * rounding tie from a mistake).                                             */
void oracle_skip_stats(const double* q, const double* k, long long* counts,
                       int B, int H, int Nq, int Nk, int d,
                       double scale, int causal, const int* q_index,
                       double lo, double hi, double alo, double ahi, double near) {
    long long total = 0, below = 0, above = 0, abelow = 0, aabove = 0, nnear = 0;
    for (int bh = 0; bh < B * H; ++bh) {
        for (int i = 0; i < Nq; ++i) {
            const double* qi = q + ((size_t)bh * Nq + i) * d;
            const double* kb = k + (size_t)bh * Nk * d;
            int nv = n_visible(q_global(q_index, i), Nk, causal);
            double s_prev = 0.0, lnw = 0.0;
            for (int j = 0; j < nv; ++j) {
                double s = dot_scaled(qi, kb + (size_t)j * d, d, scale);
                if (j > 0) {
                    double diff = s - s_prev;
                    double x = diff + lnw;             /* argument of Eq. (w-last) */
                    ++total;
                    if (diff <= lo) ++below;
                    else if (diff >= hi) ++above;
                    if (x <= alo) ++abelow;
                    else if (x >= ahi) ++aabove;
                    if (fabs(diff - lo) < near || fabs(diff - hi) < near ||
                        fabs(x - alo) < near || fabs(x - ahi) < near) ++nnear;
                    double w;
                    flashd_weight_step(0, s, s_prev, lnw, &w, &lnw);
                } else {
                    lnw = 0.0;
                }
                s_prev = s;
            }
        }
    }
    counts[0] = total; counts[1] = below; counts[2] = above;
    counts[3] = abelow; counts[4] = aabove; counts[5] = nnear;
}

/* ------------------------------------------------------------------------ */
/* Sec. IV-B: Algorithm 3 with the sigmoid and the natural logarithm replaced
 * by continuous piece-wise linear (PWL) approximations, and the sigmoid input
 * confined to a range [lo, hi] (the paper: 8 segments each, range [-6, 11]).
 *
 * A PWL function is given by n_seg + 1 nodes (x_0 < ... < x_n, y_0 .. y_n):
 * linear between neighbouring nodes, equal to the end value outside [x_0, x_n]
 * ("no computation is required outside this range").  The paper does not print
 * its coefficients, so the tables are inputs here.  n_seg = 0 selects the exact
 * function instead (sigma, resp. ln; with both exact, ln w is taken as
 * ln sigma(x), so that lo = -inf, hi = +inf reproduces oracle_attn_flashd).   */
double oracle_pwl_eval(const double* xs, const double* ys, int n_seg, double x) {
    if (x <= xs[0]) return ys[0];
    if (x >= xs[n_seg]) return ys[n_seg];
    int m = 0;
    while (m + 1 < n_seg && x >= xs[m + 1]) ++m;          /* segment with xs[m] <= x < xs[m+1] */
    return ys[m] + (x - xs[m]) * (ys[m + 1] - ys[m]) / (xs[m + 1] - xs[m]);
}

/* The carried state is the paper's (s_{i-1}, ln w_{i-1}, o_{i-1}).  Per key,
 * with x = s_i - s_{i-1} + ln w_{i-1} (argument of Eq. (w-last)):
 *   range_mode 0 (saturate): x is clamped to [lo, hi]; w = SIG(x); ln w = LN(w).
 *   range_mode 1 (bypass, Sec. III-C read on x): x < lo: the key is bypassed -
 *       no output update and the state stays as it was, which is the recurrence
 *       over the key sequence with that key removed; x > hi: w = 1, the output
 *       is replaced by v_i (the recurrence restarted at key i); otherwise as in
 *       mode 0.
 * counts (nullable, [3]) receives the number of bypassed keys, of replacements,
 * and of steps whose x lies within `near` of lo or hi (where the fp32 device
 * code may decide differently).                                              */
void oracle_attn_flashd_pwl(const double* q, const double* k, const double* v, double* o,
                            int B, int H, int Nq, int Nk, int d,
                            double scale, int causal, const int* q_index,
                            int sig_n, const double* sig_x, const double* sig_y,
                            int ln_n, const double* ln_x, const double* ln_y,
                            double lo, double hi, int range_mode, double near,
                            long long* counts) {
    long long n_skip = 0, n_repl = 0, n_near = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1) reduction(+ : n_skip, n_repl, n_near)
    for (int bh = 0; bh < B * H; ++bh) {
        for (int i = 0; i < Nq; ++i) {
            const double* qi = q + ((size_t)bh * Nq + i) * d;
            const double* kb = k + (size_t)bh * Nk * d;
            const double* vb = v + (size_t)bh * Nk * d;
            double* oi = o + ((size_t)bh * Nq + i) * d;
            int nv = n_visible(q_global(q_index, i), Nk, causal);
            double s_prev = 0.0, lnw = 0.0;
            for (int c = 0; c < d; ++c) oi[c] = (nv > 0) ? 0.0 : NAN;
            for (int j = 0; j < nv; ++j) {
                double s = dot_scaled(qi, kb + (size_t)j * d, d, scale);
                const double* vj = vb + (size_t)j * d;
                double w;
                if (j == 0) {
                    w = 1.0; lnw = 0.0;
                } else {
                    double x = s - s_prev + lnw;
                    if (fabs(x - lo) < near || fabs(x - hi) < near) ++n_near;
                    if (range_mode == 1 && x < lo) { ++n_skip; continue; }
                    if (range_mode == 1 && x > hi) {
                        ++n_repl; w = 1.0; lnw = 0.0;
                    } else {
                        if (x < lo) x = lo;
                        if (x > hi) x = hi;
                        w = sig_n > 0 ? oracle_pwl_eval(sig_x, sig_y, sig_n, x) : sigmoid(x);
                        if (ln_n > 0) lnw = oracle_pwl_eval(ln_x, ln_y, ln_n, w);
                        else lnw = sig_n > 0 ? log(w) : log_sigmoid(x);
                    }
                }
                for (int c = 0; c < d; ++c) oi[c] = oi[c] + (vj[c] - oi[c]) * w;
                s_prev = s;
            }
        }
    }
    if (counts) { counts[0] = n_skip; counts[1] = n_repl; counts[2] = n_near; }
}
