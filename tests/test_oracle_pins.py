"""Pins of the CPU oracle against things other than itself: values worked out
by hand from the paper's closed forms (tests/golden), 50-digit brute force,
library routines for the special cases that reduce to them, closed forms and
invariants.  None of these tests needs a GPU."""
import itertools
import math
from fractions import Fraction

import mpmath
import numpy as np
import pytest
import scipy.special

import oracle
from conftest import read_golden

mpmath.mp.dps = 50


# --------------------------------------------------------------------------
# helpers that do NOT use the oracle
# --------------------------------------------------------------------------
def brute_force(q, k, v, scale, causal):
    """Sec. II-A definition in 50-digit arithmetic, no max subtraction."""
    B, H, Nq, d = q.shape
    Nk = k.shape[2]
    out = np.zeros((B, H, Nq, d))
    lse = np.zeros((B, H, Nq))
    for b, h, i in itertools.product(range(B), range(H), range(Nq)):
        nv = min(i + 1, Nk) if causal else Nk
        s = [mpmath.mpf(scale) * sum(mpmath.mpf(float(q[b, h, i, c])) * mpmath.mpf(float(k[b, h, j, c]))
                                     for c in range(d)) for j in range(nv)]
        e = [mpmath.e ** x for x in s]
        Z = sum(e)
        for c in range(d):
            out[b, h, i, c] = float(sum(e[j] * mpmath.mpf(float(v[b, h, j, c])) for j in range(nv)) / Z)
        lse[b, h, i] = float(mpmath.log(Z))
    return out, lse


def one_head(scores, values):
    """q, k, v (d = len(values[0]) >= 1) such that s_i = scores[i] with scale 1:
    q = e_0, k_i = scores[i] * e_0."""
    n = len(scores)
    d = len(values[0])
    q = np.zeros((1, 1, 1, d)); q[0, 0, 0, 0] = 1.0
    k = np.zeros((1, 1, n, d)); k[0, 0, :, 0] = scores
    v = np.asarray(values, dtype=np.float64).reshape(1, 1, n, d)
    return q, k, v


def all_formulations(q, k, v, scale, causal, q_index=None):
    yield "naive", oracle.attn_naive(q, k, v, scale, causal, q_index)
    yield "alg1", oracle.attn_alg1(q, k, v, scale, causal, q_index)
    yield "alg2", oracle.attn_alg2(q, k, v, scale, causal, q_index)
    yield "flashd", oracle.attn_flashd(q, k, v, scale, causal, q_index)
    yield "flashd_blend1", oracle.attn_flashd(q, k, v, scale, causal, q_index, blend_form=1)
    yield "tiled3", oracle.attn_tiled(q, k, v, scale, causal, q_index, tile=3, num_splits=2)


# --------------------------------------------------------------------------
# golden fixtures (hand-derived from the paper's closed forms)
# --------------------------------------------------------------------------
def test_two_key_worked_example():
    g = read_golden("worked_example_two_keys.txt")
    s = [math.log(float(a)) for a in g["exp_s"]]
    v = [[float(x) for x in g["v1"]], [float(x) for x in g["v2"]]]
    w = oracle.flashd_weights(s)
    assert w[0] == float(g["w1"][0])
    assert abs(w[1] - float(g["w2"][0])) < 1e-15
    assert abs((1 - w[1]) - float(g["one_minus_w2"][0])) < 1e-15
    # o_1 = v_1: run with only the first key
    q, k, vv = one_head(s[:1], v[:1])
    for name, o in all_formulations(q, k, vv, 1.0, False):
        assert np.allclose(o[0, 0, 0], [float(x) for x in g["o1"]], atol=1e-15), name
    q, k, vv = one_head(s, v)
    for name, o in all_formulations(q, k, vv, 1.0, False):
        assert np.allclose(o[0, 0, 0], [float(x) for x in g["o2"]], rtol=0, atol=1e-14), name


def test_ln_integer_scores_exact_rationals():
    g = read_golden("ln_integer_scores.txt")
    a = [int(x) for x in g["a"]]
    s = [math.log(x) for x in a]
    v = [[float(x) for x in g[f"v{i}"]] for i in range(len(a))]
    # the fixture itself is consistent (pure rational arithmetic, no oracle)
    assert [Fraction(x, sum(a)) for x in a] == g["f"]
    assert [Fraction(a[i], sum(a[: i + 1])) for i in range(len(a))] == g["w"]
    w = oracle.flashd_weights(s)
    assert np.allclose(w, [float(x) for x in g["w"]], rtol=0, atol=2e-16 * 8)
    q, k, vv = one_head(s, v)
    o, lse, f = oracle.attn_naive(q, k, vv, 1.0, return_lse=True, return_weights=True)
    assert np.allclose(f[0, 0, 0], [float(x) for x in g["f"]], rtol=0, atol=1e-15)
    assert abs(lse[0, 0, 0] - math.log(sum(a))) < 1e-14
    for name, o in all_formulations(q, k, vv, 1.0, False):
        assert np.allclose(o[0, 0, 0], [float(x) for x in g["attn"]], rtol=0, atol=1e-13), name
    # causal: query rows 0, 1, 2 of a square problem see prefixes 1, 2, 3
    n = 3
    qc = np.zeros((1, 1, n, 2)); qc[0, 0, :, 0] = 1.0
    kc = k[:, :, :n]; vc = vv[:, :, :n]
    for name, o in all_formulations(qc, kc, vc, 1.0, True):
        for i in range(n):
            want = [float(x) for x in g[f"attn_prefix{i + 1}"]]
            assert np.allclose(o[0, 0, i], want, rtol=0, atol=1e-13), (name, i)


# --------------------------------------------------------------------------
# brute force at 50 digits
# --------------------------------------------------------------------------
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("shape", [(1, 1, 1, 1, 1), (1, 2, 3, 5, 2), (2, 1, 6, 6, 4), (1, 1, 4, 8, 3)])
def test_brute_force_50_digits(shape, causal):
    B, H, Nq, Nk, d = shape
    rng = np.random.default_rng(1234 + Nq * 7 + Nk)
    q = rng.normal(size=(B, H, Nq, d)) * 2
    k = rng.normal(size=(B, H, Nk, d)) * 2
    v = rng.normal(size=(B, H, Nk, d))
    scale = 0.7
    want, want_lse = brute_force(q, k, v, scale, causal)
    for name, o in all_formulations(q, k, v, scale, causal):
        assert np.abs(o - want).max() < 1e-13, name
    _, lse = oracle.attn_naive(q, k, v, scale, causal, return_lse=True)
    assert np.abs(lse - want_lse).max() < 1e-13
    _, lse = oracle.attn_flashd(q, k, v, scale, causal, return_lse=True)
    assert np.abs(lse - want_lse).max() < 1e-12
    _, lse = oracle.attn_tiled(q, k, v, scale, causal, tile=2, num_splits=3, return_lse=True)
    assert np.abs(lse - want_lse).max() < 1e-12


def test_brute_force_large_logits():
    """Scores in the hundreds: brute force has no overflow at 50 digits."""
    s = [310.0, -250.5, 305.25, 12.0, 309.0, -700.0, 311.5]
    rng = np.random.default_rng(5)
    v = rng.normal(size=(len(s), 3))
    q, k, vv = one_head(s, v)
    want, _ = brute_force(q, k, vv, 1.0, False)
    for name, o in all_formulations(q, k, vv, 1.0, False):
        assert np.abs(o - want).max() < 1e-12, name


# --------------------------------------------------------------------------
# library special cases
# --------------------------------------------------------------------------
def test_against_scipy_softmax_and_matmul():
    rng = np.random.default_rng(7)
    B, H, Nq, Nk, d = 2, 3, 17, 29, 8
    q = rng.normal(size=(B, H, Nq, d)); k = rng.normal(size=(B, H, Nk, d)); v = rng.normal(size=(B, H, Nk, d))
    scale = 1 / math.sqrt(d)
    S = scale * np.einsum("bhic,bhjc->bhij", q, k)
    want = scipy.special.softmax(S, axis=-1) @ v
    want_lse = scipy.special.logsumexp(S, axis=-1)
    o, lse, f = oracle.attn_naive(q, k, v, scale, return_lse=True, return_weights=True)
    assert np.abs(o - want).max() < 1e-13
    assert np.abs(lse - want_lse).max() < 1e-13
    assert np.abs(f - scipy.special.softmax(S, axis=-1)).max() < 1e-14
    for name, o in all_formulations(q, k, v, scale, False):
        assert np.abs(o - want).max() < 1e-12, name
    # causal: mask with -inf before the library softmax
    Sm = np.where(np.arange(Nk)[None, :] <= np.arange(Nq)[:, None], S, -np.inf)
    want = scipy.special.softmax(Sm, axis=-1) @ v
    for name, o in all_formulations(q, k, v, scale, True):
        assert np.abs(o - want).max() < 1e-12, name


def test_identity_values_return_the_weight_vector():
    rng = np.random.default_rng(11)
    n = 6
    s = rng.normal(size=n) * 3
    q = np.zeros((1, 1, 1, n)); q[0, 0, 0, 0] = 1
    k = np.zeros((1, 1, n, n)); k[0, 0, :, 0] = s
    v = np.eye(n).reshape(1, 1, n, n)
    want = scipy.special.softmax(s)
    for name, o in all_formulations(q, k, v, 1.0, False):
        assert np.abs(o[0, 0, 0] - want).max() < 1e-14, name


# --------------------------------------------------------------------------
# closed forms of the weight: Eq. (w-basic), Eq. (w), Eq. (w-last)
# --------------------------------------------------------------------------
def test_weight_closed_forms():
    rng = np.random.default_rng(3)
    s = rng.normal(size=40) * 5
    w = oracle.flashd_weights(s)
    sm = [mpmath.mpf(float(x)) for x in s]
    # Eq. (w-basic): w_i = e^{s_i} / sum_{j<=i} e^{s_j}
    for i in range(len(s)):
        want = mpmath.e ** sm[i] / sum(mpmath.e ** sm[j] for j in range(i + 1))
        assert abs(w[i] - float(want)) < 1e-14
    # Eq. (w): w_i = w_{i-1} / (w_{i-1} + e^{s_{i-1} - s_i}), w_1 = 1
    wi = mpmath.mpf(1)
    for i in range(1, len(s)):
        wi = wi / (wi + mpmath.e ** (sm[i - 1] - sm[i]))
        assert abs(w[i] - float(wi)) < 1e-14
    assert np.all(w > 0) and np.all(w <= 1) and w[0] == 1.0


def test_equal_scores_give_running_mean():
    n = 50
    w = oracle.flashd_weights(np.full(n, 2.5))
    assert np.allclose(w, 1.0 / np.arange(1, n + 1), rtol=1e-13, atol=0)
    rng = np.random.default_rng(2)
    v = rng.normal(size=(n, 4))
    q, k, vv = one_head([2.5] * n, v)
    for name, o in all_formulations(q, k, vv, 1.0, False):
        assert np.abs(o[0, 0, 0] - v.mean(axis=0)).max() < 1e-14, name


def test_weight_curve_is_a_shifted_sigmoid():
    """Fig. 2: as a function of s_i - s_{i-1} the weight is the sigmoid shifted
    right by -ln w_{i-1}; it crosses 1/2 at s_i - s_{i-1} = -ln w_{i-1}, and for
    w_{i-1} = 0.99 it is close to the plain sigmoid."""
    # scores (0, ln(1/3)) give w_2 = 1/4, so w_3 = 1/2 at s_3 - s_2 = ln 4
    a = math.log(1 / 3)
    w = oracle.flashd_weights([0.0, a, a + math.log(4.0)])
    assert abs(w[1] - 0.25) < 1e-15 and abs(w[2] - 0.5) < 1e-15
    # w_2 = 0.99 when s_2 - s_1 = ln 99
    for delta in np.linspace(-8, 12, 41):
        w = oracle.flashd_weights([0.0, math.log(99.0), math.log(99.0) + delta])
        assert abs(w[1] - 0.99) < 1e-15
        assert abs(w[2] - 1 / (1 + math.exp(-delta))) < 0.0026
        assert abs(w[2] - 1 / (1 + math.exp(-(delta + math.log(0.99))))) < 1e-15


def test_printed_sign_of_alg3_does_not_reproduce_softmax():
    """Algorithm 3 prints '- ln w_{i-1}' where Eq. (w-last) has '+'.  With
    ln w_1 = 0 the two agree for N <= 2 and differ from N = 3 on; only '+'
    reproduces the definition."""
    rng = np.random.default_rng(9)
    v = rng.normal(size=(3, 2))
    s = [0.3, -0.4, 0.9]
    for n in (1, 2):
        q, k, vv = one_head(s[:n], v[:n])
        want = oracle.attn_naive(q, k, vv, 1.0)
        assert np.abs(oracle.attn_flashd(q, k, vv, 1.0, variant=2) - want).max() < 1e-15
    q, k, vv = one_head(s, v)
    want, _ = brute_force(q, k, vv, 1.0, False)
    assert np.abs(oracle.attn_flashd(q, k, vv, 1.0, variant=0) - want).max() < 1e-15
    assert np.abs(oracle.attn_flashd(q, k, vv, 1.0, variant=2) - want).max() > 1e-2


# --------------------------------------------------------------------------
# invariants
# --------------------------------------------------------------------------
def implied_weights(w):
    """c_i = w_i * prod_{j>i} (1 - w_j): the coefficient of v_i in o_N."""
    n = len(w)
    c = np.zeros(n)
    for i in range(n):
        c[i] = w[i] * np.prod(1.0 - w[i + 1:])
    return c


def test_implied_weights_are_softmax():
    rng = np.random.default_rng(21)
    for scale in (1.0, 8.0, 40.0):
        s = rng.normal(size=30) * scale
        c = implied_weights(oracle.flashd_weights(s))
        assert abs(c.sum() - 1) < 1e-13
        assert np.all(c >= 0)
        assert np.abs(c - scipy.special.softmax(s)).max() < 1e-13


@pytest.mark.parametrize("causal", [False, True])
def test_convex_hull_shift_and_permutation(causal):
    rng = np.random.default_rng(33)
    B, H, N, d = 1, 2, 24, 5
    q = rng.normal(size=(B, H, N, d)) * 3; k = rng.normal(size=(B, H, N, d)) * 3
    v = rng.normal(size=(B, H, N, d))
    base = oracle.attn_flashd(q, k, v, 1.0, causal)
    if not causal:
        lo = v.min(axis=2, keepdims=True); hi = v.max(axis=2, keepdims=True)
        assert np.all(base >= lo - 1e-12) and np.all(base <= hi + 1e-12)
        perm = rng.permutation(N)
        for name, o in all_formulations(q, k[:, :, perm], v[:, :, perm], 1.0, False):
            assert np.abs(o - base).max() < 1e-12, name
    # adding a constant to every logit of a row: append a coordinate that
    # contributes q_extra * k_extra = C to every score
    for C in (1e3, -1e3, 3e5):
        q2 = np.concatenate([q, np.ones((B, H, N, 1))], axis=-1)
        k2 = np.concatenate([k, np.full((B, H, N, 1), C)], axis=-1)
        v2 = np.concatenate([v, np.zeros((B, H, N, 1))], axis=-1)
        for fn in (oracle.attn_naive, oracle.attn_flashd, oracle.attn_alg1, oracle.attn_tiled):
            o = fn(q2, k2, v2, 1.0, causal)[..., :d]
            assert np.abs(o - base).max() < 1e-9 * max(1.0, abs(C) / 1e3), (fn.__name__, C)


def test_causal_row_equals_truncated_noncausal_and_tail_padding():
    rng = np.random.default_rng(44)
    B, H, Nq, Nk, d = 1, 2, 9, 6, 4          # Nq > Nk: rows >= Nk see every key
    q = rng.normal(size=(B, H, Nq, d)); k = rng.normal(size=(B, H, Nk, d)); v = rng.normal(size=(B, H, Nk, d))
    for fn in (oracle.attn_naive, oracle.attn_flashd, oracle.attn_alg1, oracle.attn_alg2, oracle.attn_tiled):
        oc = fn(q, k, v, 0.5, True)
        for i in range(Nq):
            n = min(i + 1, Nk)
            want = oracle.attn_naive(q[:, :, i:i + 1], k[:, :, :n], v[:, :, :n], 0.5, False)
            assert np.abs(oc[:, :, i:i + 1] - want).max() < 1e-13, (fn.__name__, i)
    # q_index: a sample of rows gives the same rows as the full problem
    full = oracle.attn_naive(q, k, v, 0.5, True)
    rows = [0, 3, 8]
    part = oracle.attn_naive(q[:, :, rows], k, v, 0.5, True, q_index=rows)
    assert np.array_equal(part, full[:, :, rows])
    part = oracle.attn_flashd(q[:, :, rows], k, v, 0.5, True, q_index=rows)
    assert np.abs(part - full[:, :, rows]).max() < 1e-13


# --------------------------------------------------------------------------
# group form: tiles, splits, prefixes
# --------------------------------------------------------------------------
def test_tiled_equals_definition_for_every_tile_and_split():
    rng = np.random.default_rng(55)
    B, H, Nq, Nk, d = 1, 1, 4, 13, 3
    q = rng.normal(size=(B, H, Nq, d)) * 4; k = rng.normal(size=(B, H, Nk, d)) * 4
    v = rng.normal(size=(B, H, Nk, d))
    for causal in (False, True):
        want, want_lse = brute_force(q, k, v, 1.0, causal)
        for tile in range(1, Nk + 2):
            for S in (1, 2, 3, 5, 13, 16):
                o, lse = oracle.attn_tiled(q, k, v, 1.0, causal, tile=tile, num_splits=S, return_lse=True)
                assert np.abs(o - want).max() < 1e-12, (causal, tile, S)
                assert np.abs(lse - want_lse).max() < 1e-12, (causal, tile, S)


def test_split_partials_are_attention_over_their_keys_and_prefix_merges():
    rng = np.random.default_rng(66)
    B, H, Nq, Nk, d, S = 1, 2, 3, 20, 4, 4
    q = rng.normal(size=(B, H, Nq, d)) * 2; k = rng.normal(size=(B, H, Nk, d)) * 2
    v = rng.normal(size=(B, H, Nk, d))
    o, po, pL = oracle.attn_tiled(q, k, v, 1.0, tile=3, num_splits=S, return_partials=True)
    per = Nk // S
    for sidx in range(S):
        ks = slice(sidx * per, (sidx + 1) * per)
        want, want_lse = brute_force(q, k[:, :, ks], v[:, :, ks], 1.0, False)
        assert np.abs(po[:, :, :, sidx] - want).max() < 1e-13
        assert np.abs(pL[:, :, :, sidx] - want_lse).max() < 1e-13
    for n in range(1, S + 1):   # a prefix of the splits is attention over that key prefix
        merged, lse = oracle.split_merge(po[:, :, :, :n], pL[:, :, :, :n], return_lse=True)
        want, want_lse = brute_force(q, k[:, :, : n * per], v[:, :, : n * per], 1.0, False)
        assert np.abs(merged - want).max() < 1e-13
        assert np.abs(lse - want_lse).max() < 1e-13
    # the merge does not depend on the order of the splits
    perm = [2, 0, 3, 1]
    merged = oracle.split_merge(po[:, :, :, perm], pL[:, :, :, perm])
    assert np.abs(merged - o).max() < 1e-13
    # an empty split (L = -inf) is ignored
    po2 = np.concatenate([np.zeros_like(po[:, :, :, :1]), po], axis=3)
    pL2 = np.concatenate([np.full_like(pL[:, :, :, :1], -np.inf), pL], axis=3)
    assert np.array_equal(oracle.split_merge(po2, pL2), oracle.split_merge(po, pL))


# --------------------------------------------------------------------------
# stability (Sec. III-C): large drops and rises of the score
# --------------------------------------------------------------------------
def test_large_score_drops_and_rises():
    v = np.array([[1.0, 0.0], [0.0, 1.0], [5.0, 5.0], [-3.0, 2.0]])
    for s in ([200.0, 0.0, 150.0, 149.0], [1000.0, 0.0, 990.0, 1001.0], [0.0, -2000.0, 3.0, -1.0]):
        q, k, vv = one_head(s, v)
        want, _ = brute_force(q, k, vv, 1.0, False)
        for name, o in all_formulations(q, k, vv, 1.0, False):
            assert np.all(np.isfinite(o)), name
            assert np.abs(o - want).max() < 1e-12, name


def test_linear_domain_weight_freezes_after_underflow():
    """Why the carried quantity is ln w: a weight kept as a number in [0,1]
    underflows to 0 after a drop of more than ~745 (fp64), its logarithm is
    -inf, and every later weight stays 0 although a later key dominates."""
    s = [1000.0, 0.0, 2000.0]
    v = np.array([[1.0], [2.0], [3.0]])
    q, k, vv = one_head(s, v)
    want, _ = brute_force(q, k, vv, 1.0, False)
    assert abs(want[0, 0, 0, 0] - 3.0) < 1e-12
    assert abs(oracle.attn_flashd(q, k, vv, 1.0, variant=0)[0, 0, 0, 0] - 3.0) < 1e-12
    assert abs(oracle.attn_flashd(q, k, vv, 1.0, variant=1)[0, 0, 0, 0] - 1.0) < 1e-12
    w = oracle.flashd_weights(s, variant=1)
    assert w[1] == 0.0 and w[2] == 0.0


# --------------------------------------------------------------------------
# skip statistic (Sec. III-C static range): brute-force count
# --------------------------------------------------------------------------
def test_skip_stats_counts():
    """Static and adaptive counts against a plain Python count; the adaptive
    argument uses the closed form ln w_{i-1} = s_{i-1} - ln sum_{j<i} e^{s_j}
    (Eq. w-basic) instead of the oracle's recurrence."""
    rng = np.random.default_rng(77)
    B, H, Nq, Nk, d = 1, 2, 5, 9, 3
    q = rng.normal(size=(B, H, Nq, d)) * 4; k = rng.normal(size=(B, H, Nk, d)) * 4
    for causal in (False, True):
        total = below = above = abelow = aabove = 0
        for b, h, i in itertools.product(range(B), range(H), range(Nq)):
            nv = min(i + 1, Nk) if causal else Nk
            s = [float(np.dot(q[b, h, i], k[b, h, j])) for j in range(nv)]
            for j in range(1, nv):
                diff = s[j] - s[j - 1]
                lnw_prev = s[j - 1] - float(scipy.special.logsumexp(s[:j]))
                x = diff + lnw_prev
                total += 1
                below += diff <= -6
                above += diff >= 11
                abelow += x <= -6
                aabove += x >= 6
        got = oracle.skip_stats(q, k, 1.0, causal)
        assert got[:5] == (total, below, above, abelow, aabove)
        assert got[5] == 0
    # integer scores: thresholds hit exactly, ties count as bypassable
    qq = np.zeros((1, 1, 1, 2)); qq[0, 0, 0, 0] = 1
    kk = np.zeros((1, 1, 5, 2)); kk[0, 0, :, 0] = [0, -6, 5, 16, 16]
    got = oracle.skip_stats(qq, kk, 1.0)
    assert got[0] == 4 and got[1] == 1 and got[2] == 2     # diffs -6, 11, 11, 0
    assert got[5] >= 3
