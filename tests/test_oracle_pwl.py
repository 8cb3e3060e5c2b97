"""Pins of the oracle's PWL variant of Algorithm 3 (Sec. IV-B).

The paper prints neither its PWL coefficients nor an accuracy figure, so the
function is pinned by what fixes it independently of any table:
  * exact functions and an unbounded range reproduce the pinned per-key oracle;
  * a bypassed key is the same recurrence over the key sequence without that
    key, a replacement is the recurrence restarted at that key - checked against
    the plain definition (oracle.attn_naive) on the surviving keys;
  * saturation: a clamped argument equals running with scores shifted so that
    the argument sits on the bound;
  * interpolating tables converge to the exact-function result at second order;
  * the PWL evaluator itself against numpy.interp and at the nodes.
"""
import math

import numpy as np
import pytest

import oracle
from paper_2505_14201_b200 import pwl, synth


def small(seed, Nq=5, Nk=40, d=8, H=2):
    q, k, v = synth.random_qkv(1, H, Nq, Nk, d, seed=seed, dtype="f32")
    return q.double().numpy(), k.double().numpy(), v.double().numpy()


def test_pwl_eval_matches_interp_and_nodes():
    rng = np.random.default_rng(0)
    xs = np.sort(rng.uniform(-3, 5, 9)); ys = rng.normal(size=9)
    for x in np.concatenate([xs, rng.uniform(-6, 8, 200)]):
        assert oracle.pwl_eval(xs, ys, x) == pytest.approx(np.interp(x, xs, ys), abs=1e-14)
    assert oracle.pwl_eval(xs, ys, -100.0) == ys[0] and oracle.pwl_eval(xs, ys, 100.0) == ys[-1]
    # one segment through two points is the line
    assert oracle.pwl_eval([1.0, 3.0], [2.0, -2.0], 2.5) == pytest.approx(-1.0, abs=1e-15)


@pytest.mark.parametrize("causal", [False, True])
def test_exact_functions_unbounded_range_is_algorithm3(causal):
    q, k, v = small(1)
    want = oracle.attn_flashd(q, k, v, 0.7, causal)
    for mode in (0, 1):
        got, counts = oracle.attn_flashd_pwl(q, k, v, 0.7, causal, lo=-math.inf, hi=math.inf, range_mode=mode,
                                             return_counts=True)
        assert np.array_equal(got, want)
        assert counts[:2] == (0, 0)


def scores_case(scores, d=4, seed=3):
    """One query whose scores against the keys are exactly `scores` (q = e_0, k_j = s_j e_0)."""
    n = len(scores)
    q = np.zeros((1, 1, 1, d)); q[..., 0] = 1.0
    k = np.zeros((1, 1, n, d)); k[0, 0, :, 0] = scores
    v = np.random.default_rng(seed).normal(size=(1, 1, n, d))
    return q, k, v


def test_bypassed_key_is_removed_from_the_sequence():
    # x_2 = s_2 - s_1 + ln w_1 = -9 < lo: key 2 is bypassed; keys 3, 4 stay in range
    scores = [0.0, -9.0, 0.5, -1.0]
    q, k, v = scores_case(scores)
    got, counts = oracle.attn_flashd_pwl(q, k, v, 1.0, lo=-6.0, hi=11.0, range_mode=1, return_counts=True)
    keep = [0, 2, 3]
    want = oracle.attn_naive(q, k[:, :, keep], v[:, :, keep], 1.0)
    assert counts[0] == 1 and counts[1] == 0
    assert np.abs(got - want).max() < 1e-14
    # and it is NOT the full softmax (the dropped key has weight ~ e^-9 / Z)
    full = oracle.attn_naive(q, k, v, 1.0)
    assert 1e-6 < np.abs(got - full).max() < 1e-3


def test_replacement_restarts_the_recurrence():
    # x_3 = 14 - 0.5 + ln w_2 > 11: the output is replaced by v_3 and the prefix is forgotten
    scores = [0.0, 0.5, 14.0, 13.0, 12.5]
    q, k, v = scores_case(scores)
    got, counts = oracle.attn_flashd_pwl(q, k, v, 1.0, lo=-6.0, hi=11.0, range_mode=1, return_counts=True)
    assert counts[:2] == (0, 1)
    want = oracle.attn_naive(q, k[:, :, 2:], v[:, :, 2:], 1.0)
    assert np.abs(got - want).max() < 1e-14


def test_saturation_equals_argument_on_the_bound():
    # two keys: o = v_1 + (v_2 - v_1) sigma(clamp(s_2 - s_1)); clamped to lo = -2
    q, k, v = scores_case([0.0, -5.0])
    got = oracle.attn_flashd_pwl(q, k, v, 1.0, lo=-2.0, hi=11.0, range_mode=0)
    w = 1.0 / (1.0 + math.exp(2.0))
    want = v[0, 0, 0] + (v[0, 0, 1] - v[0, 0, 0]) * w
    assert np.abs(got[0, 0, 0] - want).max() < 1e-15
    # a third key sees ln w_2 = ln sigma(-2), not ln sigma(-5)
    q, k, v = scores_case([0.0, -5.0, -4.0])
    got = oracle.attn_flashd_pwl(q, k, v, 1.0, lo=-2.0, hi=11.0, range_mode=0)
    w2 = w
    x3 = -4.0 - (-5.0) + math.log(w2)
    w3 = 1.0 / (1.0 + math.exp(-max(x3, -2.0)))
    o2 = v[0, 0, 0] + (v[0, 0, 1] - v[0, 0, 0]) * w2
    want = o2 + (v[0, 0, 2] - o2) * w3
    assert np.abs(got[0, 0, 0] - want).max() < 1e-14


def test_interpolating_tables_converge_at_second_order():
    q, k, v = small(5, Nk=60)
    lo, hi = -3.0, 11.0                 # ln stays away from its singularity: w >= sigma(-3) = 0.047
    wl, wh = pwl.ln_range(lo)
    exact = oracle.attn_flashd_pwl(q, k, v, 0.5, lo=lo, hi=hi, range_mode=0)
    errs = []
    for n in (64, 128, 256, 512):
        sig = pwl.sampled_pwl(pwl.sigmoid, lo, hi, n)
        ln = pwl.sampled_pwl(np.log, wl, wh, n)
        got = oracle.attn_flashd_pwl(q, k, v, 0.5, sig=sig, ln=ln, lo=lo, hi=hi, range_mode=0)
        errs.append(np.abs(got - exact).max())
    assert errs[-1] < 2e-4, errs
    # halving the node spacing divides the error by about 4 (second order): 64 over three halvings
    assert all(a > b for a, b in zip(errs, errs[1:])), errs
    assert 25.0 < errs[0] / errs[-1] < 200.0, errs


def test_fitted_tables_are_what_the_paper_describes():
    sig, ln = pwl.paper_tables()
    assert len(sig[0]) == 9 and len(ln[0]) == 9
    assert sig[0][0] == -6.0 and sig[0][-1] == 11.0
    assert np.all(np.diff(sig[0]) > 0) and np.all(np.diff(ln[0]) > 0)
    assert pwl.max_error(sig, pwl.sigmoid, *pwl.SIGMOID_RANGE) < 0.03
    assert pwl.max_error(ln, np.log, *pwl.ln_range()) < 0.3
    # a least-squares fit with free breakpoints beats the uniform interpolant
    uni = pwl.sampled_pwl(pwl.sigmoid, -6.0, 11.0, 8)
    assert pwl.max_error(sig, pwl.sigmoid, -6.0, 11.0) < pwl.max_error(uni, pwl.sigmoid, -6.0, 11.0)
