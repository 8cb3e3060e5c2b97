"""Property tests of the oracle: every formulation of the paper agrees with
the Sec. II-A definition on random small problems, logits in the hundreds
included, and the results are finite."""
import numpy as np
from hypothesis import given, settings, strategies as st

import oracle


@settings(max_examples=60, deadline=None)
@given(st.integers(1, 3), st.integers(1, 9), st.integers(1, 12), st.integers(1, 5),
       st.sampled_from([0.1, 1.0, 30.0, 300.0]), st.booleans(), st.integers(0, 2 ** 31 - 1),
       st.integers(1, 7), st.integers(1, 5))
def test_formulations_agree(BH, Nq, Nk, d, spread, causal, seed, tile, splits):
    rng = np.random.default_rng(seed)
    q = rng.normal(size=(1, BH, Nq, d)) * np.sqrt(spread)
    k = rng.normal(size=(1, BH, Nk, d)) * np.sqrt(spread)
    v = rng.normal(size=(1, BH, Nk, d))
    want, want_lse = oracle.attn_naive(q, k, v, 1.0, causal, return_lse=True)
    assert np.all(np.isfinite(want))
    tol = 1e-10
    got, lse = oracle.attn_flashd(q, k, v, 1.0, causal, return_lse=True)
    assert np.abs(got - want).max() < tol
    assert np.abs(lse - want_lse).max() < tol * max(1.0, np.abs(want_lse).max())
    assert np.abs(oracle.attn_flashd(q, k, v, 1.0, causal, blend_form=1) - want).max() < tol
    assert np.abs(oracle.attn_alg1(q, k, v, 1.0, causal) - want).max() < tol
    assert np.abs(oracle.attn_alg2(q, k, v, 1.0, causal) - want).max() < tol
    got, lse = oracle.attn_tiled(q, k, v, 1.0, causal, tile=tile, num_splits=splits, return_lse=True)
    assert np.abs(got - want).max() < tol
    assert np.abs(lse - want_lse).max() < tol * max(1.0, np.abs(want_lse).max())
    # tile size 1 with one split walks the keys one at a time like Alg. 3
    got = oracle.attn_tiled(q, k, v, 1.0, causal, tile=1, num_splits=1)
    assert np.abs(got - want).max() < tol
