"""GPU parity of the PWL variant of Algorithm 3 (Sec. IV-B) against the oracle's
PWL variant, on the same seeded inputs and the same tables.

Both sides evaluate the same continuous PWL functions (the float32 nodes are
given to the oracle exactly); the device interpolates and blends in fp32, the
oracle in fp64.  Tolerance: max-abs 2e-4 for fp32 inputs and fp32 output when no
step of the oracle lies within 1e-4 of a range bound; a step that close may be
decided differently in fp32, which changes one weight by at most about
sigma(lo) = 0.25 %, so such cases are held to 1e-2 and their counts to the
number of near-bound steps.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2505_14201_b200 import pwl, synth

from test_gpu_parity import f32_scale, ok_status

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tables():
    return pwl.paper_tables()


def run_both(fd, q, k, v, sc, causal, sig, ln, lo, hi, mode):
    want, wc = oracle.attn_flashd_pwl(q, k, v, sc, causal, sig=sig, ln=ln, lo=lo, hi=hi, range_mode=mode,
                                      return_counts=True)
    got, gc = fd.flashd_attn_fwd_pwl(q.cuda(), k.cuda(), v.cuda(), sc, causal, sig=sig, ln=ln, lo=lo, hi=hi,
                                     range_mode=mode, out_dtype=torch.float32, return_counts=True)
    ok_status(fd)
    return got.double().cpu().numpy(), gc, want, wc


def test_exact_tables_unbounded_range_is_the_per_key_kernel(flashd_lib):
    q, k, v = synth.random_qkv(1, 3, 70, 150, 64, seed=11, dtype="f32", device="cuda")
    sc = f32_scale(64)
    for causal in (False, True):
        a = flashd_lib.flashd_attn_fwd_pwl(q, k, v, sc, causal, lo=-math.inf, hi=math.inf)
        b = flashd_lib.flashd_attn_fwd_perkey(q, k, v, sc, causal)
        assert torch.equal(a, b)


@pytest.mark.parametrize("shape", [(1, 2, 33, 300, 64, False, "f32"), (2, 2, 128, 128, 128, True, "f32"),
                                   (1, 3, 40, 1000, 32, False, "bf16"), (1, 1, 17, 257, 256, True, "bf16")])
@pytest.mark.parametrize("mode", [0, 1])
def test_fitted_tables_match_the_oracle(flashd_lib, tables, shape, mode):
    B, H, Nq, Nk, d, causal, dt = shape
    sig, ln = tables
    q, k, v = synth.random_qkv(B, H, Nq, Nk, d, seed=900 + Nk + mode, dtype=dt)
    sc = f32_scale(d)
    got, gc, want, wc = run_both(flashd_lib, q, k, v, sc, causal, sig, ln, -6.0, 11.0, mode)
    err = np.abs(got - want).max()
    if wc[2] == 0:
        assert gc == wc[:2], (gc, wc)
        assert err <= 2e-4, err
    else:
        assert abs(gc[0] - wc[0]) <= wc[2] and abs(gc[1] - wc[1]) <= wc[2], (gc, wc)
        assert err <= 1e-2, err
    if mode == 0:
        assert gc == (0, 0)


def test_exact_functions_with_bypass_on_stress_inputs(flashd_lib):
    """Large logits: many bypasses and replacements; exact sigma / ln so that only the range rule acts."""
    q, k, v = synth.random_qkv(1, 2, 64, 512, 64, seed=31, dtype="f32", q_gain=4.0, k_gain=4.0, outlier_every=64,
                               outlier_gain=8.0)
    sc = f32_scale(64)
    got, gc, want, wc = run_both(flashd_lib, q, k, v, sc, False, None, None, -6.0, 11.0, 1)
    assert wc[0] > 1000 and wc[1] > 10          # the rule fires
    assert abs(gc[0] - wc[0]) <= wc[2] and abs(gc[1] - wc[1]) <= wc[2], (gc, wc)
    assert np.abs(got - want).max() <= (2e-4 if wc[2] == 0 else 1e-2)


def test_malformed_tables_are_rejected(flashd_lib):
    q, k, v = synth.random_qkv(1, 1, 4, 8, 64, seed=1, dtype="f32", device="cuda")
    bad = [([0.0, 0.0, 1.0], [0.0, 0.5, 1.0]),                  # nodes not strictly increasing
           (list(range(70)), list(range(70))),                  # too many segments
           ([0.0, float("nan")], [0.0, 1.0])]
    for tab in bad:
        with pytest.raises(flashd_lib.FlashdError) as ei:
            flashd_lib.flashd_attn_fwd_pwl(q, k, v, 0.1, sig=tab)
        assert ei.value.status == 2
    with pytest.raises(flashd_lib.FlashdError) as ei:
        flashd_lib.flashd_attn_fwd_pwl(q, k, v, 0.1, lo=3.0, hi=-3.0)
    assert ei.value.status == 2
