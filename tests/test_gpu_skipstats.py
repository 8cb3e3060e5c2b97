"""GPU parity of the bypassable-update statistic (Sec. III-C / V-B) against the
CPU oracle.  Counts are integers: they must match exactly.  Both sides take the
decisions in fp64; the only admissible differences are steps that the oracle
reports as lying within 1e-4 of a threshold (the kernel's carried ln w has
fp32 terms), and the tests assert that bound."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2505_14201_b200 import synth

pytestmark = pytest.mark.gpu


def f32_scale(d):
    return float(np.float32(1.0 / math.sqrt(d)))


@pytest.mark.parametrize("shape", [(1, 2, 40, 70, 64, "bf16"), (2, 3, 130, 257, 128, "bf16"), (1, 2, 33, 50, 32, "f32"),
                                   (1, 1, 9, 300, 256, "bf16"), (1, 1, 1, 1, 64, "bf16")])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("gain", [1.0, 4.0])
def test_skip_stats_match_oracle(flashd_lib, shape, causal, gain):
    B, H, Nq, Nk, d, dt = shape
    q, k, _ = synth.random_qkv(B, H, Nq, Nk, d, seed=300 + Nk, dtype=dt, q_gain=gain, k_gain=gain,
                               outlier_every=16 if gain > 1 else 0, outlier_gain=8.0)
    sc = f32_scale(d)
    want = oracle.skip_stats(q, k, sc, causal)
    got = flashd_lib.flashd_skip_stats(q.cuda(), k.cuda(), sc, causal)
    near = want[5]
    assert got[0] == want[0]
    for a, b in zip(got[1:], want[1:5]):
        assert abs(a - b) <= near, (got, want)
    if near == 0:
        assert got == want[:5]
    # other thresholds
    want = oracle.skip_stats(q, k, sc, causal, lo=-2.0, hi=3.0, alo=-1.0, ahi=0.5)
    got = flashd_lib.flashd_skip_stats(q.cuda(), k.cuda(), sc, causal, lo=-2.0, hi=3.0, alo=-1.0, ahi=0.5)
    assert got[0] == want[0]
    for a, b in zip(got[1:], want[1:5]):
        assert abs(a - b) <= want[5], (got, want)


def test_skip_stats_exact_ties(flashd_lib):
    """Integer scores: the differences hit the thresholds exactly; ties count."""
    s = torch.tensor([0.0, -6.0, 5.0, 16.0, 16.0, 2.0, 13.0])
    q = torch.zeros(1, 1, 3, 32); q[..., 0] = 1
    k = torch.zeros(1, 1, 7, 32); k[0, 0, :, 0] = s
    for causal in (False, True):
        want = oracle.skip_stats(q, k, 1.0, causal)
        got = flashd_lib.flashd_skip_stats(q.cuda(), k.cuda(), 1.0, causal)
        assert got[:3] == want[:3]
    got = flashd_lib.flashd_skip_stats(q.cuda(), k.cuda(), 1.0, False)
    assert got[0] == 18 and got[1] == 3 * 2 and got[2] == 3 * 3     # diffs -6, 11, 11, 0, -14, 11 per row


def test_skip_stats_validation(flashd_lib):
    q, k, _ = synth.random_qkv(1, 1, 4, 4, 64, seed=1, device="cuda")
    L = flashd_lib.lib()
    cnt = torch.zeros(5, dtype=torch.int64, device="cuda")
    import ctypes
    vp = ctypes.c_void_p
    assert L.flashd_skip_stats(vp(q.data_ptr()), vp(k.data_ptr()), vp(0), 0, 1, 1, 4, 4, 64, 0.1, 0, -6, 11, -6, 6, None) == 1
    assert L.flashd_skip_stats(vp(q.data_ptr()), vp(k.data_ptr()), vp(cnt.data_ptr()), 0, 1, 1, 4, 4, 48, 0.1, 0, -6, 11, -6, 6, None) == 3
    assert L.flashd_skip_stats(vp(q.data_ptr()), vp(k.data_ptr()), vp(cnt.data_ptr()), 0, 1, 1, 4, 4, 64, 0.1, 0, 11, -6, -6, 6, None) == 2
