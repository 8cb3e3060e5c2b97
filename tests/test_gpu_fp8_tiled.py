"""GPU parity of the tiled tensor-core forward with E4M3 operands against the fp64 oracle.

The stored E4M3 values of q, k, v are the inputs (the oracle widens them exactly).  The one
approximation beyond the bf16 kernel is the rounding of the per-tile weights to E4M3 for the
P V product: at most 2^-4 relative per weight (2^-10 absolute in the subnormal range), so an
output element may differ from the exact one by 2^-4 * sum_j f_j |v_j| + 2^-6; sum_j f_j |v_j|
is the oracle's output for |V|.  A second, looser-than-measured guard on the mean error keeps
a gross loss of accuracy from hiding under that bound."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_14201_b200 import synth

from test_gpu_parity import f32_scale, ok_status

pytestmark = pytest.mark.gpu

F8 = torch.float8_e4m3fn


def fp8_qkv(B, H, Nq, Nk, d, seed, **kw):
    q, k, v = synth.random_qkv(B, H, Nq, Nk, d, seed=seed, **kw)
    return q.to(F8), k.to(F8), v.to(F8)


def check(got32, q, k, v, sc, causal, what, mean_tol=6e-3):
    want = oracle.attn_naive(q, k, v, sc, causal)
    bound = oracle.attn_naive(q, k, v.float().abs().to(F8), sc, causal) * 2.0 ** -4 + 2.0 ** -6
    g = got32.double().cpu().numpy()
    assert np.all(np.isfinite(g)), what
    err = np.abs(g - want)
    assert np.all(err <= bound), (what, float((err - bound).max()), float(err.max()))
    assert err.mean() <= mean_tol, (what, err.mean())
    return err


@pytest.mark.parametrize("shape", [
    (1, 1, 128, 128, False), (1, 2, 256, 256, True), (2, 3, 200, 200, True), (1, 2, 1, 1, False),
    (1, 2, 300, 1000, False), (1, 1, 1000, 300, True), (1, 4, 777, 777, True), (2, 2, 1024, 1024, False),
    (1, 160, 256, 384, True),                      # more work items than SMs
])
def test_fp8_tiled_shapes(flashd_lib, shape):
    B, H, Nq, Nk, causal = shape
    d = 128
    q, k, v = fp8_qkv(B, H, Nq, Nk, d, seed=500 + Nq + Nk)
    sc = f32_scale(d)
    got32, lse = flashd_lib.flashd_attn_fwd_fp8(q.cuda(), k.cuda(), v.cuda(), sc, causal, out_dtype=torch.float32,
                                                return_lse=True)
    ok_status(flashd_lib)
    check(got32, q, k, v, sc, causal, shape)
    _, want_lse = oracle.attn_naive(q, k, v, sc, causal, return_lse=True)
    assert np.abs(lse.double().cpu().numpy() - want_lse).max() <= 2e-3
    got16 = flashd_lib.flashd_attn_fwd_fp8(q.cuda(), k.cuda(), v.cuda(), sc, causal)
    assert torch.equal(got16, got32.to(torch.bfloat16))      # the bf16 output is the rounding of the fp32 one


@pytest.mark.parametrize("shape", [(1, 1, 128, 128, False), (1, 2, 256, 256, True), (2, 3, 200, 333, False),
                                   (1, 2, 1, 1, False), (1, 4, 777, 777, True), (1, 200, 130, 260, True)])
def test_fp8_tiled_hidden_size_256(flashd_lib, shape):
    B, H, Nq, Nk, causal = shape
    d = 256
    q, k, v = fp8_qkv(B, H, Nq, Nk, d, seed=700 + Nq + Nk)
    sc = f32_scale(d)
    got32 = flashd_lib.flashd_attn_fwd_fp8(q.cuda(), k.cuda(), v.cuda(), sc, causal, out_dtype=torch.float32)
    ok_status(flashd_lib)
    check(got32, q, k, v, sc, causal, shape)


def test_equal_scores_give_the_mean_of_every_code(flashd_lib):
    """K = 0: every weight is exactly 1 (representable), so the output is the plain mean of the V
    rows and only fp32 accumulation rounds.  V runs through all 254 finite E4M3 codes."""
    d, Nk = 128, 256
    codes = (torch.arange(Nk * d, dtype=torch.int64) * 37 % 256).to(torch.uint8)
    codes[(codes & 0x7f) == 0x7f] = 0x10           # the two NaN codes
    v = codes.view(F8).reshape(1, 1, Nk, d).contiguous()
    k = torch.zeros(1, 1, Nk, d).to(F8)
    q = torch.ones(1, 1, 130, d).to(F8)
    got = flashd_lib.flashd_attn_fwd_fp8(q.cuda(), k.cuda(), v.cuda(), 1.0, False, out_dtype=torch.float32)
    ok_status(flashd_lib)
    want = v.double().mean(dim=2, keepdim=True).expand(1, 1, 130, d).numpy()
    scale_ = np.abs(v.double().numpy()).mean()
    assert np.abs(got.double().cpu().numpy() - want).max() <= 1e-5 * scale_ * Nk ** 0.5 + 1e-4


def test_large_logits_and_dominant_keys(flashd_lib):
    """Stress recipe (gains on q, k; outlier keys): rows dominated by one key have weight 1 for
    it exactly; no overflow, no NaN."""
    d = 128
    q, k, v = fp8_qkv(1, 2, 512, 512, d, seed=77, q_gain=4.0, k_gain=4.0, outlier_every=64, outlier_gain=8.0)
    sc = f32_scale(d)
    got = flashd_lib.flashd_attn_fwd_fp8(q.cuda(), k.cuda(), v.cuda(), sc, True, out_dtype=torch.float32)
    ok_status(flashd_lib)
    check(got, q, k, v, sc, True, "stress")


def test_rejects_other_head_sizes(flashd_lib):
    q, k, v = fp8_qkv(1, 1, 128, 128, 64, seed=1)
    with pytest.raises(flashd_lib.FlashdError):
        flashd_lib.flashd_attn_fwd_fp8(q.cuda(), k.cuda(), v.cuda(), 0.1, False)
