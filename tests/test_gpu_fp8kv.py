"""GPU parity of the split-K decode with FP8-E4M3 K/V against the fp64 oracle.

The stored E4M3 values are the inputs: the oracle receives them widened exactly,
so the expected output is the plain definition on those values and the
tolerance is the bf16-output tolerance of the bf16 split-K path (the device
arithmetic is the same fp32 arithmetic).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_14201_b200 import synth

from test_gpu_parity import check_bf16, f32_scale, ok_status

pytestmark = pytest.mark.gpu


def fp8_inputs(B, H, Nq, Nk, d, seed, **kw):
    q, k, v = synth.random_qkv(B, H, Nq, Nk, d, seed=seed, **kw)
    return q, k.to(torch.float8_e4m3fn), v.to(torch.float8_e4m3fn)


def test_every_e4m3_code_is_widened_exactly(flashd_lib):
    """One key per head: the output is that key's V row, so all 256 codes pass through the
    device's widening; NaN codes (0x7f, 0xff) are left out of the comparison."""
    codes = torch.arange(256, dtype=torch.uint8)
    v = codes.view(torch.float8_e4m3fn).reshape(1, 2, 1, 128).contiguous()
    k = torch.zeros(1, 2, 1, 128).to(torch.float8_e4m3fn)
    q = torch.ones(1, 2, 1, 128, dtype=torch.bfloat16)
    got = flashd_lib.flashd_attn_fwd_splitk_fp8kv(q.cuda(), k.cuda(), v.cuda(), 1.0, 1)
    ok_status(flashd_lib)
    want = v.float()
    ok = ~torch.isnan(want)
    assert ok.sum() == 254
    # every finite E4M3 value is a bf16 value (3 mantissa bits, exponent range inside bf16's)
    assert torch.equal(got.cpu().float()[ok], want[ok])


@pytest.mark.parametrize("shape", [(1, 1, 1, 1, 128, 1), (2, 3, 1, 129, 128, 1), (1, 4, 1, 1000, 128, 3),
                                   (1, 2, 3, 2500, 128, 4), (2, 2, 1, 2048, 64, 4), (1, 3, 2, 777, 64, 2),
                                   (1, 1, 1, 9, 64, 8), (1, 300, 1, 600, 128, 2)])
def test_fp8kv_shapes(flashd_lib, shape):
    B, H, Nq, Nk, d, S = shape
    q, k, v = fp8_inputs(B, H, Nq, Nk, d, seed=1200 + Nk)
    sc = f32_scale(d)
    want, want_lse = oracle.attn_naive(q, k, v, sc, return_lse=True)
    qc, kc, vc = q.cuda(), k.cuda(), v.cuda()
    ws = flashd_lib.flashd_splitk_partial_fp8kv(qc, kc, vc, sc, S)
    ok_status(flashd_lib)
    got32, lse = flashd_lib.flashd_splitk_combine(ws, B, H, Nq, d, S, out_dtype=torch.float32, return_lse=True)
    assert np.abs(got32.double().cpu().numpy() - want).max() <= 2e-3
    assert np.abs(lse.double().cpu().numpy() - want_lse).max() <= 1e-3
    got = flashd_lib.flashd_attn_fwd_splitk_fp8kv(qc, kc, vc, sc, S)
    check_bf16(got, want, shape)
    assert torch.equal(got, got32.to(torch.bfloat16))
    auto = flashd_lib.flashd_attn_fwd_splitk_fp8kv(qc, kc, vc, sc, 0)
    check_bf16(auto, want, shape)


def test_fp8kv_matches_bf16_path_on_the_same_values(flashd_lib):
    """E4M3 values are bf16 values: the bf16 kernel on the widened tensors is the same function."""
    q, k, v = fp8_inputs(1, 4, 1, 5000, 128, seed=7)
    sc = f32_scale(128)
    a = flashd_lib.flashd_attn_fwd_splitk_fp8kv(q.cuda(), k.cuda(), v.cuda(), sc, 4)
    b = flashd_lib.flashd_attn_fwd_splitk(q.cuda(), k.to(torch.bfloat16).cuda(), v.to(torch.bfloat16).cuda(), sc, 4)
    ok_status(flashd_lib)
    assert (a.float() - b.float()).abs().max().item() <= 4e-3


def test_fp8kv_large_logits(flashd_lib):
    q, k, v = fp8_inputs(1, 4, 1, 3000, 128, seed=31, q_gain=4.0, k_gain=4.0, outlier_every=64, outlier_gain=8.0)
    sc = f32_scale(128)
    want = oracle.attn_naive(q, k, v, sc)
    got = flashd_lib.flashd_attn_fwd_splitk_fp8kv(q.cuda(), k.cuda(), v.cuda(), sc, 6)
    ok_status(flashd_lib)
    check_bf16(got, want)
