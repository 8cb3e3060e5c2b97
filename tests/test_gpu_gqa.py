"""GPU parity of the grouped-query split-K decode (G query heads share one K/V
head) against the fp64 oracle.  The oracle has no grouped form: the attention
function of each query head is unchanged, so the expected output is the plain
definition evaluated with that head's shared K and V.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_14201_b200 import synth

from test_gpu_parity import check_bf16, f32_scale, ok_status

pytestmark = pytest.mark.gpu


def gqa_inputs(B, Hkv, G, Nk, d, seed, **kw):
    """q [B,Hkv*G,1,d], k/v [B,Hkv,Nk,d]: independent draws for queries and keys."""
    q, _, _ = synth.random_qkv(B, Hkv * G, 1, 1, d, seed=seed, **{a: b for a, b in kw.items() if a.startswith("q_")})
    _, k, v = synth.random_qkv(B, Hkv, 1, Nk, d, seed=seed + 1, **{a: b for a, b in kw.items() if not a.startswith("q_")})
    return q, k, v


def oracle_gqa(q, k, v, G, sc, **kw):
    return oracle.attn_naive(q, k.repeat_interleave(G, dim=1), v.repeat_interleave(G, dim=1), sc, **kw)


GQA_SHAPES = [
    # B, Hkv, G, Nk, d, S
    (1, 1, 1, 1, 128, 1),          # a single key: o = v
    (1, 1, 8, 15, 128, 1),         # fewer keys than one warp's share
    (2, 3, 4, 129, 128, 1),        # one chunk and one key
    (1, 2, 8, 1000, 128, 3),       # ragged splits, split starts not on a chunk boundary
    (1, 2, 3, 777, 128, 4),        # G not a power of two
    (2, 2, 2, 2048, 64, 4),
    (1, 3, 8, 333, 64, 2),
    (1, 1, 5, 4100, 64, 8),
    (1, 2, 8, 10, 128, 4),         # per-split 3 keys; the last split holds one key
    (1, 1, 7, 9, 64, 8),           # ceil(9/8) = 2 keys per split: splits 5..7 are empty
    (1, 160, 4, 600, 128, 2),      # more work items than CTAs
]


@pytest.mark.parametrize("shape", GQA_SHAPES)
def test_gqa_shapes(flashd_lib, shape):
    B, Hkv, G, Nk, d, S = shape
    q, k, v = gqa_inputs(B, Hkv, G, Nk, d, seed=700 + Nk + G)
    sc = f32_scale(d)
    want, want_lse = oracle_gqa(q, k, v, G, sc, return_lse=True)
    qc, kc, vc = q.cuda(), k.cuda(), v.cuda()
    ws = flashd_lib.flashd_gqa_partial(qc, kc, vc, sc, S)
    ok_status(flashd_lib)
    assert tuple(ws.shape) == (B, Hkv * G, 1, S, d + 1)
    # which splits are empty is fixed by the split rule alone
    per = -(-Nk // S)
    nonempty = np.array([s * per < Nk for s in range(S)])
    Lp = ws[..., d].cpu().numpy()
    assert np.all(np.isfinite(Lp[..., nonempty])) and np.all(np.isneginf(Lp[..., ~nonempty]))
    got32, lse = flashd_lib.flashd_splitk_combine(ws, B, Hkv * G, 1, d, S, out_dtype=torch.float32, return_lse=True)
    e = np.abs(got32.double().cpu().numpy() - want)
    assert e.max() <= 1e-2 and e.mean() <= 1e-3, (shape, e.max(), e.mean())
    assert np.abs(lse.double().cpu().numpy() - want_lse).max() <= 1e-3
    got = flashd_lib.flashd_attn_fwd_gqa(qc, kc, vc, sc, S)
    ok_status(flashd_lib)
    check_bf16(got, want, shape)
    assert torch.equal(got, got32.to(torch.bfloat16))
    auto = flashd_lib.flashd_attn_fwd_gqa(qc, kc, vc, sc, 0)
    check_bf16(auto, want, shape)
    # the first split alone is the attention over the first ceil(Nk/S) keys
    if S > 1:
        pre = flashd_lib.flashd_splitk_combine(ws[:, :, :, :1].contiguous(), B, Hkv * G, 1, d, 1,
                                               out_dtype=torch.float32)
        wantp = oracle_gqa(q, k[:, :, :per], v[:, :, :per], G, sc)
        assert np.abs(pre.double().cpu().numpy() - wantp).max() <= 1e-2


MULTI_Q_SHAPES = [
    # B, Hkv, G, Nq, Nk, d, S, causal
    (1, 2, 2, 4, 500, 128, 3, True),
    (2, 2, 4, 2, 1000, 128, 4, True),
    (1, 1, 1, 8, 100, 64, 2, True),
    (1, 2, 2, 3, 300, 128, 2, False),      # G*Nq = 6, no mask among the positions
    (1, 1, 2, 4, 4, 64, 1, True),          # Nk = Nq: the first position sees one key
    (1, 1, 1, 8, 9, 64, 8, True),          # 2 keys per split: most splits are empty for the early positions
    (1, 40, 2, 4, 2100, 128, 4, True),     # more work items than CTAs
]


@pytest.mark.parametrize("shape", MULTI_Q_SHAPES)
def test_gqa_several_query_positions(flashd_lib, shape):
    """A decode step over the last Nq positions: position iq sees keys 0 .. Nk-Nq+iq."""
    B, Hkv, G, Nq, Nk, d, S, causal = shape
    q, _, _ = synth.random_qkv(B, Hkv * G, Nq, 1, d, seed=800 + Nk)
    _, k, v = synth.random_qkv(B, Hkv, 1, Nk, d, seed=801 + Nk)
    sc = f32_scale(d)
    q_index = [Nk - Nq + iq for iq in range(Nq)]
    want, want_lse = oracle.attn_naive(q, k.repeat_interleave(G, dim=1), v.repeat_interleave(G, dim=1), sc, causal,
                                       q_index=q_index, return_lse=True)
    qc, kc, vc = q.cuda(), k.cuda(), v.cuda()
    ws = flashd_lib.flashd_gqa_partial(qc, kc, vc, sc, S, causal=causal)
    ok_status(flashd_lib)
    assert tuple(ws.shape) == (B, Hkv * G, Nq, S, d + 1)
    # a partial state is empty exactly when its split holds no visible key of that position
    per = -(-Nk // S)
    Lp = ws[..., d].cpu().numpy()
    for iq in range(Nq):
        lim = (Nk - Nq + iq + 1) if causal else Nk
        for sp in range(S):
            nonempty = sp * per < min(lim, Nk)
            assert np.all(np.isfinite(Lp[:, :, iq, sp])) == nonempty and (nonempty or np.all(np.isneginf(Lp[:, :, iq, sp])))
    got32, lse = flashd_lib.flashd_splitk_combine(ws, B, Hkv * G, Nq, d, S, out_dtype=torch.float32, return_lse=True)
    e = np.abs(got32.double().cpu().numpy() - want)
    assert e.max() <= 1e-2 and e.mean() <= 1e-3, (shape, e.max(), e.mean())
    assert np.abs(lse.double().cpu().numpy() - want_lse).max() <= 1e-3
    got = flashd_lib.flashd_attn_fwd_gqa(qc, kc, vc, sc, S, causal=causal)
    ok_status(flashd_lib)
    assert torch.equal(got, got32.to(torch.bfloat16))
    check_bf16(got, want, shape)


def test_gqa_matches_single_query_path_on_repeated_heads(flashd_lib):
    """Same function, two data paths: the grouped kernel on shared heads and the
    single-query split-K kernel on explicitly repeated heads agree to rounding."""
    B, Hkv, G, Nk, d = 1, 4, 8, 5000, 128
    q, k, v = gqa_inputs(B, Hkv, G, Nk, d, seed=77)
    sc = f32_scale(d)
    a = flashd_lib.flashd_attn_fwd_gqa(q.cuda(), k.cuda(), v.cuda(), sc, 4)
    b = flashd_lib.flashd_attn_fwd_splitk(q.cuda(), k.repeat_interleave(G, dim=1).contiguous().cuda(),
                                          v.repeat_interleave(G, dim=1).contiguous().cuda(), sc, 4)
    ok_status(flashd_lib)
    assert (a.float() - b.float()).abs().max().item() <= 1e-2


def test_gqa_large_logits_and_negative_scale(flashd_lib):
    B, Hkv, G, Nk, d = 1, 2, 8, 3000, 128
    q, k, v = gqa_inputs(B, Hkv, G, Nk, d, seed=31, q_gain=4.0, k_gain=4.0, outlier_every=64, outlier_gain=8.0)
    for sc in (f32_scale(d), -f32_scale(d)):
        want = oracle_gqa(q, k, v, G, sc)
        got = flashd_lib.flashd_attn_fwd_gqa(q.cuda(), k.cuda(), v.cuda(), sc, 6)
        ok_status(flashd_lib)
        check_bf16(got, want, sc)


def test_gqa_rejects_bad_arguments(flashd_lib):
    q, k, v = gqa_inputs(1, 1, 16, 64, 128, seed=1)
    with pytest.raises(flashd_lib.FlashdError) as ei:
        flashd_lib.flashd_attn_fwd_gqa(q.cuda(), k.cuda(), v.cuda(), 0.1, 1)
    assert ei.value.status == 3
    q, k, v = gqa_inputs(1, 1, 4, 64, 128, seed=1)
    with pytest.raises(flashd_lib.FlashdError) as ei:
        flashd_lib.flashd_gqa_partial(q.cuda(), k.cuda(), v.cuda(), 0.1, 2,
                                      workspace=torch.empty(16, dtype=torch.float32, device="cuda"))
    assert ei.value.status == 5
    with pytest.raises(ValueError):
        flashd_lib.flashd_attn_fwd_gqa(q[:, :3].contiguous().cuda(), torch.cat([k, k], 1).cuda(),
                                       torch.cat([v, v], 1).cuda(), 0.1, 1)
    # G * Nq beyond the limit, and more causal positions than keys
    q9, _, _ = synth.random_qkv(1, 3, 3, 1, 128, seed=2)
    _, k1, v1 = synth.random_qkv(1, 1, 1, 64, 128, seed=3)
    with pytest.raises(flashd_lib.FlashdError) as ei:
        flashd_lib.flashd_attn_fwd_gqa(q9.cuda(), k1.cuda(), v1.cuda(), 0.1, 1)
    assert ei.value.status == 3
    q4, _, _ = synth.random_qkv(1, 1, 4, 1, 128, seed=2)
    with pytest.raises(flashd_lib.FlashdError) as ei:
        flashd_lib.flashd_attn_fwd_gqa(q4.cuda(), k1[:, :, :2].contiguous().cuda(), v1[:, :, :2].contiguous().cuda(), 0.1, 1,
                                       causal=True)
    assert ei.value.status == 2


def test_gqa_long_context_sampled(flashd_lib):
    """Long-context grouped decode in the library's own launch configuration
    (131072 keys, 8 K/V heads, groups of 8); two K/V heads recomputed by the oracle."""
    B, Hkv, G, Nk, d = 2, 8, 8, 131072, 128
    g = torch.Generator(device="cuda").manual_seed(5)
    q = torch.randn(B, Hkv * G, 1, d, generator=g, device="cuda").to(torch.bfloat16)
    k = torch.randn(B, Hkv, Nk, d, generator=g, device="cuda").to(torch.bfloat16)
    v = torch.randn(B, Hkv, Nk, d, generator=g, device="cuda").to(torch.bfloat16)
    sc = f32_scale(d)
    got = flashd_lib.flashd_attn_fwd_gqa(q, k, v, sc, 0)
    ok_status(flashd_lib)
    for (b, h) in [(0, 0), (1, 7)]:
        want = oracle_gqa(q[b:b + 1, h * G:(h + 1) * G].cpu(), k[b:b + 1, h:h + 1].cpu(), v[b:b + 1, h:h + 1].cpu(), G, sc)
        check_bf16(got[b:b + 1, h * G:(h + 1) * G], want, (b, h))
