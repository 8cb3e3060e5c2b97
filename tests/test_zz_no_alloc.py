"""The allocation-free split-K entry point (flashd_attn_fwd_splitk_static).

It serves callers that cannot obtain device memory inside the call - a decode
step of a server that gave all device memory to its own pool at start-up - by
keeping the partial states in a fixed array inside the library.  The test calls
it through the C ABI twice in a row (the second problem is smaller, so stale
contents of the shared array from the first call lie next to the slots the
second one uses) and compares each result with flashd_attn_fwd_splitk, which
takes a caller workspace, within the bf16 tolerance of the other GPU tests.
This file is collected last on purpose.
"""
import math

import numpy as np
import pytest
import torch

from paper_2505_14201_b200 import synth

pytestmark = pytest.mark.gpu

BF16_MAX, BF16_MEAN = 1e-2, 1e-3


def f32_scale(d):
    return float(np.float32(1.0 / math.sqrt(d)))


def test_static_scratch_matches_workspace_entry_point_twice(flashd_lib):
    fd = flashd_lib
    cases = [(2, 8, 1, 6000, 128, 8), (1, 3, 2, 700, 64, 3)]       # B, H, Nq, Nk, d, splits
    for n, (B, H, Nq, Nk, d, S) in enumerate(cases):
        q, k, v = synth.random_qkv(B, H, Nq, Nk, d, seed=900 + n, device="cuda")
        sc = f32_scale(d)
        want = fd.flashd_attn_fwd_splitk(q, k, v, sc, S)
        o = torch.full_like(q, float("nan"))
        got = fd.flashd_attn_fwd_splitk_static(q, k, v, sc, S, o=o)
        st, detail = fd.flashd_last_device_status()
        assert st == 0, detail
        err = (got.double() - want.double()).abs()
        assert torch.isfinite(got.float()).all()
        assert err.max().item() <= BF16_MAX and err.mean().item() <= BF16_MEAN, (n, err.max().item())
        # library's own split count
        got_auto = fd.flashd_attn_fwd_splitk_static(q, k, v, sc, 0)
        want_auto = fd.flashd_attn_fwd_splitk(q, k, v, sc, 0)
        err = (got_auto.double() - want_auto.double()).abs()
        assert err.max().item() <= BF16_MAX and err.mean().item() <= BF16_MEAN


def test_static_scratch_rejects_oversized_problems(flashd_lib):
    fd = flashd_lib
    B, H, Nq, Nk, d, S = 1, 300, 1, 2048, 128, 64      # 300*64*129*4 bytes = 9.9 MB > 8 MiB
    assert B * H * Nq * S * (d + 1) * 4 > fd.STATIC_SCRATCH_BYTES
    q, k, v = synth.random_qkv(B, H, Nq, Nk, d, seed=7, device="cuda")
    n0 = fd.launch_count()
    with pytest.raises(fd.FlashdError) as ei:
        fd.flashd_attn_fwd_splitk_static(q, k, v, f32_scale(d), S)
    assert ei.value.status == 5
    assert fd.launch_count() == n0
    # the same problem with fewer splits fits
    got = fd.flashd_attn_fwd_splitk_static(q, k, v, f32_scale(d), 32)
    want = fd.flashd_attn_fwd_splitk(q, k, v, f32_scale(d), 32)
    assert (got.double() - want.double()).abs().max().item() <= BF16_MAX
