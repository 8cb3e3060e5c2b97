"""Random shapes through the tiled tensor-core forward (bf16 and E4M3 operands).

A protocol test rather than a parity test: the kernel's warp roles hand work to each other
through two dozen barriers, some of them looked at ahead of time, and work items of many
lengths follow each other on a CTA.  Every shape is run twice back to back (the second launch
overlaps the drain of the first) and must repeat bit for bit, raise no device status, and agree
with the per-key kernel (Algorithm 3 one key at a time, itself checked against the oracle in
test_gpu_parity.py) within the bf16 tolerance.  Seeded, so a failure names its shape."""
import math
import random

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

NQ = [1, 17, 128, 129, 255, 256, 257, 384, 500, 777, 1024, 1300]
NK = [1, 64, 127, 128, 129, 300, 640, 1000, 1500]


def test_random_shapes(flashd_lib):
    rnd = random.Random(1234)
    F8 = torch.float8_e4m3fn
    for it in range(150):
        d = rnd.choice([64, 128, 256])
        B = rnd.randint(1, 3)
        H = rnd.randint(1, 40 if it % 7 == 0 else 6)
        Nq = rnd.choice(NQ)
        Nk = Nq if rnd.random() < 0.6 else rnd.choice(NK)
        causal = rnd.random() < 0.5
        what = (it, d, B, H, Nq, Nk, causal)
        g = torch.Generator(device="cuda").manual_seed(it)
        q = torch.randn(B, H, Nq, d, generator=g, device="cuda").to(torch.bfloat16)
        k = torch.randn(B, H, Nk, d, generator=g, device="cuda").to(torch.bfloat16)
        v = torch.randn(B, H, Nk, d, generator=g, device="cuda").to(torch.bfloat16)
        sc = float(np.float32(1 / math.sqrt(d)))
        a = flashd_lib.flashd_attn_fwd_ex(q, k, v, sc, causal, out_dtype=torch.float32)
        a2 = flashd_lib.flashd_attn_fwd_ex(q, k, v, sc, causal, out_dtype=torch.float32)
        ref = flashd_lib.flashd_attn_fwd_perkey(q, k, v, sc, causal, out_dtype=torch.float32)
        st, detail = flashd_lib.flashd_last_device_status()
        assert st == 0, (what, detail)
        assert torch.isfinite(a).all(), what
        assert torch.equal(a, a2), what
        assert (a - ref).abs().max().item() <= 1e-2, what
        if d >= 128 and it % 3 == 0:
            q8, k8, v8 = q.to(F8), k.to(F8), v.to(F8)
            o8 = flashd_lib.flashd_attn_fwd_fp8(q8, k8, v8, sc, causal, out_dtype=torch.float32)
            o8b = flashd_lib.flashd_attn_fwd_fp8(q8, k8, v8, sc, causal, out_dtype=torch.float32)
            r8 = flashd_lib.flashd_attn_fwd_perkey(q8.to(torch.bfloat16), k8.to(torch.bfloat16), v8.to(torch.bfloat16),
                                                   sc, causal, out_dtype=torch.float32)
            st, detail = flashd_lib.flashd_last_device_status()
            assert st == 0, (what, detail)
            assert torch.isfinite(o8).all() and torch.equal(o8, o8b), what
            # E4M3 weights: 2^-4 relative per weight against values of a few units (rigorous bound in test_gpu_fp8_tiled.py)
            e8 = (o8 - r8).abs()
            assert e8.max().item() <= 0.35 and e8.mean().item() <= 8e-3, (what, e8.max().item(), e8.mean().item())
