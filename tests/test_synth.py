"""The seeded input generator: deterministic, follows its stated recipe."""
import torch

from paper_2505_14201_b200 import synth


def test_recipe_and_determinism():
    w = synth.WORKLOADS["c0"]
    q, k, v = synth.make_inputs(w)
    assert q.shape == (1, 1, 256, 64) and q.dtype == torch.float32
    g = torch.Generator().manual_seed(0)
    q2 = torch.randn(q.shape, generator=g); k2 = torch.randn(k.shape, generator=g); v2 = torch.randn(v.shape, generator=g)
    assert torch.equal(q, q2) and torch.equal(k, k2) and torch.equal(v, v2)
    assert abs(w.scale - 0.125) < 1e-12 and w.flops == 4 * 256 * 256 * 64


def test_outlier_rows_and_gains():
    q, k, v = synth.random_qkv(1, 2, 8, 130, 64, seed=3, q_gain=4.0, k_gain=4.0, outlier_every=64, outlier_gain=8.0)
    g = torch.Generator().manual_seed(3)
    q0 = torch.randn(1, 2, 8, 64, generator=g); k0 = torch.randn(1, 2, 130, 64, generator=g)
    assert torch.equal(q, (q0 * 4).to(torch.bfloat16))
    want = k0 * 4
    want[:, :, [0, 64, 128]] *= 8
    assert torch.equal(k, want.to(torch.bfloat16))
    assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16


def test_per_batch_draw_order():
    w = synth.Workload("t", 3, 2, 1, 16, 64, False, "bf16", 4, per_batch=True)
    q, k, v = synth.make_inputs(w)
    g = torch.Generator().manual_seed(4)
    q0 = torch.stack([torch.randn(2, 1, 64, generator=g) for _ in range(3)])
    k0 = torch.stack([torch.randn(2, 16, 64, generator=g) for _ in range(3)])
    assert torch.equal(q, q0.to(torch.bfloat16)) and torch.equal(k, k0.to(torch.bfloat16))


def test_workload_table_matches_the_five_configs():
    W = synth.WORKLOADS
    assert (W["c1"].B, W["c1"].H, W["c1"].Nq, W["c1"].d, W["c1"].causal) == (8, 12, 1024, 64, False)
    assert (W["c2"].B, W["c2"].H, W["c2"].Nq, W["c2"].d, W["c2"].causal) == (2, 32, 4096, 128, True)
    assert (W["c3"].Nq, W["c3"].q_gain, W["c3"].outlier_every, W["c3"].outlier_gain) == (16384, 4.0, 64, 8.0)
    assert (W["c4"].B, W["c4"].H, W["c4"].Nq, W["c4"].Nk, W["c4"].splitk) == (64, 32, 1, 32768, True)
    assert abs(W["c2"].flops - 2.749e11) / 2.749e11 < 1e-3
    assert W["c4"].kv_bytes == 34359738368
