"""Seeded synthetic attention inputs.

This module only draws random tensors; it holds none of the method's
arithmetic and is the one piece shared by the CUDA tests, the CPU oracle tests
and the benchmark.  Tensors are [B, H, N, d].

Recipe: ``g = torch.Generator(device).manual_seed(seed)``; draw Q, then K, then
V as fp32 standard normals from ``g`` (one ``randn`` call per tensor, or one per
batch element for K and V when ``per_batch`` is set, Q first, then all of K,
then all of V); multiply Q by ``q_gain`` and K by ``k_gain``; multiply key rows
``j % outlier_every == 0`` by a further ``outlier_gain``; round to the storage
dtype (round to nearest even).  Both the oracle and the kernels consume the
rounded tensors.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    Nq: int
    Nk: int
    d: int
    causal: bool
    dtype: str            # "bf16" or "f32"
    seed: int
    q_gain: float = 1.0
    k_gain: float = 1.0
    outlier_every: int = 0
    outlier_gain: float = 1.0
    splitk: bool = False
    per_batch: bool = False   # draw K and V one batch element at a time (large tensors)
    note: str = ""

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    @property
    def flops(self) -> float:
        f = 4.0 * self.B * self.H * self.Nq * self.Nk * self.d
        return f / 2 if self.causal else f

    @property
    def kv_bytes(self) -> int:
        return 2 * self.B * self.H * self.Nk * self.d * (2 if self.dtype == "bf16" else 4)


WORKLOADS = {
    "c0": Workload("c0 tiny fp32", 1, 1, 256, 256, 64, False, "f32", 0),
    "c1": Workload("c1 encoder-shaped bf16", 8, 12, 1024, 1024, 64, False, "bf16", 1),
    "c2": Workload("c2 decoder prefill bf16 causal", 2, 32, 4096, 4096, 128, True, "bf16", 2),
    "c3": Workload("c3 stability stress bf16 causal", 1, 32, 16384, 16384, 128, True, "bf16", 3,
                   q_gain=4.0, k_gain=4.0, outlier_every=64, outlier_gain=8.0),
    "c4": Workload("c4 long-context decode bf16 split-K", 64, 32, 1, 32768, 128, False, "bf16", 4,
                   splitk=True, per_batch=True),
}


def make_inputs(w: Workload, device="cpu"):
    """Returns (q, k, v) for a workload on ``device`` following the module recipe."""
    import torch
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    g = torch.Generator(device=device).manual_seed(w.seed)

    def draw(N, gain, outliers):
        if w.per_batch:
            out = torch.empty((w.B, w.H, N, w.d), dtype=dt, device=device)
            for b in range(w.B):
                x = torch.randn((w.H, N, w.d), dtype=torch.float32, device=device, generator=g)
                out[b] = _finish(x, gain, outliers, w, dt)
            return out
        x = torch.randn((w.B, w.H, N, w.d), dtype=torch.float32, device=device, generator=g)
        return _finish(x, gain, outliers, w, dt)

    q = draw(w.Nq, w.q_gain, False)
    k = draw(w.Nk, w.k_gain, True)
    v = draw(w.Nk, 1.0, False)
    return q, k, v


def _finish(x, gain, outliers, w, dt):
    if gain != 1.0:
        x = x * gain
    if outliers and w.outlier_every > 0:
        x[..., :: w.outlier_every, :] *= w.outlier_gain
    return x.to(dt)


def random_qkv(B, H, Nq, Nk, d, seed, dtype="bf16", q_gain=1.0, k_gain=1.0, outlier_every=0,
               outlier_gain=1.0, device="cpu"):
    """Small ad-hoc problem with the same recipe (used by the parity tests)."""
    w = Workload("adhoc", B, H, Nq, Nk, d, False, dtype, seed, q_gain, k_gain, outlier_every, outlier_gain)
    return make_inputs(w, device)
