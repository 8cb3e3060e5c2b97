"""ctypes front end of the FLASH-D CPU oracle (``flashd_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The oracle is a plain fp64 restatement of the paper
(FLASH-D: FlashAttention with Hidden Softmax Division) used to check the CUDA
library.  Only tests, the smoke check and the benchmark's CPU-baseline leg may
import it; the product package never does, and this module imports nothing
from the product package.

All functions take array-likes (numpy arrays or torch CPU tensors of any float
dtype, bf16 included) shaped ``[B, H, N, d]`` and return float64 numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "flashd_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math) unless it is up to date."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
           "-fno-fast-math", "-ffp-contract=off", _SRC, "-o", tmp, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_D = ctypes.POINTER(ctypes.c_double)
_I = ctypes.POINTER(ctypes.c_int)
_LL = ctypes.POINTER(ctypes.c_longlong)


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            ci, cd = ctypes.c_int, ctypes.c_double
            lib.oracle_num_threads.restype = ci
            lib.oracle_attn_naive.argtypes = [_D, _D, _D, _D, _D, _D, ci, ci, ci, ci, ci, cd, ci, _I]
            lib.oracle_attn_alg1.argtypes = [_D, _D, _D, _D, ci, ci, ci, ci, ci, cd, ci, _I]
            lib.oracle_attn_alg2.argtypes = [_D, _D, _D, _D, ci, ci, ci, ci, ci, cd, ci, _I]
            lib.oracle_attn_flashd.argtypes = [_D, _D, _D, _D, _D, ci, ci, ci, ci, ci, cd, ci, _I, ci, ci]
            lib.oracle_attn_tiled.argtypes = [_D, _D, _D, _D, _D, _D, _D, ci, ci, ci, ci, ci, cd, ci, _I, ci, ci]
            lib.oracle_split_merge.argtypes = [_D, _D, _D, _D, ci, ci, ci]
            lib.oracle_flashd_weights.argtypes = [_D, ci, _D, ci]
            lib.oracle_skip_stats.argtypes = [_D, _D, _LL, ci, ci, ci, ci, ci, cd, ci, _I, cd, cd, cd, cd, cd]
            lib.oracle_attn_flashd_pwl.argtypes = [_D, _D, _D, _D, ci, ci, ci, ci, ci, cd, ci, _I,
                                                   ci, _D, _D, ci, _D, _D, cd, cd, ci, cd, _LL]
            lib.oracle_attn_flashd_pwl.restype = None
            lib.oracle_pwl_eval.argtypes = [_D, _D, ci, cd]
            lib.oracle_pwl_eval.restype = cd
            for f in ("oracle_attn_naive", "oracle_attn_alg1", "oracle_attn_alg2",
                      "oracle_attn_flashd", "oracle_attn_tiled", "oracle_split_merge",
                      "oracle_flashd_weights", "oracle_skip_stats"):
                getattr(lib, f).restype = None
            _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops of the oracle will use."""
    return int(_load().oracle_num_threads())


def _f64(x) -> np.ndarray:
    """Exact upcast of a stored tensor (bf16 / fp32 / fp64) to contiguous float64."""
    if hasattr(x, "detach"):  # torch tensor, without importing torch here
        x = x.detach().cpu().double().numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _p(a):
    return None if a is None else a.ctypes.data_as(_D)


def _prep(q, k, v, q_index):
    q, k, v = _f64(q), _f64(k), _f64(v)
    if q.ndim != 4 or k.ndim != 4 or v.ndim != 4:
        raise ValueError("expected [B, H, N, d] arrays")
    B, H, Nq, d = q.shape
    Nk = k.shape[2]
    if k.shape != (B, H, Nk, d) or v.shape != (B, H, Nk, d):
        raise ValueError("shape mismatch between q, k, v")
    qi = None
    if q_index is not None:
        qi = np.ascontiguousarray(np.asarray(q_index, dtype=np.int32))
        if qi.shape != (Nq,):
            raise ValueError("q_index must have one entry per query row")
    return q, k, v, B, H, Nq, Nk, d, qi


def _pi(qi):
    return None if qi is None else qi.ctypes.data_as(_I)


def attn_naive(q, k, v, scale, causal=False, q_index=None, return_lse=False,
               return_weights=False):
    """Sec. II-A definition with safe softmax.  ``q_index`` gives the global row
    index of each query row passed (for the causal mask) when only a sample of
    rows is evaluated."""
    q, k, v, B, H, Nq, Nk, d, qi = _prep(q, k, v, q_index)
    o = np.empty((B, H, Nq, d))
    lse = np.empty((B, H, Nq)) if return_lse else None
    w = np.empty((B, H, Nq, Nk)) if return_weights else None
    _load().oracle_attn_naive(_p(q), _p(k), _p(v), _p(o), _p(lse), _p(w),
                              B, H, Nq, Nk, d, float(scale), int(bool(causal)), _pi(qi))
    out = (o,)
    if return_lse:
        out += (lse,)
    if return_weights:
        out += (w,)
    return out[0] if len(out) == 1 else out


def attn_alg1(q, k, v, scale, causal=False, q_index=None):
    """Algorithm 1 (baseline FlashAttention)."""
    q, k, v, B, H, Nq, Nk, d, qi = _prep(q, k, v, q_index)
    o = np.empty((B, H, Nq, d))
    _load().oracle_attn_alg1(_p(q), _p(k), _p(v), _p(o), B, H, Nq, Nk, d,
                             float(scale), int(bool(causal)), _pi(qi))
    return o


def attn_alg2(q, k, v, scale, causal=False, q_index=None):
    """Algorithm 2 (FlashAttention2, lazy division)."""
    q, k, v, B, H, Nq, Nk, d, qi = _prep(q, k, v, q_index)
    o = np.empty((B, H, Nq, d))
    _load().oracle_attn_alg2(_p(q), _p(k), _p(v), _p(o), B, H, Nq, Nk, d,
                             float(scale), int(bool(causal)), _pi(qi))
    return o


def attn_flashd(q, k, v, scale, causal=False, q_index=None, variant=0, blend_form=0,
                return_lse=False):
    """Algorithm 3 (FLASH-D) per key.  ``variant`` 0 = Eq. (w-last) carrying
    ln w (the parity reading); 1 = literal linear-domain w; 2 = Alg. 3's printed
    sign.  ``blend_form`` 0 = o + (v - o) w, 1 = o (1 - w) + v w."""
    q, k, v, B, H, Nq, Nk, d, qi = _prep(q, k, v, q_index)
    o = np.empty((B, H, Nq, d))
    lse = np.empty((B, H, Nq)) if return_lse else None
    _load().oracle_attn_flashd(_p(q), _p(k), _p(v), _p(o), _p(lse), B, H, Nq, Nk, d,
                               float(scale), int(bool(causal)), _pi(qi),
                               int(variant), int(blend_form))
    return (o, lse) if return_lse else o


def attn_tiled(q, k, v, scale, causal=False, q_index=None, tile=128, num_splits=1,
               return_lse=False, return_partials=False):
    """Group ("super-key") form: fused tile update inside a split, super-key
    merge across splits."""
    q, k, v, B, H, Nq, Nk, d, qi = _prep(q, k, v, q_index)
    o = np.empty((B, H, Nq, d))
    lse = np.empty((B, H, Nq)) if return_lse else None
    po = np.empty((B, H, Nq, num_splits, d)) if return_partials else None
    pL = np.empty((B, H, Nq, num_splits)) if return_partials else None
    _load().oracle_attn_tiled(_p(q), _p(k), _p(v), _p(o), _p(lse), _p(po), _p(pL),
                              B, H, Nq, Nk, d, float(scale), int(bool(causal)), _pi(qi),
                              int(tile), int(num_splits))
    out = (o,)
    if return_lse:
        out += (lse,)
    if return_partials:
        out += (po, pL)
    return out[0] if len(out) == 1 else out


def split_merge(partial_o, partial_L, return_lse=False):
    """Fold per-split states ``[..., S, d]`` / ``[..., S]`` in split order."""
    po, pL = _f64(partial_o), _f64(partial_L)
    S, d = po.shape[-2], po.shape[-1]
    rows = int(np.prod(po.shape[:-2], dtype=np.int64))
    if pL.shape != po.shape[:-1]:
        raise ValueError("partial_L must be partial_o without its last axis")
    o = np.empty(po.shape[:-2] + (d,))
    lse = np.empty(po.shape[:-2]) if return_lse else None
    _load().oracle_split_merge(_p(po), _p(pL), _p(o), _p(lse), rows, S, d)
    return (o, lse) if return_lse else o


def flashd_weights(s, variant=0):
    """Weights w_1..w_N of Algorithm 3 for one score vector."""
    s = _f64(s).reshape(-1)
    w = np.empty_like(s)
    _load().oracle_flashd_weights(_p(s), int(s.size), _p(w), int(variant))
    return w


def skip_stats(q, k, scale, causal=False, q_index=None, lo=-6.0, hi=11.0, alo=-6.0, ahi=6.0, near=1e-4):
    """Bypassable output updates (Sec. III-C / V-B).  Returns (steps, diff <= lo,
    diff >= hi, x <= alo, x >= ahi, steps within ``near`` of a threshold) where
    diff = s_i - s_{i-1} and x = diff + ln w_{i-1}."""
    q, k = _f64(q), _f64(k)
    B, H, Nq, d = q.shape
    Nk = k.shape[2]
    qi = None if q_index is None else np.ascontiguousarray(np.asarray(q_index, dtype=np.int32))
    counts = np.zeros(6, dtype=np.int64)
    _load().oracle_skip_stats(_p(q), _p(k), counts.ctypes.data_as(_LL), B, H, Nq, Nk, d,
                              float(scale), int(bool(causal)), _pi(qi), float(lo), float(hi),
                              float(alo), float(ahi), float(near))
    return tuple(int(c) for c in counts)


def pwl_eval(xs, ys, x) -> float:
    """Continuous piece-wise linear function through the nodes (xs, ys), saturating outside."""
    xs, ys = _f64(xs), _f64(ys)
    return float(_load().oracle_pwl_eval(_p(xs), _p(ys), len(xs) - 1, float(x)))


def attn_flashd_pwl(q, k, v, scale, causal=False, q_index=None, sig=None, ln=None, lo=-6.0, hi=11.0,
                    range_mode=0, near=1e-4, return_counts=False):
    """Sec. IV-B: Algorithm 3 with PWL sigmoid / ln.  ``sig`` and ``ln`` are (xs, ys) node
    tables or None for the exact function; ``range_mode`` 0 saturates the sigmoid argument to
    [lo, hi], 1 bypasses keys below lo and replaces the output above hi.  With
    ``return_counts`` also returns (bypassed, replaced, near-threshold) step counts."""
    q, k, v, B, H, Nq, Nk, d, qi = _prep(q, k, v, q_index)
    o = np.empty((B, H, Nq, d))
    sx, sy = (None, None) if sig is None else (_f64(sig[0]), _f64(sig[1]))
    lx, ly = (None, None) if ln is None else (_f64(ln[0]), _f64(ln[1]))
    counts = np.zeros(3, dtype=np.int64)
    _load().oracle_attn_flashd_pwl(_p(q), _p(k), _p(v), _p(o), B, H, Nq, Nk, d, float(scale),
                                   int(bool(causal)), _pi(qi),
                                   0 if sx is None else len(sx) - 1, _p(sx), _p(sy),
                                   0 if lx is None else len(lx) - 1, _p(lx), _p(ly),
                                   float(lo), float(hi), int(range_mode), float(near),
                                   counts.ctypes.data_as(_LL))
    return (o, tuple(int(c) for c in counts)) if return_counts else o
