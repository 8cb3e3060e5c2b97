"""ctypes binding with the same names as the C ABI in ``include/flashd.h``.

Tensor arguments are torch tensors; the functions pass their ``data_ptr()`` and
sizes through and raise :class:`FlashdError` on a non-zero status.  Outputs are
allocated by the caller or, when omitted, with ``torch.empty`` on the inputs'
device (torch is used for device memory and streams only).
"""
from __future__ import annotations

import ctypes
import os
import threading

BF16, F32 = 0, 1
MAX_SPLITS = 64

EXPORTED_SYMBOLS = (
    "flashd_attn_fwd", "flashd_attn_fwd_ex", "flashd_attn_fwd_f32", "flashd_attn_fwd_perkey",
    "flashd_splitk_workspace_bytes", "flashd_splitk_num_splits", "flashd_splitk_partial",
    "flashd_splitk_combine", "flashd_attn_fwd_splitk", "flashd_attn_fwd_splitk_static",
    "flashd_gqa_num_splits", "flashd_gqa_partial", "flashd_attn_fwd_gqa", "flashd_attn_fwd_pwl",
    "flashd_splitk_partial_fp8kv", "flashd_attn_fwd_splitk_fp8kv",
    "flashd_splitk_partial_paged", "flashd_attn_fwd_splitk_paged", "flashd_attn_fwd_fp8",
    "flashd_splitk_partial_paged_fp8kv", "flashd_attn_fwd_splitk_paged_fp8kv",
    "flashd_gqa_partial_paged", "flashd_attn_fwd_gqa_paged",
    "flashd_attn_fwd_host", "flashd_skip_stats", "flashd_last_device_status", "flashd_status_string", "flashd_version", "flashd_launch_count",
)

_lock = threading.Lock()
_lib = None


class FlashdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: flashd status {status} ({status_string(status)})")


def lib_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libflashd.so")


def lib() -> ctypes.CDLL:
    """Load ``libflashd.so``; raises if it has not been built (no fallback)."""
    global _lib
    with _lock:
        if _lib is None:
            path = lib_path()
            if not os.path.exists(path):
                raise FileNotFoundError(
                    f"{path} is missing: build it with `python -m paper_2505_14201_b200.build` "
                    "(nvcc, sm_100a). There is no CPU fallback.")
            L = ctypes.CDLL(path)
            vp, ci, cf, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
            fwd = [vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, ci, vp]
            L.flashd_attn_fwd.argtypes = fwd
            L.flashd_attn_fwd_f32.argtypes = fwd
            ex = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, cf, ci, vp]
            L.flashd_attn_fwd_ex.argtypes = ex
            L.flashd_attn_fwd_perkey.argtypes = ex
            L.flashd_attn_fwd_fp8.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, ci, vp]
            L.flashd_splitk_workspace_bytes.argtypes = [ci, ci, ci, ci, ci]
            L.flashd_splitk_workspace_bytes.restype = sz
            L.flashd_splitk_num_splits.argtypes = [ci, ci, ci, ci, ci]
            L.flashd_splitk_partial.argtypes = [vp, vp, vp, vp, sz, ci, ci, ci, ci, ci, cf, ci, vp]
            L.flashd_splitk_combine.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, ci, vp]
            L.flashd_attn_fwd_splitk.argtypes = [vp, vp, vp, vp, vp, sz, ci, ci, ci, ci, ci, cf, ci, vp]
            L.flashd_splitk_partial_paged.argtypes = [vp, vp, vp, vp, vp, vp, sz, ci, ci, ci, ci, ci, ci, ci, cf, ci, vp]
            L.flashd_attn_fwd_splitk_paged.argtypes = [vp, vp, vp, vp, vp, vp, vp, sz, ci, ci, ci, ci, ci, ci, ci, cf, ci, vp]
            L.flashd_splitk_partial_paged_fp8kv.argtypes = L.flashd_splitk_partial_paged.argtypes
            L.flashd_gqa_partial_paged.argtypes = [vp, vp, vp, vp, vp, vp, sz, ci, ci, ci, ci, ci, ci, ci, ci, cf, ci, ci, vp]
            L.flashd_attn_fwd_gqa_paged.argtypes = [vp, vp, vp, vp, vp, vp, vp, sz, ci, ci, ci, ci, ci, ci, ci, ci, cf, ci, ci, vp]
            L.flashd_attn_fwd_splitk_paged_fp8kv.argtypes = L.flashd_attn_fwd_splitk_paged.argtypes
            fp = ctypes.POINTER(ctypes.c_float)
            L.flashd_attn_fwd_pwl.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, cf, ci,
                                              ci, fp, fp, ci, fp, fp, cf, cf, ci, vp]
            L.flashd_gqa_num_splits.argtypes = [ci, ci, ci, ci, ci]
            L.flashd_gqa_partial.argtypes = [vp, vp, vp, vp, sz, ci, ci, ci, ci, ci, ci, cf, ci, ci, vp]
            L.flashd_attn_fwd_gqa.argtypes = [vp, vp, vp, vp, vp, sz, ci, ci, ci, ci, ci, ci, cf, ci, ci, vp]
            L.flashd_splitk_partial_fp8kv.argtypes = [vp, vp, vp, vp, sz, ci, ci, ci, ci, ci, cf, ci, vp]
            L.flashd_attn_fwd_splitk_fp8kv.argtypes = [vp, vp, vp, vp, vp, sz, ci, ci, ci, ci, ci, cf, ci, vp]
            L.flashd_attn_fwd_splitk_static.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, ci, vp]
            L.flashd_skip_stats.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, ci, cf, cf, cf, cf, vp]
            L.flashd_attn_fwd_host.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, ci, vp]
            L.flashd_last_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int)]
            L.flashd_status_string.argtypes = [ci]
            L.flashd_status_string.restype = ctypes.c_char_p
            L.flashd_version.argtypes = []
            L.flashd_launch_count.argtypes = []
            L.flashd_launch_count.restype = ctypes.c_longlong
            _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().flashd_status_string(int(status)).decode()


def version() -> int:
    return int(lib().flashd_version())


def launch_count() -> int:
    return int(lib().flashd_launch_count())


def _check(status: int, where: str):
    if status != 0:
        raise FlashdError(int(status), where)


def _stream_ptr(stream):
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return ctypes.c_void_p(stream)
    return ctypes.c_void_p(stream.cuda_stream)


def _dims(q, k, v):
    if q.dim() != 4 or k.dim() != 4 or v.dim() != 4:
        raise ValueError("q, k, v must be [B, H, N, d]")
    B, H, Nq, d = q.shape
    Nk = k.shape[2]
    if tuple(k.shape) != (B, H, Nk, d) or tuple(v.shape) != (B, H, Nk, d):
        raise ValueError("shape mismatch between q, k, v")
    if not (q.is_contiguous() and k.is_contiguous() and v.is_contiguous()):
        raise ValueError("q, k, v must be contiguous")
    return B, H, Nq, Nk, d


def _dtype_code(t):
    import torch
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise ValueError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def flashd_attn_fwd(q, k, v, scale, causal=False, o=None, stream=None):
    """bf16 tiled tensor-core forward; returns ``o`` ([B,H,Nq,d] bf16)."""
    import torch
    B, H, Nq, Nk, d = _dims(q, k, v)
    if o is None:
        o = torch.empty_like(q)
    _check(lib().flashd_attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, H, Nq, Nk, d,
                                 float(scale), int(bool(causal)), _stream_ptr(stream)), "flashd_attn_fwd")
    return o


def flashd_attn_fwd_ex(q, k, v, scale, causal=False, out_dtype=None, return_lse=False, o=None,
                       stream=None):
    import torch
    B, H, Nq, Nk, d = _dims(q, k, v)
    out_dtype = q.dtype if out_dtype is None else out_dtype
    if o is None:
        o = torch.empty(q.shape, dtype=out_dtype, device=q.device)
    lse = torch.empty((B, H, Nq), dtype=torch.float32, device=q.device) if return_lse else None
    _check(lib().flashd_attn_fwd_ex(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _dtype_code(q),
                                    _dtype_code(o), B, H, Nq, Nk, d, float(scale), int(bool(causal)),
                                    _stream_ptr(stream)), "flashd_attn_fwd_ex")
    return (o, lse) if return_lse else o


def flashd_attn_fwd_fp8(q, k, v, scale, causal=False, out_dtype=None, return_lse=False, o=None, stream=None):
    """Tiled tensor-core forward with E4M3 operands (``torch.float8_e4m3fn`` q, k, v; d = 128 or 256);
    output bf16 (default) or fp32."""
    import torch
    B, H, Nq, Nk, d = _dims(q, k, v)
    for t in (q, k, v):
        if t.dtype != torch.float8_e4m3fn:
            raise ValueError("flashd_attn_fwd_fp8 takes torch.float8_e4m3fn tensors")
    out_dtype = torch.bfloat16 if out_dtype is None else out_dtype
    if o is None:
        o = torch.empty(q.shape, dtype=out_dtype, device=q.device)
    lse = torch.empty((B, H, Nq), dtype=torch.float32, device=q.device) if return_lse else None
    _check(lib().flashd_attn_fwd_fp8(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _dtype_code(o), B, H, Nq, Nk, d,
                                     float(scale), int(bool(causal)), _stream_ptr(stream)), "flashd_attn_fwd_fp8")
    return (o, lse) if return_lse else o


def flashd_attn_fwd_f32(q, k, v, scale, causal=False, o=None, stream=None):
    """fp32 per-key forward (Algorithm 3 one key at a time)."""
    import torch
    B, H, Nq, Nk, d = _dims(q, k, v)
    if q.dtype != torch.float32:
        raise ValueError("flashd_attn_fwd_f32 takes fp32 tensors")
    if o is None:
        o = torch.empty_like(q)
    _check(lib().flashd_attn_fwd_f32(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, H, Nq, Nk, d,
                                     float(scale), int(bool(causal)), _stream_ptr(stream)), "flashd_attn_fwd_f32")
    return o


def flashd_attn_fwd_perkey(q, k, v, scale, causal=False, out_dtype=None, return_lse=False, o=None,
                           stream=None):
    import torch
    B, H, Nq, Nk, d = _dims(q, k, v)
    out_dtype = q.dtype if out_dtype is None else out_dtype
    if o is None:
        o = torch.empty(q.shape, dtype=out_dtype, device=q.device)
    lse = torch.empty((B, H, Nq), dtype=torch.float32, device=q.device) if return_lse else None
    _check(lib().flashd_attn_fwd_perkey(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _dtype_code(q),
                                        _dtype_code(o), B, H, Nq, Nk, d, float(scale), int(bool(causal)),
                                        _stream_ptr(stream)), "flashd_attn_fwd_perkey")
    return (o, lse) if return_lse else o


PWL_MAX_SEGMENTS = 64


def _host_table(tab):
    """(xs, ys) -> (n, float* x, float* y, keep-alive); None -> exact function."""
    if tab is None:
        return 0, None, None, None
    xs = [float(t) for t in tab[0]]
    ys = [float(t) for t in tab[1]]
    if len(xs) != len(ys) or len(xs) < 2:
        raise ValueError("a PWL table needs matching node lists of at least two nodes")
    ax = (ctypes.c_float * len(xs))(*xs)
    ay = (ctypes.c_float * len(ys))(*ys)
    return len(xs) - 1, ax, ay, (ax, ay)


def flashd_attn_fwd_pwl(q, k, v, scale, causal=False, sig=None, ln=None, lo=-6.0, hi=11.0, range_mode=0,
                        out_dtype=None, return_counts=False, o=None, stream=None):
    """Algorithm 3 with piece-wise linear sigmoid / ln tables (Sec. IV-B accuracy model).
    ``sig`` / ``ln``: (xs, ys) node lists or None for the exact function."""
    import torch
    B, H, Nq, Nk, d = _dims(q, k, v)
    out_dtype = q.dtype if out_dtype is None else out_dtype
    if o is None:
        o = torch.empty(q.shape, dtype=out_dtype, device=q.device)
    counts = torch.zeros(2, dtype=torch.int64, device=q.device) if return_counts else None
    sn, sx, sy, keep1 = _host_table(sig)
    ln_n, lx, ly, keep2 = _host_table(ln)
    _check(lib().flashd_attn_fwd_pwl(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(counts), _dtype_code(q),
                                     _dtype_code(o), B, H, Nq, Nk, d, float(scale), int(bool(causal)),
                                     sn, sx, sy, ln_n, lx, ly, float(lo), float(hi), int(range_mode),
                                     _stream_ptr(stream)), "flashd_attn_fwd_pwl")
    del keep1, keep2
    return (o, tuple(int(c) for c in counts.cpu())) if return_counts else o


def flashd_splitk_workspace_bytes(B, H, Nq, d, num_splits) -> int:
    return int(lib().flashd_splitk_workspace_bytes(B, H, Nq, d, num_splits))


def flashd_splitk_num_splits(B, H, Nq, Nk, d) -> int:
    return int(lib().flashd_splitk_num_splits(B, H, Nq, Nk, d))


def flashd_splitk_partial(q, k, v, scale, num_splits, workspace=None, stream=None):
    """Returns the workspace tensor ``[B,H,Nq,num_splits,d+1]`` fp32 (o_p | L_p)."""
    import torch
    B, H, Nq, Nk, d = _dims(q, k, v)
    if workspace is None:
        workspace = torch.empty((B, H, Nq, num_splits, d + 1), dtype=torch.float32, device=q.device)
    _check(lib().flashd_splitk_partial(_ptr(q), _ptr(k), _ptr(v), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), B, H, Nq, Nk, d,
                                       float(scale), int(num_splits), _stream_ptr(stream)), "flashd_splitk_partial")
    return workspace


def flashd_splitk_combine(workspace, B, H, Nq, d, num_splits, out_dtype=None, return_lse=False, o=None,
                          stream=None):
    import torch
    out_dtype = torch.bfloat16 if out_dtype is None else out_dtype
    if o is None:
        o = torch.empty((B, H, Nq, d), dtype=out_dtype, device=workspace.device)
    lse = torch.empty((B, H, Nq), dtype=torch.float32, device=workspace.device) if return_lse else None
    _check(lib().flashd_splitk_combine(_ptr(workspace), _ptr(o), _ptr(lse), B, H, Nq, d, int(num_splits),
                                       _dtype_code(o), _stream_ptr(stream)), "flashd_splitk_combine")
    return (o, lse) if return_lse else o


def flashd_attn_fwd_splitk(q, k, v, scale, num_splits=0, workspace=None, o=None, stream=None):
    """Split-K forward (partial + combine); ``num_splits <= 0`` lets the library choose."""
    import torch
    B, H, Nq, Nk, d = _dims(q, k, v)
    S = num_splits if num_splits > 0 else flashd_splitk_num_splits(B, H, Nq, Nk, d)
    if workspace is None:
        workspace = torch.empty((B, H, Nq, max(S, 1), d + 1), dtype=torch.float32, device=q.device)
    if o is None:
        o = torch.empty_like(q)
    _check(lib().flashd_attn_fwd_splitk(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), B, H, Nq, Nk, d,
                                        float(scale), int(num_splits), _stream_ptr(stream)), "flashd_attn_fwd_splitk")
    return o


def _paged_dims(q, k_pages, v_pages, block_table, seq_lens):
    import torch
    for t in (q, k_pages, v_pages, block_table, seq_lens):
        if not t.is_contiguous():
            raise ValueError("paged split-K: all tensors must be contiguous")
    if q.dim() != 4 or k_pages.dim() != 4 or tuple(v_pages.shape) != tuple(k_pages.shape):
        raise ValueError("paged split-K: q [B,H,Nq,d], k_pages / v_pages [num_pages,H,page_size,d]")
    B, H, Nq, d = q.shape
    num_pages, Hk, page_size, dk = k_pages.shape
    if Hk != H or dk != d or block_table.dim() != 2 or block_table.shape[0] != B or tuple(seq_lens.shape) != (B,):
        raise ValueError("paged split-K: shapes do not match")
    if block_table.dtype != torch.int32 or seq_lens.dtype != torch.int32:
        raise ValueError("paged split-K: block_table and seq_lens must be int32")
    return B, H, Nq, d, num_pages, page_size, block_table.shape[1]


def flashd_splitk_partial_paged(q, k_pages, v_pages, block_table, seq_lens, scale, num_splits, workspace=None,
                                stream=None):
    """Partial states ``[B,H,Nq,num_splits,d+1]`` fp32 of the split-K forward over a paged K/V pool."""
    import torch
    B, H, Nq, d, num_pages, page_size, max_pages = _paged_dims(q, k_pages, v_pages, block_table, seq_lens)
    if workspace is None:
        workspace = torch.empty((B, H, Nq, num_splits, d + 1), dtype=torch.float32, device=q.device)
    fn = lib().flashd_splitk_partial_paged_fp8kv if k_pages.dtype == torch.float8_e4m3fn else lib().flashd_splitk_partial_paged
    _check(fn(_ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(block_table), _ptr(seq_lens),
                                             _ptr(workspace), workspace.numel() * workspace.element_size(), B, H, Nq,
                                             max_pages, page_size, num_pages, d, float(scale), int(num_splits),
                                             _stream_ptr(stream)), "flashd_splitk_partial_paged")
    return workspace


def flashd_attn_fwd_splitk_paged(q, k_pages, v_pages, block_table, seq_lens, scale, num_splits=0, workspace=None,
                                 o=None, stream=None):
    """Split-K forward over a paged K/V pool with one length per sequence (partial + combine)."""
    import torch
    B, H, Nq, d, num_pages, page_size, max_pages = _paged_dims(q, k_pages, v_pages, block_table, seq_lens)
    S = num_splits if num_splits > 0 else flashd_splitk_num_splits(B, H, Nq, max_pages * page_size, d)
    if workspace is None:
        workspace = torch.empty((B, H, Nq, max(S, 1), d + 1), dtype=torch.float32, device=q.device)
    if o is None:
        o = torch.empty_like(q)
    fn = lib().flashd_attn_fwd_splitk_paged_fp8kv if k_pages.dtype == torch.float8_e4m3fn else lib().flashd_attn_fwd_splitk_paged
    _check(fn(_ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(o), _ptr(block_table), _ptr(seq_lens), _ptr(workspace),
              workspace.numel() * workspace.element_size(), B, H, Nq, max_pages, page_size, num_pages, d,
              float(scale), int(num_splits), _stream_ptr(stream)), "flashd_attn_fwd_splitk_paged")
    return o


def flashd_attn_fwd_gqa_paged(q, k_pages, v_pages, block_table, seq_lens, scale, num_splits=0, causal=False,
                              workspace=None, o=None, stream=None):
    """Grouped-query decode over a paged K/V pool (``q: [B,Hkv*G,Nq,d]``, pool ``[num_pages,Hkv,page_size,d]``)."""
    import torch
    for t in (q, k_pages, v_pages, block_table, seq_lens):
        if not t.is_contiguous():
            raise ValueError("paged grouped-query decode: all tensors must be contiguous")
    B, Hq, Nq, d = q.shape
    num_pages, Hkv, page_size, dk = k_pages.shape
    if dk != d or Hq % Hkv != 0 or tuple(v_pages.shape) != tuple(k_pages.shape) or block_table.shape[0] != B \
            or tuple(seq_lens.shape) != (B,) or block_table.dtype != torch.int32 or seq_lens.dtype != torch.int32:
        raise ValueError("paged grouped-query decode: shapes or dtypes do not match")
    G = Hq // Hkv
    max_pages = block_table.shape[1]
    S = num_splits if num_splits > 0 else flashd_gqa_num_splits(B, Hkv, G, max_pages * page_size, d)
    if workspace is None:
        workspace = torch.empty((B, Hq, Nq, max(S, 1), d + 1), dtype=torch.float32, device=q.device)
    if o is None:
        o = torch.empty_like(q)
    _check(lib().flashd_attn_fwd_gqa_paged(_ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(o), _ptr(block_table),
                                           _ptr(seq_lens), _ptr(workspace),
                                           workspace.numel() * workspace.element_size(), B, Hkv, G, Nq, max_pages,
                                           page_size, num_pages, d, float(scale), int(bool(causal)), int(num_splits),
                                           _stream_ptr(stream)), "flashd_attn_fwd_gqa_paged")
    return o


MAX_GROUP = 8


def _gqa_dims(q, k, v):
    for t in (q, k, v):
        if not (t.dim() == 4 and t.is_contiguous()):
            raise ValueError("q, k, v must be contiguous [B, H, N, d] tensors")
    B, Hq, Nq, d = q.shape
    Bk, Hkv, Nk, dk = k.shape
    if Bk != B or dk != d or tuple(v.shape) != tuple(k.shape) or Hkv == 0 or Hq % Hkv != 0:
        raise ValueError(f"grouped-query shapes do not match: q {tuple(q.shape)} k {tuple(k.shape)} v {tuple(v.shape)}")
    return B, Hkv, Hq // Hkv, Nq, Nk, d


def flashd_gqa_num_splits(B, Hkv, G, Nk, d) -> int:
    return int(lib().flashd_gqa_num_splits(B, Hkv, G, Nk, d))


def flashd_gqa_partial(q, k, v, scale, num_splits, causal=False, workspace=None, stream=None):
    """Partial states ``[B,Hkv*G,Nq,num_splits,d+1]`` fp32 of the grouped-query split-K forward."""
    import torch
    B, Hkv, G, Nq, Nk, d = _gqa_dims(q, k, v)
    if workspace is None:
        workspace = torch.empty((B, Hkv * G, Nq, num_splits, d + 1), dtype=torch.float32, device=q.device)
    _check(lib().flashd_gqa_partial(_ptr(q), _ptr(k), _ptr(v), _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), B, Hkv, G, Nq, Nk, d,
                                    float(scale), int(bool(causal)), int(num_splits), _stream_ptr(stream)),
           "flashd_gqa_partial")
    return workspace


def flashd_attn_fwd_gqa(q, k, v, scale, num_splits=0, causal=False, workspace=None, o=None, stream=None):
    """Grouped-query split-K forward: q ``[B,Hkv*G,Nq,d]`` (the last Nq positions of the
    sequence; ``causal`` masks among them), k/v ``[B,Hkv,Nk,d]``; G*Nq <= 8."""
    import torch
    B, Hkv, G, Nq, Nk, d = _gqa_dims(q, k, v)
    S = num_splits if num_splits > 0 else flashd_gqa_num_splits(B, Hkv, G, Nk, d)
    if workspace is None:
        workspace = torch.empty((B, Hkv * G, Nq, max(S, 1), d + 1), dtype=torch.float32, device=q.device)
    if o is None:
        o = torch.empty_like(q)
    _check(lib().flashd_attn_fwd_gqa(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), B, Hkv, G, Nq, Nk, d,
                                     float(scale), int(bool(causal)), int(num_splits), _stream_ptr(stream)),
           "flashd_attn_fwd_gqa")
    return o


def flashd_splitk_partial_fp8kv(q, k, v, scale, num_splits, workspace=None, stream=None):
    """Partial states of the split-K forward with E4M3 K/V (``torch.float8_e4m3fn``), q bf16."""
    import torch
    B, H, Nq, Nk, d = _dims(q, k, v)
    if workspace is None:
        workspace = torch.empty((B, H, Nq, num_splits, d + 1), dtype=torch.float32, device=q.device)
    _check(lib().flashd_splitk_partial_fp8kv(_ptr(q), _ptr(k), _ptr(v), _ptr(workspace),
                                             workspace.numel() * workspace.element_size(), B, H, Nq, Nk, d,
                                             float(scale), int(num_splits), _stream_ptr(stream)),
           "flashd_splitk_partial_fp8kv")
    return workspace


def flashd_attn_fwd_splitk_fp8kv(q, k, v, scale, num_splits=0, workspace=None, o=None, stream=None):
    """Split-K forward with E4M3 K/V: q, o bf16 ``[B,H,Nq,d]``; k, v ``torch.float8_e4m3fn``."""
    import torch
    B, H, Nq, Nk, d = _dims(q, k, v)
    if q.dtype != torch.bfloat16 or k.dtype != torch.float8_e4m3fn or v.dtype != torch.float8_e4m3fn:
        raise ValueError("expected bf16 q and float8_e4m3fn k, v")
    S = num_splits if num_splits > 0 else flashd_splitk_num_splits(B, H, Nq, Nk, d)
    if workspace is None:
        workspace = torch.empty((B, H, Nq, max(S, 1), d + 1), dtype=torch.float32, device=q.device)
    if o is None:
        o = torch.empty_like(q)
    _check(lib().flashd_attn_fwd_splitk_fp8kv(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(workspace),
                                              workspace.numel() * workspace.element_size(), B, H, Nq, Nk, d,
                                              float(scale), int(num_splits), _stream_ptr(stream)),
           "flashd_attn_fwd_splitk_fp8kv")
    return o


STATIC_SCRATCH_BYTES = 8 << 20


def flashd_attn_fwd_splitk_static(q, k, v, scale, num_splits=0, o=None, stream=None):
    """Split-K forward for callers that must not allocate device memory inside
    the call (a server's per-token decode step running under a fixed memory
    plan): the partial states go to a fixed array inside the library instead of
    a caller workspace.  Problems whose partial states exceed
    ``STATIC_SCRATCH_BYTES`` raise ``FlashdError`` (status 5).  Calls share that
    array, so they must not overlap on the GPU.  Pass ``o`` to keep this wrapper
    from allocating the output."""
    import torch
    B, H, Nq, Nk, d = _dims(q, k, v)
    if o is None:
        o = torch.empty_like(q)
    _check(lib().flashd_attn_fwd_splitk_static(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, H, Nq, Nk, d,
                                               float(scale), int(num_splits), _stream_ptr(stream)),
           "flashd_attn_fwd_splitk_static")
    return o


def flashd_attn_fwd_host(q, k, v, scale, causal=False, path=0, o=None, stream=None):
    """End-to-end call on HOST tensors (pinned for asynchronous copies); synchronises."""
    import torch
    if q.is_cuda or k.is_cuda or v.is_cuda:
        raise ValueError("flashd_attn_fwd_host takes host tensors")
    B, H, Nq, Nk, d = _dims(q, k, v)
    if o is None:
        o = torch.empty_like(q, pin_memory=True)
    _check(lib().flashd_attn_fwd_host(_ptr(q), _ptr(k), _ptr(v), _ptr(o), int(path), B, H, Nq, Nk, d,
                                      float(scale), int(bool(causal)), _stream_ptr(stream)), "flashd_attn_fwd_host")
    return o


def flashd_skip_stats(q, k, scale, causal=False, lo=-6.0, hi=11.0, alo=-6.0, ahi=6.0, stream=None):
    """Bypassable-update counts (steps, diff <= lo, diff >= hi, x <= alo, x >= ahi) as Python ints."""
    import torch
    if q.dim() != 4 or k.dim() != 4 or q.shape[:2] != k.shape[:2] or q.shape[3] != k.shape[3]:
        raise ValueError("q, k must be [B, H, N, d] with matching B, H, d")
    if not (q.is_contiguous() and k.is_contiguous()):
        raise ValueError("q, k must be contiguous")
    B, H, Nq, d = q.shape
    Nk = k.shape[2]
    counts = torch.empty(5, dtype=torch.int64, device=q.device)
    _check(lib().flashd_skip_stats(_ptr(q), _ptr(k), _ptr(counts), _dtype_code(q), B, H, Nq, Nk, d, float(scale),
                                   int(bool(causal)), float(lo), float(hi), float(alo), float(ahi),
                                   _stream_ptr(stream)), "flashd_skip_stats")
    return tuple(int(x) for x in counts.cpu().tolist())


def flashd_last_device_status(stream=None):
    """(status, [code, block, which wait, iteration]) after synchronising the stream."""
    detail = (ctypes.c_int * 4)()
    st = lib().flashd_last_device_status(_stream_ptr(stream), detail)
    return int(st), list(detail)
