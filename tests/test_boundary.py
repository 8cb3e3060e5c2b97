"""Host-side tests of the C-ABI library that need no GPU: it loads, exports
every symbol the header declares, and validates arguments before launching."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "flashd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(flashd_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(flashd_lib):
    syms = declared_symbols()
    assert len(syms) >= 14
    L = flashd_lib.lib()
    for s in syms:
        assert hasattr(L, s), s
    assert sorted(flashd_lib.EXPORTED_SYMBOLS) == syms


def test_library_does_not_link_the_oracle(flashd_lib):
    data = open(flashd_lib.lib_path(), "rb").read()
    assert b"oracle_attn" not in data
    src = os.path.join(ROOT, "paper_2505_14201_b200")
    for dirpath, _, files in os.walk(src):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text, f
                assert "liboracle" not in text, f


def test_version_and_status_strings(flashd_lib):
    assert flashd_lib.version() >= 100
    seen = {flashd_lib.status_string(i) for i in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert flashd_lib.status_string(99) == "unknown status"


def test_validation_happens_before_any_launch(flashd_lib):
    L = flashd_lib.lib()
    n0 = flashd_lib.launch_count()
    buf = (ctypes.c_char * 4096)()
    base = ctypes.addressof(buf)
    a = ctypes.c_void_p((base + 255) // 256 * 256)          # aligned fake pointer (never dereferenced)
    mis = ctypes.c_void_p(a.value + 2)
    null = ctypes.c_void_p(0)
    fwd = L.flashd_attn_fwd
    assert fwd(null, a, a, a, 1, 1, 8, 8, 64, 0.1, 0, None) == 1          # NULL
    assert fwd(a, a, a, a, 0, 1, 8, 8, 64, 0.1, 0, None) == 2             # SHAPE
    assert fwd(a, a, a, a, 1, 1, 8, -3, 64, 0.1, 0, None) == 2
    assert fwd(a, a, a, a, 1, 1, 8, 8, 64, float("nan"), 0, None) == 2
    assert fwd(a, a, a, a, 1, 1, 8, 8, 64, float("inf"), 0, None) == 2
    assert fwd(mis, a, a, a, 1, 1, 8, 8, 64, 0.1, 0, None) == 4           # ALIGN
    assert fwd(a, a, a, ctypes.c_void_p(a.value + 512), 1, 1, 8, 8, 48, 0.1, 0, None) == 3   # d unsupported
    assert fwd(a, a, a, a, 1, 1, 8, 8, 64, 0.1, 0, None) == 2             # o aliases q
    assert L.flashd_attn_fwd_f32(a, a, a, a, 1, 1, 8, 8, 48, 0.1, 0, None) == 3
    assert L.flashd_attn_fwd_perkey(a, a, a, a, None, 1, 0, 1, 1, 8, 8, 64, 0.1, 0, None) == 3  # f32 -> bf16
    # split-K: split count and workspace size
    ws_need = L.flashd_splitk_workspace_bytes(1, 1, 1, 128, 4)
    assert ws_need == 4 * 129 * 4
    part = L.flashd_splitk_partial
    assert part(a, a, a, a, ws_need, 1, 1, 1, 1024, 128, 0.1, 0, None) == 5
    assert part(a, a, a, a, ws_need, 1, 1, 1, 1024, 128, 0.1, 65, None) == 5
    assert part(a, a, a, a, ws_need, 1, 1, 1, 2, 128, 0.1, 4, None) == 5           # more splits than keys
    assert part(a, a, a, a, ws_need - 1, 1, 1, 1, 1024, 128, 0.1, 4, None) == 5    # workspace too small
    assert part(a, a, a, a, ws_need, 1, 1, 1, 1024, 96, 0.1, 4, None) == 3
    assert L.flashd_splitk_combine(null, a, None, 1, 1, 1, 128, 4, 0, None) == 1
    assert L.flashd_splitk_combine(a, a, None, 1, 1, 1, 128, 0, 0, None) == 5
    # paged split-K: (q, k_pages, v_pages, table, lens, ws, ws_bytes, B, H, Nq, max_pages, page_size, num_pages, d, scale, S)
    pp = L.flashd_splitk_partial_paged
    assert pp(a, a, a, null, a, a, ws_need, 1, 1, 1, 4, 64, 8, 128, 0.1, 4, None) == 1
    assert pp(a, a, a, a, a, a, ws_need, 1, 1, 1, 4, 0, 8, 128, 0.1, 4, None) == 2
    assert pp(a, a, a, a, a, a, ws_need, 1, 1, 1, 4, 96, 8, 128, 0.1, 4, None) == 3     # page not a multiple of the ring stage
    assert pp(a, a, a, a, a, a, ws_need, 1, 1, 1, 4, 64, 8, 64, 0.1, 4, None) == 3      # d = 64 needs pages of 128 keys
    assert pp(a, a, a, ctypes.c_void_p(a.value + 2), a, a, ws_need, 1, 1, 1, 4, 64, 8, 128, 0.1, 4, None) == 4
    assert pp(a, a, a, a, a, a, ws_need - 1, 1, 1, 1, 4, 64, 8, 128, 0.1, 4, None) == 5
    assert pp(a, a, a, a, a, a, ws_need, 1, 1, 1, 4, 64, 8, 128, 0.1, 65, None) == 5
    assert L.flashd_attn_fwd_splitk_paged(a, a, a, null, a, a, a, ws_need, 1, 1, 1, 4, 64, 8, 128, 0.1, 4, None) == 1
    assert L.flashd_splitk_partial_paged_fp8kv(a, a, a, a, a, a, ws_need, 1, 1, 1, 4, 64, 8, 128, 0.1, 4, None) == 3   # E4M3 stage = 128 keys
    # E4M3 operands on the tensor path: (q, k, v, o, lse, out_dtype, B, H, Nq, Nk, d, scale, causal)
    o2 = ctypes.c_void_p(a.value + 512)
    assert L.flashd_attn_fwd_fp8(a, a, a, o2, None, 0, 1, 1, 8, 8, 64, 0.1, 0, None) == 3
    assert L.flashd_attn_fwd_fp8(a, a, a, o2, None, 7, 1, 1, 8, 8, 128, 0.1, 0, None) == 3
    assert L.flashd_attn_fwd_fp8(a, a, a, a, None, 0, 1, 1, 8, 8, 128, 0.1, 0, None) == 2     # o aliases q
    assert L.flashd_attn_fwd_fp8(null, a, a, o2, None, 0, 1, 1, 8, 8, 128, 0.1, 0, None) == 1
    assert L.flashd_attn_fwd_host(a, a, a, a, 7, 1, 1, 8, 8, 64, 0.1, 0, None) == 3
    assert L.flashd_attn_fwd_host(a, a, a, a, 2, 1, 1, 8, 8, 64, 0.1, 1, None) == 3  # split-K is non-causal
    assert flashd_lib.launch_count() == n0


def test_split_count_heuristic(flashd_lib):
    f = flashd_lib.flashd_splitk_num_splits
    assert f(64, 32, 1, 32768, 128) == 4
    assert f(1, 1, 1, 32768, 128) == 64
    assert f(1, 1, 1, 600, 128) == 1
    assert f(64, 32, 1, 8192, 128) >= 2
    for args in [(1, 8, 1, 100000, 128), (2, 2, 3, 5000, 64)]:
        s = f(*args)
        assert 1 <= s <= 64 and s <= args[3]
    assert f(0, 1, 1, 10, 64) == 0


def test_missing_library_fails_loudly(monkeypatch, flashd_lib):
    from paper_2505_14201_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "lib_path", lambda: "/nonexistent/libflashd.so")
    with pytest.raises(FileNotFoundError):
        binding.lib()
