"""Host-only checks of the C-ABI library: it loads, exports every symbol include/s2a.h declares,
and rejects bad arguments before touching a device.  No compute calls."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "s2a.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2309_12307_b200 import build

    path = build.build()
    return ctypes.CDLL(path)


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(s2a_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = _declared_functions()
    for n in ("s2a_fwd", "s2a_bwd", "s2a_bwd_workspace_bytes", "s2a_status_string", "s2a_version"):
        assert n in names


def test_library_exports_every_declared_symbol(lib):
    for name in _declared_functions():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_names():
    from paper_2309_12307_b200 import binding

    assert sorted(binding.EXPORTS) == _declared_functions()


def test_version_and_status_strings(lib):
    lib.s2a_status_string.restype = ctypes.c_char_p
    assert lib.s2a_version() >= 100
    seen = set()
    for code in (0, -1, -2, -3, -4):
        s = lib.s2a_status_string(code)
        assert s and s not in seen
        seen.add(s)
    assert b"unknown" in lib.s2a_status_string(-99)


def test_workspace_bytes(lib):
    lib.s2a_bwd_workspace_bytes.restype = ctypes.c_size_t
    f = lib.s2a_bwd_workspace_bytes
    # D [B, H, N] in fp32, padded to 256 bytes, and 256 bytes of work counters
    assert f(1, 32768, 32, 32, 128, 8192) == 1 * 32 * 32768 * 4 + 256
    assert f(1, 1024, 4, 4, 64, 256) == 4 * 1024 * 4 + 256
    assert f(1, 1000, 4, 4, 64, 256) == 0      # N % G
    assert f(1, 1024, 6, 4, 64, 256) == 0      # H % Hkv
    assert f(0, 1024, 4, 4, 64, 256) == 0
    assert f(3, 256, 2, 1, 64, 256) % 256 == 0


def test_bad_arguments_are_rejected_without_a_device(lib):
    P = ctypes.c_void_p
    lib.s2a_fwd.argtypes = [P] * 5 + [ctypes.c_int] * 6 + [P]
    buf = (ctypes.c_char * 4096)()
    a = (ctypes.addressof(buf) + 255) & ~255  # aligned dummy address; never dereferenced on these paths
    # null pointer
    assert lib.s2a_fwd(None, a, a, a, a, 1, 1024, 4, 4, 64, 256, None) == -1
    # misaligned pointer
    assert lib.s2a_fwd(a + 2, a, a, a, a, 1, 1024, 4, 4, 64, 256, None) == -1
    # empty input
    assert lib.s2a_fwd(a, a, a, a, a, 0, 1024, 4, 4, 64, 256, None) == -1
    assert lib.s2a_fwd(a, a, a, a, a, 1, 0, 4, 4, 64, 256, None) == -1
    # ragged: N not a multiple of G; odd H; odd G; H % Hkv
    assert lib.s2a_fwd(a, a, a, a, a, 1, 1000, 4, 4, 64, 256, None) == -1
    assert lib.s2a_fwd(a, a, a, a, a, 1, 1024, 3, 3, 64, 256, None) == -1
    assert lib.s2a_fwd(a, a, a, a, a, 1, 1023, 4, 4, 64, 341, None) == -1
    assert lib.s2a_fwd(a, a, a, a, a, 1, 1024, 4, 3, 64, 256, None) == -1
    # unsupported: head dim, half a group not a multiple of 4 tokens, sequence shorter than one tile
    assert lib.s2a_fwd(a, a, a, a, a, 1, 1024, 4, 4, 96, 256, None) == -2
    assert lib.s2a_fwd(a, a, a, a, a, 1, 1200, 4, 4, 64, 100, None) == -2
    assert lib.s2a_fwd(a, a, a, a, a, 1, 1212, 4, 4, 64, 404, None) == -2
    assert lib.s2a_fwd(a, a, a, a, a, 1, 64, 4, 4, 64, 32, None) == -2
    # backward: workspace too small / missing
    lib.s2a_bwd.argtypes = [P] * 9 + [ctypes.c_int] * 6 + [P, ctypes.c_size_t, P]
    assert lib.s2a_bwd(a, a, a, a, a, a, a, a, a, 1, 1024, 4, 4, 64, 256, a, 16, None) == -1
    assert lib.s2a_bwd(a, a, a, a, a, a, a, a, a, 1, 1024, 4, 4, 64, 256, None, 1 << 20, None) == -1


def test_fast_workspace_bytes(lib):
    lib.s2a_bwd_workspace_bytes.restype = ctypes.c_size_t
    lib.s2a_bwd_workspace_bytes_fast.restype = ctypes.c_size_t
    lib.s2a_bwd_workspace_bytes_fast.argtypes = [ctypes.c_int] * 6 + [ctypes.c_size_t]
    f, g = lib.s2a_bwd_workspace_bytes, lib.s2a_bwd_workspace_bytes_fast
    mn = f(1, 32768, 32, 32, 128, 8192)
    blocks_per_unit = 64 * 65                      # T (T + 1) with T = 8192 / 128 tiles per group
    per_kv = 1 * 1 * 4 * blocks_per_unit * 16384   # B * (H / Hkv) * (N / G) units of 16 KiB blocks
    assert g(1, 32768, 32, 32, 128, 8192, 1 << 40) == mn + 32 * per_kv
    assert g(1, 32768, 32, 32, 128, 8192, mn + 3 * per_kv + 5) == mn + 3 * per_kv      # whole KV heads only
    assert g(1, 32768, 32, 32, 128, 8192, mn + per_kv - 1) == mn                       # not even one fits
    assert g(1, 32768, 32, 32, 128, 8192, 0) == mn
    assert g(1, 1000, 4, 4, 64, 256, 1 << 40) == 0                                     # invalid sizes
    # ragged groups (G / 2 not a multiple of 128): one more tile per run of the wrapped group
    T = (25000 + 127) // 128 + 1
    assert g(1, 100000, 32, 32, 128, 25000, 1 << 50) == f(1, 100000, 32, 32, 128, 25000) + 32 * 4 * T * (T + 1) * 16384
