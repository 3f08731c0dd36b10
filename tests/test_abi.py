"""CPU-only checks of the boundary: the library loads, exports what include/spf.h declares, and
rejects bad arguments on the host before anything could be launched."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def spf():
    from paper_2603_02631_b200.build import build_library
    build_library()
    import paper_2603_02631_b200 as mod
    return mod


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "spf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"SPF_API[^;(]*?\b(spf_\w+)\s*\(", text)))


def test_header_declares_the_four_entry_points():
    syms = declared_symbols()
    for name in ("spf_score", "spf_chunk_pool", "spf_select_topk", "spf_compact_spans"):
        assert name in syms


def test_library_exports_every_declared_symbol(spf):
    dll = ctypes.CDLL(spf.LIB_PATH)
    for name in declared_symbols():
        assert hasattr(dll, name), f"{name} is declared in spf.h but not exported"


def test_keep_count_rule(spf):
    assert spf.spf_keep_count(64, 0.25) == 16
    assert spf.spf_keep_count(1024, 0.10) == 103
    assert spf.spf_keep_count(4096, 0.10) == 410
    assert spf.spf_keep_count(1024, 0.05) == 52
    assert spf.spf_keep_count(10, 0.3) == 3
    assert spf.spf_keep_count(7, 1e-6) == 1
    assert spf.spf_keep_count(7, 2.0) == 7
    assert spf.spf_keep_count(0, 0.5) == 0


def test_keep_count_agrees_with_oracle(spf):
    import oracle
    for c in (1, 2, 7, 10, 100, 1024, 4096, 8191):
        for rho in (0.03, 0.06, 0.1, 0.125, 0.15, 0.2, 0.25, 0.3, 0.45, 0.5, 1.0):
            assert spf.spf_keep_count(c, rho) == oracle.keep_count(c, rho)


def test_status_strings(spf):
    assert spf.spf_status_string(0) == "ok"
    for code in (-1, -2, -3, -4, -5):
        assert spf.spf_status_string(code) not in ("", "ok", "unknown status")
    assert spf.spf_status_string(-99) == "unknown status"
    assert re.match(r"\d+\.\d+\.\d+", spf.spf_version())


def test_host_validation_rejects_before_launch(spf):
    lib = spf.lib
    # null pointers / bad sizes: every call returns INVALID_ARG without touching a device
    assert lib.spf_chunk_pool(None, 10, 13, 32, None, None) == -1
    assert "null" in spf.spf_last_error()
    assert lib.spf_chunk_pool(1 << 20, 10, 12, 32, 1 << 20, None) == -1      # even kernel
    assert lib.spf_chunk_pool(1 << 20, 0, 13, 32, 1 << 20, None) == -1       # empty prompt
    assert lib.spf_select_topk(1 << 20, 10, 11, 1 << 20, None) == -1         # k > C
    assert lib.spf_select_topk(1 << 20, 10, 0, 1 << 20, None) == -1
    assert lib.spf_compact_spans(None, 1, 32, 10, None, None, None, None, None, None, None, None, None) == -1
    assert lib.spf_score(None, None, 0, None, 0, None, None) == -1


def test_score_shape_validation(spf):
    from paper_2603_02631_b200.binding import _Prompt, _Shape
    lib = spf.lib
    layers = (ctypes.c_void_p * 2)(4096, 8192)
    lp = ctypes.cast(layers, ctypes.POINTER(ctypes.c_void_p))

    def call(shape, prompt, ws=4096, ws_bytes=1 << 30):
        arr = (_Prompt * 1)(prompt)
        return lib.spf_score(ctypes.byref(shape), arr, 1, ws, ws_bytes, None, None)

    good = _Prompt(1000, lp, 64000, 64, 4096, 4096, None)
    assert call(_Shape(2, 4, 2, 96, 8, 0.0), good) == -2                      # head_dim
    assert call(_Shape(2, 5, 2, 64, 8, 0.0), good) == -2                      # Hq % Hkv
    assert call(_Shape(2, 32, 2, 64, 8, 0.0), good) == -2                     # G * m_pad > 64
    assert call(_Shape(2, 4, 2, 64, 40, 0.0), good) == -2                     # m > 32
    assert call(_Shape(0, 4, 2, 64, 8, 0.0), good) == -1
    assert call(_Shape(2, 4, 2, 64, 8, 0.0), _Prompt(0, lp, 64000, 64, 4096, 4096, None)) == -1
    assert call(_Shape(2, 4, 2, 64, 8, 0.0), _Prompt(1000, lp, 64000, 60, 4096, 4096, None)) == -1   # stride
    bad_layers = (ctypes.c_void_p * 2)(4096, 8200)                            # not 16-byte aligned
    blp = ctypes.cast(bad_layers, ctypes.POINTER(ctypes.c_void_p))
    assert call(_Shape(2, 4, 2, 64, 8, 0.0), _Prompt(1000, blp, 64000, 64, 4096, 4096, None)) == -1
    assert call(_Shape(2, 4, 2, 64, 8, 0.0), good, ws=None) == -3             # no workspace
    assert call(_Shape(2, 4, 2, 64, 8, 0.0), good, ws=4096, ws_bytes=16) == -3
    assert "needed" in spf.spf_last_error()
    # the size query accepts the good prompt and refuses the bad shape
    arr = (_Prompt * 1)(good)
    assert lib.spf_score_workspace_bytes(ctypes.byref(_Shape(2, 4, 2, 64, 8, 0.0)), arr, 1) > 0
    assert lib.spf_score_workspace_bytes(ctypes.byref(_Shape(2, 4, 2, 96, 8, 0.0)), arr, 1) == 0


def test_compress_host_validates_before_touching_the_device(spf):
    """Host-side checks of spf_compress_host: arena size query, null pointers, small arena (nothing is launched)."""
    from paper_2603_02631_b200.binding import _SelectParams, _Shape
    shape = _Shape(2, 4, 2, 64, 8, 0.0)
    prm = _SelectParams(32, 13, 0.25)
    need = spf.lib.spf_compress_host_arena_bytes(ctypes.byref(shape), 1000, ctypes.byref(prm))
    # the arena holds at least the device copy of the key cache, queries, ids and offsets
    assert need >= 2 * 2 * 1000 * 64 * 2 + 2 * 4 * 8 * 64 * 2 + 3 * 4 * 1000
    assert spf.lib.spf_compress_host_arena_bytes(None, 1000, ctypes.byref(prm)) == 0
    assert spf.lib.spf_compress_host_arena_bytes(ctypes.byref(shape), 0, ctypes.byref(prm)) == 0
    bad = _Shape(2, 4, 2, 96, 8, 0.0)                       # head_dim 96 is outside the kernels
    assert spf.lib.spf_compress_host_arena_bytes(ctypes.byref(bad), 1000, ctypes.byref(prm)) == 0
    none = ctypes.c_void_p(None)
    rc = spf.lib.spf_compress_host(ctypes.byref(shape), 1000, None, none, none, none, none, ctypes.byref(prm), none, 0,
                                   none, none, none, none, none, none)
    assert rc == -1
