"""The shared library loads without a GPU and exports every entry point the header declares; argument checks
that return before any CUDA work behave as documented."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def war():
    from paper_2607_17299_b200.build import build
    build()
    from paper_2607_17299_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(war):
    with open(os.path.join(ROOT, "include", "war.h")) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(war_[a-z_]+)\s*\(", text))
    assert {"war_index_build", "war_index_append", "war_draft", "war_verify_attn", "war_accept"} <= declared
    lib = C.CDLL(war.LIB_PATH)
    for name in sorted(declared):
        assert getattr(lib, name) is not None, name
    assert declared == set(war.EXPORTS)                           # the binding wraps exactly what is declared


def test_status_strings(war):
    assert war.status_string(0) == "ok"
    assert "argument" in war.status_string(1)
    assert war.status_string(99) == "unknown status"


def test_workspace_size_and_shape_limits(war):
    p = war.AttnParams()
    p.B, p.N, p.Hq, p.Hkv, p.D, p.page_size, p.max_pages_per_req, p.kernel = 8, 16, 32, 8, 128, 16, 300, 0
    p.num_pages, p.scale = 4000, 0.088
    for i, s in enumerate((8 * 16 * 128, 16 * 128, 128, 1)):
        p.k_strides[i] = s
        p.v_strides[i] = s
    n = war.war_verify_attn_workspace_bytes(p)
    assert n > 0 and n % 256 == 0
    p.D = 64
    assert war.war_verify_attn_workspace_bytes(p) == 0            # unsupported head size
    p.D = 128
    p.k_strides[1] = 128                                          # token-major pool: not built
    assert war.war_verify_attn_workspace_bytes(p) == 0


def test_argument_errors_return_before_any_launch(war):
    lib = C.CDLL(war.LIB_PATH)
    lib.war_accept.restype = C.c_int
    lib.war_accept.argtypes = [C.c_void_p] * 4 + [C.c_int32] * 3 + [C.c_void_p] * 4
    assert lib.war_accept(None, None, None, None, 4, 65, 0, None, None, None, None) == 1     # N > 64
    assert lib.war_accept(None, None, None, None, 4, 8, 2, None, None, None, None) == 1      # bad mode
    assert lib.war_accept(None, None, None, None, 0, 8, 0, None, None, None, None) == 0      # empty batch
    lib.war_index_build.restype = C.c_int
    lib.war_index_build.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_void_p,
                                    C.POINTER(C.c_void_p)]
    out = C.c_void_p(None)
    assert lib.war_index_build(None, None, 0, 100, 200, 10, None, C.byref(out)) == 1        # max_depth > 128
    assert lib.war_index_build(None, None, 0, 100, 64, 1 << 31, None, C.byref(out)) == 3    # beyond int32 positions
    p = war.DraftParams(1, 40, 8, 4, 1)
    lib.war_draft.restype = C.c_int
    assert lib.war_draft(None, None, None, C.byref(p), None, None, None, None, None, None) == 1
