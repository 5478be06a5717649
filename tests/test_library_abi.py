"""CPU-side checks of the boundary: the shared library loads without a GPU, exports every symbol
the header declares, and its host-only size queries and status strings behave."""
import ctypes
import os
import re

import pytest

from paper_2608_22788_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "tailsieve.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ts_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert set(names) == set(api.EXPORTED_SYMBOLS)
    for n in names:
        assert hasattr(lib, n), n


def test_struct_layout_matches_header():
    # 8 int32, 3 int64, 1 float (+ tail padding to 8)
    assert ctypes.sizeof(api.ts_attn_params) == 64
    assert api.ts_attn_params.kv_page_stride.offset == 32
    assert api.ts_attn_params.scale.offset == 56


def test_status_strings(lib):
    assert api.status_string(0) == "TS_OK"
    assert api.status_string(-1) == "TS_ERR_INVALID_ARG"
    assert api.status_string(-5) == "TS_ERR_TIMEOUT"
    assert api.status_string(123) == "TS_ERR_UNKNOWN"


def test_workspace_queries_need_no_gpu(lib):
    g = api.AttnGeometry(256, 1, 32, 8, 128, 64, 12000, 256, 8 * 64 * 128, 128, 64 * 128, 0.0884)
    a = api.attn_workspace_bytes(g)
    s = api.splitkv_workspace_bytes(g)
    assert 0 < s < a < 64 << 20
    g17 = api.AttnGeometry(**{**g.__dict__, "q_len": 17})
    assert api.attn_workspace_bytes(g17) > a
    assert api.attn_workspace_bytes(api.AttnGeometry(**{**g.__dict__, "head_dim": 96})) == 0
    assert api.attn_workspace_bytes(api.AttnGeometry(**{**g.__dict__, "num_q_heads": 30})) == 0
    assert api.attn_workspace_bytes(api.AttnGeometry(**{**g.__dict__, "q_len": 40})) == 0     # rows > 96
    assert api.accept_workspace_bytes(16, 16, 151936) >= 16 * 17 * 8
    assert api.accept_workspace_bytes(-1, 0, 10) == 0


def test_host_side_argument_checks_need_no_gpu(lib):
    g = api.AttnGeometry(4, 1, 8, 2, 64, 16, 64, 40, 2 * 16 * 64, 64, 16 * 64, 0.125)
    p = g.c_struct()
    # null pointers are rejected before any CUDA call
    rc = lib.ts_decode_attn(ctypes.byref(p), None, None, None, None, None, None, None, 0, None)
    assert rc == -1
    p2 = api.AttnGeometry(**{**g.__dict__, "q_len": 2}).c_struct()
    assert lib.ts_decode_attn(ctypes.byref(p2), None, None, None, None, None, None, None, 0, None) == -1
    assert lib.ts_accept_greedy(None, 8, None, 1, 0, 8, None, None, None, None, 0, None) == -1
    assert lib.ts_lse_merge(ctypes.byref(p), 4, None, None, None, None, None) == -1
