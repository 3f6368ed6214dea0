"""The C-ABI library loads and exports what include/moe.h declares; host-side checks (no GPU)."""
import ctypes
import os
import re

import pytest

from paper_1701_06538_b200 import binding as B
from paper_1701_06538_b200 import build as moe_build
from paper_1701_06538_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    moe_build.build()
    return B.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "moe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moe_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 17
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(B.EXPORTS) == names


def test_struct_layouts_match_header():
    assert ctypes.sizeof(B.moe_config) == 52
    assert ctypes.sizeof(B.moe_sizes) == 14 * 8
    assert ctypes.sizeof(B.moe_ctx_layout) == 17 * 8


def test_validate_accepts_the_five_workloads_and_rejects_bad_ones(lib):
    for w in synth.CONFIGS.values():
        cfg = B.make_config(w.T, w.d, w.h, w.n, w.k, w.act, w.w_importance, w.w_load, w.a, w.k1, w.b, w.k2)
        assert B.moe_validate(cfg) == 0, w.name
        S = B.moe_query_sizes(cfg)
        assert S.R == w.T * w.k and S.ctx_bytes > 0 and S.ws_bwd_bytes >= S.ws_bytes > 0
        assert B.moe_workspace_bytes(cfg) == (S.ws_fwd_bytes, S.ws_bwd_bytes)
    ok = dict(T=16, d=64, h=64, n=8, k=2, act="f32")
    bad = [dict(ok, k=0), dict(ok, k=9), dict(ok, k=3, n=2), dict(ok, d=3), dict(ok, h=0), dict(ok, T=-1),
           dict(ok, act=7), dict(ok, n=1 << 20), dict(ok, a=2, b=3, k1=1, k2=1), dict(ok, a=2, b=4, k1=2, k2=2),
           dict(ok, d=4, act="bf16"), dict(ok, w_load=-1.0), dict(ok, flags=16),
           dict(ok, flags=B.MOE_FLAG_GATE_SCREEN_ON | B.MOE_FLAG_GATE_SCREEN_OFF)]
    for kw in bad:
        assert B.moe_validate(B.make_config(**kw)) == 1, kw
    assert B.moe_validate(B.make_config(**dict(ok, a=2, b=4, k1=1, k2=2))) == 0
    # a hierarchical layer with more experts than the routing kernels hold in shared memory: refused up front
    assert B.moe_validate(B.make_config(**dict(ok, T=64, n=128 * 128, k=4, a=128, b=128, k1=2, k2=2))) == 2
    assert lib.moe_validate(None) == 1
    assert lib.moe_status_string(5) == b"device-side wait timed out"


def test_null_pointers_are_reported_not_faulted(lib):
    cfg = B.make_config(T=16, d=64, h=64, n=8, k=2, act="f32")
    null = ctypes.c_void_p(0)
    assert lib.moe_combine(ctypes.byref(cfg), null, null, null, null, null) == 1
    assert lib.moe_gate(ctypes.byref(cfg), *([null] * 12)) == 1
    assert lib.moe_forward(ctypes.byref(cfg), *([null] * 16)) == 1
    assert lib.moe_query_sizes(ctypes.byref(cfg), None) == 1


def test_hierarchical_sizes(lib):
    w = synth.CONFIGS["c4"]
    cfg = B.make_config(w.T, w.d, w.h, w.n, w.k, w.act, 0.1, 0.1, w.a, w.k1, w.b, w.k2)
    S = B.moe_query_sizes(cfg)
    assert S.gate_cols == 64 + 2 * 64 and S.logits_elems == w.T * 192
    assert S.gates_elems == w.T * (4 + 2 + 4) and S.kth_elems == 2 * w.T * 3
    assert S.wg_elems == 512 * 64 + 64 * 512 * 64 and S.load_elems == 2 * 4096 + 128 and S.dload_elems == 64 + 4096


def test_buffer_size_check(lib):
    w = synth.CONFIGS["c2"]
    cfg = B.make_config(w.T, w.d, w.h, w.n, w.k, w.act)
    S = B.moe_query_sizes(cfg)
    for which, need in enumerate((S.ws_bytes, S.ws_fwd_bytes, S.ws_bwd_bytes, S.ctx_bytes, S.ws_adam_bytes)):
        assert B.moe_check_buffer_sizes(cfg, which, need) == 0
        assert B.moe_check_buffer_sizes(cfg, which, need - 1) == 3      # MOE_ERR_WORKSPACE
    assert B.moe_check_buffer_sizes(cfg, 9, 1 << 40) == 1
