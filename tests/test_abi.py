"""The C-ABI library loads, exports every symbol include/hga.h declares, and rejects bad
arguments on the host before anything is launched.  No GPU needed."""
import ctypes as C
import os
import re

import pytest

from paper_2607_15105_b200 import binding, build
from paper_2607_15105_b200.workloads import CONFIGS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "hga.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hga_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_functions()
    assert set(names) == set(binding.EXPORTS), names
    for n in names:
        assert getattr(lib, n) is not None
    assert lib.hga_version() == 100


def test_params_struct_layout_matches_header():
    # 13 int32 + float + int32 = 60 bytes, padded to 64 for the int64 stride arrays (4 x 3 x 8)
    assert C.sizeof(binding.HgaParams) == 64 + 96
    assert binding.HgaParams.q_stride.offset == 64


def test_status_strings(lib):
    for code in range(0, -7, -1):
        assert lib.hga_status_string(code).decode() not in ("", "unknown status")
    assert lib.hga_status_string(-99).decode() == "unknown status"


def test_bad_arguments_are_rejected_on_the_host(lib):
    cfg = CONFIGS[1]
    p = binding.make_params(cfg)
    buf = (C.c_char * 4096)()
    a = C.addressof(buf)
    a += (-a) % 16
    ptr = C.c_void_p(a)
    # NULL pointers
    assert lib.hga_build_summaries(C.byref(p), None, 0, 64, ptr, ptr, None) == -1
    assert lib.hga_attn_fwd(C.byref(p), ptr, ptr, None, ptr, ptr, ptr, ptr, None, None) == -1
    assert lib.hga_workspace_bytes(None, None, None) == -1
    # misaligned pointer
    assert lib.hga_build_summaries(C.byref(p), C.c_void_p(a + 2), 0, 64, ptr, ptr, None) == -3
    # token range not chunk aligned / out of range
    assert lib.hga_build_summaries(C.byref(p), ptr, 0, 65, ptr, ptr, None) == -2
    assert lib.hga_build_summaries(C.byref(p), ptr, 0, cfg.total_len + 64, ptr, ptr, None) == -2
    # missing / short workspace
    assert lib.hga_route(C.byref(p), ptr, ptr, ptr, ptr, ptr, ptr, None, None, None, 0, None) == -5
    assert lib.hga_route(C.byref(p), ptr, ptr, ptr, ptr, ptr, ptr, None, None, ptr, 8, None) == -5
    assert lib.hga_attn_bwd(C.byref(p), *([ptr] * 11), ptr, 8, None, None) == -5


@pytest.mark.parametrize("field,value,code", [
    ("n_q_heads", 3, -2), ("head_dim", 96, -4), ("seg_len", 0, -2), ("group", 7, -2),
    ("q_block", 96, -2), ("seg_len", 200, -2), ("total_len", 1000, -2), ("topk_chunks", -1, -2),
    ("topk_groups", 0, -2), ("sink", 32, -2), ("local", 100, -2)])
def test_shape_rules(lib, field, value, code):
    p = binding.make_params(CONFIGS[3].scaled(n_q_heads=4, n_kv_heads=2))
    setattr(p, field, value)
    assert lib.hga_workspace_bytes(C.byref(p), None, None) == code


def test_stride_rules(lib):
    cfg = CONFIGS[1]
    p = binding.make_params(cfg, k_stride=(cfg.total_len * 64 * 2, cfg.total_len * 64, 60))
    assert lib.hga_workspace_bytes(C.byref(p), None, None) == -3     # not a multiple of 8
    p = binding.make_params(cfg, k_stride=(cfg.total_len * 64 * 2, cfg.total_len * 64, 32))
    assert lib.hga_workspace_bytes(C.byref(p), None, None) == -2     # rows would overlap


def test_workspace_sizes(lib):
    for n, cfg in CONFIGS.items():
        r, b = binding.hga_workspace_bytes(binding.make_params(cfg))
        assert r >= cfg.n_items * (cfg.total_len // cfg.chunk) * 4
        assert b >= cfg.batch * cfg.n_q_heads * cfg.seg_len * 4
        assert binding.hga_step_arena_bytes(binding.make_params(cfg)) > r + b
