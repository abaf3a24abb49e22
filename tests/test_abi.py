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


def _ws(lib, p):
    r, b = C.c_size_t(), C.c_size_t()
    rc = lib.hga_workspace_bytes(C.byref(p), C.byref(r), C.byref(b))
    return rc, r.value, b.value


def test_flag_rules_on_the_host(lib):
    """Variant flags are validated before anything touches the device."""
    from dataclasses import replace
    cfg = CONFIGS[1]
    ok = lambda flags, c=cfg: _ws(lib, binding.make_params(c, flags=flags))[0]
    assert ok(0) == 0
    assert ok(binding.HGA_FLAG_SCORE_MEAN) == 0 and ok(binding.HGA_FLAG_SCORE_LSE) == 0
    assert ok(binding.HGA_FLAG_SCORE_MEAN | binding.HGA_FLAG_SCORE_LSE) == -4      # at most one aggregator
    assert ok(1 << 9) == -4                                                          # unknown flag bit
    for bit in range(7, 32):                                                         # every bit hga.h does not define
        assert ok(1 << bit if bit < 31 else -(1 << 31)) == -4, bit
    # generation shapes need their flag: q_block below the chunk, unaligned history and length
    dec = replace(cfg, total_len=1003, seg_len=3, q_block=3)
    assert ok(0, dec) == -2
    assert ok(binding.HGA_FLAG_DECODE, dec) == 0
    # the global group budget keeps one bit per (opened chunk, group) slot: at most 4096
    big = replace(cfg, chunk=64, group=1, topk_chunks=65, total_len=8192, seg_len=512)
    assert ok(0, big) == 0 and ok(binding.HGA_FLAG_GLOBAL_GROUP_BUDGET, big) == -4


def test_workspace_sizes_follow_their_formulas(lib):
    cfg = CONFIGS[3]
    items = cfg.batch * cfg.n_kv_heads * cfg.n_q_blocks
    rc, r, b = _ws(lib, binding.make_params(cfg))
    assert rc == 0
    assert r == items * (cfg.total_len // cfg.chunk) * 4 + 16
    delta = cfg.batch * cfg.n_q_heads * cfg.seg_len * 4
    assert b == ((delta + 255) & ~255) + 16
    # global group budget: the opened chunks' group scores behind the chunk scores
    rc, r2, _ = _ws(lib, binding.make_params(cfg, flags=binding.HGA_FLAG_GLOBAL_GROUP_BUDGET))
    assert rc == 0 and r2 == r + items * cfg.topk_chunks * (cfg.chunk // cfg.group) * 4
    # bf16 gradient outputs: the fp32 dK and dV sums live in the workspace
    rc, _, b2 = _ws(lib, binding.make_params(cfg, flags=binding.HGA_FLAG_BWD_BF16_GRADS))
    assert rc == 0 and b2 == b + 2 * cfg.batch * cfg.n_kv_heads * cfg.seg_len * cfg.head_dim * 4


def test_varlen_prefix_sums_are_validated_on_the_host(lib):
    cfg = CONFIGS[1]
    p = binding.make_params(cfg)
    assert binding.hga_varlen_workspace_bytes(p, [0, 256, 512], [0, 1024, 1536]) > 0
    for cu_q, cu_k in (([0, 256], [0, 1000]),            # length not a multiple of the chunk
                       ([0, 256, 768], [0, 1024, 1280]),  # more queries than keys in the second sequence
                       ([64, 320], [0, 1024]),            # does not start at zero
                       ([0, 100], [0, 1024])):            # segment not a multiple of the query block
        with pytest.raises(binding.HgaError):
            binding.hga_varlen_workspace_bytes(p, cu_q, cu_k)
