"""ctypes loader for the fp64 CPU oracle of HGA (hga_oracle.c) -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library never does.  `build()` compiles the C source with gcc.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hga_oracle.c")
_LIB = os.path.join(_HERE, "libhga_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (gcc -O2 -fopenmp) if the shared object is missing or stale."""
    hdr = os.path.join(_HERE, "hga_oracle.h")
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(hdr)))
    if force or stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class RefParams(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "batch", "n_q_heads", "n_kv_heads", "head_dim", "total_len", "seg_len", "chunk",
        "group", "q_block", "topk_chunks", "topk_groups", "sink", "local")] + [
        ("softmax_scale", C.c_double), ("global_group_budget", C.c_int32), ("score_agg", C.c_int32), ("decode", C.c_int32)]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.hga_ref_f64_to_bf16.restype = C.c_uint16
        _lib.hga_ref_f64_to_bf16.argtypes = [C.c_double]
        _lib.hga_ref_bf16_to_f64.restype = C.c_double
        _lib.hga_ref_bf16_to_f64.argtypes = [C.c_uint16]
    return _lib


SCORE_AGG = {"max": 0, "mean": 1, "lse": 2}


def params(cfg, softmax_scale: float = 0.0, global_group_budget: bool = False, score_agg: str = "max") -> RefParams:
    """Build the oracle's parameter block from any object with the HGA shape fields."""
    return RefParams(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.total_len,
                     cfg.seg_len, cfg.chunk, cfg.group, cfg.q_block, cfg.topk_chunks,
                     cfg.topk_groups, cfg.sink, cfg.local, softmax_scale, int(global_group_budget),
                     SCORE_AGG[score_agg], int(bool(getattr(cfg, "decode", False))))


def _p(a, dtype):
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags.c_contiguous, (
        "oracle arrays must be C-contiguous %s" % dtype)
    return a.ctypes.data_as(C.c_void_p)


def _items(items):
    if items is None:
        return None, None, 0
    arr = np.ascontiguousarray(items, dtype=np.int32)
    return arr, arr.ctypes.data_as(C.c_void_p), int(arr.size)


def _ok(rc, what):
    if rc != 0:
        raise RuntimeError("oracle %s failed with code %d" % (what, rc))


def kg_eff(cfg) -> int:
    return min(cfg.topk_groups, cfg.chunk // cfg.group)


def f64_to_bf16(x: float) -> int:
    return int(lib().hga_ref_f64_to_bf16(float(x)))


def window(cfg, qb: int):
    ls, se = C.c_int32(), C.c_int32()
    _ok(lib().hga_ref_window(C.byref(params(cfg)), C.c_int32(qb), C.byref(ls), C.byref(se)), "window")
    return ls.value, se.value


def routed_tokens(cfg, qb: int, group_ids) -> np.ndarray:
    gi = np.ascontiguousarray(group_ids, dtype=np.int32)
    out = np.empty(cfg.sink + gi.size * cfg.group + cfg.local + cfg.q_block + cfg.chunk, np.int32)
    n = lib().hga_ref_routed_tokens(C.byref(params(cfg)), C.c_int32(qb), _p(gi, np.int32),
                                    C.c_int32(gi.size), _p(out, np.int32))
    if n < 0:
        raise RuntimeError("oracle routed_tokens failed with code %d" % n)
    return out[:n].copy()


def build_summaries(cfg, K, tok_begin=None, tok_end=None, chunk_sum=None, group_sum=None):
    B, Hkv, L, d = cfg.batch, cfg.n_kv_heads, cfg.total_len, cfg.head_dim
    if chunk_sum is None:
        chunk_sum = np.zeros((B, Hkv, L // cfg.chunk, d), np.uint16)
    if group_sum is None:
        group_sum = np.zeros((B, Hkv, L // cfg.group, d), np.uint16)
    tb = 0 if tok_begin is None else tok_begin
    te = (L // cfg.chunk) * cfg.chunk if tok_end is None else tok_end
    _ok(lib().hga_ref_build_summaries(C.byref(params(cfg)), _p(K, np.uint16), C.c_int32(tb),
                                      C.c_int32(te), _p(chunk_sum, np.uint16),
                                      _p(group_sum, np.uint16)), "build_summaries")
    return chunk_sum, group_sum


def route(cfg, Q, chunk_sum, group_sum, items=None, want_scores=False, global_group_budget=False,
          score_agg="max"):
    B, Hkv, nqb = cfg.batch, cfg.n_kv_heads, cfg.seg_len // cfg.q_block
    kc, kge, per = cfg.topk_chunks, kg_eff(cfg), cfg.chunk // cfg.group
    chunk_idx = np.full((B, Hkv, nqb, kc), -1, np.int32)
    group_idx = np.full((B, Hkv, nqb, kc * kge), -1, np.int32)
    n_groups = np.zeros((B, Hkv, nqb), np.int32)
    cs = gs = None
    if want_scores:
        cs = np.full((B, Hkv, nqb, cfg.total_len // cfg.chunk), -np.inf, np.float64)
        gs = np.full((B, Hkv, nqb, kc * per), -np.inf, np.float64)
    keep, ip, n = _items(items)
    _ok(lib().hga_ref_route(C.byref(params(cfg, 0.0, global_group_budget, score_agg)), _p(Q, np.uint16), _p(chunk_sum, np.uint16),
                            _p(group_sum, np.uint16), _p(chunk_idx, np.int32),
                            _p(group_idx, np.int32), _p(n_groups, np.int32), _p(cs, np.float64),
                            _p(gs, np.float64), ip, C.c_int32(n)), "route")
    out = {"chunk_idx": chunk_idx, "group_idx": group_idx, "n_groups": n_groups}
    if want_scores:
        out["chunk_scores"], out["group_scores"] = cs, gs
    return out


def attn_fwd(cfg, Q, K, V, group_idx, n_groups, items=None, softmax_scale=0.0):
    B, Hq, S, d = cfg.batch, cfg.n_q_heads, cfg.seg_len, cfg.head_dim
    O = np.zeros((B, Hq, S, d), np.float64)
    LSE = np.zeros((B, Hq, S), np.float64)
    keep, ip, n = _items(items)
    _ok(lib().hga_ref_attn_fwd(C.byref(params(cfg, softmax_scale)), _p(Q, np.uint16),
                               _p(K, np.uint16), _p(V, np.uint16), _p(group_idx, np.int32),
                               _p(n_groups, np.int32), _p(O, np.float64), _p(LSE, np.float64),
                               ip, C.c_int32(n)), "attn_fwd")
    return O, LSE


def attn_bwd(cfg, Q, K, V, dO, group_idx, n_groups, items=None, softmax_scale=0.0):
    B, Hq, Hkv, S, d = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seg_len, cfg.head_dim
    dQ = np.zeros((B, Hq, S, d), np.float64)
    dK = np.zeros((B, Hkv, S, d), np.float64)
    dV = np.zeros((B, Hkv, S, d), np.float64)
    keep, ip, n = _items(items)
    _ok(lib().hga_ref_attn_bwd(C.byref(params(cfg, softmax_scale)), _p(Q, np.uint16),
                               _p(K, np.uint16), _p(V, np.uint16), _p(dO, np.uint16),
                               _p(group_idx, np.int32), _p(n_groups, np.int32),
                               _p(dQ, np.float64), _p(dK, np.float64), _p(dV, np.float64),
                               ip, C.c_int32(n)), "attn_bwd")
    return dQ, dK, dV


def attn_fwd_f64(cfg, Q, K, V, group_idx, n_groups, items=None, softmax_scale=0.0):
    """attn_fwd on real-valued (float64) Q, K, V: the same code, for finite differences."""
    B, Hq, S, d = cfg.batch, cfg.n_q_heads, cfg.seg_len, cfg.head_dim
    O = np.zeros((B, Hq, S, d), np.float64)
    LSE = np.zeros((B, Hq, S), np.float64)
    keep, ip, n = _items(items)
    _ok(lib().hga_ref_attn_fwd_f64(C.byref(params(cfg, softmax_scale)), _p(Q, np.float64),
                                   _p(K, np.float64), _p(V, np.float64), _p(group_idx, np.int32),
                                   _p(n_groups, np.int32), _p(O, np.float64),
                                   _p(LSE, np.float64), ip, C.c_int32(n)), "attn_fwd_f64")
    return O, LSE


def attn_bwd_f64(cfg, Q, K, V, dO, group_idx, n_groups, items=None, softmax_scale=0.0):
    B, Hq, Hkv, S, d = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seg_len, cfg.head_dim
    dQ = np.zeros((B, Hq, S, d), np.float64)
    dK = np.zeros((B, Hkv, S, d), np.float64)
    dV = np.zeros((B, Hkv, S, d), np.float64)
    keep, ip, n = _items(items)
    _ok(lib().hga_ref_attn_bwd_f64(C.byref(params(cfg, softmax_scale)), _p(Q, np.float64),
                                   _p(K, np.float64), _p(V, np.float64), _p(dO, np.float64),
                                   _p(group_idx, np.int32), _p(n_groups, np.int32),
                                   _p(dQ, np.float64), _p(dK, np.float64), _p(dV, np.float64),
                                   ip, C.c_int32(n)), "attn_bwd_f64")
    return dQ, dK, dV


def num_threads() -> int:
    return int(lib().hga_ref_num_threads())
