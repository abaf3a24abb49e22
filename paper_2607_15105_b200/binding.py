"""Thin ctypes binding of libhga.so: the same names as the C ABI, argument marshalling only.

Every step of the path runs in the library's CUDA kernels; torch is used for device memory
and streams.  Loading fails loudly when the shared object has not been built -- there is no
CPU fallback.  Tensors: bf16 data are `torch.bfloat16` CUDA tensors, index outputs int32.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhga.so")

HGA_FLAG_BWD_ACCUMULATE = 1
HGA_FLAG_GENERIC_KERNELS = 2
HGA_FLAG_GLOBAL_GROUP_BUDGET = 4
HGA_FLAG_SCORE_MEAN = 8
HGA_FLAG_SCORE_LSE = 16
HGA_FLAG_DECODE = 32
HGA_FLAG_BWD_BF16_GRADS = 64
HGA_STATUS_BAD_INDEX = 1
HGA_STATUS_WAIT_TIMEOUT = 2

HGA_ROUTE_STATIC_SCRATCH_BYTES = 4 << 20

EXPORTS = ("hga_build_summaries", "hga_route", "hga_route_static", "hga_attn_fwd", "hga_attn_bwd",
           "hga_workspace_bytes", "hga_step_host", "hga_step_arena_bytes", "hga_tbptt_walk", "hga_varlen_step",
           "hga_varlen_workspace_bytes", "hga_status_string",
           "hga_version", "hga_last_cuda_error", "hga_kernel_launch_count", "hga_kernel_launch_count_by_family",
           "hga_selftest_bounded_wait")

# kernel families of hga_kernel_launch_count_by_family
(HGA_KERNELS_SUMMARIES, HGA_KERNELS_ROUTE_TENSOR, HGA_KERNELS_ROUTE_GENERIC, HGA_KERNELS_FWD_TENSOR,
 HGA_KERNELS_FWD_GENERIC, HGA_KERNELS_BWD_TENSOR, HGA_KERNELS_BWD_GENERIC, HGA_KERNELS_AUX) = range(8)
HGA_KERNELS_FAMILIES = 8


class HgaParams(C.Structure):
    _fields_ = ([(n, C.c_int32) for n in (
        "batch", "n_q_heads", "n_kv_heads", "head_dim", "total_len", "seg_len", "chunk", "group",
        "q_block", "topk_chunks", "topk_groups", "sink", "local")]
        + [("softmax_scale", C.c_float), ("flags", C.c_int32), ("summary_len", C.c_int32)]
        + [(n, C.c_int64 * 3) for n in ("q_stride", "k_stride", "v_stride", "o_stride")])


class HgaError(RuntimeError):
    def __init__(self, call, status):
        self.status = status
        msg = lib().hga_status_string(status).decode()
        extra = ""
        if status == -6:
            extra = " (cudaError %d)" % lib().hga_last_cuda_error()
        super().__init__("%s failed: %s [%d]%s" % (call, msg, status, extra))


_lib = None


def lib():
    """Load libhga.so (once).  Raises if it is missing: build it with `python -m
    paper_2607_15105_b200.build` or `__graft_entry__.build()`."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libhga.so is not built (%s missing); there is no fallback path" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        L.hga_status_string.restype = C.c_char_p
        L.hga_status_string.argtypes = [C.c_int]
        L.hga_kernel_launch_count.restype = C.c_int64
        L.hga_kernel_launch_count_by_family.restype = C.c_int64
        L.hga_kernel_launch_count_by_family.argtypes = [C.c_int]
        L.hga_selftest_bounded_wait.argtypes = [C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p]
        vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
        pp = C.POINTER(HgaParams)
        L.hga_build_summaries.argtypes = [pp, vp, i32, i32, vp, vp, vp]
        L.hga_route.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.hga_route_static.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp]
        L.hga_attn_fwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.hga_attn_bwd.argtypes = [pp] + [vp] * 12 + [sz, vp, vp]
        L.hga_workspace_bytes.argtypes = [pp, C.POINTER(sz), C.POINTER(sz)]
        L.hga_step_arena_bytes.argtypes = [pp, C.POINTER(sz)]
        L.hga_step_host.argtypes = [pp] + [vp] * 13 + [sz, vp, vp]
        L.hga_tbptt_walk.argtypes = [pp] + [vp] * 15 + [sz, vp, vp]
        L.hga_varlen_step.argtypes = [pp, C.c_int32] + [vp] * 17 + [sz, vp, vp]
        L.hga_varlen_workspace_bytes.argtypes = [pp, C.c_int32, vp, vp, C.POINTER(sz)]
        _lib = L
    return _lib


def make_params(cfg, softmax_scale: float = 0.0, flags: int = 0, q_stride=None, k_stride=None,
                v_stride=None, o_stride=None, summary_len: int = 0) -> HgaParams:
    """hga_params from any object with the HGA shape fields (e.g. workloads.HgaConfig)."""
    if getattr(cfg, "decode", False):
        flags |= HGA_FLAG_DECODE
    p = HgaParams(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.total_len,
                  cfg.seg_len, cfg.chunk, cfg.group, cfg.q_block, cfg.topk_chunks,
                  cfg.topk_groups, cfg.sink, cfg.local, softmax_scale, flags, summary_len)
    for name, s in (("q_stride", q_stride), ("k_stride", k_stride), ("v_stride", v_stride),
                    ("o_stride", o_stride)):
        if s is not None:
            setattr(p, name, (C.c_int64 * 3)(*s))
    return p


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return C.c_void_p(t)
    return C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _check(call, rc):
    if rc != 0:
        raise HgaError(call, rc)


def _strides(t):
    """element strides (batch, head, token) of a 4-D tensor whose last axis is contiguous"""
    assert t.dim() == 4 and t.stride(3) == 1
    return (t.stride(0), t.stride(1), t.stride(2))


def params_for(cfg, Q=None, K=None, V=None, O=None, softmax_scale=0.0, flags=0) -> HgaParams:
    """make_params with the strides read off the given tensors (dense ones give zeros)."""
    def st(t):
        return None if t is None or t.is_contiguous() else _strides(t)
    return make_params(cfg, softmax_scale, flags, st(Q), st(K), st(V), st(O))


def hga_version() -> int:
    return lib().hga_version()


def hga_kernel_launch_count() -> int:
    return int(lib().hga_kernel_launch_count())


def hga_kernel_launch_counts() -> list:
    """Launch counts per kernel family (index = HGA_KERNELS_*)."""
    return [int(lib().hga_kernel_launch_count_by_family(f)) for f in range(HGA_KERNELS_FAMILIES)]


def hga_selftest_bounded_wait(cycle_limit, status_word, waited_cycles=None, stream=None):
    """Runs the library's bounded on-chip wait on a barrier nothing completes (see hga.h)."""
    _check("hga_selftest_bounded_wait", lib().hga_selftest_bounded_wait(
        int(cycle_limit), _ptr(status_word), _ptr(waited_cycles), _stream(stream)))


def hga_workspace_bytes(p: HgaParams):
    r, b = C.c_size_t(), C.c_size_t()
    _check("hga_workspace_bytes", lib().hga_workspace_bytes(C.byref(p), C.byref(r), C.byref(b)))
    return r.value, b.value


def hga_step_arena_bytes(p: HgaParams) -> int:
    n = C.c_size_t()
    _check("hga_step_arena_bytes", lib().hga_step_arena_bytes(C.byref(p), C.byref(n)))
    return n.value


def hga_build_summaries(p, K, tok_begin, tok_end, chunk_sum, group_sum, stream=None):
    _check("hga_build_summaries", lib().hga_build_summaries(
        C.byref(p), _ptr(K), tok_begin, tok_end, _ptr(chunk_sum), _ptr(group_sum), _stream(stream)))


def hga_route(p, Q, chunk_sum, group_sum, chunk_idx, group_idx, n_groups, workspace,
              chunk_scores=None, group_scores=None, stream=None):
    nbytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check("hga_route", lib().hga_route(
        C.byref(p), _ptr(Q), _ptr(chunk_sum), _ptr(group_sum), _ptr(chunk_idx), _ptr(group_idx),
        _ptr(n_groups), _ptr(chunk_scores), _ptr(group_scores), _ptr(workspace), nbytes,
        _stream(stream)))


def hga_route_static(p, Q, chunk_sum, group_sum, chunk_idx, group_idx, n_groups, stream=None):
    """hga_route for callers that may not allocate device memory: no workspace argument, the
    scratch is a fixed array inside the library (HGA_ROUTE_STATIC_SCRATCH_BYTES per GPU).
    Problems whose routing scratch exceeds that size are refused with HGA_ERR_WORKSPACE.
    Calls on one device share the array: do not let two of them overlap on the GPU, and make
    the first call on a device outside any stream capture."""
    _check("hga_route_static", lib().hga_route_static(
        C.byref(p), _ptr(Q), _ptr(chunk_sum), _ptr(group_sum), _ptr(chunk_idx), _ptr(group_idx),
        _ptr(n_groups), _stream(stream)))


def hga_attn_fwd(p, Q, K, V, group_idx, n_groups, O, LSE, status_word=None, stream=None):
    _check("hga_attn_fwd", lib().hga_attn_fwd(
        C.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(group_idx), _ptr(n_groups), _ptr(O), _ptr(LSE),
        _ptr(status_word), _stream(stream)))


def hga_attn_bwd(p, Q, K, V, O, LSE, dO, group_idx, n_groups, dQ, dK, dV, workspace,
                 status_word=None, stream=None):
    nbytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check("hga_attn_bwd", lib().hga_attn_bwd(
        C.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(LSE), _ptr(dO), _ptr(group_idx),
        _ptr(n_groups), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(workspace), nbytes, _ptr(status_word),
        _stream(stream)))


def hga_step_host(p, Q_host, Kseg_host, Vseg_host, dO_host, K_dev, V_dev, chunk_sum, group_sum,
                  O_host, dQ_host, dK_host, dV_host, arena, status_word=None, stream=None):
    """Host tensors are CPU (ideally pinned) torch tensors; *_dev / summaries / arena are CUDA."""
    nbytes = arena.numel() * arena.element_size()
    _check("hga_step_host", lib().hga_step_host(
        C.byref(p), _ptr(Q_host), _ptr(Kseg_host), _ptr(Vseg_host), _ptr(dO_host), _ptr(K_dev),
        _ptr(V_dev), _ptr(chunk_sum), _ptr(group_sum), _ptr(O_host), _ptr(dQ_host), _ptr(dK_host),
        _ptr(dV_host), _ptr(arena), nbytes, _ptr(status_word), _stream(stream)))


def hga_tbptt_walk(p, Q, K, V, dO, chunk_sum, group_sum, chunk_idx, group_idx, n_groups, O, LSE, dQ,
                   dK, dV, workspace, status_word=None, stream=None):
    """One layer over a whole sequence, segment by segment (all tensors CUDA; see hga.h)."""
    nbytes = workspace.numel() * workspace.element_size()
    _check("hga_tbptt_walk", lib().hga_tbptt_walk(
        C.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(chunk_sum), _ptr(group_sum),
        _ptr(chunk_idx), _ptr(group_idx), _ptr(n_groups), _ptr(O), _ptr(LSE), _ptr(dQ), _ptr(dK),
        _ptr(dV), _ptr(workspace), nbytes, _ptr(status_word), _stream(stream)))


def _host_i32(a):
    arr = np.ascontiguousarray(a, dtype=np.int32)
    return arr, arr.ctypes.data_as(C.c_void_p)


def hga_varlen_workspace_bytes(p, cu_q, cu_k) -> int:
    q, qp = _host_i32(cu_q)
    k, kp = _host_i32(cu_k)
    n = C.c_size_t()
    _check("hga_varlen_workspace_bytes", lib().hga_varlen_workspace_bytes(C.byref(p), len(q) - 1, qp, kp, C.byref(n)))
    return n.value


def hga_varlen_step(p, cu_q, cu_k, Q, K, V, dO, chunk_sum, group_sum, chunk_idx, group_idx, n_groups, O, LSE,
                    dQ, dK, dV, workspace, status_word=None, stream=None):
    """One layer step over packed variable-length sequences (cu_q / cu_k are host prefix sums; see hga.h)."""
    q, qp = _host_i32(cu_q)
    k, kp = _host_i32(cu_k)
    nbytes = workspace.numel() * workspace.element_size()
    _check("hga_varlen_step", lib().hga_varlen_step(
        C.byref(p), len(q) - 1, qp, kp, _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(chunk_sum), _ptr(group_sum),
        _ptr(chunk_idx), _ptr(group_idx), _ptr(n_groups), _ptr(O), _ptr(LSE), _ptr(dQ), _ptr(dK), _ptr(dV),
        _ptr(workspace), nbytes, _ptr(status_word), _stream(stream)))


class HgaLayerBuffers:
    """Device buffers of one HGA layer step for `cfg`, allocated once with torch.

    Holds no arithmetic: it sizes and owns the tensors the C ABI reads and writes.
    """

    def __init__(self, cfg, device="cuda", backward=True, want_scores=False, flags=0):
        self.cfg = cfg
        self.p = make_params(cfg, flags=flags)
        B, Hq, Hkv, d = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
        L, S, nqb = cfg.total_len, cfg.seg_len, cfg.seg_len // cfg.q_block
        kge, per = min(cfg.topk_groups, cfg.chunk // cfg.group), cfg.chunk // cfg.group
        bf, dev = torch.bfloat16, device
        self.chunk_sum = torch.zeros(B, Hkv, L // cfg.chunk, d, dtype=bf, device=dev)
        self.group_sum = torch.zeros(B, Hkv, L // cfg.group, d, dtype=bf, device=dev)
        self.chunk_idx = torch.full((B, Hkv, nqb, cfg.topk_chunks), -1, dtype=torch.int32, device=dev)
        self.group_idx = torch.full((B, Hkv, nqb, cfg.topk_chunks * kge), -1, dtype=torch.int32, device=dev)
        self.n_groups = torch.zeros(B, Hkv, nqb, dtype=torch.int32, device=dev)
        self.O = torch.zeros(B, Hq, S, d, dtype=bf, device=dev)
        self.LSE = torch.zeros(B, Hq, S, dtype=torch.float32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        rb, bb = hga_workspace_bytes(self.p)
        self.route_ws = torch.empty(rb, dtype=torch.uint8, device=dev)
        self.chunk_scores = self.group_scores = None
        if want_scores:
            self.chunk_scores = torch.zeros(B, Hkv, nqb, L // cfg.chunk, dtype=torch.float32, device=dev)
            self.group_scores = torch.zeros(B, Hkv, nqb, cfg.topk_chunks * per, dtype=torch.float32, device=dev)
        self.backward = backward
        if backward:
            self.dQ = torch.zeros(B, Hq, S, d, dtype=bf, device=dev)
            gdt = bf if (self.p.flags & HGA_FLAG_BWD_BF16_GRADS) else torch.float32
            self.dK = torch.zeros(B, Hkv, S, d, dtype=gdt, device=dev)
            self.dV = torch.zeros(B, Hkv, S, d, dtype=gdt, device=dev)
            self.bwd_ws = torch.empty(bb, dtype=torch.uint8, device=dev)

    # the four steps, in path order
    def build_summaries(self, K, tok_begin=None, tok_end=None, stream=None):
        tb = self.cfg.total_len - self.cfg.seg_len if tok_begin is None else tok_begin
        te = self.cfg.total_len if tok_end is None else tok_end
        hga_build_summaries(self.p, K, tb, te, self.chunk_sum, self.group_sum, stream)

    def route(self, Q, stream=None):
        hga_route(self.p, Q, self.chunk_sum, self.group_sum, self.chunk_idx, self.group_idx,
                  self.n_groups, self.route_ws, self.chunk_scores, self.group_scores, stream)

    def attn_fwd(self, Q, K, V, group_idx=None, n_groups=None, stream=None):
        hga_attn_fwd(self.p, Q, K, V, self.group_idx if group_idx is None else group_idx,
                     self.n_groups if n_groups is None else n_groups, self.O, self.LSE,
                     self.status, stream)

    def attn_bwd(self, Q, K, V, dO, group_idx=None, n_groups=None, stream=None):
        hga_attn_bwd(self.p, Q, K, V, self.O, self.LSE, dO,
                     self.group_idx if group_idx is None else group_idx,
                     self.n_groups if n_groups is None else n_groups, self.dQ, self.dK, self.dV,
                     self.bwd_ws, self.status, stream)

    def step(self, Q, K, V, dO=None, stream=None):
        """One pass of the whole hot path over resident device tensors."""
        self.build_summaries(K, stream=stream)
        self.route(Q, stream)
        self.attn_fwd(Q, K, V, stream=stream)
        if dO is not None:
            self.attn_bwd(Q, K, V, dO, stream=stream)
