"""Parity of the CUDA library (through the C ABI) with the CPU oracle, on the same seeded
inputs: element by element at sizes the oracle finishes in seconds, on sampled items at the
benchmark's full sizes, plus the edge cases of the method."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_15105_b200 import binding
from paper_2607_15105_b200.workloads import CONFIGS, HgaConfig, bf16_bits_to_f64, make_inputs

from hga_testlib import (TOL_GRAD, TOL_LSE, TOL_O, bf16_to_f64, bits_of, check_grads, check_routing,
                         item_rows, rel_fro, to_dev)

pytestmark = pytest.mark.gpu

FLAG_SETS = [0, binding.HGA_FLAG_GENERIC_KERNELS]


def small(**kw):
    base = dict(name="small", batch=2, n_q_heads=4, n_kv_heads=2, head_dim=128, total_len=1536,
                seg_len=512, chunk=64, group=8, q_block=64, topk_chunks=5, topk_groups=3,
                sink=64, local=128, topics=16, needles=4, backward=True, seed=11)
    base.update(kw)
    return HgaConfig(**base)


SMALL_CASES = {
    "d128_hist": small(),
    "d64_tiny": CONFIGS[1],
    "no_history_ragged_budget": small(total_len=1024, seg_len=1024, batch=1, topk_chunks=8),
    "bq128_c128_g16": small(chunk=128, group=16, q_block=128, total_len=2048, seg_len=512,
                            sink=128, local=256, topk_chunks=4, topk_groups=4, topics=0, needles=0),
    "bq128_c64": small(q_block=128, total_len=1280, seg_len=256, n_q_heads=2, n_kv_heads=2),
    "gqa8": small(n_q_heads=8, n_kv_heads=1, batch=1, total_len=1024, seg_len=256),
}


class Case:
    """Inputs on host and device plus the oracle's results for one configuration."""

    def __init__(self, cfg, items=None, need_bwd=True):
        self.cfg = cfg
        self.x = make_inputs(cfg)
        self.items = items
        x = self.x
        self.Q, self.K, self.V = to_dev(x["Q"]), to_dev(x["K"]), to_dev(x["V"])
        self.dO = to_dev(x["dO"]) if "dO" in x else None
        self.cs, self.gs = oracle.build_summaries(cfg, x["K"])
        self.ref = oracle.route(cfg, x["Q"], self.cs, self.gs, items=items, want_scores=True)
        self.gi = torch.from_numpy(self.ref["group_idx"]).cuda()
        self.ng = torch.from_numpy(self.ref["n_groups"]).cuda()


_cases = {}


def get_case(name):
    if name not in _cases:
        _cases[name] = Case(SMALL_CASES[name])
    return _cases[name]


# ------------------------------------------------------------------ summaries

@pytest.mark.parametrize("name", list(SMALL_CASES))
def test_summaries_bit_exact(name):
    c = get_case(name)
    cfg = c.cfg
    buf = binding.HgaLayerBuffers(cfg, backward=False)
    buf.build_summaries(c.K, 0, cfg.total_len)
    torch.cuda.synchronize()
    assert np.array_equal(bits_of(buf.chunk_sum), c.cs)
    assert np.array_equal(bits_of(buf.group_sum), c.gs)


def test_summaries_partial_range_keeps_history():
    c = get_case("d128_hist")
    cfg = c.cfg
    buf = binding.HgaLayerBuffers(cfg, backward=False)
    buf.chunk_sum.view(torch.int16).fill_(0x1234)
    buf.group_sum.view(torch.int16).fill_(0x1234)
    buf.build_summaries(c.K)            # active range only
    torch.cuda.synchronize()
    hc, hg = cfg.history // cfg.chunk, cfg.history // cfg.group
    cs, gs = bits_of(buf.chunk_sum), bits_of(buf.group_sum)
    assert np.all(cs[:, :, :hc] == 0x1234) and np.array_equal(cs[:, :, hc:], c.cs[:, :, hc:])
    assert np.all(gs[:, :, :hg] == 0x1234) and np.array_equal(gs[:, :, hg:], c.gs[:, :, hg:])


# ------------------------------------------------------------------ routing

@pytest.mark.parametrize("flags", FLAG_SETS)
@pytest.mark.parametrize("name", list(SMALL_CASES))
def test_route_matches_oracle(name, flags):
    c = get_case(name)
    cfg = c.cfg
    buf = binding.HgaLayerBuffers(cfg, backward=False, want_scores=True, flags=flags)
    buf.chunk_sum.copy_(to_dev(c.cs))
    buf.group_sum.copy_(to_dev(c.gs))
    buf.route(c.Q)
    torch.cuda.synchronize()
    n, ec, eg = check_routing(cfg, c.ref, buf.chunk_idx.cpu().numpy(), buf.group_idx.cpu().numpy(),
                              buf.n_groups.cpu().numpy())
    assert ec <= max(1, n // 10) and eg <= max(1, n // 5), (n, ec, eg)
    # optional score outputs: fp32 accumulation of exact products vs the oracle's fp64
    cs = buf.chunk_scores.cpu().numpy().astype(np.float64)
    fin = np.isfinite(c.ref["chunk_scores"])
    assert np.array_equal(np.isfinite(cs), fin)
    assert np.max(np.abs(cs[fin] - c.ref["chunk_scores"][fin]), initial=0) < 2e-4


# ------------------------------------------------------------------ attention

@pytest.mark.parametrize("flags", FLAG_SETS)
@pytest.mark.parametrize("name", list(SMALL_CASES))
def test_attention_fwd_bwd_on_oracle_indices(name, flags):
    c = get_case(name)
    cfg, x = c.cfg, c.x
    buf = binding.HgaLayerBuffers(cfg, flags=flags)
    buf.attn_fwd(c.Q, c.K, c.V, c.gi, c.ng)
    buf.attn_bwd(c.Q, c.K, c.V, c.dO, c.gi, c.ng)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    O, LSE = oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], c.ref["group_idx"], c.ref["n_groups"])
    dQ, dK, dV = oracle.attn_bwd(cfg, x["Q"], x["K"], x["V"], x["dO"], c.ref["group_idx"], c.ref["n_groups"])
    assert np.max(np.abs(bf16_to_f64(buf.O) - O)) <= TOL_O
    assert np.max(np.abs(buf.LSE.cpu().numpy().astype(np.float64) - LSE)) <= TOL_LSE
    check_grads((bf16_to_f64(buf.dQ), buf.dK.cpu().numpy().astype(np.float64),
                 buf.dV.cpu().numpy().astype(np.float64)), (dQ, dK, dV), name)


@pytest.mark.parametrize("flags", FLAG_SETS)
def test_whole_path_end_to_end(flags):
    # build -> route -> fwd -> bwd on the GPU's own summaries and indices
    c = get_case("d128_hist")
    cfg, x = c.cfg, c.x
    buf = binding.HgaLayerBuffers(cfg, flags=flags)
    buf.build_summaries(c.K, 0, cfg.total_len)
    buf.route(c.Q)
    buf.attn_fwd(c.Q, c.K, c.V)
    buf.attn_bwd(c.Q, c.K, c.V, c.dO)
    torch.cuda.synchronize()
    gi, ng = buf.group_idx.cpu().numpy(), buf.n_groups.cpu().numpy()
    check_routing(cfg, c.ref, buf.chunk_idx.cpu().numpy(), gi, ng)
    O, _ = oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], gi, ng)     # oracle on the GPU's indices
    dQ, dK, dV = oracle.attn_bwd(cfg, x["Q"], x["K"], x["V"], x["dO"], gi, ng)
    assert np.max(np.abs(bf16_to_f64(buf.O) - O)) <= TOL_O
    assert rel_fro(bf16_to_f64(buf.dQ), dQ) <= TOL_GRAD
    assert rel_fro(buf.dK.cpu().numpy().astype(np.float64), dK) <= TOL_GRAD
    assert rel_fro(buf.dV.cpu().numpy().astype(np.float64), dV) <= TOL_GRAD


# ------------------------------------------------------------------ edge cases

@pytest.mark.parametrize("flags", FLAG_SETS)
def test_full_budget_equals_dense_causal(flags):
    cfg = small(batch=1, total_len=768, seg_len=512, topk_chunks=12, topk_groups=8)
    x = make_inputs(cfg)
    Q, K, V, dO = (to_dev(x[n]) for n in ("Q", "K", "V", "dO"))
    buf = binding.HgaLayerBuffers(cfg, flags=flags)
    buf.build_summaries(K, 0, cfg.total_len)
    buf.route(Q)
    buf.attn_fwd(Q, K, V)
    buf.attn_bwd(Q, K, V, dO)
    torch.cuda.synchronize()
    q = torch.from_numpy(bf16_bits_to_f64(x["Q"])).requires_grad_(True)
    k = torch.from_numpy(bf16_bits_to_f64(x["K"])).requires_grad_(True)
    v = torch.from_numpy(bf16_bits_to_f64(x["V"])).requires_grad_(True)
    H, L = cfg.history, cfg.total_len
    mask = torch.tril(torch.ones(L, L, dtype=torch.bool))[H:]
    o = torch.nn.functional.scaled_dot_product_attention(
        q, k.repeat_interleave(cfg.gqa, 1), v.repeat_interleave(cfg.gqa, 1), attn_mask=mask)
    (o * torch.from_numpy(bf16_bits_to_f64(x["dO"]))).sum().backward()
    assert np.max(np.abs(bf16_to_f64(buf.O) - o.detach().numpy())) <= TOL_O
    assert rel_fro(bf16_to_f64(buf.dQ), q.grad.numpy()) <= TOL_GRAD
    assert rel_fro(buf.dK.cpu().numpy().astype(np.float64), k.grad[:, :, H:].numpy()) <= TOL_GRAD
    assert rel_fro(buf.dV.cpu().numpy().astype(np.float64), v.grad[:, :, H:].numpy()) <= TOL_GRAD


@pytest.mark.parametrize("flags", FLAG_SETS)
def test_zero_budget_and_single_block(flags):
    cfg = small(batch=1, n_q_heads=2, n_kv_heads=1, total_len=64, seg_len=64, topk_chunks=0)
    x = make_inputs(cfg)
    Q, K, V, dO = (to_dev(x[n]) for n in ("Q", "K", "V", "dO"))
    buf = binding.HgaLayerBuffers(cfg, flags=flags)
    buf.step(Q, K, V, dO)
    torch.cuda.synchronize()
    assert int(buf.n_groups.sum().item()) == 0
    gi = np.zeros((1, 1, 1, 0), np.int32)
    ng = np.zeros((1, 1, 1), np.int32)
    O, LSE = oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], gi, ng)
    dQ, dK, dV = oracle.attn_bwd(cfg, x["Q"], x["K"], x["V"], x["dO"], gi, ng)
    assert np.max(np.abs(bf16_to_f64(buf.O) - O)) <= TOL_O
    assert rel_fro(bf16_to_f64(buf.dQ), dQ) <= TOL_GRAD
    assert rel_fro(buf.dK.cpu().numpy().astype(np.float64), dK) <= TOL_GRAD
    assert rel_fro(buf.dV.cpu().numpy().astype(np.float64), dV) <= TOL_GRAD


@pytest.mark.parametrize("flags", FLAG_SETS)
def test_invalid_indices_are_skipped_and_reported(flags):
    c = get_case("d128_hist")
    cfg, x = c.cfg, c.x
    gi = c.ref["group_idx"].copy()
    ng = c.ref["n_groups"].copy()
    clean_gi, clean_ng = gi.copy(), ng.copy()
    # item (0, 0, last block): duplicate its first entry in place of the second, and point
    # the last one past the end of the sequence; the valid remainder is what must be used
    last = cfg.n_q_blocks - 1
    n = int(ng[0, 0, last])
    keep = [int(m) for m in gi[0, 0, last, :n]]
    gi[0, 0, last, 1] = keep[0]
    gi[0, 0, last, n - 1] = cfg.total_len // cfg.group + 5
    valid = [keep[0]] + keep[2:n - 1]
    clean_gi[0, 0, last] = -1
    clean_gi[0, 0, last, :len(valid)] = valid
    clean_ng[0, 0, last] = len(valid)
    buf = binding.HgaLayerBuffers(cfg, flags=flags)
    buf.attn_fwd(c.Q, c.K, c.V, torch.from_numpy(gi).cuda(), torch.from_numpy(ng).cuda())
    torch.cuda.synchronize()
    assert int(buf.status.item()) & binding.HGA_STATUS_BAD_INDEX
    O, _ = oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], clean_gi, clean_ng)
    assert np.max(np.abs(bf16_to_f64(buf.O) - O)) <= TOL_O


@pytest.mark.parametrize("flags", FLAG_SETS)
def test_strided_inputs(flags):
    # Q/K/V/dO as slices of wider buffers (packed projections): same results as dense
    c = get_case("d128_hist")
    cfg = c.cfg
    d = cfg.head_dim

    def widen(t):
        wide = torch.zeros(*t.shape[:3], 2 * d + 8, dtype=t.dtype, device=t.device)
        wide[..., 8:8 + d] = t
        return wide[..., 8:8 + d]

    Qs, Ks, Vs, dOs = widen(c.Q), widen(c.K), widen(c.V), widen(c.dO)
    dense = binding.HgaLayerBuffers(cfg, flags=flags)
    dense.attn_fwd(c.Q, c.K, c.V, c.gi, c.ng)
    dense.attn_bwd(c.Q, c.K, c.V, c.dO, c.gi, c.ng)
    st = binding.HgaLayerBuffers(cfg, flags=flags)
    st.O = widen(torch.zeros_like(dense.O))
    st.dQ = widen(torch.zeros_like(dense.dQ))
    st.p = binding.params_for(cfg, Q=Qs, K=Ks, V=Vs, O=st.O, flags=flags)
    st.build_summaries(Ks, 0, cfg.total_len)
    st.attn_fwd(Qs, Ks, Vs, c.gi, c.ng)
    st.attn_bwd(Qs, Ks, Vs, dOs, c.gi, c.ng)
    torch.cuda.synchronize()
    assert np.array_equal(bits_of(st.chunk_sum), c.cs) and np.array_equal(bits_of(st.group_sum), c.gs)
    assert torch.equal(st.O.contiguous(), dense.O) and torch.equal(st.LSE, dense.LSE)
    assert torch.equal(st.dQ.contiguous(), dense.dQ)
    assert rel_fro(st.dK.cpu().numpy(), dense.dK.cpu().numpy()) < 1e-5


def test_bwd_accumulate_flag():
    c = get_case("d64_tiny")
    cfg = c.cfg
    buf = binding.HgaLayerBuffers(cfg)
    buf.attn_fwd(c.Q, c.K, c.V, c.gi, c.ng)
    buf.attn_bwd(c.Q, c.K, c.V, c.dO, c.gi, c.ng)
    once = buf.dK.clone()
    buf.p = binding.make_params(cfg, flags=binding.HGA_FLAG_BWD_ACCUMULATE)
    buf.attn_bwd(c.Q, c.K, c.V, c.dO, c.gi, c.ng)
    torch.cuda.synchronize()
    assert rel_fro(buf.dK.cpu().numpy(), 2 * once.cpu().numpy()) < 1e-5


def test_summaries_do_not_leak_into_attention():
    # summaries only select: scribbling over them after routing leaves O bit-identical
    c = get_case("d128_hist")
    buf = binding.HgaLayerBuffers(c.cfg, backward=False)
    buf.build_summaries(c.K, 0, c.cfg.total_len)
    buf.route(c.Q)
    buf.attn_fwd(c.Q, c.K, c.V)
    first = buf.O.clone()
    buf.chunk_sum.normal_()
    buf.group_sum.normal_()
    buf.attn_fwd(c.Q, c.K, c.V)
    torch.cuda.synchronize()
    assert torch.equal(first, buf.O)


def test_step_host_matches_device_path():
    c = get_case("d128_hist")
    cfg, x = c.cfg, c.x
    H = cfg.history
    dev = binding.HgaLayerBuffers(cfg)
    dev.build_summaries(c.K, 0, cfg.total_len)
    dev.route(c.Q)
    dev.attn_fwd(c.Q, c.K, c.V)
    dev.attn_bwd(c.Q, c.K, c.V, c.dO)
    # host entry point: history resident on the device, the segment arrives from the host
    host = binding.HgaLayerBuffers(cfg)
    host.build_summaries(c.K, 0, H)
    Kd, Vd = c.K.clone(), c.V.clone()
    Kd[:, :, H:].zero_()
    Vd[:, :, H:].zero_()
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).pin_memory()
    Qh, dOh = pin(x["Q"]), pin(x["dO"])
    Kh, Vh = pin(x["K"][:, :, H:]), pin(x["V"][:, :, H:])
    Oh, dQh = torch.empty_like(Qh).pin_memory(), torch.empty_like(Qh).pin_memory()
    dKh = torch.empty(cfg.batch, cfg.n_kv_heads, cfg.seg_len, cfg.head_dim).pin_memory()
    dVh = torch.empty_like(dKh).pin_memory()
    arena = torch.empty(binding.hga_step_arena_bytes(host.p), dtype=torch.uint8, device="cuda")
    binding.hga_step_host(host.p, Qh, Kh, Vh, dOh, Kd, Vd, host.chunk_sum, host.group_sum, Oh, dQh,
                          dKh, dVh, arena, host.status)
    torch.cuda.synchronize()
    assert torch.equal(Kd, c.K) and torch.equal(Vd, c.V)
    assert torch.equal(host.chunk_sum, dev.chunk_sum) and torch.equal(host.group_sum, dev.group_sum)
    assert torch.equal(Oh, dev.O.cpu()) and torch.equal(dQh, dev.dQ.cpu())
    assert rel_fro(dKh.numpy(), dev.dK.cpu().numpy()) < 1e-5
    assert rel_fro(dVh.numpy(), dev.dV.cpu().numpy()) < 1e-5


def test_forward_is_deterministic_and_launches_are_counted():
    c = get_case("d128_hist")
    buf = binding.HgaLayerBuffers(c.cfg)
    before = binding.hga_kernel_launch_count()
    buf.step(c.Q, c.K, c.V, c.dO)
    first = (buf.O.clone(), buf.LSE.clone(), buf.dQ.clone(), buf.group_idx.clone())
    buf.step(c.Q, c.K, c.V, c.dO)
    torch.cuda.synchronize()
    assert binding.hga_kernel_launch_count() - before >= 2 * 4
    assert all(torch.equal(a, b) for a, b in zip(first, (buf.O, buf.LSE, buf.dQ, buf.group_idx)))


@pytest.mark.parametrize("flags", FLAG_SETS)
@pytest.mark.parametrize("name", ["d128_hist", "bq128_c128_g16", "d64_tiny"])
def test_bf16_gradient_outputs(name, flags):
    """HGA_FLAG_BWD_BF16_GRADS: dK/dV leave as bf16; the sums still run in fp32, so the result is the
    fp32 result rounded once (compared with it to bf16 precision, and with the oracle)."""
    c = get_case(name)
    cfg = c.cfg
    outs = {}
    for extra in (0, binding.HGA_FLAG_BWD_BF16_GRADS):
        buf = binding.HgaLayerBuffers(cfg, flags=flags | extra)
        buf.attn_fwd(c.Q, c.K, c.V, c.gi, c.ng)
        before = binding.hga_kernel_launch_counts()
        buf.attn_bwd(c.Q, c.K, c.V, c.dO, c.gi, c.ng)
        torch.cuda.synchronize()
        assert int(buf.status.item()) == 0
        ran = [b - a for a, b in zip(before, binding.hga_kernel_launch_counts())]
        # one conversion launch for both tensors, behind either kernel family
        tensor = flags == 0 and cfg.head_dim == 128
        assert ran[binding.HGA_KERNELS_AUX] == (1 if extra else 0), ran
        assert (ran[binding.HGA_KERNELS_BWD_TENSOR] == 2) == tensor, ran
        outs[extra] = (buf.dQ.clone(), buf.dK.clone(), buf.dV.clone())
    (dQ32, dK32, dV32), (dQ16, dK16, dV16) = outs[0], outs[binding.HGA_FLAG_BWD_BF16_GRADS]
    assert dK16.dtype == torch.bfloat16 and dV16.dtype == torch.bfloat16
    assert torch.equal(dQ32, dQ16)
    for a32, a16 in ((dK32, dK16), (dV32, dV16)):
        ref = a32.double()
        err = (a16.double() - ref).abs()
        # one rounding to 8 significant bits, plus the run-to-run wobble of the fp32 atomics
        assert bool((err <= ref.abs() * 2.0 ** -8 + 1e-5).all())
    x = c.x
    _, dK_ref, dV_ref = oracle.attn_bwd(cfg, x["Q"], x["K"], x["V"], x["dO"], c.ref["group_idx"], c.ref["n_groups"])
    assert rel_fro(bf16_to_f64(dK16), dK_ref) <= TOL_GRAD
    assert rel_fro(bf16_to_f64(dV16), dV_ref) <= TOL_GRAD


def test_bf16_gradients_reject_accumulate():
    cfg = SMALL_CASES["d128_hist"]
    p = binding.make_params(cfg, flags=binding.HGA_FLAG_BWD_BF16_GRADS | binding.HGA_FLAG_BWD_ACCUMULATE)
    buf = binding.HgaLayerBuffers(cfg)
    c = get_case("d128_hist")
    with pytest.raises(binding.HgaError):
        binding.hga_attn_bwd(p, c.Q, c.K, c.V, buf.O, buf.LSE, c.dO, c.gi, c.ng, buf.dQ, buf.dK, buf.dV,
                             torch.empty(1 << 24, dtype=torch.uint8, device="cuda"), buf.status)
