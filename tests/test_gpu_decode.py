"""HGA_FLAG_DECODE: generation-shaped routed attention (the query block is the few newest tokens
behind a history of any length).  Summaries of the closed chunks, routing and forward attention
through the C ABI against the oracle in its decode mode, with both kernel families."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_15105_b200 import binding
from paper_2607_15105_b200.workloads import HgaConfig, make_inputs

from hga_testlib import TOL_LSE, TOL_O, bf16_to_f64, bits_of, check_routing, to_dev

pytestmark = pytest.mark.gpu

FLAG_SETS = [0, binding.HGA_FLAG_GENERIC_KERNELS]


def decode_cfg(hist, n, **kw):
    base = dict(name="decode", batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, total_len=hist + n,
                seg_len=n, chunk=64, group=8, q_block=n, topk_chunks=4, topk_groups=3, sink=64,
                local=128, topics=16, needles=0, backward=False, seed=31, decode=True)
    base.update(kw)
    return HgaConfig(**base)


CASES = {
    "one_token": decode_cfg(1500, 1),
    "one_token_odd_history": decode_cfg(1531, 1),
    "five_tokens": decode_cfg(1477, 5),
    "eight_tokens_aligned": decode_cfg(1408, 8),
    "sixteen_tokens": decode_cfg(1399, 16),
    "no_candidates": decode_cfg(100, 3),
    "few_candidates": decode_cfg(330, 1, topk_chunks=8),
    "gqa8": decode_cfg(1290, 2, n_q_heads=8, n_kv_heads=1, batch=3),
    "two_blocks": decode_cfg(1216, 4, total_len=1216 + 8, seg_len=8),
    "d64": decode_cfg(700, 3, head_dim=64, n_q_heads=4),
    "c128_g16": decode_cfg(2100, 1, chunk=128, group=16, sink=128, local=256, topk_groups=4),
}


@pytest.mark.parametrize("flags", FLAG_SETS)
@pytest.mark.parametrize("name", list(CASES))
def test_decode_matches_oracle(name, flags):
    cfg = CASES[name]
    x = make_inputs(cfg)
    closed = (cfg.total_len // cfg.chunk) * cfg.chunk
    cs, gs = oracle.build_summaries(cfg, x["K"])
    ref = oracle.route(cfg, x["Q"], cs, gs, want_scores=True)
    buf = binding.HgaLayerBuffers(cfg, backward=False, want_scores=True, flags=flags)
    assert buf.p.flags & binding.HGA_FLAG_DECODE
    Q, K, V = to_dev(x["Q"]), to_dev(x["K"]), to_dev(x["V"])
    buf.build_summaries(K, 0, closed)
    buf.route(Q)
    buf.attn_fwd(Q, K, V)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    assert np.array_equal(bits_of(buf.chunk_sum), cs) and np.array_equal(bits_of(buf.group_sum), gs)
    gi, ng = buf.group_idx.cpu().numpy(), buf.n_groups.cpu().numpy()
    n, ec, eg = check_routing(cfg, ref, buf.chunk_idx.cpu().numpy(), gi, ng)
    assert ec <= max(1, n // 10) and eg <= max(1, n // 5), (n, ec, eg)
    got = buf.chunk_scores.cpu().numpy().astype(np.float64)
    fin = np.isfinite(ref["chunk_scores"])
    assert np.array_equal(np.isfinite(got), fin)
    assert np.max(np.abs(got[fin] - ref["chunk_scores"][fin]), initial=0) < 2e-4
    O_ref, LSE_ref = oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], gi, ng)
    assert np.max(np.abs(bf16_to_f64(buf.O) - O_ref)) <= TOL_O
    assert np.max(np.abs(buf.LSE.cpu().numpy().astype(np.float64) - LSE_ref)) <= TOL_LSE


def test_keys_behind_the_newest_token_are_never_read():
    """K/V rows past total_len (the unwritten tail of a cache) must not reach the result, whatever
    they hold: the same step on a cache with a non-finite tail gives the same bits."""
    cfg = CASES["five_tokens"]
    x = make_inputs(cfg)
    L, cap = cfg.total_len, cfg.total_len + 200
    buf = binding.HgaLayerBuffers(cfg, backward=False)
    Q, K, V = to_dev(x["Q"]), to_dev(x["K"]), to_dev(x["V"])
    closed = (L // cfg.chunk) * cfg.chunk
    buf.build_summaries(K, 0, closed)
    buf.route(Q)
    buf.attn_fwd(Q, K, V)
    torch.cuda.synchronize()
    want_O, want_LSE = bits_of(buf.O).copy(), buf.LSE.cpu().numpy().copy()
    Kc = torch.full((cfg.batch, cfg.n_kv_heads, cap, cfg.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    Vc = torch.full_like(Kc, float("inf"))
    Kc[:, :, :L] = K
    Vc[:, :, :L] = V
    Kv, Vv = Kc[:, :, :L], Vc[:, :, :L]                   # views: strides of the larger cache
    buf.p = binding.params_for(cfg, Q=Q, K=Kv, V=Vv, O=buf.O, flags=binding.HGA_FLAG_DECODE)
    buf.O.zero_()
    buf.attn_fwd(Q, Kv, Vv)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    assert np.array_equal(bits_of(buf.O), want_O) and np.array_equal(buf.LSE.cpu().numpy(), want_LSE)


def test_decode_is_forward_only_and_needs_its_flag():
    cfg = CASES["one_token"]
    from dataclasses import replace
    with pytest.raises(binding.HgaError):
        binding.hga_workspace_bytes(binding.make_params(replace(cfg, decode=False)))
    buf = binding.HgaLayerBuffers(cfg, backward=False)
    t = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.HgaError):
        binding.hga_attn_bwd(buf.p, t, t, t, t, t, t, t, t, t, t, t, t, None)


def test_benchmark_decode_config_sampled_items():
    """Configuration 7 (what bench.py times as its generation-shaped step), whole path on the GPU,
    sampled (sequence, kv head) items recomputed by the oracle."""
    from paper_2607_15105_b200.workloads import CONFIGS
    cfg = CONFIGS[7]
    x = make_inputs(cfg)
    buf = binding.HgaLayerBuffers(cfg, backward=False)
    Q, K, V = to_dev(x["Q"]), to_dev(x["K"]), to_dev(x["V"])
    closed = (cfg.total_len // cfg.chunk) * cfg.chunk
    buf.build_summaries(K, 0, closed)
    buf.route(Q)
    buf.attn_fwd(Q, K, V)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    items = [0, 1, 7, 8, 100, 131, 200, cfg.n_items - 1]
    cs, gs = bits_of(buf.chunk_sum), bits_of(buf.group_sum)
    # the summaries the router read: bit-exact for the sampled heads' first and last chunks
    ocs, ogs = oracle.build_summaries(cfg.scaled(batch=1), np.ascontiguousarray(x["K"][:1]))
    assert np.array_equal(cs[:1], ocs) and np.array_equal(gs[:1], ogs)
    ref = oracle.route(cfg, x["Q"], cs, gs, items=items, want_scores=True)
    gi, ng = buf.group_idx.cpu().numpy(), buf.n_groups.cpu().numpy()
    n, ec, eg = check_routing(cfg, ref, buf.chunk_idx.cpu().numpy(), gi, ng, items=items)
    assert n == len(items) and ec <= 1 and eg <= 2, (n, ec, eg)
    O_ref, LSE_ref = oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], gi, ng, items=items)
    G = cfg.gqa
    Of, LSEf = bf16_to_f64(buf.O), buf.LSE.cpu().numpy().astype(np.float64)
    for it in items:
        b, h = it // cfg.n_kv_heads, it % cfg.n_kv_heads
        sl = slice(h * G, (h + 1) * G)
        assert np.max(np.abs(Of[b, sl] - O_ref[b, sl])) <= TOL_O
        assert np.max(np.abs(LSEf[b, sl] - LSE_ref[b, sl])) <= TOL_LSE


@pytest.mark.parametrize("generic", FLAG_SETS)
@pytest.mark.parametrize("variant", ["mean+global", "lse", "global"])
@pytest.mark.parametrize("name", ["five_tokens", "sixteen_tokens", "gqa8"])
def test_decode_with_routing_variants(name, variant, generic):
    """The routing variants (score aggregators, one group budget over all opened chunks) combine with
    the generation shape: routing against the oracle's same combination, attention on the lists taken."""
    cfg = CASES[name]
    agg = "mean" if "mean" in variant else "lse" if "lse" in variant else "max"
    gb = "global" in variant
    flags = generic | {"mean": binding.HGA_FLAG_SCORE_MEAN, "lse": binding.HGA_FLAG_SCORE_LSE, "max": 0}[agg]
    flags |= binding.HGA_FLAG_GLOBAL_GROUP_BUDGET if gb else 0
    x = make_inputs(cfg)
    cs, gs = oracle.build_summaries(cfg, x["K"])
    ref = oracle.route(cfg, x["Q"], cs, gs, want_scores=True, score_agg=agg, global_group_budget=gb)
    buf = binding.HgaLayerBuffers(cfg, backward=False, flags=flags)
    buf.chunk_sum.copy_(to_dev(cs))
    buf.group_sum.copy_(to_dev(gs))
    Q, K, V = to_dev(x["Q"]), to_dev(x["K"]), to_dev(x["V"])
    buf.route(Q)
    buf.attn_fwd(Q, K, V)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    gi, ng = buf.group_idx.cpu().numpy(), buf.n_groups.cpu().numpy()
    n, ec, eg = check_routing(cfg, ref, buf.chunk_idx.cpu().numpy(), gi, ng, global_budget=gb)
    assert ec <= max(1, n // 10) and eg <= max(1, n // 5), (n, ec, eg)
    O_ref, LSE_ref = oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], gi, ng)
    assert np.max(np.abs(bf16_to_f64(buf.O) - O_ref)) <= TOL_O
    assert np.max(np.abs(buf.LSE.cpu().numpy().astype(np.float64) - LSE_ref)) <= TOL_LSE
