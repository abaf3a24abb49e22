"""Seeded random shapes through the whole path (both kernel families) against the oracle: head counts,
head_dim, chunk/group/query-block sizes, budgets, window sizes (including none), history lengths.
Each case is small enough for the oracle to recompute everything."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_15105_b200 import binding
from paper_2607_15105_b200.workloads import HgaConfig, make_inputs

from hga_testlib import TOL_GRAD, TOL_LSE, TOL_O, bf16_to_f64, bits_of, check_routing, rel_fro, to_dev

pytestmark = pytest.mark.gpu


def draw(seed):
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 128, 128]))
    hkv = int(rng.choice([1, 2]))
    gqa = int(rng.choice([1, 2, 4, 8]))
    c = int(rng.choice([64, 128]))
    g = int(rng.choice([8, 16]))
    bq = c * int(rng.choice([1, 1, 2]))
    nqb = int(rng.integers(1, 5))
    hist_blocks = int(rng.integers(0, 9))
    per = c // g
    return HgaConfig("random%d" % seed, batch=int(rng.choice([1, 2])), n_q_heads=hkv * gqa, n_kv_heads=hkv,
                     head_dim=d, total_len=(hist_blocks + nqb) * bq, seg_len=nqb * bq, chunk=c, group=g, q_block=bq,
                     topk_chunks=int(rng.integers(0, 7)), topk_groups=int(rng.integers(1, per + 1)),
                     sink=c * int(rng.integers(0, 3)), local=c * int(rng.integers(0, 3)),
                     topics=int(rng.choice([0, 8])), needles=0, backward=True, seed=500 + seed)


@pytest.mark.parametrize("flags", [0, binding.HGA_FLAG_GENERIC_KERNELS])
@pytest.mark.parametrize("seed", range(40))
def test_random_shape(seed, flags):
    cfg = draw(seed)
    x = make_inputs(cfg)
    Q, K, V, dO = to_dev(x["Q"]), to_dev(x["K"]), to_dev(x["V"]), to_dev(x["dO"])
    buf = binding.HgaLayerBuffers(cfg, flags=flags)
    buf.build_summaries(K, 0, cfg.total_len)
    buf.route(Q)
    buf.attn_fwd(Q, K, V)
    buf.attn_bwd(Q, K, V, dO)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0, cfg
    cs, gs = oracle.build_summaries(cfg, x["K"])
    assert np.array_equal(bits_of(buf.chunk_sum), cs) and np.array_equal(bits_of(buf.group_sum), gs), cfg
    ref = oracle.route(cfg, x["Q"], cs, gs, want_scores=True)
    gi, ng = buf.group_idx.cpu().numpy(), buf.n_groups.cpu().numpy()
    n, ec, eg = check_routing(cfg, ref, buf.chunk_idx.cpu().numpy(), gi, ng)
    assert ec <= max(1, n // 8) and eg <= max(1, n // 4), (cfg, n, ec, eg)
    O_ref, LSE_ref = oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], gi, ng)
    assert np.max(np.abs(bf16_to_f64(buf.O) - O_ref)) <= TOL_O, cfg
    assert np.max(np.abs(buf.LSE.cpu().numpy().astype(np.float64) - LSE_ref)) <= TOL_LSE, cfg
    dQ_ref, dK_ref, dV_ref = oracle.attn_bwd(cfg, x["Q"], x["K"], x["V"], x["dO"], gi, ng)
    assert rel_fro(bf16_to_f64(buf.dQ), dQ_ref) <= TOL_GRAD, cfg
    assert rel_fro(buf.dK.cpu().numpy().astype(np.float64), dK_ref) <= TOL_GRAD, cfg
    assert rel_fro(buf.dV.cpu().numpy().astype(np.float64), dV_ref) <= TOL_GRAD, cfg


def draw_decode(seed):
    rng = np.random.default_rng(7000 + seed)
    d = int(rng.choice([64, 128, 128]))
    hkv = int(rng.choice([1, 2]))
    gqa = int(rng.choice([1, 2, 4, 8]))
    c = int(rng.choice([64, 128]))
    g = int(rng.choice([8, 16]))
    n = int(rng.integers(1, 17))
    hist = int(rng.integers(0, 2200))
    per = c // g
    return HgaConfig("random_decode%d" % seed, batch=int(rng.choice([1, 3])), n_q_heads=hkv * gqa, n_kv_heads=hkv,
                     head_dim=d, total_len=hist + n, seg_len=n, chunk=c, group=g, q_block=n,
                     topk_chunks=int(rng.integers(0, 7)), topk_groups=int(rng.integers(1, per + 1)),
                     sink=c * int(rng.integers(0, 3)), local=c * int(rng.integers(0, 3)),
                     topics=int(rng.choice([0, 8])), needles=0, backward=False, seed=900 + seed, decode=True)


@pytest.mark.parametrize("flags", [0, binding.HGA_FLAG_GENERIC_KERNELS])
@pytest.mark.parametrize("seed", range(30))
def test_random_decode_shape(seed, flags):
    cfg = draw_decode(seed)
    closed = (cfg.total_len // cfg.chunk) * cfg.chunk
    if closed == 0:
        pytest.skip("no closed chunk: the summary buffers would be empty")
    x = make_inputs(cfg)
    Q, K, V = to_dev(x["Q"]), to_dev(x["K"]), to_dev(x["V"])
    buf = binding.HgaLayerBuffers(cfg, backward=False, flags=flags)
    buf.build_summaries(K, 0, closed)
    buf.route(Q)
    buf.attn_fwd(Q, K, V)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0, cfg
    cs, gs = oracle.build_summaries(cfg, x["K"])
    assert np.array_equal(bits_of(buf.chunk_sum), cs) and np.array_equal(bits_of(buf.group_sum), gs), cfg
    ref = oracle.route(cfg, x["Q"], cs, gs, want_scores=True)
    gi, ng = buf.group_idx.cpu().numpy(), buf.n_groups.cpu().numpy()
    n, ec, eg = check_routing(cfg, ref, buf.chunk_idx.cpu().numpy(), gi, ng)
    assert ec <= max(1, n // 8) and eg <= max(1, n // 4), (cfg, n, ec, eg)
    O_ref, LSE_ref = oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], gi, ng)
    assert np.max(np.abs(bf16_to_f64(buf.O) - O_ref)) <= TOL_O, cfg
    assert np.max(np.abs(buf.LSE.cpu().numpy().astype(np.float64) - LSE_ref)) <= TOL_LSE, cfg
