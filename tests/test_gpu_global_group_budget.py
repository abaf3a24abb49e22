"""HGA_FLAG_GLOBAL_GROUP_BUDGET: Section 2.1 item 2 read as one budget of (opened chunks x k_g)
groups over all opened chunks together.  The library's routing is compared with the oracle's
variant of the same reading, and the attention kernels run on the lists it produced (their
per-chunk counts are no longer uniform)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_15105_b200 import binding
from paper_2607_15105_b200.workloads import CONFIGS, make_inputs

from hga_testlib import (TOL_GRAD, TOL_LSE, TOL_O, bf16_to_f64, check_routing, item_rows, rel_fro, to_dev)
from test_gpu_parity import SMALL_CASES, small

pytestmark = pytest.mark.gpu

GB = binding.HGA_FLAG_GLOBAL_GROUP_BUDGET
FLAG_SETS = [GB, GB | binding.HGA_FLAG_GENERIC_KERNELS]


@pytest.mark.parametrize("flags", FLAG_SETS)
@pytest.mark.parametrize("name", list(SMALL_CASES))
def test_route_and_attention_match_oracle(name, flags):
    cfg = SMALL_CASES[name]
    x = make_inputs(cfg)
    cs, gs = oracle.build_summaries(cfg, x["K"])
    ref = oracle.route(cfg, x["Q"], cs, gs, want_scores=True, global_group_budget=True)
    buf = binding.HgaLayerBuffers(cfg, want_scores=True, flags=flags)
    buf.chunk_sum.copy_(to_dev(cs))
    buf.group_sum.copy_(to_dev(gs))
    Q, K, V, dO = to_dev(x["Q"]), to_dev(x["K"]), to_dev(x["V"]), to_dev(x["dO"])
    buf.route(Q)
    torch.cuda.synchronize()
    gi, ng = buf.group_idx.cpu().numpy(), buf.n_groups.cpu().numpy()
    n, ec, eg = check_routing(cfg, ref, buf.chunk_idx.cpu().numpy(), gi, ng, global_budget=True)
    assert ec <= max(1, n // 10) and eg <= max(1, n // 5), (n, ec, eg)
    # the variant must really differ from the per-chunk rule somewhere, or the test shows nothing
    per_chunk = oracle.route(cfg, x["Q"], cs, gs)
    if min(cfg.topk_groups, cfg.chunk // cfg.group) < cfg.chunk // cfg.group and cfg.topk_chunks > 1:
        assert not np.array_equal(per_chunk["group_idx"], ref["group_idx"])
    gsc = buf.group_scores.cpu().numpy().astype(np.float64)
    fin = np.isfinite(ref["group_scores"])
    if np.array_equal(buf.chunk_idx.cpu().numpy(), ref["chunk_idx"]):
        assert np.max(np.abs(gsc[fin] - ref["group_scores"][fin]), initial=0) < 2e-4
    # attention on the lists the library produced
    buf.attn_fwd(Q, K, V)
    buf.attn_bwd(Q, K, V, dO)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    O_ref, LSE_ref = oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], gi, ng)
    dQ_ref, dK_ref, dV_ref = oracle.attn_bwd(cfg, x["Q"], x["K"], x["V"], x["dO"], gi, ng)
    assert np.max(np.abs(bf16_to_f64(buf.O) - O_ref)) <= TOL_O
    assert np.max(np.abs(buf.LSE.cpu().numpy().astype(np.float64) - LSE_ref)) <= TOL_LSE
    assert rel_fro(bf16_to_f64(buf.dQ), dQ_ref) <= TOL_GRAD
    assert rel_fro(buf.dK.cpu().numpy().astype(np.float64), dK_ref) <= TOL_GRAD
    assert rel_fro(buf.dV.cpu().numpy().astype(np.float64), dV_ref) <= TOL_GRAD


def test_exact_ties_across_chunks_go_to_the_lowest_group_id():
    """Constant keys make every summary equal, so every group score ties: the budget must then
    fall on the lowest group ids of the opened chunks, exactly (no near-tie excuse applies)."""
    cfg = small(batch=1, n_q_heads=2, n_kv_heads=1, total_len=1024, seg_len=256, topics=0, needles=0)
    x = make_inputs(cfg)
    x["K"][...] = x["K"][0, 0, 0][None, None, None, :]
    cs, gs = oracle.build_summaries(cfg, x["K"])
    ref = oracle.route(cfg, x["Q"], cs, gs, global_group_budget=True)
    for flags in FLAG_SETS:
        buf = binding.HgaLayerBuffers(cfg, backward=False, flags=flags)
        buf.chunk_sum.copy_(to_dev(cs))
        buf.group_sum.copy_(to_dev(gs))
        buf.route(to_dev(x["Q"]))
        torch.cuda.synchronize()
        assert np.array_equal(buf.chunk_idx.cpu().numpy(), ref["chunk_idx"])
        assert np.array_equal(buf.group_idx.cpu().numpy(), ref["group_idx"])
        assert np.array_equal(buf.n_groups.cpu().numpy(), ref["n_groups"])


def test_headline_config_sampled_items():
    cfg = CONFIGS[3]
    x = make_inputs(cfg)
    cs, gs = oracle.build_summaries(cfg, x["K"])
    nqb = cfg.n_q_blocks
    items = sorted({0, 1, nqb - 1, nqb, 3 * nqb + 7, cfg.n_items - 1, cfg.n_items - nqb})
    ref = oracle.route(cfg, x["Q"], cs, gs, items=items, want_scores=True, global_group_budget=True)
    buf = binding.HgaLayerBuffers(cfg, backward=False, flags=GB)
    buf.chunk_sum.copy_(to_dev(cs))
    buf.group_sum.copy_(to_dev(gs))
    Q, K, V = to_dev(x["Q"]), to_dev(x["K"]), to_dev(x["V"])
    buf.route(Q)
    torch.cuda.synchronize()
    gi, ng = buf.group_idx.cpu().numpy(), buf.n_groups.cpu().numpy()
    n, ec, eg = check_routing(cfg, ref, buf.chunk_idx.cpu().numpy(), gi, ng, items=items, global_budget=True)
    assert n == len(items) and ec <= 1 and eg <= 2, (n, ec, eg)
    buf.attn_fwd(Q, K, V)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    O_ref, _ = oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], gi, ng, items=items)
    bi, hi, si = item_rows(cfg, items)
    assert np.max(np.abs(bf16_to_f64(buf.O)[bi, hi, si] - O_ref[bi, hi, si])) <= TOL_O


def test_budget_too_large_is_rejected():
    """The selection holds one bit per (opened chunk, group) slot: at most 4096 of them."""
    kw = dict(chunk=64, group=1, q_block=64, total_len=8192, seg_len=512, sink=64, local=64, topk_groups=2)
    binding.hga_workspace_bytes(binding.make_params(small(topk_chunks=64, **kw), flags=GB))
    with pytest.raises(binding.HgaError):
        binding.hga_workspace_bytes(binding.make_params(small(topk_chunks=65, **kw), flags=GB))
    binding.hga_workspace_bytes(binding.make_params(small(topk_chunks=65, **kw)))
