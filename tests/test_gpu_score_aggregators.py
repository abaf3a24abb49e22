"""HGA_FLAG_SCORE_MEAN / HGA_FLAG_SCORE_LSE: the query block's score of a summary as the mean or the
log-sum-exp over its rows instead of the maximum.  Routing (both routers) against the oracle's
variant of the same aggregator, and the score outputs themselves."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_15105_b200 import binding
from paper_2607_15105_b200.workloads import CONFIGS, make_inputs

from hga_testlib import check_routing, to_dev
from test_gpu_parity import SMALL_CASES, small

pytestmark = pytest.mark.gpu

AGGS = {"mean": binding.HGA_FLAG_SCORE_MEAN, "lse": binding.HGA_FLAG_SCORE_LSE}


def routed(cfg, x, cs, gs, flags, want_scores=True):
    buf = binding.HgaLayerBuffers(cfg, backward=False, want_scores=want_scores, flags=flags)
    buf.chunk_sum.copy_(to_dev(cs))
    buf.group_sum.copy_(to_dev(gs))
    buf.route(to_dev(x["Q"]))
    torch.cuda.synchronize()
    return buf


@pytest.mark.parametrize("generic", [0, binding.HGA_FLAG_GENERIC_KERNELS])
@pytest.mark.parametrize("agg", list(AGGS))
@pytest.mark.parametrize("name", list(SMALL_CASES))
def test_route_matches_oracle(name, agg, generic):
    cfg = SMALL_CASES[name]
    x = make_inputs(cfg)
    cs, gs = oracle.build_summaries(cfg, x["K"])
    ref = oracle.route(cfg, x["Q"], cs, gs, want_scores=True, score_agg=agg)
    buf = routed(cfg, x, cs, gs, AGGS[agg] | generic)
    ci = buf.chunk_idx.cpu().numpy()
    n, ec, eg = check_routing(cfg, ref, ci, buf.group_idx.cpu().numpy(), buf.n_groups.cpu().numpy())
    assert ec <= max(1, n // 10) and eg <= max(1, n // 5), (n, ec, eg)
    got = buf.chunk_scores.cpu().numpy().astype(np.float64)
    fin = np.isfinite(ref["chunk_scores"])
    assert np.array_equal(np.isfinite(got), fin)
    assert np.max(np.abs(got[fin] - ref["chunk_scores"][fin]), initial=0) < 2e-4
    if np.array_equal(ci, ref["chunk_idx"]):
        gsc = buf.group_scores.cpu().numpy().astype(np.float64)
        fin = np.isfinite(ref["group_scores"])
        assert np.max(np.abs(gsc[fin] - ref["group_scores"][fin]), initial=0) < 2e-4
    # the aggregator must matter on this input (topic-structured cases), or the test shows nothing
    # (log-sum-exp may legitimately pick the maximum's chunks where one row dominates)
    if cfg.topics and agg == "mean":
        by_max = oracle.route(cfg, x["Q"], cs, gs)
        assert not (np.array_equal(ref["chunk_idx"], by_max["chunk_idx"]) and
                    np.array_equal(ref["group_idx"], by_max["group_idx"]))


@pytest.mark.parametrize("agg", list(AGGS))
def test_headline_config_sampled_items(agg):
    cfg = CONFIGS[3]
    x = make_inputs(cfg)
    cs, gs = oracle.build_summaries(cfg, x["K"])
    nqb = cfg.n_q_blocks
    items = sorted({0, 5, nqb - 1, 2 * nqb + 3, 5 * nqb + 17, cfg.n_items - 1})
    ref = oracle.route(cfg, x["Q"], cs, gs, items=items, want_scores=True, score_agg=agg)
    buf = routed(cfg, x, cs, gs, AGGS[agg], want_scores=False)
    n, ec, eg = check_routing(cfg, ref, buf.chunk_idx.cpu().numpy(), buf.group_idx.cpu().numpy(),
                              buf.n_groups.cpu().numpy(), items=items)
    assert n == len(items) and ec <= 1 and eg <= 2, (n, ec, eg)


def test_both_aggregator_flags_are_rejected():
    p = binding.make_params(small(), flags=binding.HGA_FLAG_SCORE_MEAN | binding.HGA_FLAG_SCORE_LSE)
    with pytest.raises(binding.HgaError):
        binding.hga_workspace_bytes(p)
