"""Host-side pieces of bench.py that need no GPU: the work counts behind the roofline objects and the
measured-traffic table."""
import importlib.util
import os

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bench():
    spec = importlib.util.spec_from_file_location("hga_bench", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_traffic_table_names_its_capture(bench):
    calls, src = bench.load_traffic(3)
    assert src and src["commit"] and src["captured"]
    for call in ("hga_attn_fwd", "hga_attn_bwd"):
        assert calls[call] > 0
    # a call's figure is the sum over its kernels
    k = src["kernels"]
    total = lambda names: sum(k[n]["dram_read"] + k[n]["dram_write"] for n in names)
    assert calls["hga_attn_fwd"] == total(["k_attn_fwd_sm100"])
    assert calls["hga_attn_bwd"] == total(["k_attn_bwd_band_sm100", "k_attn_bwd_sm100"])
    assert bench.load_traffic(99) == ({}, None)


def test_route_work_counts_candidates_and_opened_groups(bench):
    from paper_2607_15105_b200.workloads import CONFIGS
    cfg = CONFIGS[3]
    flops, nbytes = bench.route_work(cfg)
    # every block of configuration 3 sees at least 221 closed candidate chunks and opens 16 chunks of 8 groups
    rows, d = cfg.gqa * cfg.q_block, cfg.head_dim
    items = cfg.batch * cfg.n_kv_heads * cfg.n_q_blocks
    assert flops >= items * 2.0 * d * rows * (221 + 16 * 8)
    assert nbytes >= items * (221 + 16 * 8) * d * 2
