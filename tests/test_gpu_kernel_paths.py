"""Paths of the tensor-core kernels that the shape sweeps do not reach by themselves, each against
the oracle: accumulation into existing dK/dV on a head_dim-128 problem (local-band kernel plus routed
sweep), chunks narrower than the band kernel's key tile (band edges fall inside a tile), an item the
router gave up on (n_groups = -1), which kernel family a call took, and the bounded on-chip wait
running out."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_15105_b200 import binding
from paper_2607_15105_b200.workloads import HgaConfig, make_inputs

from hga_testlib import TOL_LSE, TOL_O, bf16_to_f64, check_grads, rel_fro, to_dev

pytestmark = pytest.mark.gpu

FAMILY_FLAGS = [0, binding.HGA_FLAG_GENERIC_KERNELS]


def cfg_of(**kw):
    base = dict(name="paths", batch=2, n_q_heads=4, n_kv_heads=2, head_dim=128, total_len=1536, seg_len=512,
                chunk=64, group=8, q_block=64, topk_chunks=5, topk_groups=3, sink=64, local=128, topics=16,
                needles=4, backward=True, seed=29)
    base.update(kw)
    return HgaConfig(**base)


class Problem:
    def __init__(self, cfg):
        self.cfg = cfg
        self.x = x = make_inputs(cfg)
        self.Q, self.K, self.V, self.dO = (to_dev(x[n]) for n in ("Q", "K", "V", "dO"))
        cs, gs = oracle.build_summaries(cfg, x["K"])
        self.ref = oracle.route(cfg, x["Q"], cs, gs)
        self.gi_np, self.ng_np = self.ref["group_idx"], self.ref["n_groups"]
        self.gi, self.ng = torch.from_numpy(self.gi_np).cuda(), torch.from_numpy(self.ng_np).cuda()

    def oracle_fwd(self, gi=None, ng=None):
        x = self.x
        return oracle.attn_fwd(self.cfg, x["Q"], x["K"], x["V"], self.gi_np if gi is None else gi,
                               self.ng_np if ng is None else ng)

    def oracle_bwd(self, gi=None, ng=None):
        x = self.x
        return oracle.attn_bwd(self.cfg, x["Q"], x["K"], x["V"], x["dO"], self.gi_np if gi is None else gi,
                               self.ng_np if ng is None else ng)


def grads_of(buf):
    return (bf16_to_f64(buf.dQ), buf.dK.cpu().numpy().astype(np.float64), buf.dV.cpu().numpy().astype(np.float64))


def launches(fn):
    """Kernel launches per family made by fn()."""
    before = binding.hga_kernel_launch_counts()
    fn()
    return [b - a for a, b in zip(before, binding.hga_kernel_launch_counts())]


def test_accumulate_flag_on_the_tensor_core_backward():
    """HGA_FLAG_BWD_ACCUMULATE with head_dim 128: the band kernel reads, adds and stores, the sweep
    adds atomically.  Starting from dK = dV = the oracle's gradients, the result is twice them."""
    pr = Problem(cfg_of())
    cfg = pr.cfg
    dQ, dK, dV = pr.oracle_bwd()
    buf = binding.HgaLayerBuffers(cfg, flags=binding.HGA_FLAG_BWD_ACCUMULATE)
    buf.attn_fwd(pr.Q, pr.K, pr.V, pr.gi, pr.ng)
    buf.dK.copy_(torch.from_numpy(dK.astype(np.float32)))
    buf.dV.copy_(torch.from_numpy(dV.astype(np.float32)))
    n = launches(lambda: buf.attn_bwd(pr.Q, pr.K, pr.V, pr.dO, pr.gi, pr.ng))
    torch.cuda.synchronize()
    assert n[binding.HGA_KERNELS_BWD_TENSOR] >= 2 and n[binding.HGA_KERNELS_BWD_GENERIC] == 0
    assert int(buf.status.item()) == 0
    check_grads(grads_of(buf), (dQ, 2 * dK, 2 * dV), "accumulate")
    # and once more on top: three times
    buf.attn_bwd(pr.Q, pr.K, pr.V, pr.dO, pr.gi, pr.ng)
    torch.cuda.synchronize()
    check_grads(grads_of(buf), (dQ, 3 * dK, 3 * dV), "accumulate twice")


@pytest.mark.parametrize("accumulate", [False, True])
def test_band_edges_inside_a_key_tile(accumulate):
    """c = 32, local 96: the local windows start at multiples of 32, i.e. inside the band kernel's key
    tiles; routed keys of the active segment before the band get their gradients from the sweep's
    atomic adds.  dK/dV must be overwritten (or,
    with the accumulate flag, added to)."""
    pr = Problem(cfg_of(chunk=32, group=8, q_block=64, sink=64, local=96, topk_chunks=6, topk_groups=2,
                        total_len=1024, seg_len=384, seed=31))
    cfg = pr.cfg
    dQ, dK, dV = pr.oracle_bwd()
    O, LSE = pr.oracle_fwd()
    buf = binding.HgaLayerBuffers(cfg, flags=binding.HGA_FLAG_BWD_ACCUMULATE if accumulate else 0)
    buf.attn_fwd(pr.Q, pr.K, pr.V, pr.gi, pr.ng)
    if accumulate:
        buf.dK.copy_(torch.from_numpy(dK.astype(np.float32)))
        buf.dV.copy_(torch.from_numpy(dV.astype(np.float32)))
    else:
        buf.dK.fill_(7.0)      # must be overwritten, not added to
        buf.dV.fill_(-7.0)
    n = launches(lambda: buf.attn_bwd(pr.Q, pr.K, pr.V, pr.dO, pr.gi, pr.ng))
    torch.cuda.synchronize()
    assert n[binding.HGA_KERNELS_BWD_TENSOR] == 2 and n[binding.HGA_KERNELS_BWD_GENERIC] == 0
    assert int(buf.status.item()) == 0
    assert np.max(np.abs(bf16_to_f64(buf.O) - O)) <= TOL_O
    k = 2 if accumulate else 1
    check_grads(grads_of(buf), (dQ, k * dK, k * dV), "narrow chunks")


@pytest.mark.parametrize("flags", FAMILY_FLAGS)
def test_item_the_router_gave_up_on_gets_sink_and_local_only(flags):
    """n_groups = -1 is the router's mark for an item whose routing could not be completed; its index
    lists are then stale.  The attention calls must treat the item as having no routed groups (sink and
    local window only) and report HGA_STATUS_BAD_INDEX."""
    pr = Problem(cfg_of(seed=37))
    cfg = pr.cfg
    gi, ng = pr.gi_np.copy(), pr.ng_np.copy()
    marked = [(0, 1, cfg.n_q_blocks - 1), (1, 0, cfg.n_q_blocks - 2)]
    clean_gi, clean_ng = gi.copy(), ng.copy()
    rng = np.random.default_rng(5)
    for b, h, qb in marked:
        ng[b, h, qb] = -1
        gi[b, h, qb] = rng.integers(-50, 10 ** 6, size=gi.shape[-1])      # garbage: must never be read as indices
        clean_ng[b, h, qb] = 0
        clean_gi[b, h, qb] = -1
    O, LSE = pr.oracle_fwd(clean_gi, clean_ng)
    ref_grads = pr.oracle_bwd(clean_gi, clean_ng)
    buf = binding.HgaLayerBuffers(cfg, flags=flags)
    gid, ngd = torch.from_numpy(gi).cuda(), torch.from_numpy(ng).cuda()
    buf.attn_fwd(pr.Q, pr.K, pr.V, gid, ngd)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == binding.HGA_STATUS_BAD_INDEX
    assert np.max(np.abs(bf16_to_f64(buf.O) - O)) <= TOL_O
    assert np.max(np.abs(buf.LSE.cpu().numpy().astype(np.float64) - LSE)) <= TOL_LSE
    buf.status.zero_()
    buf.attn_bwd(pr.Q, pr.K, pr.V, pr.dO, gid, ngd)
    torch.cuda.synchronize()
    assert int(buf.status.item()) & ~binding.HGA_STATUS_BAD_INDEX == 0
    check_grads(grads_of(buf), ref_grads, "n_groups = -1")


@pytest.mark.parametrize("flags", FAMILY_FLAGS)
def test_late_dominant_key_raises_the_softmax_reference_mid_sweep(flags):
    """A key late in the routed order (the last position of the local window before the block) whose
    logit lies ~98 binary orders above every other key's: the forward kernel, which takes the exponentials
    of later tiles against the reference of earlier ones, must notice that this tile alone would leave
    the exponent range and fall back to the tile's own maximum.  Exact answer: O ~ that key's value row."""
    cfg = cfg_of(seed=41, batch=1)
    x = make_inputs(cfg)
    from paper_2607_15105_b200.workloads import f32_to_bf16_bits
    H, Bq = cfg.history, cfg.q_block
    K = x["K"].copy()
    Q = x["Q"].copy()
    one = lambda v: f32_to_bf16_bits(np.array([v], np.float32))[0]
    for h in range(cfg.n_kv_heads):
        K[0, h, :, 0] = 0                                   # component 0 belongs to the planted pair alone
    qb = cfg.n_q_blocks - 1                                 # the last block, both kv heads: no later block sees the key
    kpos = H + qb * Bq - 1
    K[0, :, kpos, 0] = one(48.0)
    Q[0, :, qb * Bq:(qb + 1) * Bq, 0] = one(16.0)           # 16 * 48 / sqrt(128) = 67.9 nats = 98 in log2
    x = dict(x, K=K, Q=Q)
    cs, gs = oracle.build_summaries(cfg, K)
    ref = oracle.route(cfg, Q, cs, gs)
    gi, ng = ref["group_idx"], ref["n_groups"]
    O, LSE = oracle.attn_fwd(cfg, Q, K, x["V"], gi, ng)
    buf = binding.HgaLayerBuffers(cfg, backward=False, flags=flags)
    buf.attn_fwd(to_dev(Q), to_dev(K), to_dev(x["V"]), torch.from_numpy(gi).cuda(), torch.from_numpy(ng).cuda())
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    assert float(LSE.max()) > 60.0                          # the planted logit is really there
    assert np.max(np.abs(bf16_to_f64(buf.O) - O)) <= TOL_O
    assert np.max(np.abs(buf.LSE.cpu().numpy().astype(np.float64) - LSE)) <= TOL_LSE


def test_backward_next_to_another_stream_never_misses_a_barrier_phase():
    """The backward kernels hand tiles over through mbarrier phases; a waiter that is late must still
    find the phase it waits for.  Running the backward while another stream keeps the GPU busy (the
    way hga_tbptt_walk overlaps one segment's backward with the next segment's forward) stretches those
    delays: every call must finish in its usual time with a clean status word, and with the same dQ."""
    import time
    pr = Problem(cfg_of(batch=1, n_q_heads=32, n_kv_heads=8, total_len=4096, seg_len=2048, topk_chunks=16,
                        topk_groups=4, topics=64, needles=8, seed=43))
    cfg = pr.cfg
    a, b = binding.HgaLayerBuffers(cfg), binding.HgaLayerBuffers(cfg)
    for buf in (a, b):
        buf.build_summaries(pr.K, 0, cfg.total_len)
        buf.route(pr.Q)
        buf.attn_fwd(pr.Q, pr.K, pr.V)
    a.attn_bwd(pr.Q, pr.K, pr.V, pr.dO)
    torch.cuda.synchronize()
    first = a.dQ.clone()
    side = torch.cuda.Stream()
    for it in range(25):
        t0 = time.time()
        for _ in range(8):
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                a.attn_bwd(pr.Q, pr.K, pr.V, pr.dO)
            b.build_summaries(pr.K)
            b.route(pr.Q)
            b.attn_fwd(pr.Q, pr.K, pr.V)
            torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        assert time.time() - t0 < 0.25, "a bounded wait ran out (each takes about half a second)"
        assert int(a.status.item()) == 0 and int(b.status.item()) == 0
    assert torch.equal(a.dQ, first)


def test_kernel_families_are_counted_per_call():
    pr = Problem(cfg_of())
    cfg = pr.cfg
    T = binding
    for flags, fams in ((0, (T.HGA_KERNELS_ROUTE_TENSOR, T.HGA_KERNELS_FWD_TENSOR, T.HGA_KERNELS_BWD_TENSOR)),
                        (T.HGA_FLAG_GENERIC_KERNELS, (T.HGA_KERNELS_ROUTE_GENERIC, T.HGA_KERNELS_FWD_GENERIC,
                                                      T.HGA_KERNELS_BWD_GENERIC))):
        buf = binding.HgaLayerBuffers(cfg, flags=flags)
        total0 = binding.hga_kernel_launch_count()
        n = launches(lambda: buf.step(pr.Q, pr.K, pr.V, pr.dO))
        torch.cuda.synchronize()
        assert n[T.HGA_KERNELS_SUMMARIES] == 1
        assert all(n[f] >= 1 for f in fams), n
        assert sum(n) == sum(n[f] for f in fams) + 1, n       # nothing from the other family
        assert binding.hga_kernel_launch_count() - total0 == sum(n)
    assert binding.lib().hga_kernel_launch_count_by_family(99) == -1


def test_bounded_wait_runs_out_and_reports():
    """A wait on a barrier nothing completes, with a limit of 2^20 SM cycles (about half a millisecond):
    the kernel must return, set HGA_STATUS_WAIT_TIMEOUT, and leave the context usable."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    limit = 1 << 20
    binding.hga_selftest_bounded_wait(limit, status, waited)
    torch.cuda.synchronize()
    assert int(status.item()) == binding.HGA_STATUS_WAIT_TIMEOUT
    assert limit <= int(waited.item()) < 64 * limit
    # the context still works, and a status word that already holds a bit keeps it
    status.fill_(binding.HGA_STATUS_BAD_INDEX)
    binding.hga_selftest_bounded_wait(1 << 16, status)
    torch.cuda.synchronize()
    assert int(status.item()) == binding.HGA_STATUS_BAD_INDEX | binding.HGA_STATUS_WAIT_TIMEOUT
    assert float(torch.ones(8, device="cuda").sum().item()) == 8.0
    with pytest.raises(binding.HgaError):
        binding.hga_selftest_bounded_wait(0, status)
    with pytest.raises(binding.HgaError):
        binding.hga_selftest_bounded_wait((1 << 24) + 1, status)
