"""hga_route_static: the routing entry point for callers that may not allocate device memory
(plug-ins running under a locked or exhausted framework allocator, loops that must never enter
cudaMalloc, processes with a start-up memory budget).  Its scratch is a fixed array inside the
library, so the test checks, through the C ABI, that it selects exactly what hga_route selects
-- twice in a row, because the array keeps the previous call's contents -- and that it refuses
a problem larger than the array.  Collected last on purpose: a run that stops at the first
failure has then already run every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2607_15105_b200 import binding
from paper_2607_15105_b200.workloads import CONFIGS, HgaConfig, make_inputs

pytestmark = pytest.mark.gpu


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _route_both_ways(cfg, seed_shift=0, flags=0):
    """Indices from hga_route (caller workspace) and from hga_route_static (no allocation)."""
    x = make_inputs(cfg.scaled(seed=cfg.seed + seed_shift), with_dO=False)
    Q, K = _dev(x["Q"]), _dev(x["K"])
    ref = binding.HgaLayerBuffers(cfg, backward=False, want_scores=True, flags=flags)
    ref.build_summaries(K, 0, cfg.total_len)
    ref.route(Q)
    # every buffer the static call touches exists before it runs; the call itself gets no workspace
    chunk_idx = torch.full_like(ref.chunk_idx, -7)
    group_idx = torch.full_like(ref.group_idx, -7)
    n_groups = torch.full_like(ref.n_groups, -7)
    binding.hga_route_static(ref.p, Q, ref.chunk_sum, ref.group_sum, chunk_idx, group_idx, n_groups)
    torch.cuda.synchronize()
    return ref, (chunk_idx, group_idx, n_groups)


def test_static_route_matches_route_on_two_calls_in_a_row():
    # two different problems back to back: the second call finds the first one's scores in the
    # shared array and must not be influenced by them (indices are integers: exact equality)
    small = HgaConfig("static_small", 2, 4, 2, 128, 1536, 512, 64, 8, 64, 5, 3, 64, 128,
                      topics=16, needles=4, backward=False, seed=23)
    for cfg, shift in ((CONFIGS[3], 0), (small, 0), (CONFIGS[3], 1)):
        # against hga_route running the same (shape-generic) kernels: exact
        ref, (ci, gi, ng) = _route_both_ways(cfg, shift, flags=binding.HGA_FLAG_GENERIC_KERNELS)
        assert torch.equal(ci, ref.chunk_idx)
        assert torch.equal(gi, ref.group_idx)
        assert torch.equal(ng, ref.n_groups)
        assert int(ng.min()) >= 0
        # against hga_route's default kernels (another fp32 summation order): the routing
        # tolerance of the parity tests -- sets may differ only at score gaps below 1e-3
        dflt, (ci, gi, ng) = _route_both_ways(cfg, shift)
        assert torch.equal(ng, dflt.n_groups)
        _same_up_to_near_ties(cfg, dflt, ci.cpu().numpy(), gi.cpu().numpy())


def _same_up_to_near_ties(cfg, ref, ci, gi, gap=1e-3):
    r_ci, r_gi = ref.chunk_idx.cpu().numpy(), ref.group_idx.cpu().numpy()
    cs, gs = ref.chunk_scores.cpu().numpy(), ref.group_scores.cpu().numpy()
    per = cfg.chunk // cfg.group
    flat = lambda a: a.reshape(-1, a.shape[-1])
    for it, (a, b, c, d, sc, sg) in enumerate(zip(flat(r_ci), flat(ci), flat(r_gi), flat(gi), flat(cs), flat(gs))):
        sa, sb = set(a[a >= 0].tolist()), set(b[b >= 0].tolist())
        assert len(sa) == len(sb)
        if sa != sb:
            kth = min(sc[j] for j in sa)
            assert all(abs(sc[j] - kth) < gap for j in sa ^ sb), (it, sa ^ sb)
        ga, gb = set(c[c >= 0].tolist()), set(d[d >= 0].tolist())
        for r, j in enumerate(sorted(sa)):
            if j not in sb:
                continue
            ca, cb = {m for m in ga if m // per == j}, {m for m in gb if m // per == j}
            if ca != cb:
                s = sg[r * per:(r + 1) * per]
                kth = min(s[m - j * per] for m in ca)
                assert all(abs(s[m - j * per] - kth) < gap for m in ca ^ cb), (it, j, ca ^ cb)


def test_static_route_allocates_nothing_after_its_first_call():
    """The first call on a device makes CUDA place the library's fixed array in device memory; from the
    second call on, the free device memory is the same before and after a call (no allocation, no free),
    on a shape the fused router takes and on one that needs the array."""
    small = HgaConfig("static_small", 2, 4, 2, 128, 1536, 512, 64, 8, 64, 5, 3, 64, 128,
                      topics=16, needles=4, backward=False, seed=23)
    odd = HgaConfig("static_g16", 1, 2, 1, 64, 1024, 256, 64, 16, 64, 4, 2, 64, 64,
                    topics=8, needles=0, backward=False, seed=24)     # 4 groups per chunk: CUDA-core router + the array
    for cfg in (small, odd):
        x = make_inputs(cfg, with_dO=False)
        Q, K = _dev(x["Q"]), _dev(x["K"])
        buf = binding.HgaLayerBuffers(cfg, backward=False)
        buf.build_summaries(K, 0, cfg.total_len)
        call = lambda: binding.hga_route_static(buf.p, Q, buf.chunk_sum, buf.group_sum, buf.chunk_idx,
                                                buf.group_idx, buf.n_groups)
        before = binding.hga_kernel_launch_counts()
        call()                                   # may be the device's first call: set-up happens here
        torch.cuda.synchronize()
        ran = [b - a for a, b in zip(before, binding.hga_kernel_launch_counts())]
        tensor = cfg is small
        assert (ran[binding.HGA_KERNELS_ROUTE_TENSOR] == 1) == tensor, ran
        assert (ran[binding.HGA_KERNELS_ROUTE_GENERIC] > 0) == (not tensor), ran
        free0 = torch.cuda.mem_get_info()[0]
        for _ in range(3):
            call()
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free0
        buf.route(Q)                             # hga_route with a caller workspace selects the same
        ref = (buf.chunk_idx.clone(), buf.group_idx.clone(), buf.n_groups.clone())
        call()
        torch.cuda.synchronize()
        assert all(torch.equal(a, b) for a, b in zip(ref, (buf.chunk_idx, buf.group_idx, buf.n_groups)))


def test_static_route_refuses_problems_beyond_its_array():
    # 8 sequences of the 128K evaluation shape need 16 MiB of scores: more than the fixed array
    big = CONFIGS[4].scaled(batch=8)
    p = binding.make_params(big)
    need, _ = binding.hga_workspace_bytes(p)
    assert need > binding.HGA_ROUTE_STATIC_SCRATCH_BYTES
    dummy = torch.zeros(64, dtype=torch.int32, device="cuda")
    before = binding.hga_kernel_launch_count()
    rc = binding.lib().hga_route_static(C.byref(p), C.c_void_p(dummy.data_ptr()), C.c_void_p(dummy.data_ptr()),
                                        C.c_void_p(dummy.data_ptr()), C.c_void_p(dummy.data_ptr()),
                                        C.c_void_p(dummy.data_ptr()), C.c_void_p(dummy.data_ptr()), None)
    assert rc == -5                                      # HGA_ERR_WORKSPACE
    assert binding.hga_kernel_launch_count() == before   # nothing was launched
    # the largest benchmark shapes do fit
    for n in (3, 4, 5):
        assert binding.hga_workspace_bytes(binding.make_params(CONFIGS[n]))[0] <= binding.HGA_ROUTE_STATIC_SCRATCH_BYTES
