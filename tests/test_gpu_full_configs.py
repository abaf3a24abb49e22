"""The benchmark configurations at full size, in the launch configuration bench.py times:
the whole path runs on the GPU; the oracle recomputes sampled items (all query blocks of one
(batch, kv head) so that its dK/dV rows are complete, plus a few scattered items)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_15105_b200 import binding
from paper_2607_15105_b200.workloads import CONFIGS, make_inputs

from hga_testlib import (TOL_GRAD, TOL_GRAD_ROW, TOL_LSE, TOL_O, bf16_to_f64, bits_of, check_routing,
                         item_rows, rel_fro, row_err_ratio, to_dev)

pytestmark = pytest.mark.gpu


def sample_items(cfg, full_head, extra, seed):
    """All items of one (b, h) plus `extra` random others."""
    nqb = cfg.n_q_blocks
    b, h = full_head
    head = [((b * cfg.n_kv_heads + h) * nqb) + qb for qb in range(nqb)]
    rng = np.random.default_rng(seed)
    rest = [int(i) for i in rng.choice(cfg.n_items, size=min(extra, cfg.n_items), replace=False)]
    return head, sorted(set(head) | set(rest))


# routed keys per item (a data-independent count) for the last query block of each config
ROUTED_KEYS_LAST_BLOCK = {1: 320, 2: 512, 3: 768, 4: 768, 5: 2560, 6: 768}
# per configuration: (items that may carry an excused chunk, chunks that may carry an excused group).  Observed
# on the sampled items: none on any configuration (the counts are printed); one is allowed for a change of
# accumulation order, two on the i.i.d. configuration 5, where near ties are the most likely.
EXCUSED_BOUNDS = {1: (1, 1), 2: (1, 1), 3: (1, 1), 4: (1, 1), 5: (2, 2), 6: (1, 1)}


@pytest.mark.parametrize("n,full_head,extra", [(1, (0, 0), 4), (2, (0, 5), 12), (3, (0, 3), 12),
                                               (4, (0, 6), 0), (5, (2, 5), 0), (6, (0, 1), 8)])
def test_config_against_oracle(n, full_head, extra):
    cfg = CONFIGS[n]
    x = make_inputs(cfg)
    Q, K, V = to_dev(x["Q"]), to_dev(x["K"]), to_dev(x["V"])
    dO = to_dev(x["dO"]) if cfg.backward else None
    buf = binding.HgaLayerBuffers(cfg, backward=cfg.backward)
    # history summaries come from earlier segments; the step itself adds the active range
    buf.build_summaries(K, 0, cfg.history)
    before = binding.hga_kernel_launch_counts()
    buf.step(Q, K, V, dO)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    # which kernels ran: the tensor-core router and forward on every configuration, the tensor-core
    # backward wherever head_dim is 128 (configuration 1 has head_dim 64: its backward is the CUDA-core one)
    ran = [b - a for a, b in zip(before, binding.hga_kernel_launch_counts())]
    T = binding
    assert ran[T.HGA_KERNELS_ROUTE_TENSOR] == 1 and ran[T.HGA_KERNELS_ROUTE_GENERIC] == 0, ran
    assert ran[T.HGA_KERNELS_FWD_TENSOR] == 1 and ran[T.HGA_KERNELS_FWD_GENERIC] == 0, ran
    if cfg.backward:
        tensor_bwd = cfg.head_dim == 128
        assert (ran[T.HGA_KERNELS_BWD_TENSOR] >= 2) == tensor_bwd and (ran[T.HGA_KERNELS_BWD_GENERIC] == 0) == tensor_bwd, ran
    head, items = sample_items(cfg, full_head, extra, seed=n)
    if n == 4:
        head, items = [], head[::2]          # forward only: 16 items are plenty

    # summaries: bit exact, everywhere
    cs, gs = oracle.build_summaries(cfg, x["K"])
    assert np.array_equal(bits_of(buf.chunk_sum), cs)
    assert np.array_equal(bits_of(buf.group_sum), gs)

    # routing on the sampled items
    ref = oracle.route(cfg, x["Q"], cs, gs, items=items, want_scores=True)
    gi, ng = buf.group_idx.cpu().numpy(), buf.n_groups.cpu().numpy()
    checked, ec, eg = check_routing(cfg, ref, buf.chunk_idx.cpu().numpy(), gi, ng, items=items)
    print("config %d: %d items checked, %d with an excused chunk, %d chunks with an excused group" % (n, checked, ec, eg))
    # near ties (score gap < 1e-3 at the k-th place) are rare where keys have topic structure; the i.i.d.
    # configuration 5 is the near-tie-heavy one (about one block in ten has such a gap at the chunk level)
    max_ec, max_eg = EXCUSED_BOUNDS[n]
    assert ec <= max_ec and eg <= max_eg, (checked, ec, eg)
    # data-independent counts, everywhere
    keys = cfg.sink + ng[:, :, -1] * cfg.group + cfg.local + cfg.q_block
    assert np.all(keys == ROUTED_KEYS_LAST_BLOCK[n])

    # attention on the GPU's own indices (the oracle takes the same lists)
    O, LSE = oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], gi, ng, items=items)
    bi, hi, si = item_rows(cfg, items)
    assert np.max(np.abs(bf16_to_f64(buf.O)[bi, hi, si] - O[bi, hi, si])) <= TOL_O
    assert np.max(np.abs(buf.LSE.cpu().numpy().astype(np.float64)[bi, hi, si] - LSE[bi, hi, si])) <= TOL_LSE
    if not cfg.backward:
        return
    # dK/dV rows are complete only for the (b, h) whose every query block was recomputed
    b, h = full_head
    dQ, dKo, dVo = oracle.attn_bwd(cfg, x["Q"], x["K"], x["V"], x["dO"], gi, ng, items=head)
    rest = sorted(set(items) - set(head))
    if rest:
        dQ += oracle.attn_bwd(cfg, x["Q"], x["K"], x["V"], x["dO"], gi, ng, items=rest)[0]   # disjoint rows
    for name, got, want in (("dQ", bf16_to_f64(buf.dQ)[bi, hi, si], dQ[bi, hi, si]),
                            ("dK", buf.dK[b, h].cpu().numpy().astype(np.float64), dKo[b, h]),
                            ("dV", buf.dV[b, h].cpu().numpy().astype(np.float64), dVo[b, h])):
        fro, row = rel_fro(got, want), row_err_ratio(got, want)
        print("config %d %s: rel. Frobenius %.2e, row ratio %.2f" % (n, name, fro, row))
        assert fro <= TOL_GRAD and row <= TOL_GRAD_ROW, (name, fro, row)
    # rows of the active segment that no query block routes to get exactly zero
    H = cfg.history
    touched = np.zeros(cfg.seg_len, bool)
    for qb in range(cfg.n_q_blocks):
        tok = oracle.routed_tokens(cfg, qb, gi[b, h, qb, :ng[b, h, qb]])
        touched[tok[tok >= H] - H] = True
    if (~touched).any():
        assert float(buf.dK[b, h][torch.from_numpy(~touched).cuda()].abs().max()) == 0.0


def test_config3_bf16_gradient_outputs_at_full_size():
    """HGA_FLAG_BWD_BF16_GRADS at configuration 3, in the launch configuration bench.py times: the two
    tensor-core kernels sum in fp32 in the workspace and ONE conversion launch (released early by the sweep)
    rounds both tensors, so dK/dV must equal the fp32 call's result rounded once."""
    cfg = CONFIGS[3]
    x = make_inputs(cfg)
    Q, K, V, dO = (to_dev(x[k]) for k in ("Q", "K", "V", "dO"))
    res = {}
    for extra in (0, binding.HGA_FLAG_BWD_BF16_GRADS):
        buf = binding.HgaLayerBuffers(cfg, flags=extra)
        buf.build_summaries(K, 0, cfg.history)
        buf.step(Q, K, V, None)
        before = binding.hga_kernel_launch_counts()
        buf.attn_bwd(Q, K, V, dO, buf.group_idx, buf.n_groups)
        torch.cuda.synchronize()
        assert int(buf.status.item()) == 0
        ran = [b - a for a, b in zip(before, binding.hga_kernel_launch_counts())]
        assert ran[binding.HGA_KERNELS_BWD_TENSOR] == 2 and ran[binding.HGA_KERNELS_AUX] == (1 if extra else 0), ran
        res[extra] = (buf.dQ.clone(), buf.dK.clone(), buf.dV.clone())
    (dQ32, dK32, dV32), (dQ16, dK16, dV16) = res[0], res[binding.HGA_FLAG_BWD_BF16_GRADS]
    assert dK16.dtype == torch.bfloat16 and dV16.dtype == torch.bfloat16
    assert torch.equal(dQ32, dQ16)
    for a32, a16 in ((dK32, dK16), (dV32, dV16)):
        ref = a32.double()
        err = (a16.double() - ref).abs()
        # one rounding to 8 significant bits, plus the run-to-run wobble of the fp32 atomics
        assert bool((err <= ref.abs() * 2.0 ** -8 + 1e-5).all())
        assert float(a16.double().abs().max()) > 0.0
