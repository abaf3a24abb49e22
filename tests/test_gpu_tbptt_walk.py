"""hga_tbptt_walk (one layer over a whole sequence, segment by segment, Section 2.2) against the
oracle run separately on every segment's problem (total_len = (s+1)*S, history s*S)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_15105_b200 import binding
from paper_2607_15105_b200.workloads import HgaConfig, make_inputs

from hga_testlib import (TOL_GRAD, TOL_LSE, TOL_O, bf16_to_f64, bits_of, check_routing, rel_fro, to_dev)

pytestmark = pytest.mark.gpu


def seq_cfg(total_len, seg_len, **kw):
    base = dict(name="walk", batch=2, n_q_heads=4, n_kv_heads=2, head_dim=128, total_len=total_len,
                seg_len=seg_len, chunk=64, group=8, q_block=64, topk_chunks=4, topk_groups=3,
                sink=64, local=128, topics=16, needles=0, backward=True, seed=23)
    base.update(kw)
    return HgaConfig(**base)


@pytest.mark.parametrize("backward", [True, False, "bf16_grads"])
def test_walk_matches_oracle_segment_by_segment(backward):
    L, S = 1536, 512
    n_seg = L // S
    full = seq_cfg(L, L)                    # generator view: every token is a query
    x = make_inputs(full)
    Q, K, V, dO = x["Q"], x["K"], x["V"], x["dO"]
    cfg = seq_cfg(L, S)                     # the walk's parameters: segments of S tokens
    B, Hq, Hkv, d = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    nqb, kc, kge = S // cfg.q_block, cfg.topk_chunks, min(cfg.topk_groups, cfg.chunk // cfg.group)
    bf16_grads = backward == "bf16_grads"
    p = binding.make_params(cfg, flags=binding.HGA_FLAG_BWD_BF16_GRADS if bf16_grads else 0)
    dev = "cuda"
    Qd, Kd, Vd, dOd = to_dev(Q), to_dev(K), to_dev(V), to_dev(dO)
    cs = torch.zeros(B, Hkv, L // cfg.chunk, d, dtype=torch.bfloat16, device=dev)
    gs = torch.zeros(B, Hkv, L // cfg.group, d, dtype=torch.bfloat16, device=dev)
    ci = torch.full((n_seg, B, Hkv, nqb, kc), -7, dtype=torch.int32, device=dev)
    gi = torch.full((n_seg, B, Hkv, nqb, kc * kge), -7, dtype=torch.int32, device=dev)
    ng = torch.full((n_seg, B, Hkv, nqb), -7, dtype=torch.int32, device=dev)
    O = torch.zeros(B, Hq, L, d, dtype=torch.bfloat16, device=dev)
    LSE = torch.zeros(n_seg, B, Hq, S, dtype=torch.float32, device=dev)
    dQ = torch.zeros_like(O) if backward else None
    dK = torch.zeros(n_seg, B, Hkv, S, d, dtype=torch.bfloat16 if bf16_grads else torch.float32, device=dev) if backward else None
    dV = torch.zeros_like(dK) if backward else None
    r_bytes, b_bytes = binding.hga_workspace_bytes(p)
    ws = torch.empty(r_bytes + b_bytes + 512, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    binding.hga_tbptt_walk(p, Qd, Kd, Vd, dOd if backward else None, cs, gs, ci, gi, ng, O, LSE, dQ, dK, dV,
                           ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0

    # summaries of the whole sequence: bit-exact
    ocs, ogs = oracle.build_summaries(full, K)
    assert np.array_equal(bits_of(cs), ocs) and np.array_equal(bits_of(gs), ogs)

    Of = bf16_to_f64(O)
    dQf = bf16_to_f64(dQ) if backward else None
    for s in range(n_seg):
        cfg_s = seq_cfg((s + 1) * S, S)
        Ls = (s + 1) * S
        Qs = np.ascontiguousarray(Q[:, :, s * S:Ls])
        Ks, Vs = np.ascontiguousarray(K[:, :, :Ls]), np.ascontiguousarray(V[:, :, :Ls])
        cs_s, gs_s = oracle.build_summaries(cfg_s, Ks)
        ref = oracle.route(cfg_s, Qs, cs_s, gs_s, want_scores=True)
        gi_s, ng_s = gi[s].cpu().numpy(), ng[s].cpu().numpy()
        n, ec, eg = check_routing(cfg_s, ref, ci[s].cpu().numpy(), gi_s, ng_s)
        assert ec <= max(1, n // 10) and eg <= max(1, n // 5), (s, n, ec, eg)
        # attention parity on the routing the library actually took
        O_ref, LSE_ref = oracle.attn_fwd(cfg_s, Qs, Ks, Vs, gi_s, ng_s)
        assert np.max(np.abs(Of[:, :, s * S:Ls] - O_ref)) <= TOL_O, s
        assert np.max(np.abs(LSE[s].cpu().numpy().astype(np.float64) - LSE_ref)) <= TOL_LSE, s
        if backward:
            dOs = np.ascontiguousarray(dO[:, :, s * S:Ls])
            dQ_ref, dK_ref, dV_ref = oracle.attn_bwd(cfg_s, Qs, Ks, Vs, dOs, gi_s, ng_s)
            assert rel_fro(dQf[:, :, s * S:Ls], dQ_ref) <= TOL_GRAD, s
            assert rel_fro(dK[s].double().cpu().numpy(), dK_ref) <= TOL_GRAD, s
            assert rel_fro(dV[s].double().cpu().numpy(), dV_ref) <= TOL_GRAD, s


def test_walk_rejects_bad_arguments():
    cfg = seq_cfg(1536, 512)
    p = binding.make_params(cfg)
    t = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.HgaError):          # workspace too small
        binding.hga_tbptt_walk(p, t, t, t, None, t, t, t, t, t, t, t, None, None, None, t)
    bad = binding.make_params(seq_cfg(1536, 1024))  # total_len not a multiple of seg_len
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.HgaError):
        binding.hga_tbptt_walk(bad, t, t, t, None, t, t, t, t, t, t, t, None, None, None, ws)
