"""hga_varlen_step: packed sequences of different lengths (prefix-sum convention) against the oracle run
on every sequence by itself."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_15105_b200 import binding
from paper_2607_15105_b200.workloads import HgaConfig, make_inputs

from hga_testlib import TOL_GRAD, TOL_LSE, TOL_O, bits_of, check_routing, rel_fro

pytestmark = pytest.mark.gpu

SEQS = [(1536, 512), (640, 640), (2048, 256), (1024, 128)]      # (L_i, S_i): with history, none, long, short


def seq_cfg(L, S, seed):
    return HgaConfig("varlen", batch=1, n_q_heads=4, n_kv_heads=2, head_dim=128, total_len=L, seg_len=S,
                     chunk=64, group=8, q_block=64, topk_chunks=4, topk_groups=3, sink=64, local=128,
                     topics=16, needles=0, backward=True, seed=seed)


def pack_tokens(parts):
    """per-sequence [1, H, T, d] arrays -> token-major packed [sum T, H, d]"""
    return np.ascontiguousarray(np.concatenate([a[0].transpose(1, 0, 2) for a in parts], axis=0))


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("mode", ["fwd+bwd", "fwd", "bf16_grads", "generic"])
def test_varlen_matches_oracle_per_sequence(mode):
    cfgs = [seq_cfg(L, S, 41 + i) for i, (L, S) in enumerate(SEQS)]
    xs = [make_inputs(c) for c in cfgs]
    cu_q = np.cumsum([0] + [S for _, S in SEQS]).astype(np.int32)
    cu_k = np.cumsum([0] + [L for L, _ in SEQS]).astype(np.int32)
    c0 = cfgs[0]
    Hq, Hkv, d, kc, kge = c0.n_q_heads, c0.n_kv_heads, c0.head_dim, c0.topk_chunks, c0.kg_eff
    backward = mode != "fwd"
    flags = {"bf16_grads": binding.HGA_FLAG_BWD_BF16_GRADS, "generic": binding.HGA_FLAG_GENERIC_KERNELS}.get(mode, 0)
    p = binding.make_params(c0, flags=flags)
    Q, K, V, dO = (dev_bf16(pack_tokens([x[k] for x in xs])) for k in ("Q", "K", "V", "dO"))
    n_q, n_k = int(cu_q[-1]), int(cu_k[-1])
    cs = torch.zeros(Hkv, n_k // c0.chunk, d, dtype=torch.bfloat16, device="cuda")
    gs = torch.zeros(Hkv, n_k // c0.group, d, dtype=torch.bfloat16, device="cuda")
    # resident state: history summaries of every sequence (from the oracle; the active ranges are built by the call)
    ocs, ogs = [], []
    for c, x in zip(cfgs, xs):
        a, b = oracle.build_summaries(c, x["K"])
        ocs.append(a)
        ogs.append(b)
        h_c, h_g = c.history // c.chunk, c.history // c.group
    for i, c in enumerate(cfgs):
        r0c, r0g = int(cu_k[i]) // c.chunk, int(cu_k[i]) // c.group
        h_c, h_g = c.history // c.chunk, c.history // c.group
        cs[:, r0c:r0c + h_c] = dev_bf16(ocs[i][0, :, :h_c])
        gs[:, r0g:r0g + h_g] = dev_bf16(ogs[i][0, :, :h_g])
    items = Hkv * n_q // c0.q_block
    ci = torch.full((items, kc), -7, dtype=torch.int32, device="cuda")
    gi = torch.full((items, kc * kge), -7, dtype=torch.int32, device="cuda")
    ng = torch.full((items,), -7, dtype=torch.int32, device="cuda")
    O = torch.zeros(n_q, Hq, d, dtype=torch.bfloat16, device="cuda")
    LSE = torch.zeros(Hq * n_q, dtype=torch.float32, device="cuda")
    gdt = torch.bfloat16 if mode == "bf16_grads" else torch.float32
    dQ = torch.zeros_like(O) if backward else None
    dK = torch.zeros(Hkv * n_q * d, dtype=gdt, device="cuda") if backward else None
    dV = torch.zeros_like(dK) if backward else None
    ws = torch.empty(binding.hga_varlen_workspace_bytes(p, cu_q, cu_k) + 256, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.hga_varlen_step(p, cu_q, cu_k, Q, K, V, dO if backward else None, cs, gs, ci, gi, ng, O, LSE, dQ, dK, dV,
                            ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for i, (c, x) in enumerate(zip(cfgs, xs)):
        q0, q1, k0 = int(cu_q[i]), int(cu_q[i + 1]), int(cu_k[i])
        S, nqb = c.seg_len, c.n_q_blocks
        r0c, r0g = k0 // c.chunk, k0 // c.group
        assert np.array_equal(bits_of(cs[:, r0c:r0c + c.total_len // c.chunk]), ocs[i][0])
        assert np.array_equal(bits_of(gs[:, r0g:r0g + c.total_len // c.group]), ogs[i][0])
        it0 = Hkv * q0 // c.q_block
        ci_i = ci[it0:it0 + Hkv * nqb].cpu().numpy().reshape(1, Hkv, nqb, kc)
        gi_i = gi[it0:it0 + Hkv * nqb].cpu().numpy().reshape(1, Hkv, nqb, kc * kge)
        ng_i = ng[it0:it0 + Hkv * nqb].cpu().numpy().reshape(1, Hkv, nqb)
        ref = oracle.route(c, x["Q"], ocs[i], ogs[i], want_scores=True)
        n, ec, eg = check_routing(c, ref, ci_i, gi_i, ng_i)
        assert ec <= max(1, n // 10) and eg <= max(1, n // 5), (i, n, ec, eg)
        O_ref, LSE_ref = oracle.attn_fwd(c, x["Q"], x["K"], x["V"], gi_i, ng_i)
        O_i = O[q0:q1].double().cpu().numpy().transpose(1, 0, 2)[None]
        assert np.max(np.abs(O_i - O_ref)) <= TOL_O, i
        LSE_i = LSE[Hq * q0:Hq * q1].cpu().numpy().astype(np.float64).reshape(1, Hq, S)
        assert np.max(np.abs(LSE_i - LSE_ref)) <= TOL_LSE, i
        if backward:
            dQ_ref, dK_ref, dV_ref = oracle.attn_bwd(c, x["Q"], x["K"], x["V"], x["dO"], gi_i, ng_i)
            dQ_i = dQ[q0:q1].double().cpu().numpy().transpose(1, 0, 2)[None]
            assert rel_fro(dQ_i, dQ_ref) <= TOL_GRAD, i
            blk = slice(Hkv * d * q0, Hkv * d * q1)
            assert rel_fro(dK[blk].double().cpu().numpy().reshape(1, Hkv, S, d), dK_ref) <= TOL_GRAD, i
            assert rel_fro(dV[blk].double().cpu().numpy().reshape(1, Hkv, S, d), dV_ref) <= TOL_GRAD, i


def test_varlen_rejects_bad_prefix_sums():
    c = seq_cfg(1536, 512, 41)
    p = binding.make_params(c)
    with pytest.raises(binding.HgaError):        # a sequence whose length is not a multiple of the chunk
        binding.hga_varlen_workspace_bytes(p, [0, 512], [0, 1500])
    with pytest.raises(binding.HgaError):        # more queries than keys
        binding.hga_varlen_workspace_bytes(p, [0, 512, 1024], [0, 1536, 1792])
    with pytest.raises(binding.HgaError):        # does not start at zero
        binding.hga_varlen_workspace_bytes(p, [64, 576], [0, 1536])
