"""Helpers shared by the parity tests: moving the seeded inputs to the device and comparing
the CUDA library's outputs with the CPU oracle's.  No method arithmetic lives here."""
import numpy as np
import torch

import oracle

SCORE_GAP = 1e-3   # routing: an index may differ only where the score gap to the k-th is below this
TOL_O = 1e-2       # attention forward: max abs error on O (unit-scale bf16 inputs)
TOL_LSE = 1e-3     # attention forward: max abs error on LSE
TOL_GRAD = 2e-2    # backward: relative Frobenius error per gradient tensor
# backward, per row (one query row of dQ, one key row of dK / dV): the Frobenius bound alone would let one
# wholly wrong row in ~2000 pass.  The kernels feed bf16 P and dS to the tensor core (relative rounding 2^-9
# per term, signs random) and round dQ once to bf16; a row whose terms cancel carries the rounding error of
# the terms, not of the sum, so the error is measured against |row| + the tensor's RMS row norm.  Measured
# worst rows sit near 4 (heavy cancellation); a wholly wrong row of typical size gives >= 64.
TOL_GRAD_ROW = 16.0  # max over rows of |err_row| / (2^-8 * (|ref_row| + rms row norm of ref))


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bfloat16 tensor (same bits)."""
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def rel_fro(a: np.ndarray, ref: np.ndarray) -> float:
    den = float(np.linalg.norm(ref.ravel()))
    num = float(np.linalg.norm((a - ref).ravel()))
    return num / den if den > 0 else num


def row_err_ratio(a: np.ndarray, ref: np.ndarray) -> float:
    """max over rows (last axis = head_dim) of |a_row - ref_row| / (2^-8 * (|ref_row| + rms row norm))."""
    a2, r2 = a.reshape(-1, a.shape[-1]), ref.reshape(-1, ref.shape[-1])
    err = np.linalg.norm(a2 - r2, axis=1)
    nrm = np.linalg.norm(r2, axis=1)
    rms = float(np.sqrt(np.mean(nrm ** 2)))
    if rms == 0.0:
        return float(err.max(initial=0.0) > 0) * np.inf if err.size else 0.0
    return float(np.max(err / (2.0 ** -8 * (nrm + rms)), initial=0.0))


def check_grads(got, ref, what=""):
    """got / ref: (dQ, dK, dV) as float64 arrays of equal shapes.  Frobenius and per-row bounds."""
    for name, a, r in zip(("dQ", "dK", "dV"), got, ref):
        fro, row = rel_fro(a, r), row_err_ratio(a, r)
        assert fro <= TOL_GRAD, (what, name, "rel fro", fro)
        assert row <= TOL_GRAD_ROW, (what, name, "row ratio", row)


def check_routing(cfg, ref, chunk_idx, group_idx, n_groups, items=None, global_budget=False):
    """Compare GPU routing with the oracle's (ref holds oracle indices and fp64 scores).

    Index sets must be equal, except that an index in the symmetric difference is excused
    when its oracle score lies within SCORE_GAP of the oracle's k-th best score; set sizes
    must match.  Groups are compared inside chunks both sides selected; with global_budget (one
    budget over all opened chunks) the whole group sets are compared, against the oracle's
    N-th best group score, for the items whose chunk sets agree.
    Returns (items checked, items with an excused chunk, chunks with an excused group).
    """
    per, kge = cfg.chunk // cfg.group, min(cfg.topk_groups, cfg.chunk // cfg.group)
    nqb, Hkv = cfg.n_q_blocks, cfg.n_kv_heads
    all_items = range(cfg.n_items) if items is None else items
    exc_c = exc_g = 0
    for item in all_items:
        qb = item % nqb
        h = (item // nqb) % Hkv
        b = item // (nqb * Hkv)
        o_c = [int(j) for j in ref["chunk_idx"][b, h, qb] if j >= 0]
        g_c = [int(j) for j in chunk_idx[b, h, qb] if j >= 0]
        assert len(o_c) == len(g_c), (item, o_c, g_c)
        assert g_c == sorted(set(g_c)), ("chunk list not ascending/unique", item, g_c)
        ls, se = oracle.window(cfg, qb)
        assert all(se <= j * cfg.chunk and (j + 1) * cfg.chunk <= ls for j in g_c), (item, g_c)
        sc = ref["chunk_scores"][b, h, qb]
        if set(o_c) != set(g_c):
            kth = min(sc[j] for j in o_c)
            for j in set(o_c) ^ set(g_c):
                assert abs(sc[j] - kth) < SCORE_GAP, ("chunk not excused", item, j, sc[j], kth)
            exc_c += 1
        ng = int(n_groups[b, h, qb])
        assert ng == len(g_c) * kge, (item, ng)
        g_g = [int(m) for m in group_idx[b, h, qb, :ng]]
        assert g_g == sorted(set(g_g)) and np.all(group_idx[b, h, qb, ng:] == -1), (item, g_g)
        if global_budget:
            assert all(m // per in g_c for m in g_g), (item, g_g)
            o_set = {int(m) for m in ref["group_idx"][b, h, qb] if m >= 0}
            if set(o_c) == set(g_c) and o_set != set(g_g):
                sg = ref["group_scores"][b, h, qb]
                slot = lambda m: o_c.index(m // per) * per + m % per
                nth = min(sg[slot(m)] for m in o_set)
                for m in o_set ^ set(g_g):
                    assert abs(sg[slot(m)] - nth) < SCORE_GAP, ("group not excused", item, m)
                exc_g += 1
            continue
        for r, j in enumerate(o_c):
            if j not in g_c:
                continue
            o_set = {int(m) for m in ref["group_idx"][b, h, qb] if m >= 0 and m // per == j}
            g_set = {m for m in g_g if m // per == j}
            assert len(g_set) == kge, (item, j, g_set)
            if o_set != g_set:
                sg = ref["group_scores"][b, h, qb, r * per:(r + 1) * per]
                kth = min(sg[m - j * per] for m in o_set)
                for m in o_set ^ g_set:
                    assert abs(sg[m - j * per] - kth) < SCORE_GAP, ("group not excused", item, m)
                exc_g += 1
    return len(list(all_items)), exc_c, exc_g


def item_rows(cfg, items):
    """(b, hq, s) index arrays of every query row belonging to the listed items."""
    G, Bq, nqb, Hkv = cfg.gqa, cfg.q_block, cfg.n_q_blocks, cfg.n_kv_heads
    bs, hs, ss = [], [], []
    for item in items:
        qb = item % nqb
        h = (item // nqb) % Hkv
        b = item // (nqb * Hkv)
        for a in range(G):
            bs.append(np.full(Bq, b))
            hs.append(np.full(Bq, h * G + a))
            ss.append(qb * Bq + np.arange(Bq))
    return np.concatenate(bs), np.concatenate(hs), np.concatenate(ss)
