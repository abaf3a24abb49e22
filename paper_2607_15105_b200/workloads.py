"""Seeded synthetic workloads for Hierarchical Global Attention (HGA).

This module only *draws inputs*: it knows the tensor shapes of an HGA layer step and
plants structure in the keys and queries (topics shared by a chunk, needle groups that
match one query block).  It holds none of the method's arithmetic (no summaries, no
scores, no selection, no attention) and is the one module that both the CPU oracle's
tests and the CUDA path's tests/benchmark may use, so that both sides see the same bits.

The data stand in for the paper's workloads by shape and structure only: documents
whose neighbouring tokens share a topic (long-form text, Section 3 "Experimental
Setup") and planted key/query matches (retrieval, Section 4.6).  No dataset item is
reproduced.

Tensors are bf16 bit patterns held in ``numpy.uint16`` arrays:
  Q, dO : [B, Hq,  S, d]   (the S active-segment rows; row t is position H + t)
  K, V  : [B, Hkv, L, d]   (history first, active segment last)
"""
from __future__ import annotations

from dataclasses import dataclass, replace
import numpy as np

__all__ = ["HgaConfig", "CONFIGS", "get_config", "make_inputs", "f32_to_bf16_bits",
           "bf16_bits_to_f32", "bf16_bits_to_f64"]


@dataclass(frozen=True)
class HgaConfig:
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    total_len: int      # L
    seg_len: int        # S (active, differentiable rows = queries)
    chunk: int          # c
    group: int          # g
    q_block: int        # Bq
    topk_chunks: int    # k_c
    topk_groups: int    # k_g per opened chunk
    sink: int
    local: int          # W
    topics: int         # 0 = i.i.d. keys/queries
    needles: int        # planted key-group / query-block matches
    backward: bool
    seed: int
    decode: bool = False   # generation-shaped: q_block = the few newest tokens, any history length

    @property
    def history(self) -> int:
        return self.total_len - self.seg_len

    @property
    def gqa(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_q_blocks(self) -> int:
        return self.seg_len // self.q_block

    @property
    def n_items(self) -> int:
        return self.batch * self.n_kv_heads * self.n_q_blocks

    @property
    def kg_eff(self) -> int:
        return min(self.topk_groups, self.chunk // self.group)

    @property
    def tokens_per_step(self) -> int:
        return self.batch * self.seg_len

    def scaled(self, **kw) -> "HgaConfig":
        return replace(self, **kw)


# The five benchmark configurations (seed = 1337 + configuration number), plus a sixth in the
# paper's own default routing shape: eight selected chunks opened whole (k_g = c/g), Section 3 / Table 1.
CONFIGS = {
    1: HgaConfig("cfg1_tiny_1k", 1, 2, 1, 64, 1024, 256, 64, 8, 64, 4, 4, 64, 64,
                 topics=8, needles=0, backward=True, seed=1338),
    2: HgaConfig("cfg2_qwen3_8b_2k", 1, 32, 8, 128, 2048, 2048, 64, 8, 64, 8, 4, 64, 128,
                 topics=64, needles=0, backward=True, seed=1339),
    3: HgaConfig("cfg3_qwen3_8b_16k_tbptt", 1, 32, 8, 128, 16384, 2048, 64, 8, 64, 16, 4, 64, 128,
                 topics=256, needles=32, backward=True, seed=1340),
    4: HgaConfig("cfg4_qwen3_8b_128k_eval", 1, 32, 8, 128, 131072, 2048, 64, 8, 64, 16, 4, 64, 128,
                 topics=1024, needles=32, backward=False, seed=1341),
    5: HgaConfig("cfg5_stress_b4_64k", 4, 32, 8, 128, 65536, 4096, 128, 16, 128, 32, 4, 128, 256,
                 topics=0, needles=0, backward=True, seed=1342),
    6: HgaConfig("cfg6_paper_default_16k", 1, 32, 8, 128, 16384, 2048, 64, 8, 64, 8, 8, 64, 128,
                 topics=256, needles=32, backward=True, seed=1343),
    # generation-shaped: 32 sequences, one new token each behind 16 379 resident tokens (not a multiple of
    # anything), the routing shape of configuration 3
    7: HgaConfig("cfg7_decode_b32_16k", 32, 32, 8, 128, 16380, 1, 64, 8, 1, 16, 4, 64, 128,
                 topics=256, needles=0, backward=False, seed=1344, decode=True),
}


def get_config(n: int) -> HgaConfig:
    return CONFIGS[n]


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns the 16-bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


_KEY_TOPIC_GAIN = 1.5     # keys   = N(0, I) + 1.5 * topic(chunk)
_QUERY_TOPIC_GAIN = 3.0   # queries = N(0, I) + 3.0 * (topic_a + topic_b)
_NEEDLE_GAIN = 8.0        # needle keys / probe queries = N(0, I) + 8 * w


def make_inputs(cfg: HgaConfig, with_dO: bool | None = None) -> dict:
    """Draw Q, K, V (and dO) for one layer step of ``cfg`` from ``cfg.seed``.

    Returns a dict with uint16 arrays "Q", "K", "V", optionally "dO", and "needles":
    a list of (batch, kv_head, q_block, group_id) for the planted matches.
    One random stream per (batch, kv head), spawned from the seed, drawn in a fixed order.
    """
    if with_dO is None:
        with_dO = cfg.backward
    B, Hq, Hkv, d = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    L, S, c, g, Bq = cfg.total_len, cfg.seg_len, cfg.chunk, cfg.group, cfg.q_block
    G, H, nqb, nch = cfg.gqa, cfg.history, cfg.n_q_blocks, -(-cfg.total_len // cfg.chunk)
    Q = np.empty((B, Hq, S, d), np.uint16)
    K = np.empty((B, Hkv, L, d), np.uint16)
    V = np.empty((B, Hkv, L, d), np.uint16)
    dO = np.empty((B, Hq, S, d), np.uint16) if with_dO else None
    needles = []
    streams = np.random.SeedSequence(cfg.seed).spawn(B * Hkv)
    for b in range(B):
        for h in range(Hkv):
            rng = np.random.Generator(np.random.PCG64(streams[b * Hkv + h]))
            k = rng.standard_normal((L, d), dtype=np.float32)
            q = rng.standard_normal((G, S, d), dtype=np.float32)
            if cfg.topics > 0:
                U = rng.standard_normal((cfg.topics, d)).astype(np.float32)
                U /= np.linalg.norm(U, axis=1, keepdims=True)
                tau = rng.integers(0, cfg.topics, nch)
                k += _KEY_TOPIC_GAIN * np.repeat(U[tau], c, axis=0)[:L]
                for qb in range(nqb):
                    # a block follows the topics of two earlier chunks (of two random
                    # topics when nothing precedes it)
                    n_prev = (H + qb * Bq) // c
                    if n_prev > 0:
                        ta, tb = tau[rng.integers(0, n_prev, 2)]
                    else:
                        ta, tb = rng.integers(0, cfg.topics, 2)
                    q[:, qb * Bq:(qb + 1) * Bq] += _QUERY_TOPIC_GAIN * (U[ta] + U[tb])
            # needle n belongs to query block n (mod nqb) and lives on kv head n mod Hkv
            for n in range(cfg.needles):
                if n % Hkv != h:
                    continue
                qb = n % nqb
                lo = cfg.sink // g
                hi = (H + qb * Bq - cfg.local - c) // g      # well before the local window
                if hi <= lo:
                    continue
                m = int(rng.integers(lo, hi))
                w = rng.standard_normal(d).astype(np.float32)
                w /= np.linalg.norm(w)
                k[m * g:(m + 1) * g] = rng.standard_normal((g, d), dtype=np.float32) + _NEEDLE_GAIN * w
                q[:, qb * Bq:(qb + 1) * Bq] += _NEEDLE_GAIN * w
                needles.append((b, h, qb, m))
            K[b, h] = f32_to_bf16_bits(k)
            del k
            V[b, h] = f32_to_bf16_bits(rng.standard_normal((L, d), dtype=np.float32))
            Q[b, h * G:(h + 1) * G] = f32_to_bf16_bits(q)
            del q
            if with_dO:
                dO[b, h * G:(h + 1) * G] = f32_to_bf16_bits(rng.standard_normal((G, S, d), dtype=np.float32))
    out = {"Q": Q, "K": K, "V": V, "needles": needles}
    if with_dO:
        out["dO"] = dO
    return out
