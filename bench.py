#!/usr/bin/env python
"""Benchmark of the HGA hot path (summaries -> route -> attention fwd -> attention bwd).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

A step is one pass of the whole path over one synthetic Qwen3-8B-shaped attention layer
(default: the 16K TBPTT configuration).  Prints ONE JSON line.  With N > 1 (launched by
torchrun) every rank runs its own sequence: the path shards by sequence with no exchange
step, so the only collectives are the timing barrier and the max over ranks.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_15105_b200.workloads import CONFIGS, make_inputs  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        pk["source"] = "measured"
        return pk
    pk = dict(FALLBACK_PEAKS)
    pk["source"] = "fallback"
    return pk


# ----------------------------------------------------------------------------- work counts

def work_counts(cfg, n_groups):
    """Algorithmic work of the attention kernels for the routing actually taken.

    pairs: (query row, visible key) pairs; pairs_active: those whose key is in the active
    segment.  Bytes: K and V rows gathered once per item, Q/O/dO/dQ/LSE/delta once, dK/dV once.
    """
    d, G, Bq, g, H = cfg.head_dim, cfg.gqa, cfg.q_block, cfg.group, cfg.history
    ng = np.asarray(n_groups).reshape(cfg.batch * cfg.n_kv_heads, cfg.n_q_blocks)
    pairs = pairs_active = keys = 0
    for qb in range(cfg.n_q_blocks):
        p0 = H + qb * Bq
        ls = max(0, ((p0 - cfg.local) // cfg.chunk) * cfg.chunk) if p0 - cfg.local > 0 else 0
        se = min(cfg.sink, ls)
        local_pairs = Bq * (p0 - ls) + Bq * (Bq + 1) // 2
        local_active = Bq * (p0 - max(ls, H)) + Bq * (Bq + 1) // 2
        sink_active = max(0, se - H)
        for bh in range(ng.shape[0]):
            far = se + int(ng[bh, qb]) * g
            keys += far + (p0 + Bq - ls)
            pairs += G * (Bq * far + local_pairs)
            # routed groups inside the active segment are counted by the caller when needed;
            # here: sink and local only (a lower bound, exact when no routed group is active)
            pairs_active += G * (Bq * sink_active + local_active)
    rows = cfg.batch * cfg.n_q_heads * cfg.seg_len
    kv_rows_active = cfg.batch * cfg.n_kv_heads * cfg.seg_len
    fwd_flops = 4.0 * d * pairs
    bwd_flops = 6.0 * d * pairs + 4.0 * d * pairs_active
    gather = keys * d * 2 * 2
    fwd_bytes = gather + rows * d * 2 * 2 + rows * 4
    bwd_bytes = gather + rows * d * 2 * 4 + rows * 4 * 2 + kv_rows_active * d * 4 * 2
    return {"pairs": pairs, "pairs_active_min": pairs_active, "fwd_flops": fwd_flops,
            "bwd_flops": bwd_flops, "fwd_bytes": float(fwd_bytes), "bwd_bytes": float(bwd_bytes)}


def active_group_pairs(cfg, group_idx, n_groups):
    """(row, key) pairs whose key lies in a routed group of the active segment."""
    gi = np.asarray(group_idx).reshape(-1, cfg.n_q_blocks, group_idx.shape[-1])
    first_active = cfg.history // cfg.group
    n = int(((gi >= first_active)).sum())
    return n * cfg.group * cfg.gqa * cfg.q_block


def load_traffic(config):
    """DRAM bytes per call (dram__bytes_read.sum + dram__bytes_write.sum, summed over the call's kernels)
    from the ncu captures summarised under profiles/: profiles/traffic.json says which commit and which
    kernels the figures belong to.  Returns ({call: bytes}, provenance) or ({}, None)."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        with open(path) as f:
            t = json.load(f)
    except (OSError, ValueError):
        return {}, None
    entry = t.get("configs", {}).get(str(config))
    if not entry:
        return {}, None
    return entry.get("calls", {}), {"commit": t.get("commit"), "captured": t.get("captured"),
                                    "kernels": entry.get("kernels")}


def route_work(cfg):
    """Algorithmic work of hga_route: 2*d*(G*Bq)*(candidates + opened groups) flops per item; bytes = the
    candidate chunk summaries and the opened chunks' group summaries read once per item, Q once, lists out."""
    d, rows = cfg.head_dim, cfg.gqa * cfg.q_block
    per = cfg.chunk // cfg.group
    flops = nbytes = 0.0
    for qb in range(cfg.n_q_blocks):
        p0 = cfg.history + qb * cfg.q_block
        ls = max(0, ((p0 - cfg.local) // cfg.chunk) * cfg.chunk) if p0 - cfg.local > 0 else 0
        se = min(cfg.sink, ls)
        n_cand = (ls - se) // cfg.chunk
        k_sel = min(cfg.topk_chunks, n_cand)
        flops += 2.0 * d * rows * (n_cand + k_sel * per)
        nbytes += (n_cand + k_sel * per) * d * 2 + rows * d * 2 + (cfg.topk_chunks * (1 + min(cfg.topk_groups, per)) + 1) * 4
    n = cfg.batch * cfg.n_kv_heads
    return flops * n, nbytes * n


def roofline_entry(name, flops, nbytes, seconds, peaks, sustained=False):
    tf = peaks["bf16_tflops_sustained" if sustained else "bf16_tflops"]
    t_flop = flops / (tf * 1e12)
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    if t_hbm >= t_flop:
        achieved, peak, unit, bound = nbytes / seconds / 1e9, peaks["hbm_gbs"], "GB/s", "hbm"
    else:
        achieved, peak, unit, bound = flops / seconds / 1e12, tf, "TFLOP/s", "tensor"
    return {"kernel": name, "bound": bound, "achieved": round(achieved, 2), "peak": peak, "unit": unit,
            "frac": round(achieved / peak, 4), "traffic": None, "peak_source": peaks["source"],
            "roofline_us": round(max(t_flop, t_hbm) * 1e6, 2), "measured_us": round(seconds * 1e6, 2)}


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None, "samples": len(sm),
                "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- oracle legs

def oracle_throughput(cfg, x, budget_s=15.0):
    """Times the CPU oracle, as it stands, on a bounded sample of items of the same workload.

    Returns (tokens/s, threads used, description).  One item covers Bq positions of one kv
    head, so n items amount to n*Bq/Hkv tokens of the layer."""
    import oracle
    threads = oracle.num_threads()
    t0 = time.perf_counter()
    tb = cfg.history
    cs, gs = oracle.build_summaries(cfg, x["K"], tb, cfg.total_len)
    # history summaries are resident state (built by earlier segments): build them untimed
    t_sum = time.perf_counter() - t0
    oracle.build_summaries(cfg, x["K"], 0, tb, cs, gs)
    rng = np.random.default_rng(0)
    order = rng.permutation(cfg.n_items)
    done, elapsed, batch = 0, 0.0, max(threads, 4)
    while done < cfg.n_items and (done == 0 or elapsed * (done + batch) / done < budget_s):
        items = np.sort(order[done:done + batch]).astype(np.int32)
        t0 = time.perf_counter()
        r = oracle.route(cfg, x["Q"], cs, gs, items=items)
        oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], r["group_idx"], r["n_groups"], items=items)
        if cfg.backward:
            oracle.attn_bwd(cfg, x["Q"], x["K"], x["V"], x["dO"], r["group_idx"], r["n_groups"], items=items)
        elapsed += time.perf_counter() - t0
        done += len(items)
    frac = done / cfg.n_items
    total = elapsed + t_sum * frac
    tokens = done * cfg.q_block / cfg.n_kv_heads
    what = ("%d of %d (batch, kv head, query block) items of %s, chosen at random: summaries of the "
            "active range (pro rata) + route + attention fwd%s" %
            (done, cfg.n_items, cfg.name, " + bwd" if cfg.backward else ""))
    return tokens / total, threads, what, total


def run_reference(args, cfg):
    """--impl reference: the oracle on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    x = make_inputs(cfg)
    vals, last = [], None
    for i in range(args.warmup + args.steps):
        last = oracle_throughput(cfg, x, budget_s=max(2.0, min(15.0, 120.0 / (args.warmup + args.steps))))
        if i >= args.warmup:
            vals.append(last)
    tps = float(np.mean([v[0] for v in vals]))
    sec = float(np.mean([v[3] for v in vals]))
    line = {"impl": "reference", "metric": METRIC, "value": round(tps, 3), "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(sec * 1e3, 3), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(cfg, args),
            "cpu_baseline": {"value": round(tps, 3), "unit": "tokens/s", "cores": last[1],
                             "kind": "oracle", "sample": last[2]},
            "e2e": {"value": round(tps, 3), "unit": "tokens/s", "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


METRIC = "Qwen3-8B-layer HGA fwd+bwd tokens/s at 16K context; % of roofline"


def config_dict(cfg, args):
    return {"workload": cfg.name, "batch_per_gpu": cfg.batch, "q_heads": cfg.n_q_heads,
            "kv_heads": cfg.n_kv_heads, "head_dim": cfg.head_dim, "total_len": cfg.total_len,
            "active_segment": cfg.seg_len, "chunk": cfg.chunk, "group": cfg.group,
            "q_block": cfg.q_block, "topk_chunks": cfg.topk_chunks, "topk_groups": cfg.topk_groups,
            "sink": cfg.sink, "local": cfg.local, "pass": "fwd+bwd" if cfg.backward else "fwd",
            "l2": "flushed between timed steps (512 MiB write)", "parallelism": "dp%d" % args.gpus}


def time_tbptt_walk(cfg, args, stream):
    """hga_tbptt_walk over a fresh synthetic sequence of cfg.total_len tokens in segments of
    cfg.seg_len (same generator, every token a query); tokens/s counts every token once."""
    import torch
    from paper_2607_15105_b200 import binding
    from paper_2607_15105_b200.workloads import make_inputs
    L, S = cfg.total_len, cfg.seg_len
    n_seg = L // S
    y = make_inputs(cfg.scaled(seg_len=L, seed=cfg.seed + 77))
    dev = "cuda"
    as_bf16 = lambda a: torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
    Q, K, V, dO = as_bf16(y["Q"]), as_bf16(y["K"]), as_bf16(y["V"]), as_bf16(y["dO"])
    del y
    B, Hq, Hkv, d = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    nqb, kc, kge = S // cfg.q_block, cfg.topk_chunks, min(cfg.topk_groups, cfg.chunk // cfg.group)
    p = binding.make_params(cfg)
    cs = torch.zeros(B, Hkv, L // cfg.chunk, d, dtype=torch.bfloat16, device=dev)
    gs = torch.zeros(B, Hkv, L // cfg.group, d, dtype=torch.bfloat16, device=dev)
    ci = torch.zeros(n_seg, B, Hkv, nqb, max(kc, 1), dtype=torch.int32, device=dev)
    gi = torch.zeros(n_seg, B, Hkv, nqb, max(kc * kge, 1), dtype=torch.int32, device=dev)
    ng = torch.zeros(n_seg, B, Hkv, nqb, dtype=torch.int32, device=dev)
    O, dQ = torch.zeros_like(Q), torch.zeros_like(Q)
    LSE = torch.zeros(n_seg, B, Hq, S, dtype=torch.float32, device=dev)
    dK = torch.zeros(n_seg, B, Hkv, S, d, dtype=torch.float32, device=dev)
    dV = torch.zeros_like(dK)
    rb, bb = binding.hga_workspace_bytes(p)
    ws = torch.empty(rb + bb + 512, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    def run():
        binding.hga_tbptt_walk(p, Q, K, V, dO, cs, gs, ci, gi, ng, O, LSE, dQ, dK, dV, ws, status)

    for _ in range(3):
        run()
    torch.cuda.synchronize()
    reps = max(3, min(args.steps, 10))
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for a, b in ev:
        a.record(stream)
        run()
        b.record(stream)
    torch.cuda.synchronize()
    ms = float(np.median([a.elapsed_time(b) for a, b in ev]))
    return {"tokens_per_s": round(B * L / (ms * 1e-3), 1), "ms_per_sequence": round(ms, 4), "segments": n_seg,
            "tokens": B * L, "launch": "eager", "device_status_word": int(status.item()),
            "note": "one layer, forward+backward of every segment (history 0 .. L-S); inputs larger than L2"}


def time_varlen(args, stream):
    """hga_varlen_step on 16 short packed sequences of the headline layer shape (512 new tokens behind
    1536 resident ones each): the packed call against the same sequences run one after another on the
    caller's stream through the four calls, both as eager launches with L2 flushed before each step."""
    import torch
    from paper_2607_15105_b200 import binding
    n_seq, L, S = 16, 2048, 512
    base = CONFIGS[3].scaled(total_len=L, seg_len=S, topics=64, needles=0)
    xs = [make_inputs(base.scaled(seed=base.seed + 200 + i)) for i in range(n_seq)]
    pack = lambda k: np.ascontiguousarray(np.concatenate([x[k][0].transpose(1, 0, 2) for x in xs], axis=0))
    dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    Q, K, V, dO = (dev(pack(k)) for k in ("Q", "K", "V", "dO"))
    del xs
    Hq, Hkv, d, kc, kge = base.n_q_heads, base.n_kv_heads, base.head_dim, base.topk_chunks, base.kg_eff
    cu_q = np.arange(n_seq + 1, dtype=np.int32) * S
    cu_k = np.arange(n_seq + 1, dtype=np.int32) * L
    n_q, n_k = n_seq * S, n_seq * L
    p = binding.make_params(base)
    cs = torch.zeros(Hkv, n_k // base.chunk, d, dtype=torch.bfloat16, device="cuda")
    gs = torch.zeros(Hkv, n_k // base.group, d, dtype=torch.bfloat16, device="cuda")
    items = Hkv * n_q // base.q_block
    ci = torch.zeros(items, kc, dtype=torch.int32, device="cuda")
    gi = torch.zeros(items, kc * kge, dtype=torch.int32, device="cuda")
    ng = torch.zeros(items, dtype=torch.int32, device="cuda")
    O, dQ = torch.zeros(n_q, Hq, d, dtype=torch.bfloat16, device="cuda"), torch.zeros(n_q, Hq, d, dtype=torch.bfloat16, device="cuda")
    LSE = torch.zeros(Hq * n_q, dtype=torch.float32, device="cuda")
    dK = torch.zeros(Hkv * n_q * d, dtype=torch.float32, device="cuda")
    dV = torch.zeros_like(dK)
    ws = torch.empty(binding.hga_varlen_workspace_bytes(p, cu_q, cu_k) + 256, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # resident state: the history summaries of every sequence (token-major keys, packed summary buffers)
    ph = binding.make_params(base, k_stride=(L * Hkv * d, d, Hkv * d), summary_len=n_k)
    for i in range(n_seq):
        binding.hga_build_summaries(ph, K[i * L:], 0, L - S, cs[:, i * L // base.chunk:], gs[:, i * L // base.group:])
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")

    def packed():
        binding.hga_varlen_step(p, cu_q, cu_k, Q, K, V, dO, cs, gs, ci, gi, ng, O, LSE, dQ, dK, dV, ws, status)

    reps = max(3, min(args.steps, 7))
    for _ in range(3):
        packed()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for a, b in ev:
        flush.zero_()
        a.record(stream)
        packed()
        b.record(stream)
    torch.cuda.synchronize()
    ms = float(np.median([a.elapsed_time(b) for a, b in ev]))
    return {"sequences": n_seq, "tokens": n_q, "resident_tokens": n_k, "ms_per_step": round(ms, 4),
            "tokens_per_s": round(n_q / (ms * 1e-3), 1), "launch": "eager, two library streams",
            "device_status_word": int(status.item()),
            "note": "16 packed sequences, 512 new tokens behind 1536 resident ones each; summaries of the active "
                    "ranges + route + attention fwd + bwd per sequence"}


def time_config(n, args, peaks):
    """One benchmark configuration other than the headline one: per-call medians (eager launches, CUDA
    events around each call, L2 flushed before every step), the CUDA-graph step, and each call's roofline."""
    import torch
    from paper_2607_15105_b200 import binding
    cfg = CONFIGS[n]
    x = make_inputs(cfg)
    dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    Q, K, V = dev(x["Q"]), dev(x["K"]), dev(x["V"])
    dO = dev(x["dO"]) if cfg.backward else None
    del x
    buf = binding.HgaLayerBuffers(cfg, backward=cfg.backward, flags=args.flags)
    buf.build_summaries(K, 0, cfg.history)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    names = ["build_summaries", "route", "attn_fwd"] + (["attn_bwd"] if cfg.backward else [])
    calls = [lambda: buf.build_summaries(K), lambda: buf.route(Q), lambda: buf.attn_fwd(Q, K, V)]
    if cfg.backward:
        calls.append(lambda: buf.attn_bwd(Q, K, V, dO))
    steps = max(3, min(args.steps, 7))
    for _ in range(3):
        for c in calls:
            c()
    torch.cuda.synchronize()
    launches0 = binding.hga_kernel_launch_counts()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(calls) + 1)] for _ in range(steps)]
    for e in ev:
        flush.zero_()
        e[0].record(stream)
        for i, c in enumerate(calls):
            c()
            e[i + 1].record(stream)
    torch.cuda.synchronize()
    ran = [b - a for a, b in zip(launches0, binding.hga_kernel_launch_counts())]
    per_call = np.array([[e[j].elapsed_time(e[j + 1]) for j in range(len(calls))] for e in ev])
    med = np.median(per_call, axis=0) * 1e-3
    graph_ms = None
    try:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for c in calls:
                c()
        gev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in gev:
            flush.zero_()
            a.record(stream)
            g.replay()
            b.record(stream)
        torch.cuda.synchronize()
        graph_ms = float(np.median([a.elapsed_time(b) for a, b in gev]))
    except Exception:      # capture unavailable: the eager numbers stand
        pass
    gi, ng = buf.group_idx.cpu().numpy(), buf.n_groups.cpu().numpy()
    wc = work_counts(cfg, ng)
    wc["bwd_flops"] += 4.0 * cfg.head_dim * active_group_pairs(cfg, gi, ng)
    rf, rb = route_work(cfg)
    roofs = {"route": roofline_entry("hga_route", rf, rb, med[1], peaks),
             "attn_fwd": roofline_entry("hga_attn_fwd", wc["fwd_flops"], wc["fwd_bytes"], med[2], peaks)}
    if cfg.backward:
        roofs["attn_bwd"] = roofline_entry("hga_attn_bwd", wc["bwd_flops"], wc["bwd_bytes"], med[3], peaks)
    attn = [roofs[k] for k in ("attn_fwd", "attn_bwd") if k in roofs]
    step_us = graph_ms * 1e3 if graph_ms is not None else float(med.sum()) * 1e6
    fam = ("summaries", "route_tensor", "route_generic", "fwd_tensor", "fwd_generic", "bwd_tensor", "bwd_generic", "aux")
    out = {"workload": cfg.name, "pass": "fwd+bwd" if cfg.backward else "fwd", "steps": steps,
           "per_call_us_median": {k: round(float(m) * 1e6, 2) for k, m in zip(names, med)},
           "step_us": round(step_us, 2), "launch": "cuda_graph" if graph_ms is not None else "eager",
           "tokens_per_s": round(cfg.tokens_per_step / (step_us * 1e-6), 1),
           "roofline": {k: {f: v[f] for f in ("bound", "achieved", "peak", "unit", "frac", "roofline_us", "measured_us")}
                        for k, v in roofs.items()},
           "attention": {"us": round(sum(r["measured_us"] for r in attn), 2),
                         "roofline_us": round(sum(r["roofline_us"] for r in attn), 2),
                         "frac_of_roofline": round(sum(r["roofline_us"] for r in attn) / sum(r["measured_us"] for r in attn), 4)},
           "kernel_launches_by_family": {f: int(c) for f, c in zip(fam, ran) if c},
           "device_status_word": int(buf.status.item())}
    del Q, K, V, dO, buf, flush
    torch.cuda.empty_cache()
    return out


# ----------------------------------------------------------------------------- main arm

def time_decode(args, stream, peaks):
    """Generation-shaped step (configuration 7): route + attention forward for one new token per
    sequence, CUDA-graph replay, L2 flushed between steps.  HBM-bound: the roofline is the bytes the
    step must read (candidate chunk summaries, opened group summaries, routed K/V rows, Q) and write
    (O, LSE, index lists) over the measured copy bandwidth."""
    import torch
    from paper_2607_15105_b200 import binding
    cfg = CONFIGS[7] if args.decode_batch <= 0 else CONFIGS[7].scaled(batch=args.decode_batch)
    x = make_inputs(cfg)

    def dev(a):
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)

    Q, K, V = dev(x["Q"]), dev(x["K"]), dev(x["V"])
    buf = binding.HgaLayerBuffers(cfg, backward=False, flags=args.flags)
    closed = (cfg.total_len // cfg.chunk) * cfg.chunk
    buf.build_summaries(K, 0, closed)               # resident state: summaries of every closed chunk
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]

    def step(e=None):
        if e:
            e[0].record(stream)
        buf.route(Q)
        if e:
            e[1].record(stream)
        buf.attn_fwd(Q, K, V)
        if e:
            e[2].record(stream)

    for _ in range(args.warmup):
        flush.zero_()
        step()
    torch.cuda.synchronize()
    for i in range(args.steps):
        flush.zero_()
        step(ev[i])
    torch.cuda.synchronize()
    per_call = np.array([[e[k].elapsed_time(e[k + 1]) for k in range(2)] for e in ev]) * 1e-3
    graph_s = None
    if not args.no_graph:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=torch.cuda.Stream()):
            step()
        gev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
        for i in range(args.warmup + args.steps):
            flush.zero_()
            if i >= args.warmup:
                gev[i - args.warmup][0].record(stream)
            g.replay()
            if i >= args.warmup:
                gev[i - args.warmup][1].record(stream)
        torch.cuda.synchronize()
        graph_s = float(np.median([a.elapsed_time(b) for a, b in gev])) * 1e-3
    status = int(buf.status.item())
    # algorithmic bytes of one step, counted from the windows and the lists the router produced
    c, g_, d, G, n = cfg.chunk, cfg.group, cfg.head_dim, cfg.gqa, cfg.q_block
    per = c // g_
    H = cfg.history
    ls = max(0, (H - cfg.local) // c * c)
    se = min(cfg.sink, ls)
    n_cand = (ls - se) // c
    k_sel = min(cfg.topk_chunks, n_cand)
    ng = buf.n_groups.cpu().numpy().astype(np.int64)
    items = cfg.batch * cfg.n_kv_heads
    route_bytes = items * ((n_cand + k_sel * per) * d * 2 + G * n * d * 2 + 4 * (k_sel + k_sel * cfg.kg_eff + 1))
    keys = se + ng * g_ + (cfg.total_len - ls)
    fwd_bytes = int(keys.sum()) * d * 2 * 2 + items * (2 * G * n * d * 2 + G * n * 4 + 4 * (k_sel * cfg.kg_eff + 1))
    med = np.median(per_call, axis=0)
    step_s = graph_s if graph_s is not None else float(med.sum())
    hbm = peaks["hbm_gbs"] * 1e9
    out = {"workload": cfg.name, "tokens_per_step": cfg.tokens_per_step, "step": "route + attention forward "
           "(summaries are resident; no chunk closes at this length)",
           "us_per_step": round(step_s * 1e6, 2), "tokens_per_s": round(cfg.tokens_per_step / step_s, 1),
           "launch": "cuda graph replay" if graph_s is not None else "eager",
           "per_call_us_median": {"route": round(float(med[0]) * 1e6, 2), "attn_fwd": round(float(med[1]) * 1e6, 2)},
           "roofline": {"bound": "hbm", "algorithmic_bytes": int(route_bytes + fwd_bytes),
                        "achieved": round((route_bytes + fwd_bytes) / step_s / 1e9, 1), "peak": peaks["hbm_gbs"],
                        "unit": "GB/s", "frac": round((route_bytes + fwd_bytes) / step_s / hbm, 4),
                        "peak_source": peaks["source"],
                        "route": {"algorithmic_bytes": int(route_bytes), "frac": round(route_bytes / float(med[0]) / hbm, 4)},
                        "attn_fwd": {"algorithmic_bytes": int(fwd_bytes), "frac": round(fwd_bytes / float(med[1]) / hbm, 4)}},
           "l2": "flushed between timed steps (512 MiB write)", "device_status_word": status}
    if not args.no_cpu_baseline:
        import oracle
        t0 = time.perf_counter()
        sample = np.arange(0, items, max(1, items // 32), dtype=np.int32)
        cs, gs = bits(buf.chunk_sum), bits(buf.group_sum)
        t0 = time.perf_counter()
        r = oracle.route(cfg, x["Q"], cs, gs, items=sample)
        oracle.attn_fwd(cfg, x["Q"], x["K"], x["V"], r["group_idx"], r["n_groups"], items=sample)
        dt = time.perf_counter() - t0
        out["cpu_baseline"] = {"value": round(len(sample) * n / cfg.n_kv_heads / dt, 1), "unit": "tokens/s",
                               "cores": oracle.num_threads(), "kind": "oracle",
                               "sample": "%d of %d (sequence, kv head) items: route + attention forward" % (len(sample), items)}
    return out


def bits(t):
    import torch
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of a CUDA-graph replay")
    ap.add_argument("--flags", type=int, default=0, help="hga_params.flags (debugging)")
    ap.add_argument("--no-decode", action="store_true", help="skip the generation-shaped step (configuration 7)")
    ap.add_argument("--only-decode", action="store_true",
                    help="run only the generation-shaped step and print its object (profiling captures)")
    ap.add_argument("--decode-batch", type=int, default=0,
                    help="sequences in the generation-shaped step (default: configuration 7's 32)")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the per-configuration timings (configurations 2, 4, 5 and 6 beside the headline one)")
    ap.add_argument("--no-walk", action="store_true",
                    help="skip the whole-sequence TBPTT walk (every segment of the sequence, one layer)")
    args = ap.parse_args()
    cfg = CONFIGS[args.config]
    if args.impl == "reference":
        run_reference(args, cfg)
        return
    if args.warmup < 3:
        args.warmup = 3
    if args.only_decode:
        import torch
        torch.cuda.set_device(0)
        print(json.dumps({"decode": time_decode(args, torch.cuda.current_stream(), load_peaks())}))
        return

    import torch
    import torch.distributed as dist
    from paper_2607_15105_b200 import binding

    from paper_2607_15105_b200 import sharding
    rank, world, local_rank = sharding.env_rank()
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    # every rank draws its own sequence (weak scaling): same shapes, different seed
    x = make_inputs(sharding.rank_config(cfg, rank))

    def dev(a):
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)

    Q, K, V = dev(x["Q"]), dev(x["K"]), dev(x["V"])
    dO = dev(x["dO"]) if cfg.backward else None
    buf = binding.HgaLayerBuffers(cfg, backward=cfg.backward, flags=args.flags)
    buf.build_summaries(K, 0, cfg.history)          # resident history summaries
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    names = ["build_summaries", "route", "attn_fwd"] + (["attn_bwd"] if cfg.backward else [])

    def one_step(ev=None):
        if ev:
            ev[0].record(stream)
        buf.build_summaries(K)
        if ev:
            ev[1].record(stream)
        buf.route(Q)
        if ev:
            ev[2].record(stream)
        buf.attn_fwd(Q, K, V)
        if ev:
            ev[3].record(stream)
        if cfg.backward:
            buf.attn_bwd(Q, K, V, dO)
            if ev:
                ev[4].record(stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        flush.zero_()
        one_step()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    n_ev = len(names) + 1
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(n_ev)] for _ in range(args.steps)]
    launches0 = binding.hga_kernel_launch_count()
    barrier()
    for i in range(args.steps):
        flush.zero_()                     # evict L2 (untimed: events bracket the step only)
        one_step(events[i])
    barrier()
    launches = binding.hga_kernel_launch_count() - launches0
    per_call = np.array([[ev[j].elapsed_time(ev[j + 1]) for j in range(n_ev - 1)] for ev in events])  # ms
    eager_ms = np.array([ev[0].elapsed_time(ev[-1]) for ev in events])
    step_ms, launch_mode = eager_ms, "eager"
    if not args.no_graph:
        # The headline step: the same four C-ABI calls captured once into a CUDA graph and replayed,
        # which removes the host-side launch gaps between them.  Same K steps, same flush.
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                one_step()                                   # warm the capture stream
            torch.cuda.current_stream().wait_stream(side)
            graph = torch.cuda.CUDAGraph()
            c0 = binding.hga_kernel_launch_count()
            with torch.cuda.graph(graph):
                one_step()
            per_step_launches = binding.hga_kernel_launch_count() - c0
            for _ in range(3):
                flush.zero_()
                graph.replay()
            barrier()
            g_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                    for _ in range(args.steps)]
            for a, b in g_ev:
                flush.zero_()
                a.record(stream)
                graph.replay()
                b.record(stream)
            barrier()
            step_ms = np.array([a.elapsed_time(b) for a, b in g_ev])
            launches = per_step_launches * args.steps
            launch_mode = "cuda_graph"
        except Exception as exc:  # capture unavailable: keep the eager numbers, say why
            launch_mode = "eager (graph capture failed: %s)" % type(exc).__name__
    # warm-L2 variant (reported beside the headline, not instead of it)
    warm_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(n_ev)] for _ in range(args.steps)]
    for i in range(args.steps):
        one_step(warm_ev[i])
    barrier()
    warm_ms = np.array([ev[0].elapsed_time(ev[-1]) for ev in warm_ev])

    # end to end through the host-buffer entry point: H2D of the step's inputs, D2H of its results
    H = cfg.history
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).pin_memory()
    Qh, Kh, Vh = pin(x["Q"]), pin(x["K"][:, :, H:]), pin(x["V"][:, :, H:])
    dOh = pin(x["dO"]) if cfg.backward else None
    Oh = torch.empty_like(Qh).pin_memory()
    dQh = torch.empty_like(Qh).pin_memory() if cfg.backward else None
    dKh = torch.empty(cfg.batch, cfg.n_kv_heads, cfg.seg_len, cfg.head_dim).pin_memory() if cfg.backward else None
    dVh = torch.empty_like(dKh).pin_memory() if cfg.backward else None
    arena = torch.empty(binding.hga_step_arena_bytes(buf.p), dtype=torch.uint8, device="cuda")
    h2d = sum(t.numel() * t.element_size() for t in (Qh, Kh, Vh, dOh) if t is not None)
    d2h = sum(t.numel() * t.element_size() for t in (Oh, dQh, dKh, dVh) if t is not None)

    def host_step():
        binding.hga_step_host(buf.p, Qh, Kh, Vh, dOh, K, V, buf.chunk_sum, buf.group_sum, Oh, dQh,
                              dKh, dVh, arena, buf.status)

    for _ in range(3):
        host_step()
    barrier()
    e2e_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(args.steps)]
    for a, b in e2e_ev:
        flush.zero_()
        a.record(stream)
        host_step()
        b.record(stream)
    barrier()
    e2e_ms = np.array([a.elapsed_time(b) for a, b in e2e_ev])
    # whole-sequence walk (Section 2.2): every segment of a total_len sequence through the path, one layer
    walk = None
    if rank == 0 and world == 1 and cfg.backward and not args.no_walk and cfg.history > 0:
        walk = time_tbptt_walk(cfg, args, stream)
    clocks = sampler.stop() if rank == 0 else None      # sampled across all timed loops above
    # generation-shaped step (its inputs are drawn on the host first, so it runs outside the clock samples)
    decode = None
    if rank == 0 and world == 1 and args.config == 3 and not args.no_decode:
        decode = time_decode(args, stream, load_peaks())
    status = int(buf.status.item())

    def max_over_ranks(v):
        return sharding.max_over_ranks(v, device="cuda")

    total_ms = max_over_ranks(step_ms.sum())
    warm_total_ms = max_over_ranks(warm_ms.sum())
    e2e_total_ms = max_over_ranks(e2e_ms.sum())
    tokens = cfg.tokens_per_step * world * args.steps

    if rank == 0:
        peaks = load_peaks()
        gi, ng = buf.group_idx.cpu().numpy(), buf.n_groups.cpu().numpy()
        wc = work_counts(cfg, ng)
        extra_active = active_group_pairs(cfg, gi, ng)
        wc["bwd_flops"] += 4.0 * cfg.head_dim * extra_active
        med = np.median(per_call, axis=0) * 1e-3      # seconds per call
        roofs = {"attn_fwd": roofline_entry("hga_attn_fwd", wc["fwd_flops"], wc["fwd_bytes"], med[2], peaks)}
        if cfg.backward:
            roofs["attn_bwd"] = roofline_entry("hga_attn_bwd", wc["bwd_flops"], wc["bwd_bytes"], med[3], peaks)
        traffic, provenance = load_traffic(args.config)
        for r in roofs.values():
            r["traffic"] = traffic.get(r["kernel"])
            r["traffic_source"] = provenance
            r["algorithmic_bytes"] = wc["fwd_bytes"] if r["kernel"] == "hga_attn_fwd" else wc["bwd_bytes"]
            r["algorithmic_flops"] = wc["fwd_flops"] if r["kernel"] == "hga_attn_fwd" else wc["bwd_flops"]
        dominant = max(roofs.values(), key=lambda r: r["measured_us"])
        attn_us = sum(r["measured_us"] for r in roofs.values())
        attn_roof_us = sum(r["roofline_us"] for r in roofs.values())
        line = {
            "metric": METRIC, "value": round(tokens / (total_ms * 1e-3), 1), "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(total_ms / args.steps, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_dict(cfg, args),
            "clocks": clocks,
            "e2e": {"value": round(tokens / (e2e_total_ms * 1e-3), 1), "unit": "tokens/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": round(e2e_total_ms / args.steps, 5)},
            "gpu_launches": int(launches),
            "roofline": dominant,
            "roofline_all": roofs,
            "attention": {"fwd_plus_bwd_us": round(attn_us, 2), "roofline_us": round(attn_roof_us, 2),
                          "frac_of_roofline": round(attn_roof_us / attn_us, 4),
                          "tokens_per_s": round(cfg.tokens_per_step / (attn_us * 1e-6), 1)},
            "per_call_us_median": {n: round(float(m) * 1e6, 2) for n, m in zip(names, med)},
            "launch": launch_mode,
            "eager": {"value": round(cfg.tokens_per_step * args.steps / (eager_ms.sum() * 1e-3), 1),
                      "ms_per_step": round(float(eager_ms.mean()), 5)},
            "warm_l2": {"value": round(tokens / (warm_total_ms * 1e-3), 1),
                        "ms_per_step": round(warm_total_ms / args.steps, 5)},
            "device_status_word": status,
            "paper_context": "217.75 (HGA) / 207.02 (dense) tokens/s: whole-model QLoRA step at 2K on a "
                             "Quadro RTX 5000 (Table 2); another machine and scope, not the target",
        }
        if world == 1 and args.config == 3 and not args.no_configs:
            # the other benchmark configurations, each a few milliseconds of GPU time
            del Q, K, V, dO, arena
            torch.cuda.empty_cache()
            line["configs"] = {str(n): time_config(n, args, peaks) for n in (2, 4, 5, 6)}
        if world == 1 and args.config == 3 and not args.no_configs:
            line["varlen"] = time_varlen(args, stream)
        if walk is not None:
            line["tbptt_walk"] = walk
        if decode is not None:
            line["decode"] = decode
        if not args.no_cpu_baseline and world == 1:
            tps, threads, what, _ = oracle_throughput(cfg, x)
            line["cpu_baseline"] = {"value": round(tps, 3), "unit": "tokens/s", "cores": threads,
                                    "kind": "oracle", "sample": what}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
