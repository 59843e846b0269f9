#!/usr/bin/env python
"""Benchmark of the CompKV decode step (append + compensated sparse decode) at 128K context.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workload: benchmark configs[2] -- Llama-3-8B-shaped layer, batch 4, 32 query / 8 KV heads,
head_dim 128, bf16 paged KV, 131072 prefilled tokens per sequence, block size 16, budget 2048
tokens; every step appends one token per sequence (summary update) and decodes one query.
Seeded synthetic inputs.  One JSON line on stdout (rank 0).

A "step" is ckv_append + ckv_decode (summary update, summary scan, scoring + top-k, exact attention
on the selected blocks, compensation merge).  The one-off prefill summary build and the dense
baseline are timed separately and reported in the same line.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "sparse decode-attn us/step at 128K ctx (append + decode, batch 4)"
UNIT = "us/step"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
PAPER_CONTEXT = {"speedup_vs_full": 6.85, "hardware": "NVIDIA H100 80GB HBM3, CPU-offload pipeline, batch 1",
                 "setting": "128K endpoint, budget 512, r=4 (1.456 ms vs 9.966 ms)", "note": "context only"}
# DRAM traffic (reads + writes) per algorithmic byte of the summary-scan kernel, from the committed ncu capture
# (profiles/ckv_scan_kernel_llama8b_128k_b4.md): 206.06 MB read + 10.15 MB written for the 205.5 MB of summaries the
# step reads (mean keys hi + lo, mean values hi, variances).
SCAN_TRAFFIC_RATIO = (206.06 + 10.15) / 205.5
# What is stored and multiplied (the line's `dtype`): K/V pages are bf16; mean keys and mean values keep fp32
# precision as split bf16 pairs (hi = bf16(x), lo = bf16(x - hi), relative error <= 2^-18), variances are fp32; the
# decode step reads the mean keys as pairs and the mean values as their hi halves; the contractions run on bf16
# tensor-core tiles (mma.sync) with fp32 accumulation, everything else is fp32.
DTYPE = ("bf16 mma operands (bf16 K/V; summaries stored as split-bf16 pairs hi+lo, rel. error 2^-18, the step reading "
         "mean keys hi+lo and mean values hi; fp32 variances), fp32 accumulate")


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period: float = 0.002):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2.0)
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def workload(total_steps: int, args=None):
    """The bench workload: configs[2] of the baseline file (synth.CONFIGS[3]) unless overridden for a sweep point."""
    from paper_2609_26300_b200 import synth
    w = synth.CONFIGS[getattr(args, "config", 3) if args is not None else 3].with_(decode_steps=total_steps)
    if args is not None:
        over = {}
        if args.block_size:
            over["block_size"] = args.block_size
        if args.budget:
            over["budget_tokens"] = args.budget
        if args.var_groups:
            over["var_groups"] = args.var_groups
        if over:
            w = w.with_(**over)
    return w


def describe(w, default: bool) -> str:
    head = "configs[2] " if default else "sweep point of "
    ctx = "ctx %d" % w.ctx if w.ctx_min is None else "ctx %d..%d (ragged)" % (w.ctx_min, w.ctx)
    return ("%s%s: batch %d, %dq/%dkv heads, d%d, %s (+ appended tokens), block %d, budget %d, r=%d, "
            "fp32-precision summaries stored as split bf16 pairs (mean values read as hi halves when r = 4), bf16 paged KV"
            % (head, w.name, w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, ctx, w.block_size, w.budget_tokens,
               w.var_groups))


def step_inputs(w, n_steps: int):
    """Per-step queries and appended rows as numpy arrays [steps][...] (bf16 values in float32)."""
    from paper_2609_26300_b200 import synth
    q = np.stack([synth.queries(w, t) for t in range(n_steps)])
    k_new = np.zeros((n_steps, w.batch, w.num_kv_heads, w.head_dim), np.float32)
    v_new = np.zeros_like(k_new)
    for s in range(w.batch):
        for h in range(w.num_kv_heads):
            kt, vt = synth.unit_tail(w, s, h)
            k_new[:, s, h] = kt[:n_steps]
            v_new[:, s, h] = vt[:n_steps]
    return q, k_new, v_new


def oracle_sample_setup(w):
    """Inputs of the oracle's sample: every KV head of sequence 0, prefill + the appended rows."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import compkv_oracle as O
    from paper_2609_26300_b200 import synth
    heads = list(range(w.num_kv_heads))
    cores = min(os.cpu_count() or 1, len(heads))
    with ThreadPoolExecutor(cores) as ex:
        kv = list(ex.map(lambda h: synth.unit_kv(w, 0, h), heads))
        n0 = int(synth.seq_lens(w)[0])
        stats = list(ex.map(lambda i: O.stats(kv[i][0][:n0], kv[i][1][:n0], w.block_size, w.var_groups), heads))
    return kv, stats, n0, cores


def oracle_dense_step(w, kv, n0, cores, step: int):
    """The oracle's dense attention over the same sample units (Eq. 12 with every block selected); wall seconds."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import compkv_oracle as O
    from paper_2609_26300_b200 import synth
    q = synth.queries(w, step)[0]
    n = n0 + step + 1
    G = w.group
    t0 = time.perf_counter()
    with ThreadPoolExecutor(cores) as ex:
        list(ex.map(lambda h: O.dense(q[h * G:(h + 1) * G], kv[h][0][:n], kv[h][1][:n]), range(len(kv))))
    return time.perf_counter() - t0


def sweep_config5(dev, peak, steps: int = 16):
    """Benchmark configs[4]: batch 1, 128K context, block size {16, 32, 64} x budget {512, 1024, 2048, 4096} and
    the stats build per block size, against the dense decode of the same cache.  One cache for all points; every
    point is ckv_step captured as a CUDA graph, 3 warm-up + `steps` timed replays, L2 flushed before each."""
    import torch
    from paper_2609_26300_b200 import binding, synth
    base = synth.CONFIGS[5].with_(decode_steps=400)
    k_pool, v_pool, table, lens0 = synth.make_pools(base, threads=min(8, os.cpu_count() or 1))
    k_pool, v_pool, table = k_pool.to(dev), v_pool.to(dev), table.to(dev)
    n0 = int(lens0.max())
    max_len = n0 + 400
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    clean = torch.zeros(64 << 20, dtype=torch.float32, device=dev)
    q = torch.from_numpy(synth.queries(base, 0)).to(torch.bfloat16).to(dev)
    kn, vn = (torch.from_numpy(a).to(torch.bfloat16).to(dev) for a in synth.appended_rows(base, 0))
    points, builds = [], []
    dense_us = None
    for bs in synth.SWEEP_BLOCK_SIZES:
        w = base.with_(block_size=bs)
        lens = lens0.clone().to(dev)
        max_blocks = synth.pages_per_seq(w) * w.page_size // bs
        ckv = binding.CompKV(w.num_q_heads, w.num_kv_heads, w.batch, max_blocks, k_pool.shape[0], block_size=bs,
                             var_groups=w.var_groups, device=str(dev))
        ms = []
        for i in range(4):
            flush.zero_(); clean.sum()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); ckv.stats_build(k_pool, v_pool, table, lens, n0); e1.record()
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        b_us = float(np.median(ms[1:])) * 1e3
        b_bytes = n0 * w.num_kv_heads * 2 * w.head_dim * 2 + required_bytes(w, [n0], 0, stored=True)[0]
        builds.append({"block_size": bs, "us": b_us, "bytes": b_bytes, "gbs": b_bytes / (b_us * 1e-6) / 1e9,
                       "frac_of_peak": b_bytes / (b_us * 1e-6) / 1e9 / peak})
        if dense_us is None:
            dms = []
            for i in range(6):
                flush.zero_(); clean.sum()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); ckv.dense_decode(q, k_pool, v_pool, table, lens, max_len); e1.record()
                torch.cuda.synchronize()
                dms.append(e0.elapsed_time(e1))
            dense_us = float(np.median(dms[2:])) * 1e3
        for budget in synth.SWEEP_BUDGETS:
            outs = ckv.alloc_outputs(w.batch, budget)
            ckv.step(q, kn, vn, k_pool, v_pool, table, lens, max_len, budget, outs)   # eager warm-up
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                ckv.step(q, kn, vn, k_pool, v_pool, table, lens, max_len, budget, outs)
            ev = []
            for i in range(3 + steps):
                flush.zero_(); clean.sum()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); g.replay(); e1.record()
                ev.append((e0, e1))
            torch.cuda.synchronize()
            us = float(np.mean([a.elapsed_time(b) for a, b in ev[3:]])) * 1e3
            sel = outs[3].cpu().numpy()
            stats_b, sel_b = required_bytes(w, lens.cpu().numpy(), sel * bs)
            req = stats_b + sel_b
            points.append({"block_size": bs, "budget": budget, "us_per_step": us, "required_bytes": req,
                           "hbm_gbs": req / (us * 1e-6) / 1e9, "frac_of_peak": req / (us * 1e-6) / 1e9 / peak,
                           "speedup_vs_dense": dense_us / us})
            del g
        assert ckv.read_status() == 0
        del ckv
    del k_pool, v_pool, flush, clean
    torch.cuda.empty_cache()
    return {"workload": "configs[4]: batch 1, 32q/8kv heads, d128, ctx 131072, block {16,32,64} x budget {512,1024,2048,4096}",
            "steps_per_point": steps, "dense_us": dense_us, "dense_bytes": n0 * 8 * 2 * 128 * 2,
            "points": points, "stats_build": builds}


def oracle_step(w, kv, stats, n0, cores, step: int):
    """One oracle decode step (summary update, scores, selection, compensated attention) on the sample units.
    Returns wall seconds; stats are advanced in place."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import compkv_oracle as O
    from paper_2609_26300_b200 import synth
    q = synth.queries(w, step)[0]
    n = n0 + step + 1
    G = w.group

    def one(h):
        K, V = kv[h][0][:n], kv[h][1][:n]
        stats[h] = O.append(stats[h], K, V)
        O.decode_unit(q[h * G:(h + 1) * G], K, V, stats[h], w.budget_tokens)

    t0 = time.perf_counter()
    with ThreadPoolExecutor(cores) as ex:
        list(ex.map(one, range(len(kv))))
    return time.perf_counter() - t0


def required_bytes(w, lens, sel_tokens_per_unit, mean_bytes: int = 4, stored: bool = False):
    """Bytes one decode step must read: every block summary once, plus K and V of the selected tokens.

    With the default layout (full-precision summaries, four variance groups) the step reads the mean values as their
    bf16 hi halves: 2 bytes per coordinate instead of 4.  stored=True counts the summaries as they are stored (what
    the stats build and the chunked prefill write)."""
    value_bytes = 2 if (not stored and mean_bytes == 4 and w.var_groups == 4) else mean_bytes
    stats = 0
    for n in lens:
        x = -(-int(n) // w.block_size)
        stats += w.num_kv_heads * x * (w.head_dim * (mean_bytes + value_bytes) + 4 * w.var_groups)
    sel = int(np.sum(sel_tokens_per_unit)) * 2 * w.head_dim * 2
    return stats, sel


def reference_arm(args):
    """Times the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from oracle import compkv_oracle as O  # noqa: F401
    w = workload(args.warmup + args.steps)
    kv, stats, n0, cores = oracle_sample_setup(w)
    scale = w.batch   # the sample is one of `batch` equally sized sequences
    for t in range(args.warmup):
        oracle_step(w, kv, stats, n0, cores, t)
    times = [oracle_step(w, kv, stats, n0, cores, args.warmup + t) for t in range(args.steps)]
    us = float(np.mean(times)) * 1e6 * scale
    sample = ("CPU oracle (fp64, plain C) decode step on the %d KV heads of sequence 0 (1 of %d sequences), "
              "wall time x %d" % (w.num_kv_heads, w.batch, scale))
    line = {"impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            # the same workload string as the other arm's line (the oracle works on it in fp64; how the CUDA path stores
            # its summaries is part of that string because it is part of the workload's name there)
            "config": {"workload": describe(w, True), "sample": sample},
            "cpu_baseline": {"value": us, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--profile-steps", type=int, default=48)
    ap.add_argument("--e2e-steps", type=int, default=48)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the batch-1 128K sweep (configs[4])")
    # sweep points (the default line is configs[2]; these leave the metric's workload)
    ap.add_argument("--config", type=int, default=3, choices=[1, 2, 3, 4, 5], help="synth.CONFIGS index")
    ap.add_argument("--block-size", type=int, default=0)
    ap.add_argument("--budget", type=int, default=0)
    ap.add_argument("--var-groups", type=int, default=0)
    ap.add_argument("--layers", type=int, default=8, help="layers of the stacked-cache measurement (0 or 1: skip)")
    ap.add_argument("--stat-bf16", action="store_true", help="bf16 mean keys / mean values (half the summary bytes)")
    args = ap.parse_args()
    if args.impl == "reference":
        return reference_arm(args)

    import torch
    from paper_2609_26300_b200 import binding, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    torch.cuda.set_device(local)
    from paper_2609_26300_b200.replicas import Replicas
    rep = Replicas(device=torch.device("cuda", local))
    dist = rep.dist

    W, K, KP, KE = max(args.warmup, 3), args.steps, args.profile_steps, args.e2e_steps
    total = W + K + KP + KE + W + 2 * min(K, 64) + 16   # + the stacked-layers measurement
    w = workload(total, args)
    is_default = args.config == 3 and not (args.block_size or args.budget or args.var_groups or args.stat_bf16)
    dev = torch.device("cuda", local)

    # ---- inputs: every rank holds a full replica of the workload (the path does not shard) ----
    k_pool, v_pool, table, lens = synth.make_pools(w, threads=min(8, os.cpu_count() or 1))
    q_np, kn_np, vn_np = step_inputs(w, total)
    max_blocks = synth.pages_per_seq(w) * w.page_size // w.block_size   # the table row holds whole blocks
    ckv = binding.CompKV(w.num_q_heads, w.num_kv_heads, w.batch, max_blocks, k_pool.shape[0],
                         block_size=w.block_size, var_groups=w.var_groups, device=str(dev),
                         stat_bf16=int(args.stat_bf16))
    k_pool, v_pool, table, lens = (t.to(dev) for t in (k_pool, v_pool, table, lens))
    q_all = torch.from_numpy(q_np).to(torch.bfloat16).to(dev)
    kn_all = torch.from_numpy(kn_np).to(torch.bfloat16).to(dev)
    vn_all = torch.from_numpy(vn_np).to(torch.bfloat16).to(dev)
    n0 = int(lens.max())
    max_len = n0 + total
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    clean = torch.zeros(64 << 20, dtype=torch.float32, device=dev)
    outputs = ckv.alloc_outputs(w.batch, w.budget_tokens)

    def l2_flush():
        # write a buffer larger than L2, then read another one: L2 ends up holding clean lines of neither
        # the cache nor the summaries, so the timed step neither hits in L2 nor pays for dirty write-backs
        flush.zero_()
        clean.sum()

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- prefill summary build (timed separately) ----
    build_ms = []
    for i in range(5):
        l2_flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); ckv.stats_build(k_pool, v_pool, table, lens, n0); e1.record()
        torch.cuda.synchronize()
        build_ms.append(e0.elapsed_time(e1))
    build_us = float(np.median(build_ms[2:])) * 1e3
    build_bytes = sum(int(n) for n in lens.tolist()) * w.num_kv_heads * 2 * w.head_dim * 2 + \
        required_bytes(w, lens.tolist(), 0, 2 if args.stat_bf16 else 4, stored=True)[0]

    # ---- chunked prefill of the same cache from contiguous rows (pages + summaries in one pass), timed separately:
    # the rows are gathered from the pools, so the call rewrites what is already there ----
    prefill = None
    if is_default:
        tok = n0
        pages = table[:, :(tok + w.page_size - 1) // w.page_size].long()
        k_src = k_pool[pages].permute(0, 1, 3, 2, 4).reshape(w.batch, -1, w.num_kv_heads, w.head_dim)[:, :tok].contiguous()
        v_src = v_pool[pages].permute(0, 1, 3, 2, 4).reshape(w.batch, -1, w.num_kv_heads, w.head_dim)[:, :tok].contiguous()
        pf_ms = []
        for i in range(4):
            cur = torch.zeros_like(lens)
            l2_flush()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); ckv.prefill(k_pool, v_pool, table, cur, k_src, v_src, lens, tok); e1.record()
            torch.cuda.synchronize()
            pf_ms.append(e0.elapsed_time(e1))
        assert torch.equal(cur, lens) and ckv.read_status() == 0
        pf_us = float(np.median(pf_ms[1:])) * 1e3
        pf_bytes = 2 * (build_bytes - required_bytes(w, lens.tolist(), 0, stored=True)[0]) + required_bytes(w, lens.tolist(), 0, stored=True)[0]
        prefill = {"us": pf_us, "gbs": pf_bytes / (pf_us * 1e-6) / 1e9, "bytes": pf_bytes,
                   "note": "ckv_prefill: rows read once, written to their pages, summaries from the same pass"}
        del k_src, v_src
        torch.cuda.empty_cache()

    # ---- one step as a CUDA graph over static input buffers ----
    sq, sk, sv = q_all[0].clone(), kn_all[0].clone(), vn_all[0].clone()
    step = 0

    def eager_step(t):
        ckv.step(q_all[t], kn_all[t], vn_all[t], k_pool, v_pool, table, lens, max_len, w.budget_tokens, outputs)

    for _ in range(W):           # untimed eager warm-up (also pages in the kernels before capture)
        eager_step(step); step += 1
    torch.cuda.synchronize()
    launches0 = ckv.launch_count()
    graph = torch.cuda.CUDAGraph()
    sq.copy_(q_all[step]); sk.copy_(kn_all[step]); sv.copy_(vn_all[step])
    with torch.cuda.graph(graph):
        ckv.step(sq, sk, sv, k_pool, v_pool, table, lens, max_len, w.budget_tokens, outputs)
    launches_per_step = ckv.launch_count() - launches0
    # capture does not execute: seq_lens is unchanged, the captured step runs on replay

    def graph_step(t, ev=None):
        sq.copy_(q_all[t]); sk.copy_(kn_all[t]); sv.copy_(vn_all[t])
        l2_flush()
        if ev is not None:
            ev[0].record()
        graph.replay()
        if ev is not None:
            ev[1].record()

    for _ in range(W):
        graph_step(step); step += 1
    sync_all()
    sampler = ClockSampler(local)
    sampler.start()
    events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    t_wall0 = time.perf_counter()
    for i in range(K):
        graph_step(step, events[i]); step += 1
    sync_all()
    t_wall = time.perf_counter() - t_wall0
    clocks = sampler.stop()
    step_ms = np.array([a.elapsed_time(b) for a, b in events])
    ms_per_step = float(step_ms.mean())
    sel_cnt = outputs[3].cpu().numpy()
    lens_now = lens.cpu().numpy()
    stats_b, sel_b = required_bytes(w, lens_now, sel_cnt * w.block_size, 2 if args.stat_bf16 else 4)
    stats_stored_b = required_bytes(w, lens_now, 0, 2 if args.stat_bf16 else 4, stored=True)[0]
    assert ckv.read_status() == 0

    # ---- per-kernel durations (events between the launches), L2 flushed before each step ----
    stage = np.zeros((KP, 5))
    for i in range(KP):
        l2_flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); ckv.append(k_pool, v_pool, table, lens, kn_all[step], vn_all[step]); e1.record()
        _, ms = ckv.decode_profile(q_all[step], k_pool, v_pool, table, lens, max_len, w.budget_tokens, outputs)
        stage[i, 0] = e0.elapsed_time(e1)
        stage[i, 1:] = ms
        step += 1
    stage_us = stage[KP // 4:].mean(0) * 1e3
    scan_eager_us = float(stage_us[1])

    # ---- the dominant kernel alone: back-to-back launches between two events (its summaries exceed L2, so every
    # launch streams them from HBM); this is the duration the roofline figure uses ----
    l2_flush()
    ckv.scan_profile(q_all[step - 1], lens, max_len, 4)
    scan_us = float(np.median([ckv.scan_profile(q_all[step - 1], lens, max_len, 16) for _ in range(5)])) * 1e3

    # ---- the same graph replayed without the flush (warm L2: what stays resident is at most 126 MB of the last
    # things touched; the summaries alone are 273 MB) ----
    warm = []
    for i in range(min(K, 64)):
        sq.copy_(q_all[step]); sk.copy_(kn_all[step]); sv.copy_(vn_all[step])
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); graph.replay(); e1.record()
        warm.append((e0, e1)); step += 1
    torch.cuda.synchronize()
    warm_us = float(np.median([a.elapsed_time(b) for a, b in warm][len(warm) // 4:])) * 1e3

    # ---- steady-state decode: replays queued back to back inside ONE pair of events (fixed inputs, the cache still
    # grows by a token per step), so that the launch of a step overlaps the end of the one before it ----
    n_pipe = min(K, 64)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(n_pipe):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    pipe_us = e0.elapsed_time(e1) * 1e3 / n_pipe
    step += n_pipe

    # ---- a stack of layers: L independent caches (device copies of the same values in different memory), one step
    # of each per token, back to back with no flush -- every layer's summaries and pages are cold because the other
    # layers' 2.7 GB each went through L2 since they were last touched ----
    multi = None
    if args.layers > 1:
        try:
            layers = []
            for li in range(args.layers):
                kp, vp, ln = k_pool.clone(), v_pool.clone(), lens.clone()
                ck = binding.CompKV(w.num_q_heads, w.num_kv_heads, w.batch, max_blocks, k_pool.shape[0],
                                    block_size=w.block_size, var_groups=w.var_groups, device=str(dev),
                                    stat_bf16=int(args.stat_bf16))
                ck.stats_build(kp, vp, table, ln, int(ln.max()))
                outs = ck.alloc_outputs(w.batch, w.budget_tokens)
                ck.step(sq, sk, sv, kp, vp, table, ln, max_len, w.budget_tokens, outs)   # eager warm-up
                layers.append((ck, kp, vp, ln, outs))
            torch.cuda.synchronize()
            g_all = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_all):
                for ck, kp, vp, ln, outs in layers:
                    ck.step(sq, sk, sv, kp, vp, table, ln, max_len, w.budget_tokens, outs)
            n_tok = 8
            for _ in range(3):
                g_all.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(n_tok):
                g_all.replay()
            e1.record()
            torch.cuda.synchronize()
            assert all(ck.read_status() == 0 for ck, *_ in layers)
            multi = {"layers": args.layers, "tokens": n_tok,
                     "us_per_layer_step": e0.elapsed_time(e1) * 1e3 / (n_tok * args.layers),
                     "note": "one CUDA graph holding one ckv_step per layer, replayed per token; no flush: each "
                             "layer owns its own cache, summaries and workspace"}
            del layers, g_all
            torch.cuda.empty_cache()
        except RuntimeError as e:   # not enough device memory for the stack
            multi = {"layers": args.layers, "error": str(e)[:120]}

    # ---- dense decode attention over the same cache ----
    dense_ms = []
    dout = torch.empty_like(outputs[0])
    for i in range(12):
        l2_flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); ckv.dense_decode(q_all[step - 1], k_pool, v_pool, table, lens, max_len, dout, outputs[1]); e1.record()
        torch.cuda.synchronize()
        dense_ms.append(e0.elapsed_time(e1))
    dense_us = float(np.median(dense_ms[3:])) * 1e3
    dense_bytes = int(lens_now.sum()) * w.num_kv_heads * 2 * w.head_dim * 2

    # ---- end to end from pinned host buffers through ckv_step_host ----
    # A decode loop's usual shape: one set of pinned staging buffers, reused every step, on a stream of the caller's
    # own.  The step's inputs are written into the staging buffers inside the timed region (48 KB of host copies).
    kcap = w.budget_tokens // w.block_size
    hq_all = torch.from_numpy(q_np).to(torch.bfloat16)
    hk_all = torch.from_numpy(kn_np).to(torch.bfloat16)
    hv_all = torch.from_numpy(vn_np).to(torch.bfloat16)
    hq = torch.empty(w.batch, w.num_q_heads, w.head_dim, dtype=torch.bfloat16).pin_memory()
    hk = torch.empty(w.batch, w.num_kv_heads, w.head_dim, dtype=torch.bfloat16).pin_memory()
    hv = torch.empty_like(hk).pin_memory()
    ho = torch.empty(w.batch, w.num_q_heads, w.head_dim, dtype=torch.bfloat16).pin_memory()
    hi = torch.empty(w.batch, w.num_kv_heads, kcap, dtype=torch.int32).pin_memory()
    hc = torch.empty(w.batch, w.num_kv_heads, dtype=torch.int32).pin_memory()
    e2e_stream = torch.cuda.Stream()
    hq_np, hk_np, hv_np = (t.view(torch.int16).numpy() for t in (hq, hk, hv))            # pinned staging, as numpy views
    src_q, src_k, src_v = (t.view(torch.int16).numpy() for t in (hq_all, hk_all, hv_all))
    e2e_s = []
    with torch.cuda.stream(e2e_stream):
        for i in range(KE):
            l2_flush()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            np.copyto(hq_np, src_q[step]); np.copyto(hk_np, src_k[step]); np.copyto(hv_np, src_v[step])
            ckv.step_host(hq, hk, hv, k_pool, v_pool, table, lens, max_len, w.budget_tokens, ho, hi, hc)
            e2e_s.append(time.perf_counter() - t0)
            step += 1
    torch.cuda.synchronize()
    e2e_us = float(np.mean(e2e_s[KE // 4:])) * 1e6
    h2d = hq.numel() * 2 + hk.numel() * 2 + hv.numel() * 2
    d2h = ho.numel() * 2 + hi.numel() * 4 + hc.numel() * 4
    assert ckv.read_status() == 0

    # ---- max over ranks ----
    ms_per_step, e2e_us, scan_us, dense_us, scan_eager_us, warm_us, pipe_us = rep.max_over_ranks(
        [ms_per_step, e2e_us, scan_us, dense_us, scan_eager_us, warm_us, pipe_us])
    us_per_step = ms_per_step * 1e3

    if rank != 0:
        rep.close()
        return 0

    peak, peak_kind = measured_peak()
    req = stats_b + sel_b
    step_gbs = req / (us_per_step * 1e-6) / 1e9
    scan_gbs = stats_b / (scan_us * 1e-6) / 1e9
    line = {
        "metric": METRIC if is_default else "sparse decode-attn us/step (append + decode)", "value": us_per_step, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": DTYPE, "data": "synthetic",
        "config": {"workload": describe(w, is_default).replace("fp32 summaries", "bf16 summaries") if args.stat_bf16
                   else describe(w, is_default),
                   "step": "ckv_step (summary scan with the new token's append in its tail CTAs, select, attention + merge: three launches) replayed as one CUDA graph; CUDA events around each replay",
                   "l2": "flushed between steps (256 MiB memset then 256 MiB read, outside the events); per-step inputs exceed L2",
                   "replicas": "every rank runs the whole workload (the path does not shard)",
                   "kv_storage": "bf16", "seed": w.seed},
        "us_per_step_median": float(np.median(step_ms)) * 1e3, "us_per_step_min": float(step_ms.min()) * 1e3,
        "us_per_step_warm_l2": warm_us,
        "us_per_step_back_to_back": pipe_us,
        "multi_layer": multi,
        "us_per_step_note": "value: one graph replay per event pair, L2 flushed before it (includes the launch latency "
                            "of the graph); warm_l2: same without the flush; back_to_back: 64 replays queued inside "
                            "one event pair, no flush (every step still streams its summaries, more than the 126 MB L2 holds, "
                            "through it)",
        "tokens_per_s": rep.aggregate_tokens_per_s(w.batch, us_per_step),
        "required_bytes_per_step": req, "hbm_gbs": step_gbs,
        "required_bytes_note": "summary bytes the step reads (mean keys hi + lo, variances, and -- default layout -- the "
                               "mean values' hi halves) + K/V of the selected tokens; with whole summary rows, as the "
                               "summaries are stored, the count would be required_bytes_whole_rows",
        "required_bytes_whole_rows": int(stats_stored_b + sel_b),
        "frac_of_%s_peak_on_whole_rows" % peak_kind: (stats_stored_b + sel_b) / (us_per_step * 1e-6) / 1e9 / peak,
        "frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS, "frac_of_%s_peak" % peak_kind: step_gbs / peak,
        "dense_us": dense_us, "dense_gbs": dense_bytes / (dense_us * 1e-6) / 1e9,
        "speedup_vs_dense": dense_us / us_per_step,
        "stages_us": {"append": float(stage_us[0]), "scan": float(stage_us[1]), "select": float(stage_us[2]),
                      "attention": float(stage_us[3]), "merge": float(stage_us[4]),
                      "note": "the two-call route (ckv_append, then ckv_decode) launched eagerly with events between "
                              "the kernels; in the timed ckv_step the append runs inside the scan launch, beside "
                              "the scan CTAs, so its time does not add"},
        "prefill": prefill,
        "stats_build": {"us": build_us, "gbs": build_bytes / (build_us * 1e-6) / 1e9, "bytes": build_bytes},
        "roofline": {"kernel": "ckv_scan_kernel", "bound": "hbm", "achieved": scan_gbs, "peak": peak,
                     "peak_kind": "%s copy bandwidth" % peak_kind, "unit": "GB/s", "frac": scan_gbs / peak,
                     "frac_step": step_gbs / peak, "frac_step_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS,
                     "frac_step_note": "the whole step (scan, select, attention + merge) on its required bytes; "
                                       "`frac` is the dominant kernel alone",
                     "scan_form": "the launch timed here is the decode-only form (its tail CTAs redo the last "
                                  "block's terms but append nothing); in the timed step the same launch also "
                                  "appends the new token",
                     "algorithmic_bytes": stats_b, "launch_us": scan_us,
                     "timing": "average of 16 back-to-back launches between two CUDA events on the launching stream "
                               "(median of 5 such runs); inside an eager step, between events, the same kernel "
                               "takes launch_us_in_eager_step",
                     "launch_us_in_eager_step": scan_eager_us,
                     "traffic": SCAN_TRAFFIC_RATIO * stats_b,
                     "traffic_source": "dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of this launch "
                                       "configuration (profiles/ckv_scan_kernel_llama8b_128k_b4.md: 206.06 MB + "
                                       "10.15 MB for 205.5 MB of summaries read), scaled by the algorithmic bytes"},
        "clocks": clocks,
        "e2e": {"value": e2e_us, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "call": "ckv_step_host on the caller's own stream: the step's q/k_new/v_new are written into one set of pinned staging buffers (inside the timed region), out/sel_ids/sel_cnt come back into pinned buffers; returns when the results are complete in the host buffers"},
        "gpu_launches": int(launches_per_step * K),
        "wall_s_timed_region": t_wall,
        "paper_context": PAPER_CONTEXT,
    }
    if world == 1 and is_default and not args.no_sweep:
        sw = sweep_config5(dev, peak)
        line["sweep"] = sw
        b1 = next(p for p in sw["points"] if p["block_size"] == 16 and p["budget"] == 2048)
        line["batch1_128k"] = {"workload": "configs[4] point: batch 1, ctx 131072, block 16, budget 2048 (the paper's "
                                           "latency table is batch 1 throughout)",
                               "us_per_step": b1["us_per_step"], "required_mb": b1["required_bytes"] / 1e6,
                               "frac_of_%s_peak" % peak_kind: b1["frac_of_peak"], "dense_us": sw["dense_us"],
                               "speedup_vs_dense": b1["speedup_vs_dense"]}
    if world == 1 and not args.no_cpu_baseline:
        kv, stats, n0s, cores = oracle_sample_setup(w)
        reps = 6
        oracle_step(w, kv, stats, n0s, cores, 0)
        ts = [oracle_step(w, kv, stats, n0s, cores, 1 + i) for i in range(reps)]
        cpu_us = float(np.mean(ts)) * 1e6 * w.batch
        t1 = [oracle_step(w, kv, stats, n0s, 1, 1 + reps + i) for i in range(2)]
        td = [oracle_dense_step(w, kv, n0s, cores, i) for i in range(3)]
        td1 = [oracle_dense_step(w, kv, n0s, 1, i) for i in range(1)]
        line["cpu_baseline"] = {"value": cpu_us, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "value_1thread": float(np.mean(t1)) * 1e6 * w.batch,
                                "dense_value": float(np.mean(td[1:])) * 1e6 * w.batch,
                                "dense_value_1thread": float(np.mean(td1)) * 1e6 * w.batch,
                                "host_cores": os.cpu_count(),
                                "sample": "oracle decode step (summary update, scores, top-k, compensated attention) "
                                          "on the %d KV heads of sequence 0, %d steps, wall time x %d sequences; "
                                          "dense_value: the oracle's dense attention over the same units; "
                                          "`cores` = threads used (one per KV head), the *_1thread values use one"
                                          % (w.num_kv_heads, reps, w.batch)}
    print(json.dumps(line))
    rep.close()
    return 0


if __name__ == "__main__":
    sys.exit(main())
