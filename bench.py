#!/usr/bin/env python
"""Benchmark of the LOCKS decode hot path on B200.

A "step" is one pass of the whole path over one batch of synthetic input: append the new token's
K/V, scan + score every resident page summary, share-average + top-k, sparse paged attention over
the selected pages, and the summary build of pages that just filled -- one `locks_decode_step`,
captured in a CUDA graph and replayed.  The workload is the Llama-3.1-8B-shaped configuration
(32 q heads / 8 KV heads, d 128, page 16, bf16 KV, batch 8 x 32K context, r8i4, b = 2048).

Cold caches: the step touches about 175 MB and B200's L2 holds 126 MB, so the replays cycle over
several independent "layers" (own KV cache, summaries and query), as a real model would; by the
time a layer comes round again its lines are gone.

Prints ONE JSON line: metric / value / unit, the step time over exactly K replays, `windows` (mean and spread over
three windows of 64 replays), `e2e` (the same step through the host-buffer entry point, copies included),
`roofline` (scan kernel: algorithmic bytes / measured kernel time against the measured copy bandwidth, plus the
kernel's DRAM traffic from the committed ncu capture), `cpu_baseline` (the oracle on the host cores), per-stage
times, the dense flash-decode time on the same inputs, the bulk summary build, `multi_layer_graph` (for information:
the same steps with all layers in one graph), clocks, launch count, and
`workloads`: a compact table (step, bytes, fraction of peak, dense) for one cell of each other configuration.  `--impl reference` times the CPU
oracle instead (test infrastructure; the only other place this file runs it is `cpu_baseline`).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "decode_step_us"
UNIT = "us"
FALLBACK_HBM_GBS = 6650.0


def workload(name: str):
    import locks_synth
    if name == "cfg1":
        return locks_synth.config1()
    if name == "cfg3_1m":
        return locks_synth.config3(T=1 << 20)
    if name == "cfg3_128k":
        return locks_synth.config3(T=1 << 17)
    if name.startswith("cfg2_"):          # cfg2_r8_b1024, cfg2_r2_b256, ...
        _, r, b = name.split("_")
        return locks_synth.config2(rank=int(r[1:]), budget=int(b[1:]))
    if name == "cfg3_512k":
        return locks_synth.config3(T=1 << 19)
    if name.startswith("cfg3g8_"):        # the paper's stated GLM geometry: 4 KV heads, G = 8
        T = {"128k": 1 << 17, "512k": 1 << 19, "1m": 1 << 20}[name[7:]]
        return locks_synth.config3(T=T, Hkv=4)
    if name == "cfg3_mix":               # two GLM-shaped requests of very different lengths (512K and 32K tokens)
        return locks_synth.Workload("cfg3_glm_mix_512k_32k", [1 << 19, 1 << 15], Hq=32, Hkv=2, seed=3)
    if name.startswith("cfg4_b"):
        return locks_synth.config4(batch=int(name[6:]))
    if name == "small":
        return locks_synth.Workload("small", [4096] * 2, Hq=8, Hkv=2, budget=256)
    raise SystemExit(f"unknown workload {name}")


def algorithmic_bytes(w, reserve_tokens=0):
    """Bytes the method itself must move per step: 818 B (r8i4 payload) per scored (page, KV head) for the scan,
    8192 B per selected (page, KV head) for attention."""
    payload = {8: 818, 4: 490, 2: 326}[w.rank] if w.fmt == "i4" else 4 * (128 + w.rank * 128 + 16 * w.rank)
    scan = attend = dense = 0
    for T in w.seq_lens:
        P = -(-T // w.B)
        k = min(w.k, P)
        scan += w.Hkv * max(P - 2, 0) * payload if P > w.k else 0
        attend += w.Hkv * k * w.B * w.d * 2 * 2
        dense += w.Hkv * P * w.B * w.d * 2 * 2
    return scan, attend, dense


def config_dict(w, layers, identity, partition="auto"):
    scan_b, att_b, _ = algorithmic_bytes(w)
    return {"workload": w.name, "batch_per_gpu": w.n, "context": w.seq_lens[0], "q_heads": w.Hq, "kv_heads": w.Hkv,
            "head_dim": w.d, "page": w.B, "rank": w.rank, "budget_tokens": w.budget,
            "summary": f"r{w.rank}i4" if w.fmt == "i4" else f"r{w.rank}f32", "launch": "one CUDA graph per step",
            "block_mapping": "identity" if identity else "seeded random permutation",
            "scan_partition": partition,
            "l2": f"inputs larger than L2: replays cycle over {layers} independent layers "
                  f"({(scan_b + att_b) / 1e6:.0f} MB touched per step, L2 126 MB)"}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def recorded_traffic(wname):
    """DRAM bytes per scan launch (dram__bytes_read.sum + dram__bytes_write.sum) copied from the committed ncu
    summary of this workload, with the file it was copied from; (None, None) when no capture covers it.  The
    number is evidence about re-reads, not an input of any timing: it moves only when the kernel's memory
    access pattern changes, and the summary file names the source revision it was captured at."""
    p = os.path.join(ROOT, "profiles", "scan_dram_traffic.json")
    if os.path.exists(p):
        try:
            e = json.load(open(p)).get(wname)
            if e:
                return float(e["bytes_per_launch"]), f"profiles/{e['summary']} (captured at {e['revision']})"
        except Exception:
            pass
    return None, None


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(w, steps: int, threads: int):
    """Time the oracle's decode step (score -> select -> attend on resident summaries) on a bounded
    sample of the workload: the first `nreq` requests, full context.  Returns (us per full-batch
    step scaled from the sample, sample description, seconds spent)."""
    import numpy as np
    import torch
    import locks_synth
    import oracle
    oracle.set_threads(threads)
    nreq = 1
    ws = w.with_(seq_lens=w.seq_lens[:nreq])
    case = locks_synth.make_case(ws, device="cpu")

    def bits(t):
        t = t.contiguous()
        return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()

    sb, sh, st = case.strides
    cache = oracle.Cache(bits(case.k), bits(case.v), case.block_table.numpy(), case.seq_lens.numpy(), w.Hq,
                         strides={"shape": (case.num_blocks, w.Hkv, w.B, w.d), "block": sb, "head": sh, "token": st})
    fmt = oracle.FMT_I4 if w.fmt == "i4" else oracle.FMT_F32
    summ = oracle.build_summaries(cache, w.rank, fmt)
    q = bits(case.q)
    sm = 1.0 / math.sqrt(w.d)
    oracle.decode_step(cache, q, w.rank, fmt, summ, sm, w.k)          # warm the caches once
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.decode_step(cache, q, w.rank, fmt, summ, sm, w.k)
    dt = (time.perf_counter() - t0) / steps
    scale = w.n / nreq
    return dt * 1e6 * scale, f"{nreq} of {w.n} requests ({ws.Hkv} KV heads, full {ws.seq_lens[0]}-token context), " \
                             f"time scaled by {scale:g}", dt * steps


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    import oracle
    w = workload(args.workload)
    cores = oracle.max_threads()
    steps = max(1, min(args.steps, 5))
    us, sample, _ = oracle_sample(w, steps, cores)
    scan, attend, dense = algorithmic_bytes(w)
    line = {"impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": 1, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": config_dict(w, args.layers, args.identity_blocks, args.scan_partition),
            "cpu_baseline": {"value": us, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def stagger(w, li):
    """Start lengths of the timed run: the configuration's context minus 1 .. 16 tokens, different per request
    and layer, so that requests cross page boundaries at different steps and a typical step contains the
    summary build of the pages that fill (with every length a multiple of 16 no timed step would)."""
    return [max(1, t - 1 - ((5 * b + 3 * li) % w.B)) for b, t in enumerate(w.seq_lens)]


def measure(args, w0, K, W, L, rank, local_rank, full):
    """Build the workload on the device and time the decode step.  `full`: everything the JSON line carries;
    otherwise the compact row of the per-workload table (step, dense, stage split)."""
    import torch
    import locks_synth
    import paper_2607_24555_b200 as locks
    from paper_2607_24555_b200 import dist as ldist
    from paper_2607_24555_b200.binding import KVView, make_config

    dev = f"cuda:{local_rank}"
    NW, WSTEPS = (3, 64) if (full and not args.no_windows) else (0, 0)
    grow = (W + K + NW * WSTEPS + (K + 2) + (4 * L + 3 * K if full else 0)) // L + 24   # tokens appended per layer
    reserve = -(-grow // w0.B) + 2
    layers = []
    for li in range(L):
        w = w0.with_(seed=w0.seed * 1000 + 17 * li + 101 * rank, seq_lens=[t + reserve * w0.B for t in w0.seq_lens],
                     permute_blocks=not args.identity_blocks)
        case = locks_synth.make_case(w, device=dev)
        case.seq_lens.copy_(torch.tensor(stagger(w0, li), dtype=torch.int32, device=dev))
        layers.append(case)
    max_pages = layers[0].block_table.shape[1]
    cfg = make_config(w0.Hq, w0.Hkv, w0.rank, w0.fmt, w0.dtype, w0.n, max_pages, w0.budget)
    ctx = locks.Context(cfg, device=dev)
    ctx.locks_set_scan_partition({"auto": locks.PARTITION_AUTO, "strided": locks.PARTITION_STRIDED,
                                  "balanced": locks.PARTITION_BALANCED}[args.scan_partition])
    kvs = [KVView(c.k, c.v, c.strides, c.num_blocks, c.block_table, c.seq_lens) for c in layers]
    summs = [ctx.new_summaries(c.num_blocks) for c in layers]
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        for kv, s in zip(kvs, summs):                       # first pass also loads the kernel
            ctx.locks_build_summaries(kv, w0.n, s, stream=stream)
        stream.synchronize()
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b0.record(stream)
        for kv, s in zip(kvs, summs):
            ctx.locks_build_summaries(kv, w0.n, s, stream=stream)
        b1.record(stream)
        stream.synchronize()
    bulk_build_ms = b0.elapsed_time(b1) / L
    build_pages = sum((t // w0.B) for t in stagger(w0, 0)) * w0.Hkv
    outs = [torch.empty(w0.n, w0.Hq, w0.d, dtype=torch.bfloat16 if w0.dtype == "bf16" else torch.float32, device=dev)
            for _ in layers]
    news = [locks_synth.new_token(w0.with_(seed=w0.seed + li), li, device=dev) for li in range(L)]

    def step(li, s=None):
        kn, vn, qn = news[li]
        ctx.locks_decode_step(qn, kn, vn, kvs[li], summs[li], w0.n, outs[li], stream=s or stream)

    # ---- capture one graph per layer (after one eager step each, which also warms the kernels)
    graphs = []
    with torch.cuda.stream(stream):
        for li in range(L):
            step(li)
        stream.synchronize()
        partition = ctx.locks_last_scan_partition()
        for li in range(L):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                step(li)
            graphs.append(g)
    launches_per_step = ctx.locks_last_launch_count()
    torch.cuda.synchronize()
    done = [0]

    def run_graph_steps(n):
        for _ in range(n):
            graphs[done[0] % L].replay()
            done[0] += 1

    res = {}
    with torch.cuda.stream(stream):
        run_graph_steps(W)
        stream.synchronize()
        ldist.barrier()
        torch.cuda.synchronize()
        sampler = ClockSampler(local_rank) if rank == 0 else None
        # ---- spread: three windows of 64 replays each (the paper's own timing cell: 3 x 64 decode steps).  They
        # run first: the first summary builds of a process fetch their code from HBM (+10 us on a step), and a
        # serving process is past that after a few dozen steps.
        wins = []
        for _ in range(NW):
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            run_graph_steps(WSTEPS)
            a1.record(stream)
            stream.synchronize()
            wins.append(a0.elapsed_time(a1) / WSTEPS * 1e3)
        res["windows_us"] = wins
        ldist.barrier()
        torch.cuda.synchronize()
        # ---- timed region: exactly K graph replays between barrier + synchronize
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        run_graph_steps(K)
        e1.record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        ldist.barrier()
        res["step_ms"] = e0.elapsed_time(e1) / K
        # ---- per-kernel split: the same step captured with event-record nodes at the stage boundaries,
        # replayed K times, durations read after each replay (CUDA events on the launch stream)
        ctx.locks_profile_begin(1)
        pgraphs = []
        for li in range(L):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                step(li)
            pgraphs.append(g)
        stage_ms = {"scan": 0.0, "select": 0.0, "attend": 0.0}
        for i in range(K + 2):
            pgraphs[(done[0] + i) % L].replay()
            one = ctx.locks_profile_read(stream=stream)
            if i >= 2:
                for k_ in stage_ms:
                    stage_ms[k_] += one[k_] / K
        ctx.locks_profile_end()
        res["stage_ms"] = stage_ms
        # ---- dense flash-decode over the full cache on the same GPU (same entry point, no page table)
        for li in range(min(L, 3)):
            ctx.locks_sparse_attend(news[li][2], kvs[li], w0.n, None, None, outs[li], stream=stream)
        stream.synchronize()
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        nd = max(3, min(K, 10))
        d0.record(stream)
        for i in range(nd):
            ctx.locks_sparse_attend(news[i % L][2], kvs[i % L], w0.n, None, None, outs[i % L], stream=stream)
        d1.record(stream)
        stream.synchronize()
        res["dense_ms"] = d0.elapsed_time(d1) / nd
        res["clocks"] = sampler.stop() if sampler else None
        if full:
            # ---- for information: the same steps with all L layers captured in ONE graph, as a caller that batches a
            # model's layers would launch them (the launch gap is paid once per L steps and the next scan is
            # scheduled while the attention drains); not the headline, which keeps one graph per step
            mg = torch.cuda.CUDAGraph()
            with torch.cuda.graph(mg, stream=stream):
                for li in range(L):
                    step(li)
            reps = max(2, K // L)
            mg.replay()
            stream.synchronize()
            m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            m0.record(stream)
            for _ in range(reps):
                mg.replay()
            m1.record(stream)
            stream.synchronize()
            res["multi_layer_graph_us"] = m0.elapsed_time(m1) / (reps * L) * 1e3
            del mg
            # ---- end to end through the host-buffer entry point: H2D of q, k_new, v_new and D2H of out every step
            hq = [n[2].cpu().pin_memory() for n in news]
            hk = [n[0].cpu().pin_memory() for n in news]
            hv = [n[1].cpu().pin_memory() for n in news]
            hout = torch.empty_like(outs[0], device="cpu").pin_memory()
            for i in range(3 * L):   # every layer's arguments seen often enough for the library to cache its launch
                ctx.locks_decode_step_host(hq[i % L], hk[i % L], hv[i % L], kvs[i % L], summs[i % L], w0.n, hout, stream=stream)
            ldist.barrier()
            t0 = time.perf_counter()
            for i in range(K):
                li = (3 * L + i) % L
                ctx.locks_decode_step_host(hq[li], hk[li], hv[li], kvs[li], summs[li], w0.n, hout, stream=stream)
            res["e2e_ms"] = (time.perf_counter() - t0) * 1e3 / K
    res["status"] = ctx.locks_poll_status()
    res["launches_per_step"] = launches_per_step
    res["bulk_build_ms"] = bulk_build_ms
    res["build_pages"] = build_pages
    res["partition"] = {0: "none", 1: "strided", 2: "balanced"}.get(partition, str(partition))
    res["max_pages"] = max_pages
    ctx.close()
    del graphs, pgraphs, layers, kvs, summs, outs, news
    torch.cuda.empty_cache()
    return res


def table_row(args, name, K, W, rank, local_rank, peak):
    w = workload(name)
    r = measure(args, w, K, W, args.layers, rank, local_rank, full=False)
    scan_b, att_b, dense_b = algorithmic_bytes(w)
    step_us = r["step_ms"] * 1e3
    return {"workload": w.name, "step_us": round(step_us, 2), "algorithmic_bytes": scan_b + att_b,
            "frac_of_measured_peak": round((scan_b + att_b) / (step_us * 1e-6) / 1e9 / peak, 4),
            "dense_us": round(r["dense_ms"] * 1e3, 2),
            "stages_us": {k_: round(v * 1e3, 2) for k_, v in r["stage_ms"].items()},
            "scan_frac": round(scan_b / (r["stage_ms"]["scan"] * 1e-3) / 1e9 / peak, 4) if scan_b else None,
            "scan_partition": r["partition"], "bulk_build_ms_per_layer": round(r["bulk_build_ms"], 3),
            "device_status": r["status"]}


def run_ours(args):
    import torch
    from paper_2607_24555_b200 import dist as ldist

    rank, local_rank, world = ldist.env_rank_world()
    if world > 1:
        import torch.distributed as tdist
        tdist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    K, W = args.steps, max(args.warmup, 3)
    w0 = workload(args.workload)
    L = args.layers
    # every rank owns a full batch (weak scaling): requests are independent, no data-path collective
    r = measure(args, w0, K, W, L, rank, local_rank, full=True)
    step_ms_max = ldist.max_over_ranks(r["step_ms"], device=dev)
    e2e_ms_max = ldist.max_over_ranks(r["e2e_ms"], device=dev)
    peak, peak_kind = measured_peak()
    rows = []
    if args.table and world == 1 and rank == 0:
        for name in args.table.split(","):
            if name and workload(name).name != w0.name:
                rows.append(table_row(args, name, 16, 3, rank, local_rank, peak))
    if rank != 0:
        return
    stage_ms = r["stage_ms"]
    scan_b, att_b, dense_b = algorithmic_bytes(w0)
    scan_gbs = scan_b / (stage_ms["scan"] * 1e-3) / 1e9
    esz = 2 if w0.dtype == "bf16" else 4
    h2d = w0.n * (w0.Hq + 2 * w0.Hkv) * w0.d * esz
    d2h = w0.n * w0.Hq * w0.d * esz
    cores = os.cpu_count() or 1
    cpu_us = cpu_sample = None
    if not args.no_cpu_baseline:
        import oracle
        cores = oracle.max_threads()
        cpu_us, cpu_sample, _ = oracle_sample(w0, 5, cores)
    wins = r["windows_us"]
    build_bytes = r["build_pages"] * (4096 + 818)
    traffic, traffic_src = recorded_traffic(w0.name)
    cfg_d = config_dict(w0, L, args.identity_blocks, r["partition"])
    cfg_d["start_lengths"] = "context minus 1..16 tokens, staggered per request and layer: steps include the summary " \
                             "build of the pages that fill"
    cfg_d["order"] = "W warm-up replays, three 64-replay windows (reported under `windows`), then the K timed replays"
    line = {
        "metric": METRIC, "value": step_ms_max * 1e3, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": step_ms_max, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if w0.dtype == "bf16" else "f32", "data": "synthetic",
        "config": cfg_d,
        "e2e": {"value": e2e_ms_max * 1e3, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": r["launches_per_step"] * K,
        "clocks": r["clocks"],
        "roofline": {"bound": "hbm", "kernel": "scan_i4_kernel", "achieved": scan_gbs, "peak": peak, "unit": "GB/s",
                     "frac": scan_gbs / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                     "traffic_source": traffic_src,
                     "algorithmic_bytes_per_launch": scan_b, "launch_us": stage_ms["scan"] * 1e3},
        "step_roofline": {"algorithmic_bytes": scan_b + att_b, "achieved": (scan_b + att_b) / (step_ms_max * 1e-3) / 1e9,
                          "frac": (scan_b + att_b) / (step_ms_max * 1e-3) / 1e9 / peak, "unit": "GB/s",
                          "frac_of_8000": (scan_b + att_b) / (step_ms_max * 1e-3) / 1e9 / 8000.0},
        "multi_layer_graph": {"layers_per_graph": L, "us_per_step": r.get("multi_layer_graph_us")},
        "windows": {"replays_per_window": 64, "us_per_step": [round(x, 3) for x in wins],
                    "mean_us": statistics.mean(wins) if wins else None,
                    "sd_us": statistics.stdev(wins) if len(wins) > 1 else None},
        "stages_us": {k_: v * 1e3 for k_, v in stage_ms.items()},
        "dense_flash_decode": {"us": r["dense_ms"] * 1e3, "bytes": dense_b,
                               "achieved_gbs": dense_b / (r["dense_ms"] * 1e-3) / 1e9,
                               "speedup_of_step": r["dense_ms"] / step_ms_max},
        "bulk_build_ms_per_layer": r["bulk_build_ms"],
        "bulk_build": {"ms_per_layer": r["bulk_build_ms"], "page_heads": r["build_pages"], "algorithmic_bytes": build_bytes,
                       "achieved_gbs": build_bytes / (r["bulk_build_ms"] * 1e-3) / 1e9,
                       "frac": build_bytes / (r["bulk_build_ms"] * 1e-3) / 1e9 / peak},
        "device_status": r["status"],
        "workloads": rows,
        "cpu_baseline": ({"value": cpu_us, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": cpu_sample}
                         if cpu_us is not None else None),
    }
    print(json.dumps(line))


def run_diagnostics(args):
    """Selection fidelity on the synthetic workloads (the paper's App. B metrics): for the summary's own score, the
    exact-LSE arm and the rival scorers, all under the same share-average selection, measured against exact page
    masses by the library's own kernels.  Prints one JSON line."""
    import torch
    import locks_synth
    import paper_2607_24555_b200 as locks
    from paper_2607_24555_b200.binding import KVView, make_config
    dev = "cuda:0"
    rows = []
    cells = [("cfg0_tiny", locks_synth.config0()), ("cfg1_llama_8x32k", locks_synth.config1().with_(carriers=16)),
             ("cfg2_qwen_32x16k_r8_b1024", locks_synth.config2(rank=8, budget=1024)),
             ("cfg2_qwen_32x16k_r2_b256", locks_synth.config2(rank=2, budget=256)),
             ("cfg1_soft_queries", locks_synth.config1().with_(q_scale=0.25, carriers=0))]
    for name, w in cells:
        case = locks_synth.make_case(w, device=dev)
        max_pages = case.block_table.shape[1]
        ctx = locks.Context(make_config(w.Hq, w.Hkv, w.rank, w.fmt, w.dtype, w.n, max_pages, w.budget), device=dev)
        kv = KVView(case.k, case.v, case.strides, case.num_blocks, case.block_table, case.seq_lens)
        summ = ctx.new_summaries(case.num_blocks)
        ctx.locks_build_summaries(kv, w.n, summ)
        mk = lambda: (torch.zeros(w.n, w.Hkv, w.k, dtype=torch.int32, device=dev), torch.zeros(w.n, w.Hkv, dtype=torch.int32, device=dev))
        ids_e, cnt_e = mk()
        mass = torch.zeros(w.n, w.Hq, max_pages, dtype=torch.float32, device=dev)
        ctx.locks_select_exact(case.q, kv, w.n, ids_e, cnt_e, mass)
        ncar = max((len(c) for c in case.carrier_pages), default=0)
        marked = None
        if ncar:
            marked = torch.full((w.n, ncar), -1, dtype=torch.int32, device=dev)
            for b, cps in enumerate(case.carrier_pages):
                marked[b, :len(cps)] = torch.tensor(cps, dtype=torch.int32, device=dev)
        row = {"workload": name, "budget_tokens": w.budget, "rank": w.rank, "carriers_per_request": ncar, "scorers": {}}
        arms = [("exact_lse", None), ("locks_summary", 0), ("moment_core", locks.SCORER_MOMENT),
                ("centroid_only", locks.SCORER_CENTROID), ("envelope_quest", locks.SCORER_ENVELOPE)]
        for label, sc in arms:
            ids, cnt = mk()
            if sc is None:
                ids, cnt = ids_e, cnt_e
            elif sc == 0:
                ctx.locks_select(case.q, summ, kv, w.n, ids, cnt)
            else:
                ctx.locks_select_rival(sc, case.q, summ, kv, w.n, ids, cnt)
            qual = torch.zeros(w.n, w.Hkv, 4, dtype=torch.float32, device=dev)
            ctx.locks_selection_quality(mass, kv, w.n, ids, cnt, ids_e, cnt_e, qual, marked_pages=marked)
            torch.cuda.synchronize()
            m = qual.mean(dim=(0, 1)).tolist()
            row["scorers"][label] = {"gamma": round(m[0], 4), "gamma_c": round(m[1], 4), "recall": round(m[2], 4),
                                     "needle": round(m[3], 4) if ncar else None}
        # ---- the combine rules of the paper's GQA ablation (App. D) on the summary's scores: mass kept by each rule's
        # page tables (mean over the query heads); the per-head arm keeps one table per query head
        row["combine_rules"] = {}
        if w.G > 1:
            for label, rule in (("share_average", locks.COMBINE_SHARE_AVG), ("group_max", locks.COMBINE_GROUP_MAX),
                                ("group_mass", locks.COMBINE_GROUP_MASS), ("per_head", locks.COMBINE_PER_HEAD)):
                per_head = rule == locks.COMBINE_PER_HEAD
                c2 = locks.Context(make_config(w.Hq, w.Hkv, w.rank, w.fmt, w.dtype, w.n, max_pages, w.budget, combine=rule), device=dev)
                H = w.Hq if per_head else w.Hkv
                ids = torch.zeros(w.n, H, w.k, dtype=torch.int32, device=dev)
                cnt = torch.zeros(w.n, H, dtype=torch.int32, device=dev)
                c2.locks_select(case.q, summ, kv, w.n, ids, cnt)
                # the metrics kernel of a context whose groups are single heads reads a table per query head
                cq = locks.Context(make_config(w.Hq, w.Hq, w.rank, w.fmt, w.dtype, w.n, max_pages, w.budget), device=dev) if per_head else ctx
                qual = torch.zeros(w.n, H, 4, dtype=torch.float32, device=dev)
                cq.locks_selection_quality(mass, kv, w.n, ids, cnt, ids, cnt, qual, marked_pages=marked)
                torch.cuda.synchronize()
                m = qual.mean(dim=(0, 1)).tolist()
                row["combine_rules"][label] = {"gamma": round(m[0], 4), "gamma_c": round(m[1], 4)}
                if per_head:
                    cq.close()
                c2.close()
        rows.append(row)
        ctx.close()
        del case, summ, mass
        torch.cuda.empty_cache()
    print(json.dumps({"diagnostics": "selection fidelity against exact page masses (App. B metrics), synthetic keys",
                      "rows": rows}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=48)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg1")
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--table", default="cfg2_r8_b1024,cfg3_1m,cfg4_b8",
                    help="comma-separated workloads measured compactly (few steps) for the `workloads` table of the "
                         "JSON line; empty: none")
    ap.add_argument("--scan-partition", default="auto", choices=["auto", "strided", "balanced"],
                    help="how the scan deals pages to its warps (auto: the library follows the lengths)")
    ap.add_argument("--identity-blocks", action="store_true",
                    help="logical page i of a request sits in consecutive physical blocks (default: seeded permutation)")
    ap.add_argument("--no-windows", action="store_true", help="skip the three 64-replay windows (short profiling runs)")
    ap.add_argument("--diagnostics", action="store_true",
                    help="print the selection-fidelity table (gamma, gamma_c, recall, needle per scorer) instead of timing")
    args = ap.parse_args()
    if args.diagnostics:
        run_diagnostics(args)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
