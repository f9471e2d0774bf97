#!/usr/bin/env python
"""Benchmark of the HybridKV decode hot path on B200.

A *step* is one autoregressive decode step of attention over the hybrid-compressed KV cache of the
whole model: one hkv_decode_attn per layer (chunk score + top-k for dynamic heads, split-K
flash-decode over static and selected dynamic KV, merge), layers in sequence on one stream, captured
once in a CUDA graph.  Default workload: the 28-layer, batch-4, 24K-32K-token video-like
configuration ("cfg2": static fraction 0.6, budget 10 %, chunk 64) with seeded synthetic inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]

Prints ONE JSON line (rank 0).  `value` = algorithmic HBM bytes per step (512 B per retained token
+ 256 B per chunk mean) summed over all ranks / step time; `us_per_step` is the step latency.
Under torchrun every rank runs its own replica of the workload (different seed): weak scaling, no
data-path collective.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

FALLBACK_HBM_GBS = 6650.0          # earlier measurement on this machine, used only without MEASURED_PEAKS.json
NOMINAL_HBM_GBS = 8000.0           # nominal HBM3e bandwidth of a B200, the second denominator reported
N_LAYERS = {"cfg0": 1, "cfg1": 28, "cfg2": 28, "cfg3": 28, "cfg4": 1}
N_QUERY_SETS = 8                   # distinct seeded queries per layer, rotated step by step
STATS_REPLAYS = 500                # per-step CUDA-event pairs behind median / min / mean


def kernel_revision() -> str:
    """Identifies the decode kernel's code (comments and blank space do not count): ncu counters are only quoted
    for the revision they were taken on."""
    import hashlib
    import re
    h = hashlib.sha256()
    for f in ("hkv_decode.cu", "hkv_device.cuh", "hkv_internal.h"):
        text = open(os.path.join(ROOT, "paper_2604_05887_b200", "csrc", f)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        text = re.sub(r"//[^\n]*", "", text)
        h.update(" ".join(text.split()).encode())
    return h.hexdigest()[:12]


def ncu_traffic(workload: str):
    """DRAM bytes per launch of the decode kernel (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu
    capture summarised in profiles/decode_kernel_traffic.txt: lines `workload revision bytes`.  None when no
    line matches the kernel as it is now (the counters then belong to an older kernel)."""
    path = os.path.join(ROOT, "profiles", "decode_kernel_traffic.txt")
    if not os.path.exists(path):
        return None
    rev = kernel_revision()
    for line in open(path):
        f = line.split()
        if len(f) >= 3 and not line.startswith("#") and f[0] == workload and f[1] == rev:
            return float(f[2])
    return None


def layer_inputs(workload: str, layer: int, seed: int, threads: int, n_steps: int = 1):
    """One layer of a workload with `n_steps` seeded decode queries (L.q[0 .. n_steps))."""
    import hkv_inputs as hi
    if workload == "cfg0":
        return hi.cfg0(seed=seed, layer=layer, n_steps=n_steps)
    if workload == "cfg1":
        return hi.cfg1(layer, seed=seed, n_steps=n_steps, threads=threads)
    if workload == "cfg2":
        return hi.cfg2(layer, seed=seed, n_steps=n_steps, threads=threads)
    if workload == "cfg3":
        return hi.cfg3(layer, seed=seed, n_steps=n_steps, threads=threads)
    if workload == "cfg4":
        return hi.cfg4(0.10, 0.5, 32, seed=seed, layer=layer, n_steps=n_steps, threads=threads)
    raise SystemExit(f"unknown workload {workload}")


WORKLOAD_TEXT = {
    "cfg0": "1 layer, B=1, 2048 tokens, 2 static / 2 dynamic heads, budget 10%, chunk 32",
    "cfg1": "28 layers, B=1, 16384 tokens (image blocks), static fraction 0.5, budget 10%, chunk 32",
    "cfg2": "28 layers, B=4, 24K-32K tokens (64 frames x 500 video-like), static fraction 0.6, budget 10%, chunk 64",
    "cfg3": "28 layers, B=8, 50000 tokens, static fraction 0.4, budget 5%, chunk 32, planted chunks",
    "cfg4": "1 layer, B=16, 32768 tokens, cell budget 10% / static fraction 0.5 / chunk 32",
}


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML every few milliseconds while the timed
    regions run (reading only)."""

    def __init__(self, index: int, period_s: float = 0.005):
        self.index, self.period, self.rows, self.stop, self.thread = index, period_s, [], False, None

    def __enter__(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = None
            try:
                import torch
                uuid = str(torch.cuda.get_device_properties(self.index).uuid)
            except Exception:
                pass
            self.h = None
            if uuid:
                for cand in (f"GPU-{uuid}", uuid):
                    try:
                        self.h = pynvml.nvmlDeviceGetHandleByUUID(cand)
                        break
                    except Exception:
                        pass
            if self.h is None:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_sm = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.thread = threading.Thread(target=self._run, daemon=True)
            self.thread.start()
        except Exception:
            self.thread = None
        return self

    def _run(self):
        nv = self.nv
        while not self.stop:
            try:
                self.rows.append((nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM),
                                  nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                                  if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons")
                                  else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)))
            except Exception:
                pass
            time.sleep(self.period)

    def __exit__(self, *a):
        self.stop = True
        if self.thread:
            self.thread.join(timeout=1)

    def summary(self):
        if not self.rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        bits = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}
        seen = 0
        for _, r in self.rows:
            seen |= int(r)
        return {"sm_mhz": statistics.median(c for c, _ in self.rows), "sm_max_mhz": float(self.max_sm),
                "reasons": sorted(n for n, b in bits.items() if seen & b), "samples": len(self.rows),
                "how": "NVML, every 5 ms during the timed regions"}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy read+write)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def oracle_decode_timing(L, budget_s: float):
    """Times the oracle's decode step (score + select + attend, all heads of one layer) as it stands."""
    from oracle import hkv_oracle as o
    dyn = [(b, h) for b in range(L.batch) for h in range(L.n_kv_heads)]
    # compression is set-up for the decode timing; window scores are skipped through a score override
    ts = np.zeros((L.batch, L.n_kv_heads, L.max_seq_len), dtype=np.float32)
    ts[:] = np.linspace(1.0, 0.0, L.max_seq_len, dtype=np.float32)[None, None, :]
    oc = o.compress_layer(L, token_scores=ts, only=dyn)
    t0, n = time.perf_counter(), 0
    while True:
        o.decode_layer(L, oc, L.q[0])
        n += 1
        if time.perf_counter() - t0 > budget_s or n >= 50:
            break
    return (time.perf_counter() - t0) / n, n


def layer_algo_bytes(L) -> int:
    """512 B per retained token + 256 B per chunk mean (host arithmetic on the plan inputs)."""
    tot = 0
    cs = L.chunk_size
    for b in range(L.batch):
        C = int(L.seq_lens[b])
        for h in range(L.n_kv_heads):
            bud = min(int(L.budgets[b, h]), C)
            if L.head_type[b, h] == 0:
                tot += 512 * bud
            else:
                nch = (C + cs - 1) // cs
                k = min(nch, (bud + cs - 1) // cs)
                tot += 512 * min(k * cs, C) + 256 * nch
    return tot


def measure_classification(L, dev, n_text: int = 256):
    """hkv_classify_heads on one layer's keys with `n_text` text-token queries per sequence (the step before the
    budgets and the compression; not part of the decode metric)."""
    import torch
    import hkv_inputs as hi
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import to_device_bf16
    q_text, counts = hi.text_queries(L, n_text, ragged=False)
    cfg = hkv.hkv_config(batch=L.batch, n_q_heads=L.n_q_heads, n_kv_heads=L.n_kv_heads, head_dim=L.head_dim,
                         max_seq_len=L.max_seq_len, chunk_size=L.chunk_size, obs_window=L.obs_window,
                         softmax_scale=0.0, flags=0, append_capacity=0)
    _, ws_bytes = hkv.hkv_classify_workspace(cfg, n_text)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    scores = torch.zeros((L.batch, L.n_kv_heads), dtype=torch.float64, device=dev)
    types = torch.zeros((L.batch, L.n_kv_heads), dtype=torch.uint8, device=dev)
    k, q = to_device_bf16(L.k, dev), to_device_bf16(q_text, dev)
    times = []
    for _ in range(4):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        hkv.hkv_classify_heads(cfg, k, q, L.seq_lens, counts, 0.05, 0.9, ws, scores, types)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    rows = int(sum(int(c) for c in counts)) * L.n_q_heads
    cols = float(sum(int(c) * int(t) for c, t in zip(L.seq_lens, counts))) * L.n_q_heads   # softmax entries
    ms = min(times[1:])
    return {"what": "hkv_classify_heads, layer 0: text-centric attention rows -> top-5% sums -> score -> label",
            "text_tokens_per_sequence": n_text, "rows": rows, "ms": ms, "us_per_row": ms * 1e3 / rows,
            "logit_TFLOPs": cols * 2 * L.head_dim / (ms * 1e-3) / 1e12,
            "static_heads_at_theta_0.9": int((types == 0).sum().item()), "heads": L.batch * L.n_kv_heads}


def measure_offload(L, dev, launches: int = 10):
    """One layer with HKV_OFFLOAD_DYNAMIC (the paper's placement: dynamic heads' K/V in pinned host memory, the
    selected chunks cross PCIe inside the decode kernel): time per launch from a CUDA graph of `launches`."""
    import torch
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    lc = LayerCache(L, flags=hkv.HKV_OFFLOAD_DYNAMIC, device=dev)
    q, out = to_device_bf16(L.q[0], dev), lc.new_out()
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        for _ in range(3):
            hkv.hkv_decode_attn(lc.handle, q, out)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(launches):
                hkv.hkv_decode_attn(lc.handle, q, out)
        times = []
        for _ in range(5):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            g.replay()
            e1.record(stream)
            stream.synchronize()
            times.append(e0.elapsed_time(e1) * 1e3 / launches)
    us = min(times[1:])
    host_bytes = sum(512 * min(int(L.seq_lens[b]), -(-int(L.budgets[b, h]) // L.chunk_size) * L.chunk_size)
                     for b in range(L.batch) for h in range(L.n_kv_heads) if L.head_type[b, h] == 1)
    code, detail = hkv.hkv_last_device_error(lc.handle)
    lc.close()
    return {"what": "HKV_OFFLOAD_DYNAMIC, layer 0: dynamic heads' K/V in pinned host memory, selected chunks read over PCIe by the decode kernel",
            "us_per_launch": us, "host_bytes_per_launch": host_bytes, "pcie_GBps": host_bytes / us / 1e3,
            "device_error": [code, detail]}


class StepBench:
    """The caches of `n_layers` layers of one workload, N_QUERY_SETS seeded queries per layer, and one CUDA graph per
    query set holding one decode step (one hkv_decode_attn per layer, layers in sequence).  Step i replays the
    graph of query set i % N_QUERY_SETS, so consecutive steps select different chunks."""

    def __init__(self, workload: str, n_layers: int, seed: int, dev, time_compress: bool = False):
        import torch
        from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
        self.torch, self.workload, self.n_layers, self.dev = torch, workload, n_layers, dev
        threads = min(os.cpu_count() or 8, 32)
        self.caches, self.qs, self.outs, self.L0, self.comp_ms, self.kv_in_bytes0 = [], [], [], None, [], 0
        for layer in range(n_layers):
            L = layer_inputs(workload, layer, seed, threads, n_steps=N_QUERY_SETS)
            k_dev, v_dev = to_device_bf16(L.k, dev), to_device_bf16(L.v, dev)
            lc = LayerCache(L, device=dev, k_dev=k_dev, v_dev=v_dev)
            self.caches.append(lc)
            self.qs.append([to_device_bf16(q, dev) for q in L.q])
            self.outs.append(lc.new_out())
            if layer == 0:
                self.L0 = L
                self.kv_in_bytes0 = sum(int(c) for c in L.seq_lens) * L.n_kv_heads * 512
                if time_compress:
                    # compression proper: hkv_compress of layer 0 again with every input already on the device and
                    # the two buffers allocated beforehand, CUDA events around the C-ABI call alone
                    from paper_2604_05887_b200 import binding as hkv
                    cb, wb = hkv.hkv_plan(lc.cfg, L.seq_lens, L.head_type, L.budgets)
                    cmem = torch.empty(cb, dtype=torch.uint8, device=dev)
                    wmem = torch.empty(wb, dtype=torch.uint8, device=dev)
                    q_obs = to_device_bf16(L.q_obs, dev)
                    is_text = torch.from_numpy(np.ascontiguousarray(L.is_text)).to(dev)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    for _ in range(5):
                        torch.cuda.synchronize()
                        e0.record()
                        h2 = hkv.hkv_compress(lc.cfg, k_dev, v_dev, q_obs, None, is_text, L.seq_lens, L.head_type,
                                              L.budgets, cmem, wmem)
                        e1.record()
                        torch.cuda.synchronize()
                        self.comp_ms.append(e0.elapsed_time(e1))
                        hkv.hkv_cache_destroy(h2)
                    del cmem, wmem, q_obs, is_text
            del k_dev, v_dev
        self.stats = [c.stats for c in self.caches]
        self.algo_bytes = sum(st["algorithmic_bytes_per_step"] for st in self.stats)
        self.launches_per_step = sum(st["launches_per_decode"] for st in self.stats)
        self.graphs = []

    def step(self, qset: int):
        from paper_2604_05887_b200 import binding as hkv
        for lc, q, o_ in zip(self.caches, self.qs, self.outs):
            hkv.hkv_decode_attn(lc.handle, q[qset], o_)

    def capture(self, stream):
        torch = self.torch
        with torch.cuda.stream(stream):
            for s_ in range(N_QUERY_SETS):
                self.step(s_)
            stream.synchronize()
            for s_ in range(N_QUERY_SETS):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    self.step(s_)
                self.graphs.append(g)
            stream.synchronize()

    def per_step_us(self, stream, graphs, replays: int, flush=None):
        """One CUDA-event pair per step on the launching stream; `flush` (a buffer larger than L2) is rewritten before
        every step when the step's working set is not itself larger than L2."""
        torch = self.torch
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(replays)]
        with torch.cuda.stream(stream):
            for i in range(replays):
                if flush is not None:
                    flush.zero_()
                evs[i][0].record(stream)
                graphs[i % len(graphs)].replay()
                evs[i][1].record(stream)
            stream.synchronize()
        return [a.elapsed_time(b) * 1e3 for a, b in evs]

    def close(self):
        self.graphs = []
        for lc in self.caches:
            lc.close()
        self.caches = []


def spread(us):
    us = sorted(us)
    return {"median": statistics.median(us), "min": us[0], "mean": sum(us) / len(us), "replays": len(us)}


def measure_step_workload(workload: str, n_layers: int, seed: int, dev, peak: float, flush):
    """Another step workload through the same path: per-step events, median / min / mean."""
    import torch
    sb = StepBench(workload, n_layers, seed, dev)
    stream = torch.cuda.Stream(device=dev)
    sb.capture(stream)
    big = sb.algo_bytes > 2 * 126e6
    sb.per_step_us(stream, sb.graphs, 24, None if big else flush)
    sp = spread(sb.per_step_us(stream, sb.graphs, 200, None if big else flush))
    full = N_LAYERS[workload]
    res = {"workload": f"{workload}: {WORKLOAD_TEXT[workload]}" + (f" -- REDUCED to {n_layers} of {full} layers" if n_layers != full else ""),
           "layers": n_layers, "us_per_step": sp, "us_per_launch_median": sp["median"] / n_layers,
           "bytes_per_step": sb.algo_bytes, "achieved_GBps": sb.algo_bytes / sp["median"] / 1e3,
           "frac_of_measured_peak": sb.algo_bytes / sp["median"] / 1e3 / peak,
           "frac_of_8TBps": sb.algo_bytes / sp["median"] / 1e3 / NOMINAL_HBM_GBS,
           "l2": "a step streams more than L2 holds" if big else "L2 flushed (512 MB rewritten) before every timed step",
           "queries": f"{N_QUERY_SETS} seeded query sets rotated step by step"}
    sb.close()
    return res


def measure_other_workload(workload: str, n_caches: int, seed: int, dev, peak: float):
    """Per-launch time of the decode kernel on another workload: `n_caches` independent one-layer
    caches (distinct seeds, together larger than L2) replayed round-robin from one CUDA graph."""
    import torch
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    threads = min(os.cpu_count() or 8, 32)
    lcs, qs, outs = [], [], []
    for i in range(n_caches):
        L = layer_inputs(workload, i, seed, threads, n_steps=4)
        lc = LayerCache(L, device=dev)
        lcs.append(lc); qs.append([to_device_bf16(q, dev) for q in L.q]); outs.append(lc.new_out())
        del L
    byt = sum(lc.stats["algorithmic_bytes_per_step"] for lc in lcs) / n_caches
    stream = torch.cuda.Stream(device=dev)
    reps, replays = 4, 60
    with torch.cuda.stream(stream):
        for r in range(reps):
            for lc, q, o_ in zip(lcs, qs, outs):
                hkv.hkv_decode_attn(lc.handle, q[r], o_)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for r in range(reps):                  # every pass over the caches uses another query set
                for lc, q, o_ in zip(lcs, qs, outs):
                    hkv.hkv_decode_attn(lc.handle, q[r], o_)
        for _ in range(3):
            g.replay()
        stream.synchronize()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(replays)]
        for a, b in evs:
            a.record(stream)
            g.replay()
            b.record(stream)
        stream.synchronize()
    per = sorted(a.elapsed_time(b) * 1e3 / (reps * n_caches) for a, b in evs)
    us = statistics.median(per)
    gbs = byt / us / 1e3
    res = {"workload": f"{workload}: {WORKLOAD_TEXT[workload]}", "us_per_launch": us, "us_per_launch_min": per[0],
           "bytes_per_launch": byt,
           "achieved_GBps": gbs, "frac_of_measured_peak": gbs / peak, "frac_of_8TBps": gbs / NOMINAL_HBM_GBS,
           "how": f"{n_caches} independent caches ({byt * n_caches / 1e6:.0f} MB together, larger than L2) launched round-robin, "
                  f"{reps} passes with {reps} query sets in one CUDA graph; median over {replays} graph replays / launches"}
    for lc in lcs:
        lc.close()
    return res


def run_sweep(args):
    """The single-layer sweep (B=16, 32768 tokens): budget x static fraction x chunk size, 100 cells.
    K/V of four independent layers are generated and uploaded once; every cell re-compresses them with
    its own head types, budgets and chunk size and times the decode launch (4 caches round-robin from
    one CUDA graph, so every launch reads cold data).  Prints one JSON line with all cells."""
    import math
    import torch
    import hkv_inputs as hi
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peak, peak_src = measured_peak()
    threads = min(os.cpu_count() or 8, 32)
    n_inst = 4
    Ls, kd, vd, qs = [], [], [], []
    for i in range(n_inst):
        L = hi.cfg4(0.10, 0.5, 32, seed=args.seed + 4, layer=i, threads=threads)
        kd.append(to_device_bf16(L.k, dev)); vd.append(to_device_bf16(L.v, dev)); qs.append(to_device_bf16(L.q[0], dev))
        L.k = L.v = None          # the device copies are what the cells use
        Ls.append(L)
    stream = torch.cuda.Stream(device=dev)
    cells = []
    budgets = hi.CFG4_BUDGETS if not args.sweep_quick else (0.10, 1.00)
    fracs = hi.CFG4_STATIC_FRACTIONS if not args.sweep_quick else (0.5,)
    for bf in budgets:
        for sf in fracs:
            for cs in hi.CFG4_CHUNKS:
                lcs, outs = [], []
                for i, L in enumerate(Ls):
                    L.chunk_size = cs
                    L.head_type = hi._choose_static(args.seed + 4, i, L.batch, L.n_kv_heads, sf)
                    L.budgets = hi._budget_tokens(bf, L.seq_lens, L.n_kv_heads)
                    lc = LayerCache(L, device=dev, k_dev=kd[i], v_dev=vd[i])
                    lcs.append(lc); outs.append(lc.new_out())
                byt = sum(lc.stats["algorithmic_bytes_per_step"] for lc in lcs) / n_inst
                reps = 4 if byt < 4e8 else 2
                with torch.cuda.stream(stream):
                    for _ in range(2):
                        for lc, q, o_ in zip(lcs, qs, outs):
                            hkv.hkv_decode_attn(lc.handle, q, o_)
                    stream.synchronize()
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=stream):
                        for _ in range(reps):
                            for lc, q, o_ in zip(lcs, qs, outs):
                                hkv.hkv_decode_attn(lc.handle, q, o_)
                    for _ in range(2):
                        g.replay()
                    stream.synchronize()
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(stream)
                    for _ in range(10):
                        g.replay()
                    b.record(stream)
                    stream.synchronize()
                us = a.elapsed_time(b) * 1e3 / (10 * reps * n_inst)
                code, _ = hkv.hkv_last_device_error(lcs[0].handle)
                cells.append({"budget": bf, "static_fraction": sf, "chunk": cs, "bytes_per_launch": byt, "us_per_launch": us,
                              "GBps": byt / us / 1e3, "frac_of_measured_peak": byt / us / 1e3 / peak, "device_error": code})
                del g
                for lc in lcs:
                    lc.close()
                del lcs, outs
    best = max(c["frac_of_measured_peak"] for c in cells)
    print(json.dumps({"metric": "decode_attention_achieved_hbm_GBps", "sweep": "cfg4: 1 layer, B=16, 32768 tokens",
                      "unit": "GB/s", "peak": peak, "peak_source": peak_src, "n_cells": len(cells),
                      "best_frac_of_measured_peak": best, "cells": cells,
                      "how": "4 independent layers launched round-robin from one CUDA graph per cell; graph time / launches"}))


PHASES = [(0, "start"), (1, "pre-wait work issued"), (2, "dependency wait over"), (3, "query loads issued"),
          (4, "own chunks scored, scores sent"), (5, "all scores received"), (20, "selection: histogram, barrier"),
          (21, "selection: threshold bin found"), (22, "selection: candidates, barrier"), (23, "selection: ranked"),
          (6, "selection done (list in shared memory)"), (7, "copies issued, lists written back"),
          (14, "first tile landed"), (17, "first tile computed"), (18, "its stage re-armed"),
          (19, "warp 0: second tile landed"), (8, "warp 0: tiles done"), (9, "all warps done"),
          (16, "partials parked, barrier"), (10, "CTA partial sent to its owners"), (11, "partials received"),
          (13, "output written")]


def run_timeline(args):
    """Phase timeline of the decode kernel: the profiling build of the library (same sources, -DHKV_PROFILE)
    stamps the global nanosecond timer at the phase boundaries of every CTA; prints, for a middle layer of a
    few-layer graph of the workload, the mean and the latest stamp of every phase, dynamic and static units apart,
    relative to the end of the preceding layer."""
    import ctypes
    import torch
    from paper_2604_05887_b200 import binding as hkv, build
    lib = hkv.use_library(build.build_profile())
    lib.hkv_profile_attach.argtypes = [ctypes.c_void_p, ctypes.c_longlong]
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    torch.cuda.set_device(0)
    nl = args.layers if args.layers > 0 else 6
    threads = min(os.cpu_count() or 8, 32)
    Ls = [layer_inputs(args.workload, l, args.seed, threads) for l in range(nl)]
    caches = [LayerCache(L) for L in Ls]
    qs = [to_device_bf16(L.q[0]) for L in Ls]
    outs = [c.new_out() for c in caches]
    n_splits = [c.stats["n_splits"] for c in caches]

    def step():
        for c, q, o_ in zip(caches, qs, outs):
            hkv.hkv_decode_attn(c.handle, q, o_)
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    slots = 32
    total = sum(n_splits)
    buf = torch.zeros(total * slots, dtype=torch.int64, device="cuda")
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        step()
        s.synchronize()
        lib.hkv_profile_attach(buf.data_ptr(), total)       # the launches captured next take the regions in order
        with torch.cuda.graph(g, stream=s):
            step()
        lib.hkv_profile_attach(None, 0)
        for _ in range(3):
            g.replay()
        s.synchronize()
    raw = buf.cpu().numpy().reshape(-1, slots).astype(np.uint64)
    gt = (raw & np.uint64(0xFFFFFFFF)).astype(np.float64)          # global timer, ns (low 32 bits: 4.3 s, no wrap inside a replay)
    clk = (raw >> np.uint64(32)).astype(np.int64)                  # SM cycle counter, low 32 bits
    lay = max(1, nl - 2)
    o0 = sum(n_splits[:lay])
    sl = slice(o0, o0 + n_splits[lay])
    blk, cb, prev = gt[sl], clk[sl], gt[o0 - n_splits[lay - 1]:o0]
    prev_end = prev.max()
    dyn = blk[:, 4] > 0
    for kind, m in (("dynamic", dyn), ("static", ~dyn)):
        b, c = blk[m], cb[m]
        if not b.shape[0]:
            continue
        print(f"{kind} units: {b.shape[0]} CTAs.  us after the end of the preceding layer (global timer); SM cycles since the CTA's previous stamp")
        last_k = None
        for k, name in PHASES:
            have = b[:, k] > 0
            if not have.any():
                continue
            col = b[have, k]
            line = f"  {name:34s} mean {(col.mean() - prev_end) / 1e3:7.2f}   last {(col.max() - prev_end) / 1e3:7.2f}"
            if last_k is not None:
                both = have & (b[:, last_k] > 0)
                d = (c[both, k] - c[both, last_k]) % (1 << 32)
                line += f"   cycles mean {d.mean():8.0f}  max {d.max():8.0f}"
            print(line)
            last_k = k
    ticks = np.unique(gt[gt > 0])
    print(f"layer: first CTA start {(blk[:, 0].min() - prev_end) / 1e3:.2f}, end {(blk.max() - prev_end) / 1e3:.2f} us "
          f"after the preceding layer's end; the global timer ticks in steps of {np.diff(ticks)[:2000].min():.0f} ns")
    hkv.use_library(None)


def run_reference(args):
    """The reference arm of this tier is the CPU oracle, timed as it stands on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    threads = min(os.cpu_count() or 8, 32)
    L = layer_inputs(args.workload, 0, args.seed, threads)
    n_layers = N_LAYERS[args.workload]
    per = []
    for i in range(args.warmup + args.steps):
        dt, _ = oracle_decode_timing(L, 0.0)          # one decode of one layer per step (bounded sample)
        if i >= args.warmup:
            per.append(dt)
    t = sum(per) / len(per)
    bytes_layer = layer_algo_bytes(L)
    value = bytes_layer / t / 1e9
    sample = f"1 of {n_layers} layers per step (all {L.batch * L.n_kv_heads} heads), oracle decode_layer, step time scaled x{n_layers}"
    line = {"impl": "reference", "metric": "decode_attention_achieved_hbm_GBps", "value": value, "unit": "GB/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * n_layers * 1e3,
            "us_per_step": t * n_layers * 1e6, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": {"workload": f"{args.workload}: {WORKLOAD_TEXT[args.workload]}"},
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=list(N_LAYERS))
    ap.add_argument("--seed", type=int, default=2)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="CPU time spent on the oracle baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip the other workloads (cfg4 cell, cfg1, cfg3 reduced, cfg0) and the next rows")
    ap.add_argument("--sweep", action="store_true", help="run the 100-cell single-layer sweep (cfg4) instead of the step benchmark")
    ap.add_argument("--sweep-quick", action="store_true", help="with --sweep: only budgets 10 % and 100 % at static fraction 0.5")
    ap.add_argument("--next-rows", action="store_true",
                    help="time hkv_classify_heads and the host-offload variant on layer 0 even in a reduced (--layers) run")
    ap.add_argument("--timeline", action="store_true",
                    help="print the phase timeline of the decode kernel (profiling build of the library, --layers N layers, default 6)")
    ap.add_argument("--layers", type=int, default=0,
                    help="use only the first N layers of the workload (small case for profiler captures; "
                         "the line is then marked reduced and is not the headline number)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.sweep:
        run_sweep(args)
        return
    if args.timeline:
        run_timeline(args)
        return

    import torch
    from paper_2604_05887_b200 import binding as hkv          # raises if libhkv.so is missing: no fallback
    from paper_2604_05887_b200 import replicas

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the CUDA path has no CPU fallback)")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    peak, peak_src = measured_peak()

    # ---- the workload: every layer generated on the host, uploaded, compressed; caches stay resident ----
    n_layers = N_LAYERS[args.workload]
    if args.layers > 0:
        n_layers = min(n_layers, args.layers)
    sb = StepBench(args.workload, n_layers, args.seed + 1000 * rank, dev, time_compress=True)   # = replicas.replica_seed
    algo_bytes, L0 = sb.algo_bytes, sb.L0
    resident = sum(st["cache_bytes"] for st in sb.stats)
    big = algo_bytes > 2 * 126e6
    flush = None if big else torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.Stream(device=dev)
    sb.capture(stream)

    with torch.cuda.stream(stream):
        # end-to-end variant: every step's queries start in pinned host memory, outputs end there
        q_host = [torch.stack([q[s_].cpu() for q in sb.qs]).pin_memory() for s_ in range(N_QUERY_SETS)]
        out_host = torch.empty((n_layers,) + tuple(sb.outs[0].shape), dtype=sb.outs[0].dtype).pin_memory()
        q_all = torch.empty_like(q_host[0], device=dev)
        out_all = torch.empty_like(out_host, device=dev)
        handles = [lc.handle for lc in sb.caches]
        # the library's host-buffer entry point for a whole step: all layers' queries (pinned host) -> device, one
        # decode launch per layer, all outputs -> pinned host, every copy enqueued by the C-ABI call itself
        hkv.hkv_decode_step_host(handles, q_host[0], out_host, q_all, out_all)
        stream.synchronize()
        graphs_e2e = []
        for s_ in range(N_QUERY_SETS):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                hkv.hkv_decode_step_host(handles, q_host[s_], out_host, q_all, out_all)
            graphs_e2e.append(g)
        stream.synchronize()

        def barrier():
            torch.cuda.synchronize()
            replicas.barrier()
            torch.cuda.synchronize()

        def timed(graphs, n):
            """EXACTLY n steps between one CUDA-event pair on the launching stream; the slowest rank's time."""
            barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i in range(n):
                if flush is not None:
                    flush.zero_()
                graphs[i % len(graphs)].replay()
            b.record(stream)
            barrier()
            ms, _, _ = replicas.aggregate_step(a.elapsed_time(b), algo_bytes, dev)
            return ms

        warm = max(args.warmup, 3)
        for i in range(warm):
            sb.graphs[i % N_QUERY_SETS].replay()
        with ClockSampler(local) as clk:
            ms = timed(sb.graphs, args.steps)
            per_step = sb.per_step_us(stream, sb.graphs, 100 if args.layers > 0 else STATS_REPLAYS, flush)
            for i in range(3):
                graphs_e2e[i].replay()
            ms_e2e = timed(graphs_e2e, args.steps)
            per_step_e2e = sb.per_step_us(stream, graphs_e2e, 200, flush)

        # layers-batched figure (labelled; not the metric): every layer's cache in ONE launch.  A real model's
        # layers are sequential, so this only shows what the per-layer dependency chain costs.
        batched = None
        if n_layers <= 32:
            gb = torch.cuda.CUDAGraph()
            hkv.hkv_decode_attn_multi(handles, [q[0] for q in sb.qs], sb.outs)
            stream.synchronize()
            with torch.cuda.graph(gb, stream=stream):
                hkv.hkv_decode_attn_multi(handles, [q[0] for q in sb.qs], sb.outs)
            batched = spread(sb.per_step_us(stream, [gb], 60, flush))
        code, detail = hkv.hkv_last_device_error(sb.caches[0].handle)

    world_bytes = algo_bytes * world          # every rank runs a replica of the same size (weak scaling)
    t_step = ms * 1e-3 / args.steps
    value = world_bytes / t_step / 1e9
    # Launch duration of the dominant kernel = timed region (CUDA events on the launching stream around the
    # graph replays) / launches in it: one decode_kernel per layer and nothing else, so launch gaps are
    # charged to the kernel.
    fused_avg_s = t_step / n_layers
    achieved = (algo_bytes / n_layers) / fused_avg_s / 1e9
    t_e2e = ms_e2e * 1e-3 / args.steps
    h2d = q_host[0].numel() * q_host[0].element_size()
    d2h = out_host.numel() * out_host.element_size()
    sp = spread(per_step)
    comp_ms = min(sb.comp_ms)

    line = {
        "metric": "decode_attention_achieved_hbm_GBps", "value": value, "unit": "GB/s",
        "n_gpus": world, "steps": args.steps, "warmup": warm, "ms_per_step": t_step * 1e3,
        "us_per_step": t_step * 1e6, "us_per_step_stats": sp,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {WORKLOAD_TEXT[args.workload]}"
                   + (f" -- REDUCED to {n_layers} layers (profiling case)" if n_layers != N_LAYERS[args.workload] else ""),
                   "layers": n_layers,
                   "algorithmic_bytes_per_step": algo_bytes, "resident_cache_bytes": resident,
                   "l2": "inputs larger than L2: one step streams %.0f MB of distinct KV" % (algo_bytes / 1e6)
                   if big else "L2 flushed (512 MB rewritten) before every step, inside the timed region",
                   "queries": f"{N_QUERY_SETS} seeded query sets per layer, rotated step by step (one CUDA graph per set)",
                   "launch": "CUDA graph of one hkv_decode_attn per layer, layers in sequence",
                   "timing": f"ms_per_step: one event pair around --steps steps; us_per_step_stats: one event pair per step, "
                             f"{len(per_step)} steps",
                   "compress_ms_per_layer": comp_ms,
                   "compress_GBps_of_input_kv": sb.kv_in_bytes0 / (comp_ms * 1e-3) / 1e9,
                   "compress_how": "hkv_compress of layer 0 alone (inputs resident, buffers preallocated), CUDA events around the call, fastest of 5; GB/s = that layer's full K/V bytes / that time"},
        "frac_of_measured_peak": value / world / peak, "frac_of_8TBps": value / world / NOMINAL_HBM_GBS,
        "roofline": {"bound": "hbm", "kernel": "decode_kernel (score + top-k + flash-decode + merge, one launch per layer)",
                     "achieved": achieved, "peak": peak, "peak_source": peak_src, "unit": "GB/s",
                     "frac": achieved / peak, "frac_of_8TBps": achieved / NOMINAL_HBM_GBS,
                     "avg_launch_us": fused_avg_s * 1e6, "median_launch_us": sp["median"] / n_layers,
                     "bytes_per_launch": algo_bytes / n_layers,
                     "how": "graph step time / launches per step (CUDA events on the launching stream)",
                     "traffic": ncu_traffic(args.workload), "kernel_revision": kernel_revision(),
                     "traffic_how": "profiles/decode_kernel_traffic.txt, the row of this kernel revision (null: no capture of this revision)"},
        "e2e": {"value": world_bytes / t_e2e / 1e9, "unit": "GB/s", "us_per_step": t_e2e * 1e6,
                "us_per_step_stats": spread(per_step_e2e),
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "how": "hkv_decode_step_host: pinned host queries of all layers -> device (first layer's ahead, the rest beside the first layers), one decode launch per layer, outputs -> pinned host in four groups beside the later layers, copies enqueued by the C-ABI call, all inside the timed graph"},
        "layers_batched": None if batched is None else {
            "us_per_step": batched, "GBps": algo_bytes / batched["median"] / 1e3,
            "frac_of_measured_peak": algo_bytes / batched["median"] / 1e3 / peak,
            "label": "NOT the metric: all layers' caches in one hkv_decode_attn_multi launch (no layer-to-layer dependency)"},
        "gpu_launches": sb.launches_per_step * args.steps,
        "clocks": clk.summary(),
        "device_error": [code, detail],
        "paper_context": "paper reports 7.9x KV-memory reduction and 1.52x decode speed-up (whole model, NVIDIA L40S); no attention-only number",
    }
    stats0 = sb.stats[0]
    sb.close()
    del sb
    torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.no_extra and args.layers == 0 and args.workload == "cfg2":
        # the other workloads through the same path (one line carries all five)
        fl = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
        others = [measure_other_workload("cfg4", 4, args.seed + 4, dev, peak)]
        for wl, nl in (("cfg1", 28), ("cfg3", 8), ("cfg0", 1)):
            others.append(measure_step_workload(wl, nl, args.seed + 10, dev, peak, fl))
            torch.cuda.empty_cache()
        del fl
        line["other_workloads"] = others
        line["next_rows"] = [measure_classification(L0, dev), measure_offload(L0, dev)]
    elif rank == 0 and world == 1 and args.next_rows:
        line["next_rows"] = [measure_classification(L0, dev), measure_offload(L0, dev)]
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        dt, n = oracle_decode_timing(L0, args.cpu_seconds)
        b0 = stats0["algorithmic_bytes_per_step"]
        line["cpu_baseline"] = {"value": b0 / dt / 1e9, "unit": "GB/s", "us_per_step": dt * n_layers * 1e6,
                                "cores": blas_threads(), "kind": "oracle",
                                "sample": f"oracle decode_layer on layer 0 of {n_layers} ({L0.batch * L0.n_kv_heads} heads), "
                                          f"{n} repetitions, step time scaled x{n_layers}"}
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
