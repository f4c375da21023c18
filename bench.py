#!/usr/bin/env python
"""Benchmark of the CAKE prefill-time eviction path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 4] [--impl reference]

One step = one pass of the whole hot path over one batch of synthetic input:
for every layer score -> allocate -> evict, then one gather-compaction.  Prints
one JSON line.  The path does not shard: with N > 1 (torchrun) every rank runs
an independent replica on its own GPU ("replicas only") and the value is the
sum of tokens over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "CAKE score+evict+compact prompt tokens/s"
# DRAM bytes of one score-kernel launch at workload 4 from the ncu capture under profiles/;
# set to None whenever the kernel changes until the counters are taken again.
SCORE_KERNEL_DRAM_BYTES = 285018112 + 10838272
UNIT = "tokens/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--blocks", type=int, default=10,
                    help="timed blocks of --steps steps; the first one is the headline value, the "
                         "others show the run-to-run spread")
    ap.add_argument("--workload", type=int, default=4, help="config index 1..5 (4 = 128K Llama-3.1-8B shape)")
    ap.add_argument("--impl", default="cake", choices=["cake", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-sample-layers", type=int, default=2)
    return ap.parse_args()


# ----------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def median_between(self, t0: float, t1: float):
        """Median sampled SM clock (MHz) of the samples taken in the host-time window."""
        v = []
        for ts, ln in list(self.lines):
            if t0 <= ts <= t1:
                try:
                    v.append(float(ln.split(",")[0]))
                except ValueError:
                    pass
        v.sort()
        return v[len(v) // 2] if v else None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for _, ln in self.lines:
            p = [x.strip() for x in ln.split(",")]
            if len(p) < 6:
                continue
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except ValueError:
                continue
            for nm, val in zip(names, p[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------ CPU oracle leg
class OracleSample:
    """The oracle, as it stands, on a bounded sample of the workload: `sample_layers` full
    layers of the first request through every step of the path (score, budgets, top-k,
    compaction).  Inputs are generated once; `run()` times one pass over them.  The oracle is
    single-process NumPy: the only parallelism is the BLAS thread pool inside its matrix
    products, whose size is reported as `cores`."""

    def __init__(self, w, sample_layers: int):
        import numpy as np
        from paper_2503_12491_b200 import synth
        try:
            from threadpoolctl import threadpool_info
            self.threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        except Exception:
            self.threads = os.cpu_count() or 1
        self.w = w
        self.layers = max(1, min(sample_layers, w.n_layers))
        self.N = w.seq_lens[0]
        w1 = synth.scaled(w, seq_lens=(self.N,))
        self.qs, self.ks, self.vs = [], [], []
        for l in range(self.layers):
            q, k, v = synth.layer_inputs(w1, l, "cpu")
            self.qs.append(q[0].float().numpy().astype(np.float64))
            self.ks.append(k.float().numpy().astype(np.float64))
            self.vs.append(v.float().numpy().astype(np.float64))
        # tokens the sample stands for, in the metric's unit: `layers` of the L layers of N prompt
        # tokens are N * layers / L prompt tokens' worth of the whole path
        self.tokens = self.N * self.layers / w.n_layers
        self.desc = (f"{self.layers} of {w.n_layers} layers of request 0 (N={self.N}), every step of the "
                     f"path, float64 NumPy (single process; BLAS threads are its only parallelism); "
                     f"a pass counts as N*{self.layers}/{w.n_layers} prompt tokens")

    def run(self) -> float:
        """One timed pass; returns seconds."""
        from oracle import cake_oracle as O
        w = self.w
        t0 = time.perf_counter()
        scored = [O.score_layer(q, k, gamma=w.gamma, pool_kernel=w.pool_kernel, tau1=w.tau1, tau2=w.tau2)
                  for q, k in zip(self.qs, self.ks)]
        # the sampled layers stand for all L: they share the budget the full cascade would give them
        share = w.total_budget * self.layers // w.n_layers
        c = O.cascade([s["indicator"] for s in scored], [s["P"] for s in scored],
                      total_budget=share, window=w.window, seq_len=self.N)
        for l in range(self.layers):
            O.compact(self.ks[l], self.vs[l], c.positions[l])
        return time.perf_counter() - t0


def run_reference(args, w):
    """The reference arm: the oracle alone on the host cores.  A step is one pass over the
    bounded sample; `ms_per_step` is its measured time and `value` the prompt tokens that the
    sample stands for per second (the same number as scaling the time to all layers)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    smp = OracleSample(w, args.cpu_sample_layers)
    for _ in range(max(1, args.warmup)):
        smp.run()
    times = [smp.run() for _ in range(args.steps)]
    dt = sum(times) / len(times)
    value = smp.tokens / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": max(1, args.warmup), "ms_per_step": dt * 1e3,
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": smp.threads, "kind": "oracle",
                         "sample": smp.desc, "sample_seconds": dt,
                         "seconds_min_max": [min(times), max(times)],
                         "whole_workload_ms_extrapolated": w.total_tokens / value * 1e3},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def block_stats(ms, mhz, steps):
    """Spread of the per-step time over the repeated blocks (this rank), and time x clock."""
    srt = sorted(ms)
    med = srt[len(srt) // 2]
    known = [(m, c) for m, c in zip(ms, mhz) if c]
    out = {"n_blocks": len(ms), "steps_per_block": steps, "ms_per_step_median": med,
           "ms_per_step_min": srt[0], "ms_per_step_max": srt[-1],
           "ms_per_step_each": [round(x, 4) for x in ms],
           "sm_mhz_median_each": mhz}
    if known:
        prod = sorted(m * c for m, c in known)
        out["ms_x_mhz_median"] = prod[len(prod) // 2]
    return out


def workload_config(w):
    return {"workload": w.name, "n_layers": w.n_layers, "n_q_heads": w.n_q_heads,
            "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "seq_lens": list(w.seq_lens),
            "window": w.window, "pool_kernel": w.pool_kernel, "gamma": w.gamma,
            "total_budget": w.total_budget, "compaction": "deferred (one gather after the last stage)",
            "l2": "inputs larger than L2 (every layer's K exceeds 126 MB or the step streams > 1 GB)",
            "parallelism": "replicas only"}


# ------------------------------------------------------------- replicas
def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's time: replicas do not exchange data, only this number."""
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_rank: int, world: int, ms_step: float) -> float:
    """Whole-job throughput of `world` independent replicas that all finish within ms_step."""
    return tokens_per_rank * world / (ms_step * 1e-3)


# --------------------------------------------------------------- CUDA leg
def main():
    args = parse_args()
    from paper_2503_12491_b200 import synth
    w = synth.workload(args.workload)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2503_12491_b200 import harness, binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) if os.path.exists(
            os.path.join(ROOT, "MEASURED_PEAKS.json")) else open(os.devnull) as f:
        try:
            peaks = json.load(f)
        except Exception:
            peaks = {}
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    peak_kind = "measured" if "hbm_gbs" in peaks else "fallback"

    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w)
    rows = None
    L = w.n_layers
    esize = 4 if w.dtype == "fp32" else 2

    def step(bufs):
        cake.begin(w.cu_seqlens)
        for l in range(L):
            cake.score_layer(l, qs[l], ks[l])
            cake.allocate(l)
            cake.evict(l)
        return cake.compact(ks, vs, k_out=bufs[0], v_out=bufs[1], row_offsets=bufs[2], positions=bufs[3])

    cake.begin(w.cu_seqlens)
    rows = cake.packed_rows_bound()
    bufs = (torch.empty(rows, w.head_dim, dtype=w.torch_dtype, device="cuda"),
            torch.empty(rows, w.head_dim, dtype=w.torch_dtype, device="cuda"),
            torch.empty(len(w.seq_lens) * L + 1, dtype=torch.int64, device="cuda"),
            torch.empty(rows, dtype=torch.int32, device="cuda"))

    for _ in range(max(3, args.warmup)):
        step(bufs)
    barrier()
    if cake.status() != 0:
        raise RuntimeError(f"device status {cake.status()}")

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = binding.launch_count()
    def timed_block():
        """K steps bracketed by barrier + synchronize; (device ms, host window)."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        h0 = time.time()
        e0.record()
        for _ in range(args.steps):
            step(bufs)
        e1.record()
        barrier()
        return e0.elapsed_time(e1), (h0, time.time())

    ms_total, win0 = timed_block()                 # the headline: exactly K steps
    launches = binding.launch_count() - launches0
    # the same block again and again: how much one block moves from run to run, with the clock
    # sampled during each
    block_ms, block_mhz = [ms_total / args.steps], [sampler.median_between(*win0) if rank == 0 else None]
    for _ in range(max(0, args.blocks - 1)):
        ms_b, win = timed_block()
        block_ms.append(ms_b / args.steps)
        block_mhz.append(sampler.median_between(*win) if rank == 0 else None)
    # second pass of the same K steps with every stage bracketed by CUDA events on the
    # launching stream: gives the per-kernel durations (the brackets cost a little, so the
    # headline value comes from the first pass)
    cake.profile_enable(True)
    cake.profile_read()
    evp0, evp1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    evp0.record()
    for _ in range(args.steps):
        step(bufs)
    evp1.record()
    prof = cake.profile_read()
    ms_profiled = evp0.elapsed_time(evp1) / args.steps
    cake.profile_enable(False)
    clocks = sampler.stop() if rank == 0 else None
    ms_step = max_over_ranks(ms_total, world, "cuda") / args.steps
    value = whole_job_value(w.total_tokens, world, ms_step)

    retained_rows = int(bufs[2][-1].item())
    k_bytes = L * w.n_kv_heads * w.total_tokens * w.head_dim * esize
    q_bytes = L * len(w.seq_lens) * w.n_q_heads * w.window * w.head_dim * esize
    out_bytes = 2 * retained_rows * w.head_dim * esize
    ideal = k_bytes + q_bytes + out_bytes

    # dominant kernel: the window-score kernel (both passes in one launch);
    # algorithmic bytes per launch = one layer's K read once + its window Q
    phase_ms = {k: v["ms"] / args.steps for k, v in prof.items()}
    dom = "score"
    dom_ms = prof[dom]["ms"] / max(prof[dom]["spans"], 1)
    per_launch_bytes = (k_bytes + q_bytes) / L
    achieved = per_launch_bytes / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 else None
    step_gbps = ideal / (ms_step * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": hbm_peak,
                "unit": "GB/s", "frac": (achieved / hbm_peak) if achieved else None,
                "peak_kind": f"{peak_kind} copy bandwidth",
                "traffic": SCORE_KERNEL_DRAM_BYTES if args.workload == 4 else None,
                "traffic_source": "profiles/score_fused_kernel_llama31-8b-gqa-128k_2layers.md "
                                  "(dram__bytes_read.sum + dram__bytes_write.sum of one launch; a "
                                  "launch of the reduced case is a full-size launch)",
                "bytes_per_launch": per_launch_bytes, "ms_per_launch": dom_ms,
                "launches_timed": prof[dom]["spans"],
                "blocks": block_stats(block_ms, block_mhz, args.steps),
                "phase_ms_per_step": phase_ms, "ms_per_step_with_brackets": ms_profiled,
                "whole_step": {"ideal_bytes": ideal, "GBps": step_gbps,
                               "frac_of_measured_peak": step_gbps / hbm_peak,
                               "frac_of_8TBps_nominal": step_gbps / 8000.0}}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32",
            "data": "synthetic", "config": workload_config(w), "gpu_launches": launches,
            "roofline": roofline, "clocks": clocks}

    # ---- end to end: host-resident Q/K/V, copies inside the timed region
    if not args.no_e2e:
        line["e2e"] = e2e_leg(args, w, cake, qs, ks, vs, bufs, world, barrier)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        smp = OracleSample(w, args.cpu_sample_layers)
        dt = smp.run()
        line["cpu_baseline"] = {"value": smp.tokens / dt, "unit": UNIT, "cores": smp.threads,
                                "kind": "oracle", "sample": smp.desc, "sample_seconds": dt}
    if rank == 0:
        print(json.dumps(line), flush=True)
    cake.destroy()
    if world > 1:
        dist.destroy_process_group()


def e2e_leg(args, w, cake, qs, ks, vs, bufs, world, barrier):
    """Same step with Q/K/V in pinned host memory: every layer's queries and
    keys are copied host->device inside the timed region (double-buffered
    against the scoring of the previous layer); the values, which only the
    gather reads, stay on the host and the gather fetches their retained rows
    from there; the packed cache is read back."""
    import torch
    L = w.n_layers
    hq = [q.cpu().pin_memory() for q in qs]
    hk = [k.cpu().pin_memory() for k in ks]
    hv = [v.cpu().pin_memory() for v in vs]
    del qs[:]
    # the gather needs every layer's K/V on the device: reuse the resident tensors as the landing zone
    rows = bufs[0].shape[0]
    out_k = torch.empty(bufs[0].shape, dtype=bufs[0].dtype).pin_memory()
    out_v = torch.empty(bufs[1].shape, dtype=bufs[1].dtype).pin_memory()
    out_off = torch.empty(bufs[2].shape, dtype=torch.int64).pin_memory()
    out_pos = torch.empty(bufs[3].shape, dtype=torch.int32).pin_memory()
    dq = [torch.empty_like(hq[0], device="cuda") for _ in range(L)]
    arrived = [torch.cuda.Event() for _ in range(L)]
    copy_stream = torch.cuda.Stream()
    main = torch.cuda.current_stream()

    def step():
        cake.begin(w.cu_seqlens)
        copy_stream.wait_stream(main)              # previous step's gather has read K/V
        for l in range(L):
            with torch.cuda.stream(copy_stream):
                dq[l].copy_(hq[l], non_blocking=True)
                ks[l].copy_(hk[l], non_blocking=True)
                arrived[l].record(copy_stream)
            main.wait_event(arrived[l])
            cake.score_layer(l, dq[l], ks[l])
            cake.allocate(l)
            cake.evict(l)
        cake.compact(ks, hv, k_out=bufs[0], v_out=bufs[1], row_offsets=bufs[2], positions=bufs[3])
        out_off.copy_(bufs[2], non_blocking=True)
        main.synchronize()
        n = int(out_off[-1])
        out_k[:n].copy_(bufs[0][:n], non_blocking=True)
        out_v[:n].copy_(bufs[1][:n], non_blocking=True)
        out_pos[:n].copy_(bufs[3][:n], non_blocking=True)
        main.synchronize()
        return n

    steps = max(1, min(args.steps, 3))
    step()
    barrier()
    t0 = time.perf_counter()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(steps):
        n = step()
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1) / steps
    ms = max_over_ranks(ms, world, "cuda")
    esize = 4 if w.dtype == "fp32" else 2
    h2d = sum(x.numel() * x.element_size() for x in hq + hk) + n * w.head_dim * esize
    d2h = 2 * n * w.head_dim * esize + n * 4 + out_off.numel() * 8
    return {"value": w.total_tokens * world / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms,
            "steps": steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "note": "Q/K/V pinned on the host; Q and K copied per layer on a side stream, the retained V rows "
                    "read from host memory by the gather; packed cache read back"}


if __name__ == "__main__":
    main()
