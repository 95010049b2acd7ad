#!/usr/bin/env python
"""Benchmark of the BPTT training step: sample-timesteps/s per checkpoint strategy.

Default arm: the CUDA library on workload c4, the largest configuration of the benchmark definition
(3 recurrent LIF layers 1024-8192-8192-8192-100, T = 2000, batch 8, Double checkpointing with
remote checkpoints every 256 steps and local ones every 16), one process per GPU; with several GPUs
every rank runs an independent replica (the step does not shard: no collective).  One JSON line on
rank 0; the other workloads are timed briefly and reported under "workloads" of the same line.

`--impl reference` times the CPU oracle as it stands on the host cores, each step a bounded
sample (the first T' steps) of the same workload.
"""
from __future__ import annotations

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

import snn_workloads as wl  # noqa: E402

METRIC = "sample_timesteps_per_s"
UNIT = "sample-timesteps/s"
STRATEGY_NAME = {0: "standard", 1: "chunk", 2: "remote", 3: "double", 4: "hierarchical", 5: "double_local"}
ORACLE_SAMPLE_T = 100   # steps per oracle "step" in --impl reference


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# DRAM bytes (read + written) of one launch of a pass's kernel from one ncu capture of this workload
# (dram__bytes_read.sum + dram__bytes_write.sum; summaries under profiles/): (workload, phase) -> (kernel,
# sha256 of the kernel's source text when the counters were taken, bytes per launch).  Reported only while
# the kernel still has that text.  The backward pass of c2 now runs in bwd_segment_kernel, a cooperative launch
# of thread-block clusters that the profiler cannot launch: no counters, hence no entry.
NCU_TRAFFIC = {
    # one launch = 16 steps of one layer: 3,337,776,000 B read + 5,214,720 B written; per layer and step (less than the
    # algorithmic bytes: the first 64 MB of the matrix stay in L2 from one step to the next):
    ("c4", "bwd"): ("bwd_stream_kernel", "5a49fc56be35fd5f7a11f4fa48db838043c34b52375e31c8f755c92e20664b84",
                    (3337776000 + 5214720) // 16),
    ("c3", "bwd"): ("bwd_step_kernel", "2f4bbd76ae837e3ce2614c31b106f74f4b5e27af23b3429895c113105211be02",
                    51018240 + 43264),
    ("c4", "fwd"): ("fwd_step_kernel", "f984311eddc0b278aeb605935b3e36af28944f04d5c03dee15033512817ce1fb",
                    388252416 + 4982784),
    ("c2", "fwd"): ("fwd_resident_kernel", "0d6da12b003e9d7942f18dfc1f0a724c029951a870a748a04acca7060137967b",
                    15203584),
}


def kernel_source_sha(name: str):
    """sha256 of the text of kernel `name` in kernels.cuh: from its __global__ line to the next section rule."""
    import hashlib
    src = os.path.join(ROOT, "paper_2412_11810_b200", "csrc", "kernels.cuh")
    try:
        text = open(src).read()
    except OSError:
        return None
    at = text.find(" " + name + "(const __grid_constant__")
    if at < 0:
        return None
    start = text.rfind("__global__", 0, at)
    end = text.find("\n// ----", at)
    return hashlib.sha256(text[start:end if end > 0 else len(text)].encode()).hexdigest()


def ncu_traffic(workload: str, phase: str):
    entry = NCU_TRAFFIC.get((workload, phase))
    if not entry:
        return None
    kernel, sha, nbytes = entry
    return nbytes if sha and kernel_source_sha(kernel) == sha else None


def read_tensor_peak():
    """Dense tf32 peak in TFLOP/s: the measured bf16 figure times the nominal tf32 : bf16 ratio."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["bf16_tflops"]) * 1.1 / 2.25, "measured bf16 x 1.1/2.25"
    return 1590.0 * 1.1 / 2.25, "fallback bf16 x 1.1/2.25"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.thread, self.gpu = [], None, None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu), "-lms", "200"], stdout=subprocess.PIPE, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        self.proc.wait()
        self.thread.join(timeout=1)
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_spec(w):
    from oracle.oracle import NetSpec, leak_from_tau
    return NetSpec(w.sizes, leak_from_tau(w.tau_mem), w.theta, w.beta, w.scale(), cell=w.cell)


def time_oracle(w, d, T_sample):
    """One oracle train step on the first T_sample steps; returns seconds."""
    from oracle.oracle import Oracle
    orc = Oracle("f32")
    spec = oracle_spec(w.with_T(T_sample))
    t0 = time.perf_counter()
    orc.bptt_full(spec, d["input_dense"][:T_sample], d["targets"], d["W_ff"], d["W_rec"], d["W_out"],
                  keep_states=False)
    return time.perf_counter() - t0


def run_reference(args, rank):
    if rank != 0:
        return
    from oracle.oracle import num_threads
    w = wl.WORKLOADS[args.workload]
    Ts = min(ORACLE_SAMPLE_T, w.T)
    d = wl.make(w.with_T(Ts))
    for _ in range(args.warmup):
        time_oracle(w, d, Ts)
    times = [time_oracle(w, d, Ts) for _ in range(args.steps)]
    total = sum(times)
    value = w.B * Ts * args.steps / total
    sample = f"each step = oracle full-storage BPTT on the first {Ts} of {w.T} steps of {w.name}, full width and batch"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "sizes": list(w.sizes), "T": w.T, "B": w.B, "sample_T": Ts},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def aggregate_replicas(per_rank_ms, units_per_rank, world, dist=None, device=None):
    """Whole-job throughput of independent replicas: every rank processed units_per_rank units; the job
    took as long as its slowest rank (max over ranks of each entry of per_rank_ms).  Returns
    (list of max times in ms, list of units per second)."""
    times = [float(x) for x in per_rank_ms]
    if dist is not None and world > 1:
        import torch
        t = torch.tensor(times, dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        times = [float(x) for x in t]
    return times, [units_per_rank * world / (ms / 1e3) for ms in times]


def algorithmic_bytes(w, activity, B):
    """Bytes the method must move per launch of each step kernel (one wavefront launch = one step of
    every layer), from the per-layer figures: forward gathers the active weight rows and writes V and
    events; backward streams W_rec and the next layer's W_ff once per step and touches V and delta."""
    sz = w.sizes
    fwd = bwd = 0.0
    for l in range(1, w.L + 1):
        n_pre, n = sz[l - 1], sz[l]
        ev = activity[l - 1] * n_pre + activity[l] * n          # events per sample feeding layer l
        fwd += 4.0 * n * B * ev + 4.0 * ev * B + 8.0 * B * n + B * n / 8.0
        bwd += 4.0 * n * n + (4.0 * n * sz[l + 1] if l < w.L else 0.0) + 16.0 * B * n
    return fwd, bwd


def dw_bytes(w, activity, B, n_steps):
    """Bytes one weight-gradient launch (a segment of n_steps steps, all matrices) must move: every touched
    dW row read and written once, and one delta row read per event."""
    sz = w.sizes
    total = 0.0
    for l in range(1, w.L + 1):
        for n_pre, p in ((sz[l - 1], activity[l - 1]), (sz[l], activity[l])):
            touched = n_pre * (1.0 - (1.0 - min(p, 1.0)) ** (n_steps * B))
            total += 8.0 * sz[l] * touched + 4.0 * sz[l] * n_steps * B * p * n_pre
    return total


def host_link_probe(torch, device, nbytes=64 << 20, reps=5):
    """Pinned-memory copy bandwidth of the host link, each way: one asynchronous copy of nbytes between a
    page-locked host buffer and a device buffer, timed with CUDA events, best of reps (GB/s)."""
    host = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    dev = torch.empty(nbytes, dtype=torch.uint8, device=device)
    st = torch.cuda.Stream(device=device)
    best = {"h2d": 0.0, "d2h": 0.0}
    with torch.cuda.stream(st):
        for _ in range(reps + 1):
            for name, dst, src in (("h2d", dev, host), ("d2h", host, dev)):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(st)
                dst.copy_(src, non_blocking=True)
                e1.record(st)
                e1.synchronize()
                best[name] = max(best[name], nbytes / (e0.elapsed_time(e1) / 1e3) / 1e9)
    return {"h2d_gbs": best["h2d"], "d2h_gbs": best["d2h"], "bytes": nbytes}


def quick_measure(torch, name, device, flush, max_activity, steps=3):
    """A few steps of another workload of the benchmark definition in its own strategy (CUDA events on the
    library's stream, L2 flushed between steps): an entry of the "workloads" table, not the headline."""
    from paper_2412_11810_b200 import Session
    w = wl.WORKLOADS[name]
    d = wl.make(w, dense_input=False)
    s = Session(w.sizes, tau_mem=w.tau_mem, threshold=w.theta, surrogate_beta=w.beta, cell=w.cell,
                readout_scale=w.scale(), device=str(device))
    s.set_weights(d["W_ff"], d["W_rec"], d["W_out"])
    src = d["input_dense"] if w.cell == wl.CELL_GRADED else d["input_bits"].view(np.int32)
    bits, targets = torch.from_numpy(src).to(device), torch.from_numpy(d["targets"]).to(device)
    kw = dict(strategy=w.strategy, chunk_size=w.chunk_size, remote_chunk_size=w.remote_chunk_size,
              max_activity=max_activity)
    for _ in range(3):
        s.train_step(bits, targets, **kw)
    ms = []
    for _ in range(steps):
        flush.fill_(1)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(s.main):
            e0.record(); s.train_step(bits, targets, **kw); e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1))
    s.train_step(bits, targets, time_phases=True, **kw)
    ph = s.phase_times()
    dp, pp = s.peak_memory()
    out = {"value": w.B * w.T / (float(np.median(ms)) / 1e3), "unit": UNIT, "ms_per_step": float(np.median(ms)),
           "steps": steps, "strategy": STRATEGY_NAME[w.strategy], "chunk_size": w.chunk_size,
           "remote_chunk_size": w.remote_chunk_size, "sizes": list(w.sizes), "T": w.T, "B": w.B,
           "device_peak_bytes": dp, "pinned_peak_bytes": pp, "kernel_launches": int(s.stats().kernel_launches),
           "phases_ms": {k: v[0] for k, v in ph.items()}}
    s.close()
    return out


def run_ours(args, rank, world):
    import torch
    from paper_2412_11810_b200 import Session, binding as sb

    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    w = wl.WORKLOADS[args.workload]
    d = wl.make(w, dense_input=(rank == 0 and not args.no_cpu_baseline))
    s = Session(w.sizes, tau_mem=w.tau_mem, threshold=w.theta, surrogate_beta=w.beta, cell=w.cell,
                readout_scale=w.scale(), device=f"cuda:{local_rank}")
    s.set_weights(d["W_ff"], d["W_rec"], d["W_out"])
    if w.cell == wl.CELL_GRADED:
        bits_host = torch.from_numpy(d["input_dense"]).pin_memory()
    else:
        bits_host = torch.from_numpy(d["input_bits"].view(np.int32)).pin_memory()
    tg_host = torch.from_numpy(d["targets"]).pin_memory()
    bits, targets = bits_host.to(s.device), tg_host.to(s.device)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=s.device)   # larger than the 126 MB L2
    kw = dict(strategy=w.strategy, chunk_size=w.chunk_size, remote_chunk_size=w.remote_chunk_size,
              max_activity=args.max_activity, extra_flags=args.flags)

    def timed_steps(n, inp, tg, **extra):
        """n steps, each bracketed by CUDA events on the library's main stream; L2 flushed between."""
        ms, phases = [], []
        for _ in range(n):
            flush.fill_(1)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(s.main):
                e0.record()
                s.train_step(inp, tg, **kw, **extra)
                e1.record()
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
            if extra.get("time_phases"):
                phases.append(s.phase_times())
        return ms, phases

    timed_steps(args.warmup, bits, targets)
    barrier()
    clocks = ClockSampler(local_rank)
    if rank == 0:
        clocks.start()
    wall0 = time.perf_counter()
    ms, phases = timed_steps(args.steps, bits, targets, **({"time_phases": True} if args.profile else {}))
    barrier()
    wall = time.perf_counter() - wall0
    clk = clocks.stop() if rank == 0 else None
    # the split into passes comes from separate steps: the events around every pass cost a few per cent
    if not args.profile:
        _, phases = timed_steps(min(3, args.steps), bits, targets, time_phases=True)
    stats = s.stats()
    dev_peak, pin_peak = s.peak_memory()
    total_ms = float(sum(ms))
    # end to end: inputs start in pinned host memory, the loss comes back to the host
    if args.profile:
        e2e_total = total_ms
    else:
        timed_steps(1, bits_host, tg_host)
        e2e_ms, _ = timed_steps(max(3, args.steps // 4), bits_host, tg_host)
        e2e_total = float(sum(e2e_ms)) / len(e2e_ms) * args.steps
    (total_ms, e2e_total), (value, e2e_value) = aggregate_replicas(
        [total_ms, e2e_total], w.B * w.T * args.steps, world, dist, s.device)

    out = None
    if rank == 0:
        # measured activity per layer (input, hidden 1..L) from the stored event lists
        activity = []
        for layer in range(w.L + 1):
            off, _ = s.events(layer)
            activity.append(float(off[w.T + 1].astype(np.int64).sum()) / (w.T * w.B * w.sizes[layer]))
        fwd_b, bwd_b = algorithmic_bytes(w, activity, w.B)
        ph = {k: (sum(p[k][0] for p in phases) / len(phases), phases[0][k][1]) for k in phases[0]}
        peak, peak_kind = read_peaks()
        if ph["ffgemm"][1] > 0:
            # layer-by-layer backward order: a backward launch is one step of ONE layer and streams W_rec only
            bwd_b = sum(4.0 * n * n + 16.0 * w.B * n for n in w.sizes[1:-1]) / w.L
        dominant = max(("fwd", "refwd1", "refwd2", "bwd", "dw"), key=lambda k: ph[k][0])
        seg = {0: w.T, 1: w.chunk_size, 2: w.chunk_size, 3: w.chunk_size, 4: w.chunk_size, 5: w.chunk_size}[w.strategy]
        per_launch_bytes = {"fwd": fwd_b, "refwd1": fwd_b, "refwd2": fwd_b, "bwd": bwd_b,
                            "dw": dw_bytes(w, activity, w.B, min(seg, w.T))}.get(dominant)
        roof = None
        if per_launch_bytes and ph[dominant][1] > 0:
            kernel = {"fwd": "fwd_step_kernel<true>", "refwd1": "fwd_step_kernel<false>",
                      "refwd2": "fwd_step_kernel<false>", "bwd": "bwd_step_kernel", "dw": "dw_slab_kernel / dw_kernel"}[dominant]
            units = ph[dominant][1]
            if dominant == "fwd" and ph["fwd"][1] < w.T:
                # small spiking networks: one cooperative launch per forward operation, T steps in all;
                # the bytes are per step, so the launch count is replaced by the step count
                kernel, units = "fwd_resident_kernel / fwd_segment_kernel (per step)", w.T
            if dominant == "bwd" and ph["ffgemm"][1] > 0 and ph["bwd"][1] < w.T * w.L:
                # large networks: one cooperative launch per layer and run of 32 steps that keeps W_rec streaming;
                # the bytes are per step of one layer
                kernel, units = "bwd_stream_kernel (per layer and step)", w.T * w.L
            elif dominant == "bwd" and ph["bwd"][1] < w.T:
                # small networks: one cooperative launch per segment with the weights resident
                kernel, units = "bwd_segment_kernel (per step)", w.T
            avg_s = ph[dominant][0] / 1e3 / units
            ach = per_launch_bytes / avg_s / 1e9
            roof = {"bound": "hbm", "kernel": kernel,
                    "phase": dominant,
                    "achieved": ach, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": ach / peak,
                    "traffic": ncu_traffic(w.name, dominant), "algorithmic_bytes_per_launch": per_launch_bytes,
                    "avg_launch_us": avg_s * 1e6, "launches_per_step": ph[dominant][1]}
            if dominant == "bwd":
                # the backward step is the one dense contraction of the path (delta x W^T, fp32 result through three
                # TF32 passes): its rate against the tensor peak for tf32 (measured bf16 peak x nominal 1.1 / 2.25)
                sz = w.sizes
                if ph["ffgemm"][1] > 0:     # one layer per launch, recurrent matrix only
                    flops = 2.0 * w.B * sum(n * n for n in sz[1:-1]) / w.L
                else:
                    flops = 2.0 * w.B * sum(sz[l] * sz[l] + (sz[l] * sz[l + 1] if l < w.L else 0)
                                            for l in range(1, w.L + 1))
                tpeak, tkind = read_tensor_peak()
                roof["tensor"] = {"achieved": flops / avg_s / 1e12, "peak": tpeak, "peak_kind": tkind,
                                  "unit": "TFLOP/s", "frac": flops / avg_s / 1e12 / tpeak,
                                  "flops_per_launch": flops,
                                  "note": "fp32-equivalent flops; the kernel issues three tf32 mma.sync passes per product"}
        # the other strategies on the same workload (fewer steps), for the per-strategy table
        per_strategy = {}
        T = w.T
        K0 = w.chunk_size if w.strategy in (1, 2) else max(1, int(round(T ** 0.5)))
        Kd, Rd = (w.chunk_size, w.remote_chunk_size) if w.strategy == 3 else (16, 256)
        P0 = max(1, int(round((-(-T // K0)) ** 0.5)))          # nb_local = sqrt(number of checkpoints)
        alt = {0: (0, 0), 1: (K0, 0), 2: (K0, 0), 3: (Kd, Rd), 4: (K0, P0), 5: (Kd, Rd)}
        for strat, (K, R) in ([] if args.no_strategies else alt.items()):
            kws = dict(strategy=strat, chunk_size=K, remote_chunk_size=0 if strat == 4 else R,
                       nb_local=R if strat == 4 else 0, max_activity=args.max_activity)
            s.train_step(bits, targets, **kws)
            tms = []
            for _ in range(3):
                flush.fill_(1); torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                with torch.cuda.stream(s.main):
                    e0.record(); s.train_step(bits, targets, **kws); e1.record()
                torch.cuda.synchronize()
                tms.append(e0.elapsed_time(e1))
            st = s.stats()
            dp, pp = s.peak_memory()
            per_strategy[STRATEGY_NAME[strat]] = {
                "chunk_size": K, "remote_chunk_size": 0 if strat == 4 else R, "nb_local": R if strat == 4 else 0,
                "d2h_copies": st.d2h_copies, "h2d_copies": st.h2d_copies, "value": w.B * T / (float(np.median(tms)) / 1e3),
                "ms_per_step": float(np.median(tms)), "device_peak_bytes": dp, "pinned_peak_bytes": pp,
                "local_state_slots": st.local_state_slots, "state_bytes": st.state_bytes,
                "kernel_launches": st.kernel_launches}
        link = host_link_probe(torch, s.device)
        others = {}
        if world == 1 and not args.no_other_workloads:
            for name in sorted(wl.WORKLOADS):
                if name != w.name:
                    others[name] = quick_measure(torch, name, s.device, flush, args.max_activity)
        cpu = None
        if not args.no_cpu_baseline:
            from oracle.oracle import num_threads
            # bounded sample: a short probe sizes the number of steps so that the run takes ~20 s
            T_probe = min(8, w.T)
            per_step = time_oracle(w, d, T_probe) / T_probe
            T_s = int(min(w.T, max(T_probe, 20.0 / per_step)))
            sec = time_oracle(w, d, T_s)
            cpu = {"value": w.B * T_s / sec, "unit": UNIT, "cores": num_threads(), "kind": "oracle",
                   "sample": f"one oracle train step (full-storage BPTT) on the first {T_s} of {w.T} steps, "
                             f"full width and batch, {sec:.1f} s"}
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "sizes": list(w.sizes), "T": w.T, "B": w.B,
                       "strategy": STRATEGY_NAME[w.strategy], "chunk_size": w.chunk_size,
                       "remote_chunk_size": w.remote_chunk_size, "l2": "flushed between timed steps",
                       "parallelism": "replicas only" if world > 1 else "single gpu",
                       "measured_activity": activity},
            "clocks": clk,
            "e2e": {"value": e2e_value, "unit": UNIT,
                    "h2d_bytes_per_step": int(bits_host.numel() * 4 + tg_host.numel() * 4), "d2h_bytes_per_step": 8},
            "gpu_launches": int(stats.kernel_launches) * args.steps,
            "roofline": roof,
            "phases_ms": {k: v[0] for k, v in ph.items()}, "phase_launches": {k: v[1] for k, v in ph.items()},
            "host_link": None if not stats.d2h_copies else {
                "bytes_per_copy": int(stats.state_bytes), "d2h_copies": int(stats.d2h_copies),
                "h2d_copies": int(stats.h2d_copies),
                "d2h_gbs": stats.state_bytes * stats.d2h_copies / (ph["d2h"][0] / 1e3) / 1e9 if ph["d2h"][0] > 0 else None,
                "h2d_gbs": stats.state_bytes * stats.h2d_copies / (ph["h2d"][0] / 1e3) / 1e9 if ph["h2d"][0] > 0 else None,
                "copy_ms_per_step": ph["d2h"][0] + ph["h2d"][0],
                "peak": link, "peak_kind": "pinned 64 MiB copy each way, CUDA events, same run",
                "d2h_frac": (stats.state_bytes * stats.d2h_copies / (ph["d2h"][0] / 1e3) / 1e9 / link["d2h_gbs"])
                            if ph["d2h"][0] > 0 else None,
                "h2d_frac": (stats.state_bytes * stats.h2d_copies / (ph["h2d"][0] / 1e3) / 1e9 / link["h2d_gbs"])
                            if ph["h2d"][0] > 0 else None,
                "note": "CUDA events on the side stream around every checkpoint copy; copies overlap the passes"},
            "peak_memory": {"device_bytes": dev_peak, "pinned_bytes": pin_peak,
                            "local_state_slots": stats.local_state_slots, "state_bytes": stats.state_bytes,
                            "event_bytes": stats.event_bytes},
            "strategies": per_strategy,
            "workloads": others,
            "cpu_baseline": cpu,
            "wall_s_timed_region": wall,
        }
    s.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if out is not None:
        print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--max-activity", type=float, default=0.25)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-strategies", action="store_true", help="skip the per-strategy table")
    ap.add_argument("--no-other-workloads", action="store_true", help="skip the brief runs of the other workloads")
    ap.add_argument("--profile", action="store_true",
                    help="for a profiler: one warm-up step and one timed step of the workload, nothing else "
                         "(no end-to-end steps, strategy table, other workloads or CPU baseline); the printed "
                         "numbers are not benchmark values")
    ap.add_argument("--flags", type=int, default=0,
                    help="extra SNN_FLAG_* bits for the timed strategy, e.g. 256 = backward with one launch per step")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.profile:
        args.warmup, args.steps = 1, 1
        args.no_cpu_baseline = args.no_strategies = args.no_other_workloads = True
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        # called as a plain script: start one replica rank per GPU and let rank 0 print the line
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, world)


if __name__ == "__main__":
    main()
