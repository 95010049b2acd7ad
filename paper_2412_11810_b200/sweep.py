#!/usr/bin/env python
"""Time and peak memory of one train step against the hyper-parameters of the checkpointing strategies.

The paper's Hyperparameter Study plots time and memory against the sequence length T, the network width N,
the checkpoint interval (chunk_size), the number of local checkpoints of the hierarchical scheme (nb_local)
and the remote interval of Double Checkpointing (remote_chunk_size).  This script measures the same curves
on one GPU with synthetic spikes on a network shaped like a benchmark workload, and prints one JSON line per
point (or, with --markdown, one table per sweep).

    python paper_2412_11810_b200/sweep.py --workload c2 --markdown
"""
from __future__ import annotations

import argparse
import json
import os
import sys
from dataclasses import replace

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import snn_workloads as wl  # noqa: E402

NAMES = {0: "standard", 1: "chunk", 2: "remote", 3: "double", 4: "hierarchical", 5: "double_local"}


def measure(w, strategy, K=0, R=0, P=0, reps=3, max_activity=0.25):
    """One point: best of `reps` timed steps after one warm-up; returns a dict."""
    import torch
    from paper_2412_11810_b200 import Session

    d = wl.make(w, dense_input=False)
    s = Session(w.sizes, tau_mem=w.tau_mem, threshold=w.theta, surrogate_beta=w.beta, cell=w.cell,
                readout_scale=w.scale())
    s.set_weights(d["W_ff"], d["W_rec"], d["W_out"])
    x = d["input_dense"] if w.cell == wl.CELL_GRADED else d["input_bits"].view(np.int32)
    x = torch.from_numpy(np.ascontiguousarray(x)).to(s.device)
    tg = torch.from_numpy(d["targets"]).to(s.device)
    kw = dict(strategy=strategy, chunk_size=K, remote_chunk_size=R, nb_local=P, max_activity=max_activity)
    s.train_step(x, tg, **kw)
    ms = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(s.main):
            e0.record()
            s.train_step(x, tg, **kw)
            e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1))
    dev, pin = s.peak_memory()
    st = s.stats()
    out = {"strategy": NAMES[strategy], "sizes": list(w.sizes), "T": w.T, "B": w.B, "chunk_size": K,
           "remote_chunk_size": R, "nb_local": P, "ms_per_step": min(ms),
           "us_per_timestep": 1e3 * min(ms) / w.T, "device_peak_bytes": dev, "pinned_peak_bytes": pin,
           "state_slots": st.local_state_slots, "state_bytes": st.state_bytes, "event_bytes": st.event_bytes,
           "d2h_copies": st.d2h_copies, "h2d_copies": st.h2d_copies}
    s.close()
    del s, x
    torch.cuda.empty_cache()
    return out


def isqrt_pow2(x):
    """Power of two nearest to sqrt(x) from below."""
    k = 1
    while 4 * k * k <= x:
        k *= 2
    return k


def sweeps(base, quick):
    """Yields (sweep name, varied key, list of measure() keyword dicts)."""
    Ts = [250, 1000, 4000] if quick else [250, 500, 1000, 2000, 4000, 8000]
    pts = []
    for T in Ts:
        w = base.with_T(T)
        K = max(1, int(round(T ** 0.5)))
        Kd = 16
        Rd = min(256, max(Kd, (T // Kd) * Kd))
        n_ck = -(-T // K)
        for strat, kw in ((0, {}), (1, dict(K=K)), (2, dict(K=K)), (3, dict(K=Kd, R=Rd)),
                          (4, dict(K=K, P=max(1, int(round(n_ck ** 0.5))))), (5, dict(K=Kd, R=Rd))):
            pts.append(dict(w=w, strategy=strat, **kw))
    yield "sequence length", "T", pts
    T = 1000 if quick else 2000
    w = base.with_T(T)
    Ks = [8, 32, 128] if quick else [4, 8, 16, 32, 45, 64, 128, 256, 500]
    yield "chunk size (T = %d)" % T, "chunk_size", [dict(w=w, strategy=s, K=K) for K in Ks for s in (1, 2)]
    T = 2000 if quick else 4000
    w = base.with_T(T)
    Rs = [64, 256] if quick else [64, 128, 256, 512, 1024]
    yield "remote chunk size of Double Checkpointing (T = %d)" % T, "remote_chunk_size", \
        [dict(w=w, strategy=3, K=isqrt_pow2(R), R=R) for R in Rs]
    Ps = [1, 8] if quick else [1, 2, 4, 8, 16, 32]
    yield "local checkpoints of the hierarchical scheme (T = %d, chunk size 16)" % T, "nb_local", \
        [dict(w=w, strategy=4, K=16, P=P) for P in Ps]
    Ns = [256, 1024] if quick else [256, 512, 1024, 2048]
    T = 1000
    pts = []
    for N in Ns:
        sizes = (base.sizes[0],) + (N,) * base.L + (base.sizes[-1],)
        wn = replace(base, sizes=sizes, T=T, readout_scale=1.0 / T)
        pts += [dict(w=wn, strategy=0), dict(w=wn, strategy=1, K=32), dict(w=wn, strategy=3, K=16, R=256)]
    yield "hidden width (T = 1000)", "sizes", pts


def event_backward_table(base, T=192, K=16):
    """Dense against event-driven backward pass (SNN_SURR_TRIANGLE) on the network of `base`: per batch size and
    surrogate width the fraction of near-threshold neurons and the time of the backward steps of one train step of
    T steps (CHUNK, chunk size K), from the per-pass CUDA-event timers.  Prints a markdown table."""
    import torch
    from paper_2412_11810_b200 import Session, binding as sb

    print(f"\n## event-driven against dense backward steps ({'-'.join(map(str, base.sizes))}, T = {T}, chunk {K}, triangle surrogate)\n")
    print("| B | beta | near-threshold fraction per layer | dense: backward steps + feed-forward product ms | "
          "event-driven: backward steps ms | ratio |")
    print("|---|---|---|---|---|---|")
    for B in (1, 8, 32):
        w = replace(base, T=T, B=B, readout_scale=1.0 / T)
        d = wl.make(w, dense_input=False)
        x = torch.from_numpy(np.ascontiguousarray(d["input_bits"].view(np.int32))).cuda()
        tg = torch.from_numpy(d["targets"]).cuda()
        for beta in (3.0, 10.0):
            s = Session(w.sizes, tau_mem=w.tau_mem, threshold=w.theta, surrogate=sb.SNN_SURR_TRIANGLE,
                        surrogate_beta=beta, readout_scale=w.scale())
            s.set_weights(d["W_ff"], d["W_rec"], d["W_out"])
            s.train_step(x[:64], tg, strategy=0, forward_only=True, keep_V=True)
            near = [float(((v[1:] - w.theta).abs() * beta < 1).float().mean()) for v in s.debug_V]
            s.debug_V = None
            res = {}
            for name, flags in (("dense", 0), ("event", sb.SNN_FLAG_BACKWARD_EVENT_DRIVEN)):
                kw = dict(strategy=1, chunk_size=K, extra_flags=flags)
                s.train_step(x, tg, **kw)
                best = None
                for _ in range(2):
                    s.train_step(x, tg, time_phases=True, **kw)
                    ph = s.phase_times()
                    ms = ph["bwd"][0] + ph["ffgemm"][0]
                    best = ms if best is None else min(best, ms)
                res[name] = best
            print(f"| {B} | {beta:g} | {' / '.join(f'{100 * v:.1f} %' for v in near)} | {res['dense']:.1f} | "
                  f"{res['event']:.1f} | {res['event'] / res['dense']:.2f} |", flush=True)
            s.close()
            del s
            torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c2", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--quick", action="store_true", help="a few points per sweep")
    ap.add_argument("--markdown", action="store_true", help="tables instead of JSON lines")
    ap.add_argument("--event-backward", action="store_true",
                    help="only the table of the event-driven against the dense backward pass (triangle surrogate)")
    args = ap.parse_args()
    base = wl.WORKLOADS[args.workload]
    if args.event_backward:
        event_backward_table(base)
        return 0
    for name, key, pts in sweeps(base, args.quick):
        rows = [measure(**p) for p in pts]
        if not args.markdown:
            for r in rows:
                print(json.dumps(dict(sweep=name, **r)), flush=True)
            continue
        print(f"\n## {name}\n")
        print(f"| {key} | strategy (K, R, P) | ms per step | us per timestep | device peak MiB | pinned MiB | state slots | copies each way |")
        print("|---|---|---|---|---|---|---|---|")
        for r in rows:
            val = r["sizes"][1] if key == "sizes" else r[key]
            print(f"| {val} | {r['strategy']} ({r['chunk_size']}, {r['remote_chunk_size']}, {r['nb_local']}) | "
                  f"{r['ms_per_step']:.2f} | {r['us_per_timestep']:.2f} | {r['device_peak_bytes'] / 2**20:.0f} | "
                  f"{r['pinned_peak_bytes'] / 2**20:.1f} | {r['state_slots']} | {r['d2h_copies']} |", flush=True)
    return 0


if __name__ == "__main__":
    sys.exit(main())
