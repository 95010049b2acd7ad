#!/usr/bin/env python
"""How much longer a sequence fits under a fixed device-memory budget with Double Checkpointing.

The paper's headline claim is sequences more than ten times longer than plain BPTT at little extra
time.  This script reproduces the shape of that experiment on one GPU: under a cap on the device
workspace it finds the longest sequence full-storage BPTT (STANDARD) can train, runs it, then runs
DOUBLE at a multiple of that length under the same cap, and prints one JSON line with both times
per sample-timestep, the peak bytes and the overhead.

    python paper_2412_11810_b200/seqlen_demo.py --workload c3 --cap-gib 2 --factor 10
    python paper_2412_11810_b200/seqlen_demo.py --workload c3 --cap-gib 2 --factor 30 --spill

With --spill the DOUBLE run keeps only two remote segments' events on the device (SNN_FLAG_SPILL_EVENTS); the events of
the other segments wait in pinned host memory, so the device workspace no longer grows with the sequence.
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


def longest(fits, hi=1 << 26):
    lo = 1
    while lo < hi:
        mid = (lo + hi + 1) // 2
        lo, hi = (mid, hi) if fits(mid) else (lo, mid - 1)
    return lo


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c3", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--cap-gib", type=float, default=2.0, help="cap on the device workspace")
    ap.add_argument("--factor", type=int, default=10, help="DOUBLE runs factor x the longest STANDARD sequence")
    ap.add_argument("--max-activity", type=float, default=0.06)
    ap.add_argument("--remote-chunk", type=int, default=256)
    ap.add_argument("--chunk", type=int, default=16)
    ap.add_argument("--spill", action="store_true", help="DOUBLE spills the events of finished remote segments to pinned memory")
    args = ap.parse_args()

    import torch
    from paper_2412_11810_b200 import Session, binding as sb

    base = wl.WORKLOADS[args.workload]
    cap = int(args.cap_gib * (1 << 30))
    net = sb.snn_create(list(base.sizes), base.tau_mem, base.theta, cell=base.cell)

    dbl_flags = sb.SNN_FLAG_SPILL_EVENTS if args.spill else 0

    def fits(ck, flags=0):
        def f(T):
            try:
                return sb.snn_workspace_query(net, T, base.B, ck, args.max_activity, flags)[0] <= cap
            except sb.SnnError:
                return False
        return f

    T_std = longest(fits(sb.snn_ckpt(sb.SNN_STANDARD, 0, 0)))
    T_dbl_max = longest(fits(sb.snn_ckpt(sb.SNN_DOUBLE, args.chunk, args.remote_chunk), dbl_flags))
    sb.snn_destroy(net)
    T_dbl = args.factor * T_std
    out = {"workload": base.name, "sizes": list(base.sizes), "B": base.B, "cap_bytes": cap,
           "max_activity": args.max_activity, "T_standard_max": T_std, "T_double": T_dbl,
           "T_double_max_under_cap": T_dbl_max, "chunk_size": args.chunk, "remote_chunk_size": args.remote_chunk,
           "events_spilled": bool(args.spill)}
    if T_dbl > T_dbl_max:
        out["error"] = "DOUBLE does not fit the requested multiple under the cap"
        print(json.dumps(out))
        return 1

    w_long = replace(base, T=T_dbl, readout_scale=1.0 / T_dbl)
    d = wl.make(w_long, dense_input=False)
    s = Session(base.sizes, tau_mem=base.tau_mem, threshold=base.theta, surrogate_beta=base.beta, cell=base.cell,
                readout_scale=1.0 / T_dbl)
    s.set_weights(d["W_ff"], d["W_rec"], d["W_out"])
    x_all = d["input_dense"] if base.cell == wl.CELL_GRADED else d["input_bits"].view(np.int32)
    targets = torch.from_numpy(d["targets"]).to(s.device)
    for name, T, strat, K, R in (("standard", T_std, sb.SNN_STANDARD, 0, 0),
                                 ("double", T_dbl, sb.SNN_DOUBLE, args.chunk, args.remote_chunk)):
        x = torch.from_numpy(np.ascontiguousarray(x_all[:T])).to(s.device)
        s.device_ws = None                            # a fresh workspace of exactly the queried size
        torch.cuda.empty_cache()
        kw = dict(strategy=strat, chunk_size=K, remote_chunk_size=R, max_activity=args.max_activity,
                  extra_flags=dbl_flags if name == "double" else 0)
        s.train_step(x, targets, **kw)
        ms = []
        for _ in range(2):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(s.main):
                e0.record()
                loss = s.train_step(x, targets, **kw)
                e1.record()
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        dev, pin = s.peak_memory()
        st = s.stats()
        assert dev <= cap, (dev, cap)
        out[name] = {"T": T, "ms_per_step": min(ms), "ns_per_sample_timestep": 1e6 * min(ms) / (T * base.B),
                     "device_peak_bytes": dev, "pinned_peak_bytes": pin, "local_state_slots": st.local_state_slots,
                     "state_bytes": st.state_bytes, "event_bytes": st.event_bytes, "loss": loss,
                     "d2h_copies": st.d2h_copies, "h2d_copies": st.h2d_copies,
                     "event_window_copies": st.event_window_copies}
        del x
    out["sequence_length_ratio"] = T_dbl / T_std
    out["time_overhead_per_sample_timestep"] = (out["double"]["ns_per_sample_timestep"] /
                                                out["standard"]["ns_per_sample_timestep"] - 1.0)
    s.close()
    print(json.dumps(out))
    return 0


if __name__ == "__main__":
    sys.exit(main())
