"""Shared plumbing of the GPU parity tests: run a workload through the oracle and through the
CUDA library (via its C ABI) on the same arrays."""
import numpy as np

import snn_workloads as wl
from oracle.oracle import NetSpec, leak_from_tau

GRAD_RTOL = 1e-4     # per tensor: max |g_gpu - g_ref| <= GRAD_RTOL * max |g_ref|
V_ATOL = 1e-5        # membranes, absolute


def spec_of(w):
    return NetSpec(w.sizes, leak_from_tau(w.tau_mem), w.theta, w.beta, w.scale(), cell=w.cell)


def run_oracle(orc, w, d, **kw):
    return orc.bptt_full(spec_of(w), d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"], **kw)


def make_session(w, d):
    import torch
    from paper_2412_11810_b200 import Session
    s = Session(w.sizes, tau_mem=w.tau_mem, threshold=w.theta, surrogate_beta=w.beta, cell=w.cell,
                readout_scale=w.scale())
    s.set_weights(d["W_ff"], d["W_rec"], d["W_out"])
    if w.cell == wl.CELL_GRADED:
        bits = torch.from_numpy(d["input_dense"]).to(s.device)
    else:
        bits = torch.from_numpy(d["input_bits"].view(np.int32)).to(s.device)
    targets = torch.from_numpy(d["targets"]).to(s.device)
    return s, bits, targets


def lists_from_dense(S_tb):
    """Ascending active indices per (t, b) of a dense 0/1 array [T][B][N] (brute force)."""
    return [[np.flatnonzero(S_tb[t, b]).astype(np.uint32) for b in range(S_tb.shape[1])]
            for t in range(S_tb.shape[0])]


def assert_grads_close(gpu, ref, rtol=GRAD_RTOL):
    gff, grec, gout = gpu
    for name, a, b in ([(f"dW_ff[{l}]", gff[l], ref["dW_ff"][l]) for l in range(len(gff))]
                       + [(f"dW_rec[{l}]", grec[l], ref["dW_rec"][l]) for l in range(len(grec))]
                       + [("dW_out", gout, ref["dW_out"])]):
        scale = np.abs(b).max()
        err = np.abs(a.astype(np.float64) - b).max()
        assert err <= rtol * scale + 1e-30, f"{name}: err {err:.3e} vs scale {scale:.3e}"
        # rows no event ever touched are exactly zero on both sides
        zero_rows = ~np.any(b != 0, axis=1)
        assert np.all(a[zero_rows] == 0), f"{name}: untouched rows must be exactly zero"
