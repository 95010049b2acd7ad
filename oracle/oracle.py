"""ctypes front end of the CPU oracle (test infrastructure only).

Only tests/, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It knows nothing about the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass, field
from typing import Sequence

import numpy as np

from . import build_oracle

CELL_LIF, CELL_GRADED = 0, 1
SURR_FAST_SIGMOID, SURR_SIGMOID, SURR_TRIANGLE = 0, 1, 2


class _Params(C.Structure):
    _fields_ = [("L", C.c_int32), ("cell", C.c_int32), ("surrogate", C.c_int32), ("smooth", C.c_int32),
                ("alpha", C.c_double), ("theta", C.c_double), ("beta", C.c_double), ("scale", C.c_double)]


def leak_from_tau(tau_mem: float) -> np.float32:
    """alpha = exp(-1/tau), evaluated in double and rounded once to fp32."""
    return np.float32(np.exp(-1.0 / np.float64(tau_mem)))


@dataclass
class NetSpec:
    sizes: Sequence[int]              # N_0, N_1..N_L, N_out
    alpha: float                      # leak per step (already rounded to the working precision)
    theta: float = 1.0
    beta: float = 10.0
    scale: float = 1.0
    cell: int = CELL_LIF
    surrogate: int = SURR_FAST_SIGMOID
    smooth: bool = False
    L: int = field(init=False)

    def __post_init__(self):
        self.sizes = [int(s) for s in self.sizes]
        self.L = len(self.sizes) - 2
        assert self.L >= 1

    def c_params(self) -> _Params:
        return _Params(self.L, self.cell, self.surrogate, int(self.smooth),
                       float(self.alpha), float(self.theta), float(self.beta), float(self.scale))


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _ptr_array(arrs):
    if arrs is None:
        return None
    return (C.c_void_p * len(arrs))(*[a.ctypes.data if a is not None else None for a in arrs])


class Oracle:
    """kind='f32': canonical fp32 forward, double backward.  kind='f64': all double."""

    def __init__(self, kind: str = "f32"):
        assert kind in ("f32", "f64")
        build_oracle.build()
        self.kind = kind
        self.real = np.float32 if kind == "f32" else np.float64
        self.lib = C.CDLL(build_oracle.lib_path(kind))
        self._fwd = getattr(self.lib, f"oracle_{kind}_forward_step")
        self._bwd = getattr(self.lib, f"oracle_{kind}_backward_step")
        self._readout = getattr(self.lib, f"oracle_{kind}_readout")
        self._readout.restype = C.c_double
        self._full = getattr(self.lib, f"oracle_{kind}_bptt_full")
        self._full.restype = C.c_double
        self._compact = getattr(self.lib, f"oracle_{kind}_compact")
        self._compact.restype = C.c_int32

    def _r(self, a):
        return np.ascontiguousarray(a, dtype=self.real)

    # ---- single steps -------------------------------------------------------------------
    def forward_step(self, spec: NetSpec, S_below, S_prev, V_prev, W_ff, W_rec):
        S_below, S_prev, V_prev = self._r(S_below), self._r(S_prev), self._r(V_prev)
        W_ff, W_rec = self._r(W_ff), self._r(W_rec)
        B, N_pre = S_below.shape
        N = S_prev.shape[1]
        assert W_ff.shape == (N_pre, N) and W_rec.shape == (N, N) and V_prev.shape == (B, N)
        V = np.empty((B, N), self.real)
        S = np.empty((B, N), self.real)
        p = spec.c_params()
        self._fwd(C.byref(p), C.c_int32(B), C.c_int32(N_pre), C.c_int32(N), _ptr(S_below), _ptr(S_prev),
                  _ptr(V_prev), _ptr(W_ff), _ptr(W_rec), _ptr(V), _ptr(S))
        return V, S

    def readout(self, spec: NetSpec, c, targets, W_out):
        c, W_out = self._r(c), self._r(W_out)
        targets = np.ascontiguousarray(targets, np.int32)
        B, N_L = c.shape
        N_out = W_out.shape[1]
        logits = np.empty((B, N_out)); dlogits = np.empty((B, N_out))
        g_out = np.empty((B, N_L)); dW_out = np.empty((N_L, N_out))
        p = spec.c_params()
        loss = self._readout(C.byref(p), C.c_int32(B), C.c_int32(N_L), C.c_int32(N_out), _ptr(c),
                             _ptr(targets), _ptr(W_out), _ptr(logits), _ptr(dlogits), _ptr(g_out),
                             _ptr(dW_out))
        return float(loss), logits, dlogits, g_out, dW_out

    def backward_step(self, spec: NetSpec, V_t, S_below_t, S_prev, delta_next, delta_above, g_out,
                      W_ff_above, W_rec, dW_ff, dW_rec):
        """Returns delta^l_t; accumulates into dW_ff / dW_rec (float64, in place)."""
        V_t, S_below_t, S_prev, W_rec = self._r(V_t), self._r(S_below_t), self._r(S_prev), self._r(W_rec)
        B, N = V_t.shape
        N_pre = S_below_t.shape[1]
        N_post = 0
        if delta_above is not None:
            delta_above = np.ascontiguousarray(delta_above, np.float64)
            W_ff_above = self._r(W_ff_above)
            N_post = W_ff_above.shape[1]
            assert W_ff_above.shape[0] == N and delta_above.shape == (B, N_post)
        else:
            W_ff_above = None
        delta_next = np.ascontiguousarray(delta_next, np.float64)
        if g_out is not None:
            g_out = np.ascontiguousarray(g_out, np.float64)
        assert dW_ff.dtype == np.float64 and dW_rec.dtype == np.float64
        assert dW_ff.flags.c_contiguous and dW_rec.flags.c_contiguous
        assert dW_ff.shape == (N_pre, N) and dW_rec.shape == (N, N)
        delta = np.empty((B, N))
        p = spec.c_params()
        self._bwd(C.byref(p), C.c_int32(B), C.c_int32(N_pre), C.c_int32(N), C.c_int32(N_post), _ptr(V_t),
                  _ptr(S_below_t), _ptr(S_prev), _ptr(delta_next), _ptr(delta_above), _ptr(g_out),
                  _ptr(W_ff_above), _ptr(W_rec), _ptr(delta), _ptr(dW_ff), _ptr(dW_rec))
        return delta

    # ---- the whole training step ---------------------------------------------------------
    def bptt_full(self, spec: NetSpec, inp, targets, W_ff, W_rec, W_out, *, keep_states=True,
                  keep_delta=False, do_backward=True):
        """Full-storage BPTT.  inp [T][B][N_0].  Returns a dict with loss, logits, counts,
        V / S (lists per hidden layer, [T+1][B][N]), delta (optional, [T+2][B][N]) and the
        gradients dW_ff, dW_rec (lists), dW_out (all float64)."""
        L, sizes = spec.L, spec.sizes
        inp = self._r(inp)
        T, B, N0 = inp.shape
        assert N0 == sizes[0]
        targets = np.ascontiguousarray(targets, np.int32)
        W_ff = [self._r(w) for w in W_ff]
        W_rec = [self._r(w) for w in W_rec]
        W_out = self._r(W_out)
        for l in range(L):
            assert W_ff[l].shape == (sizes[l], sizes[l + 1]) and W_rec[l].shape == (sizes[l + 1],) * 2
        assert W_out.shape == (sizes[L], sizes[L + 1])
        V = [np.empty((T + 1, B, sizes[l + 1]), self.real) for l in range(L)] if keep_states else None
        S = [np.empty((T + 1, B, sizes[l + 1]), self.real) for l in range(L)] if keep_states else None
        D = [np.empty((T + 2, B, sizes[l + 1])) for l in range(L)] if keep_delta else None
        dW_ff = [np.empty((sizes[l], sizes[l + 1])) for l in range(L)]
        dW_rec = [np.empty((sizes[l + 1], sizes[l + 1])) for l in range(L)]
        dW_out = np.empty((sizes[L], sizes[L + 1]))
        logits = np.empty((B, sizes[L + 1]))
        counts = np.empty((B, sizes[L]), self.real)
        p = spec.c_params()
        csizes = (C.c_int32 * (L + 2))(*sizes)
        loss = self._full(C.byref(p), csizes, C.c_int32(T), C.c_int32(B), _ptr(inp), _ptr(targets),
                          _ptr_array(W_ff), _ptr_array(W_rec), _ptr(W_out), _ptr_array(V), _ptr_array(S),
                          _ptr_array(D), _ptr_array(dW_ff), _ptr_array(dW_rec), _ptr(dW_out),
                          _ptr(logits), _ptr(counts), C.c_int32(int(do_backward)))
        out = dict(loss=float(loss), logits=logits, counts=counts, V=V, S=S, delta=D)
        if do_backward:
            out.update(dW_ff=dW_ff, dW_rec=dW_rec, dW_out=dW_out)
        return out

    def compact(self, v, theta: float) -> np.ndarray:
        """Ascending indices i with v[i] > theta (brute force)."""
        v = self._r(v).ravel()
        idx = np.empty(v.size, np.int32)
        n = self._compact(_ptr(v), C.c_int32(v.size), C.c_double(theta), _ptr(idx))
        return idx[:n].copy()


def num_threads() -> int:
    """Threads the oracle's OpenMP loops will use."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    return len(os.sched_getaffinity(0))
