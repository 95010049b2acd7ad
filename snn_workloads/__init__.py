"""Seeded synthetic workloads (inputs, targets, weights) shaped like the paper's experiments.

This module only draws random numbers and packs bits.  It contains none of the
method's arithmetic, so both the CUDA library's callers and the CPU oracle's
callers can be fed the very same arrays.

Recipe (all draws from numpy.random.Generator(PCG64(seed)), in this order):
  1. weights: for each hidden layer l, W_ff^l ~ N(0, g_ff^2 / N_{l-1}) then
     W_rec^l ~ N(0, g_rec^2 / N_l); then W_out ~ N(0, 1 / N_L); all fp32, row-major
     by presynaptic neuron;
  2. input: spikes i.i.d. Bernoulli(p_in) per (t, b, i); for the graded workload
     values ~ N(0, 1) multiplied by a Bernoulli(p_in) mask;
  3. targets: uniform integers in [0, N_out).
The gains g_ff, g_rec are fixed constants per workload, chosen once (offline, by
bisection on a forward pass) so that the hidden activity lands near the level the
workload names (about 5 % for the spiking ones, about 10 % for the graded one).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Optional, Sequence

import numpy as np

STANDARD, CHUNK, REMOTE, DOUBLE = 0, 1, 2, 3
CELL_LIF, CELL_GRADED = 0, 1


@dataclass(frozen=True)
class Workload:
    name: str
    sizes: Sequence[int]        # N_0, N_1..N_L, N_out
    T: int
    B: int
    p_in: float
    seed: int
    strategy: int
    chunk_size: int = 0
    remote_chunk_size: int = 0
    cell: int = CELL_LIF
    tau_mem: float = 20.0
    theta: float = 1.0
    beta: float = 10.0
    g_ff: Sequence[float] = ()
    g_rec: Sequence[float] = ()
    readout_scale: Optional[float] = None   # None -> 1/T

    @property
    def L(self) -> int:
        return len(self.sizes) - 2

    def scale(self) -> float:
        return 1.0 / self.T if self.readout_scale is None else self.readout_scale

    def with_T(self, T: int) -> "Workload":
        """Same network and seed, shorter or longer sequence (weights do not depend on T)."""
        return replace(self, T=int(T), readout_scale=self.scale())


# The five configurations of the benchmark definition.  c1 states seed 0 and a literal
# time-summed readout (scale 1); the others use seeds 1..4 and scale 1/T so that the
# soft-max does not saturate.
WORKLOADS: Dict[str, Workload] = {
    "c1": Workload("c1", (64, 128, 10), T=100, B=4, p_in=0.05, seed=0, strategy=STANDARD,
                   g_ff=(1.0,), g_rec=(1.0,), readout_scale=1.0),
    "c2": Workload("c2", (512, 1024, 1024, 20), T=1000, B=32, p_in=0.03, seed=1, strategy=CHUNK,
                   chunk_size=32, g_ff=(2.49, 1.34), g_rec=(1.0, 1.0)),
    "c3": Workload("c3", (512, 2048, 2048, 20), T=10000, B=16, p_in=0.02, seed=2, strategy=REMOTE,
                   chunk_size=64, g_ff=(3.08, 1.32), g_rec=(1.0, 1.0)),
    "c4": Workload("c4", (1024, 8192, 8192, 8192, 100), T=2000, B=8, p_in=0.02, seed=3, strategy=DOUBLE,
                   chunk_size=16, remote_chunk_size=256, g_ff=(2.9, 1.36, 1.32), g_rec=(1.0, 1.0, 1.0)),
    "c5": Workload("c5", (1024, 4096, 4096, 50), T=4096, B=16, p_in=0.10, seed=4, strategy=DOUBLE,
                   chunk_size=16, remote_chunk_size=256, cell=CELL_GRADED, g_ff=(0.703, 0.113),
                   g_rec=(0.05, 0.05)),
}


def pack_bits(dense: np.ndarray) -> np.ndarray:
    """[..., N] array of 0/non-zero -> [..., ceil(N/32)] uint32, bit (i % 32) of word i // 32."""
    n = dense.shape[-1]
    words = (n + 31) // 32
    bits = np.zeros(dense.shape[:-1] + (words * 32,), np.uint8)
    bits[..., :n] = dense != 0
    packed = np.packbits(bits.reshape(dense.shape[:-1] + (words, 32)), axis=-1, bitorder="little")
    return np.ascontiguousarray(packed).view("<u4").reshape(dense.shape[:-1] + (words,))


def unpack_bits(packed: np.ndarray, n: int) -> np.ndarray:
    """Inverse of pack_bits: uint32 words -> uint8 [..., n]."""
    b = np.unpackbits(np.ascontiguousarray(packed).view(np.uint8), axis=-1, bitorder="little")
    return b[..., :n]


def make_weights(w: Workload, rng: np.random.Generator):
    W_ff: List[np.ndarray] = []
    W_rec: List[np.ndarray] = []
    for l in range(w.L):
        n_pre, n = w.sizes[l], w.sizes[l + 1]
        W_ff.append((rng.standard_normal((n_pre, n), dtype=np.float32)
                     * np.float32(w.g_ff[l] / np.sqrt(n_pre))).astype(np.float32))
        W_rec.append((rng.standard_normal((n, n), dtype=np.float32)
                      * np.float32(w.g_rec[l] / np.sqrt(n))).astype(np.float32))
    n_l, n_out = w.sizes[w.L], w.sizes[w.L + 1]
    W_out = (rng.standard_normal((n_l, n_out), dtype=np.float32) * np.float32(1.0 / np.sqrt(n_l)))
    return W_ff, W_rec, W_out.astype(np.float32)


def make(w: Workload, dense_input: bool = True):
    """Draw the workload.  Returns a dict with
       W_ff, W_rec (lists), W_out, targets [B] int32,
       input_bits uint32 [T][B][ceil(N_0/32)]  (spiking workloads),
       input_dense float32 [T][B][N_0]         (if dense_input, or always for the graded one)."""
    rng = np.random.Generator(np.random.PCG64(w.seed))
    W_ff, W_rec, W_out = make_weights(w, rng)
    n0 = w.sizes[0]
    out = dict(W_ff=W_ff, W_rec=W_rec, W_out=W_out)
    # drawn in slabs of time steps so that long sequences do not need a huge temporary
    slab = max(1, (1 << 24) // (w.B * n0))
    dense = np.empty((w.T, w.B, n0), np.float32) if (dense_input or w.cell == CELL_GRADED) else None
    bits = np.empty((w.T, w.B, (n0 + 31) // 32), np.uint32)
    for t0 in range(0, w.T, slab):
        t1 = min(w.T, t0 + slab)
        mask = rng.random((t1 - t0, w.B, n0), dtype=np.float32) < np.float32(w.p_in)
        if w.cell == CELL_GRADED:
            vals = rng.standard_normal((t1 - t0, w.B, n0), dtype=np.float32)
            dense[t0:t1] = np.where(mask, vals, np.float32(0))
            bits[t0:t1] = pack_bits(dense[t0:t1])
        else:
            if dense is not None:
                dense[t0:t1] = mask
            bits[t0:t1] = pack_bits(mask)
    out["input_bits"] = bits
    if dense is not None:
        out["input_dense"] = dense
    out["targets"] = rng.integers(0, w.sizes[-1], size=w.B).astype(np.int32)
    return out


def small(name: str = "tiny", sizes=(20, 24, 12, 5), T=13, B=3, p_in=0.2, seed=7, **kw) -> Workload:
    """A small workload for tests; gains default to values that give lively activity."""
    L = len(sizes) - 2
    kw.setdefault("g_ff", (2.0,) * L)
    kw.setdefault("g_rec", (1.0,) * L)
    kw.setdefault("strategy", STANDARD)
    kw.setdefault("readout_scale", 1.0 / T)
    return Workload(name, tuple(sizes), T=T, B=B, p_in=p_in, seed=seed, **kw)
