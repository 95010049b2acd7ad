"""Checkpointed BPTT executed with the oracle's single-step functions (test infrastructure).

Each routine walks the execution trace the paper draws in Fig. 1 for one strategy
(forward, re-forward_1, re-forward_2, backward) and counts what the paper's cost
models count: dense states held in local memory (Eqs. 2, 4, 6, 11) and transfers
to and from remote memory (Eqs. 7, 13).  As in the paper's Discussion, the sparse
activations of the whole sequence stay available; only the dense membrane states
are dropped and recomputed.

Strategy names are the caption names of Fig. 1: STANDARD keeps every state
("Base Implementation"), CHUNK is the section "Standard Checkpointing", REMOTE and
DOUBLE as in the sections of those names.  Sequence lengths that are not a
multiple of the interval end with a short segment.
"""
from __future__ import annotations

import numpy as np

from .oracle import NetSpec, Oracle

STANDARD, CHUNK, REMOTE, DOUBLE, HIERARCHICAL = 0, 1, 2, 3, 4


class _Tier:
    """A keyed store that counts entries held, its high-water mark, reads and writes."""

    def __init__(self):
        self.data, self.peak, self.reads, self.writes = {}, 0, 0, 0

    def put(self, key, value):
        self.data[key] = [v.copy() for v in value]
        self.writes += 1
        self.peak = max(self.peak, len(self.data))

    def get(self, key):
        self.reads += 1
        return [v.copy() for v in self.data[key]]

    def drop(self, key):
        self.data.pop(key, None)


class _Run:
    def __init__(self, orc: Oracle, spec: NetSpec, inp, targets, W_ff, W_rec, W_out):
        self.orc, self.spec = orc, spec
        self.inp = np.ascontiguousarray(inp, orc.real)
        self.targets, self.W_ff, self.W_rec, self.W_out = targets, W_ff, W_rec, W_out
        self.T, self.B, _ = self.inp.shape
        L, sizes = spec.L, spec.sizes
        # activations of every step stay stored (index 0 = initial zeros)
        self.S = [np.zeros((self.T + 1, self.B, sizes[l + 1]), orc.real) for l in range(L)]
        self.fwd_steps = 0
        self.refwd_steps = [0, 0]
        self.bwd_steps = np.zeros(self.T + 1, np.int64)
        self.dW_ff = [np.zeros((sizes[l], sizes[l + 1])) for l in range(L)]
        self.dW_rec = [np.zeros((sizes[l + 1], sizes[l + 1])) for l in range(L)]
        self.delta_next = [np.zeros((self.B, sizes[l + 1])) for l in range(L)]
        self.trace = []      # (pass name, first state index, last state index), in execution order
        self.ckpts = []      # (tier name, state index) of every checkpoint written in the forward

    def zero_state(self):
        return [np.zeros((self.B, self.spec.sizes[l + 1]), self.orc.real) for l in range(self.spec.L)]

    def step(self, V_prev, t, generate_spikes):
        """V_{t-1} -> V_t for all layers.  With generate_spikes the new activations are stored;
        without, the stored ones are used and nothing is generated (re-forward)."""
        V = []
        for l in range(self.spec.L):
            below = self.inp[t - 1] if l == 0 else self.S[l - 1][t]
            v, s = self.orc.forward_step(self.spec, below, self.S[l][t - 1], V_prev[l], self.W_ff[l],
                                         self.W_rec[l])
            if generate_spikes:
                self.S[l][t] = s
            V.append(v)
        return V

    def readout(self):
        c = np.zeros((self.B, self.spec.sizes[self.spec.L]), self.orc.real)
        for t in range(1, self.T + 1):          # same order of additions as the full-storage oracle
            c = c + self.S[-1][t]
        self.loss, self.logits, _, self.g_out, self.dW_out = self.orc.readout(self.spec, c, self.targets,
                                                                              self.W_out)

    def backward(self, V_t, t):
        L = self.spec.L
        self.bwd_steps[t] += 1
        new = [None] * L
        for l in range(L - 1, -1, -1):
            below = self.inp[t - 1] if l == 0 else self.S[l - 1][t]
            new[l] = self.orc.backward_step(
                self.spec, V_t[l], below, self.S[l][t - 1], self.delta_next[l],
                new[l + 1] if l < L - 1 else None, self.g_out if l == L - 1 else None,
                self.W_ff[l + 1] if l < L - 1 else None, self.W_rec[l], self.dW_ff[l], self.dW_rec[l])
        self.delta_next = new

    def result(self, local: _Tier, remote: _Tier, chunk_peak: int):
        return dict(loss=self.loss, logits=self.logits, dW_ff=self.dW_ff, dW_rec=self.dW_rec,
                    dW_out=self.dW_out, S=self.S, trace=self.trace, ckpts=self.ckpts,
                    stats=dict(local_states_peak=local.peak + chunk_peak, remote_states_peak=remote.peak,
                               transfers=remote.reads + remote.writes, fwd_steps=self.fwd_steps,
                               refwd1_steps=self.refwd_steps[0], refwd2_steps=self.refwd_steps[1],
                               bwd_steps=self.bwd_steps))


def bptt_checkpointed(orc: Oracle, spec: NetSpec, inp, targets, W_ff, W_rec, W_out, strategy: int,
                      chunk_size: int = 0, remote_chunk_size: int = 0, nb_local: int = 0):
    run = _Run(orc, spec, inp, targets, W_ff, W_rec, W_out)
    T = run.T
    local, remote = _Tier(), _Tier()
    K, R = chunk_size, remote_chunk_size

    if strategy == STANDARD:
        # Fig. 1 "Plain BPTT": every state kept, one forward, one backward (Eq. 2).
        V = run.zero_state()
        for t in range(1, T + 1):
            V = run.step(V, t, True); run.fwd_steps += 1
            local.put(t, V)
        run.trace.append(("forward", 0, T))
        run.readout()
        for t in range(T, 0, -1):
            run.backward(local.get(t), t)
        run.trace.append(("backward", T, 0))
        return run.result(local, remote, 0)

    assert K >= 1
    if strategy == HIERARCHICAL:
        return _hierarchical(run, local, remote, K, nb_local)
    if strategy == DOUBLE:
        assert R >= K and R % K == 0
    # ---- forward pass: keep checkpoints only ------------------------------------------------
    V = run.zero_state()
    interval = R if strategy == DOUBLE else K
    tier = local if strategy == CHUNK else remote
    tier_name = "local" if strategy == CHUNK else "remote"
    tier.put(0, V); run.ckpts.append((tier_name, 0))
    for t in range(1, T + 1):
        V = run.step(V, t, True); run.fwd_steps += 1
        if t % interval == 0 and t < T:
            tier.put(t, V); run.ckpts.append((tier_name, t))
    run.trace.append(("forward", 0, T))
    run.readout()

    def chunk_backward(t0, t1, V0):
        """Re-forward t0+1..t1 into the chunk buffer, then back-propagate t1..t0+1."""
        buf, Vt = {}, V0
        for t in range(t0 + 1, t1 + 1):
            Vt = run.step(Vt, t, False); run.refwd_steps[1 if strategy == DOUBLE else 0] += 1
            buf[t] = Vt
        run.trace.append(("reforward2" if strategy == DOUBLE else "reforward1", t0, t1))
        for t in range(t1, t0, -1):
            run.backward(buf[t], t)
        run.trace.append(("backward", t1, t0))
        return len(buf)

    chunk_peak = 0
    if strategy in (CHUNK, REMOTE):
        # Fig. 1 "Standard Checkpointing" / "Remote Checkpointing": one recomputation pass.
        for t0 in range(((T - 1) // K) * K, -1, -K):
            if strategy == REMOTE:
                local.put("loaded", remote.get(t0))      # "Load": the one local copy of Eq. 6
                V0 = local.get("loaded")
            else:
                V0 = local.get(t0)
            chunk_peak = max(chunk_peak, chunk_backward(t0, min(T, t0 + K), V0))
    else:
        # Fig. 1 "Double Checkpointing": load one remote checkpoint, recompute the local
        # checkpoints of its segment (re-forward_1), then chunk by chunk (re-forward_2).
        for r0 in range(((T - 1) // R) * R, -1, -R):
            r1 = min(T, r0 + R)
            Vt = remote.get(r0)
            local.put(r0, Vt)
            last_fine = r0 + ((r1 - 1 - r0) // K) * K
            for t in range(r0 + 1, last_fine + 1):
                Vt = run.step(Vt, t, False); run.refwd_steps[0] += 1
                if (t - r0) % K == 0:
                    local.put(t, Vt); run.ckpts.append(("local", t))
            if last_fine > r0:
                run.trace.append(("reforward1", r0, last_fine))
            for t0 in range(last_fine, r0 - 1, -K):
                chunk_peak = max(chunk_peak, chunk_backward(t0, min(r1, t0 + K), local.get(t0)))
                local.drop(t0)
    return run.result(local, remote, chunk_peak)


def _hierarchical(run: _Run, local: _Tier, remote: _Tier, K: int, P: int):
    """Section "Hierarchical Checkpointing": checkpoints every K steps live in remote memory and are
    moved nb_local = P at a time, one communication per batch; the last batch of checkpoints is
    stored locally and never moved.  Local memory: chunk_size + nb_local states (Eq. 9).  The paper's
    Eq. 10 counts the communications as 2 (nb_checkpoints / nb_local - nb_local); the text explains
    the subtracted term as the last batch that stays local, so it is read here as
    2 (number of batches - 1), each communication moving one batch."""
    assert P >= 1
    T = run.T
    n_ck = -(-T // K)
    n_b = -(-n_ck // P)
    comms = 0
    V = run.zero_state()
    batch = {}

    def add_checkpoint(t, v):
        nonlocal batch, comms
        j = (t // K) // P
        batch[t] = v
        run.ckpts.append(("remote" if j < n_b - 1 else "local", t))
        if len(batch) == P and j < n_b - 1:   # a complete batch that is not the last one leaves at once
            for tt, vv in batch.items():
                remote.put(tt, vv)
            comms += 1
            batch = {}

    add_checkpoint(0, V)
    for t in range(1, T + 1):
        V = run.step(V, t, True); run.fwd_steps += 1
        if t % K == 0 and t < T:
            add_checkpoint(t, V)
    run.trace.append(("forward", 0, T))
    run.readout()
    chunk_peak, local_peak = 0, len(batch)
    for j in range(n_b - 1, -1, -1):
        if j < n_b - 1:
            batch = {c * K: remote.get(c * K) for c in range(j * P, (j + 1) * P)}
            comms += 1
        local_peak = max(local_peak, len(batch))
        for c in range(min(n_ck, (j + 1) * P) - 1, j * P - 1, -1):
            t0, t1 = c * K, min(T, c * K + K)
            buf, Vt = {}, batch[t0]
            for t in range(t0 + 1, t1 + 1):
                Vt = run.step(Vt, t, False); run.refwd_steps[0] += 1
                buf[t] = Vt
            run.trace.append(("reforward1", t0, t1))
            for t in range(t1, t0, -1):
                run.backward(buf[t], t)
            run.trace.append(("backward", t1, t0))
            chunk_peak = max(chunk_peak, len(buf))
    res = run.result(local, remote, chunk_peak)
    res["stats"]["local_states_peak"] = local_peak + chunk_peak
    res["stats"]["transfers"] = comms
    return res
