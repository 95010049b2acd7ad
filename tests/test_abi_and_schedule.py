"""Host-side checks that need no GPU: the C-ABI library loads and exports what include/snn.h
declares, argument validation, and the schedule generator (run through the oracle's step
functions, it must reproduce full-storage BPTT bit for bit with the slot counts and transfer
counts of the paper's cost models)."""
import ctypes as C
import math
import os
import re

import numpy as np
import pytest

import snn_workloads as wl
from oracle.oracle import NetSpec, leak_from_tau
from paper_2412_11810_b200 import binding as sb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "snn.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(snn_[a-z_]+)\s*\(", header))
    assert declared == set(sb.EXPORTS)
    for name in declared:
        assert getattr(sb.lib, name) is not None


def test_binding_constants_match_the_header():
    """Flags and enumerators are spelled twice (include/snn.h and binding.py): same names, same values."""
    header = open(os.path.join(ROOT, "include", "snn.h")).read()
    flags = dict(re.findall(r"#define\s+(SNN_FLAG_[A-Z_]+)\s+(\d+)u", header))
    assert len(flags) >= 9
    for name, value in flags.items():
        assert getattr(sb, name) == int(value), name
    for name, value in re.findall(r"\b(SNN_(?:ERR_[A-Z_]+|OK|STANDARD|CHUNK|REMOTE|DOUBLE|HIERARCHICAL|DOUBLE_LOCAL|CELL_[A-Z]+|SURR_[A-Z_]+))\s*=\s*(\d+)", header):
        assert getattr(sb, name) == int(value), name
    m = re.search(r"#define\s+SNN_STATIC_WORKSPACE_BYTES\s+\((\d+)u\s*<<\s*(\d+)\)", header)
    assert m and sb.SNN_STATIC_WORKSPACE_BYTES == int(m.group(1)) << int(m.group(2))


def test_create_validates():
    net = sb.snn_create([8, 16, 4], 20.0, 1.0)
    assert abs(sb.snn_alpha(net) - float(leak_from_tau(20.0))) == 0.0
    sb.snn_destroy(net)
    for sizes, tau in (([8, 15, 4], 20.0), ([8, 16], 20.0), ([8, 0, 4], 20.0), ([8, 16, 4], 0.0),
                       ([8] + [16] * 9 + [4], 20.0)):
        with pytest.raises(sb.SnnError):
            sb.snn_create(sizes, tau, 1.0)


def test_workspace_query_and_bad_intervals():
    net = sb.snn_create([8, 16, 4], 20.0, 1.0)
    d0, p0 = sb.snn_workspace_query(net, 100, 2, sb.snn_ckpt(sb.SNN_STANDARD, 0, 0), 0.25)
    d1, p1 = sb.snn_workspace_query(net, 100, 2, sb.snn_ckpt(sb.SNN_CHUNK, 10, 0), 0.25)
    d2, p2 = sb.snn_workspace_query(net, 100, 2, sb.snn_ckpt(sb.SNN_REMOTE, 10, 0), 0.25)
    ms = 4 * 2 * 16
    assert p0 == 0 and p1 == 0 and p2 == 10 * ms
    # same event storage, different number of dense states: T+1, K + T/K, K + 2 (256-byte rounding aside);
    # the strategies that recompute also hold two words per (32 presynaptic rows, step of a chunk, sample),
    # the pairs rounded up to 64: here 2 blocks of rows
    scratch = 2 * 4 * 64 * 2
    assert abs((d0 - (d1 - scratch)) - ms * (101 - 20)) < 512 and abs((d1 - d2) - ms * (20 - 12)) < 512
    d3, p3 = sb.snn_workspace_query(net, 100, 2, sb.snn_ckpt(sb.SNN_DOUBLE, 5, 20), 0.25)
    d4, p4 = sb.snn_workspace_query(net, 100, 2, sb.snn_ckpt(sb.SNN_DOUBLE_LOCAL, 5, 20), 0.25)
    assert p3 == 5 * ms and p4 == 0 and abs((d4 - d3) - 5 * ms) < 512      # the second tier moves on device
    for ck in (sb.snn_ckpt(sb.SNN_CHUNK, 0, 0), sb.snn_ckpt(sb.SNN_DOUBLE, 4, 6), sb.snn_ckpt(sb.SNN_DOUBLE, 8, 4),
               sb.snn_ckpt(sb.SNN_HIERARCHICAL, 4, 0, 0), sb.snn_ckpt(7, 1, 1)):
        with pytest.raises(sb.SnnError):
            sb.snn_workspace_query(net, 100, 2, ck, 0.25)
    with pytest.raises(sb.SnnError):
        sb.snn_workspace_query(net, 0, 2, sb.snn_ckpt(sb.SNN_STANDARD, 0, 0), 0.25)
    sb.snn_destroy(net)


def test_train_step_rejects_bad_arguments_without_a_gpu():
    net = sb.snn_create([8, 16, 4], 20.0, 1.0)
    a = sb.snn_step_args()
    loss = C.c_float()
    assert sb.lib.snn_train_step(net, C.byref(a), C.byref(loss)) == sb.SNN_ERR_INVALID_ARG
    assert sb.lib.snn_train_step(None, C.byref(a), C.byref(loss)) == sb.SNN_ERR_INVALID_ARG
    assert "T and B" in sb.snn_last_error(net)
    sb.snn_destroy(net)


# ------------------------------------------------------------------------------------------
CASES = [(sb.SNN_STANDARD, 0, 0), (sb.SNN_CHUNK, 4, 0), (sb.SNN_CHUNK, 1, 0), (sb.SNN_CHUNK, 13, 0),
         (sb.SNN_CHUNK, 40, 0), (sb.SNN_REMOTE, 4, 0), (sb.SNN_REMOTE, 1, 0), (sb.SNN_REMOTE, 13, 0),
         (sb.SNN_DOUBLE, 2, 6), (sb.SNN_DOUBLE, 3, 3), (sb.SNN_DOUBLE, 1, 4), (sb.SNN_DOUBLE, 2, 26),
         (sb.SNN_DOUBLE, 13, 13), (sb.SNN_DOUBLE_LOCAL, 2, 6), (sb.SNN_DOUBLE_LOCAL, 3, 3),
         (sb.SNN_HIERARCHICAL, 2, 2), (sb.SNN_HIERARCHICAL, 2, 3), (sb.SNN_HIERARCHICAL, 3, 1),
         (sb.SNN_HIERARCHICAL, 1, 4), (sb.SNN_HIERARCHICAL, 4, 9), (sb.SNN_HIERARCHICAL, 13, 2)]
# the third number is remote_chunk_size, except for HIERARCHICAL where it is nb_local


def _ckpt(strategy, K, R):
    return sb.snn_ckpt(strategy, K, 0, R) if strategy == sb.SNN_HIERARCHICAL else sb.snn_ckpt(strategy, K, R, 0)


def _execute_plan(orc, spec, d, T, ops, n_local, n_remote):
    """Run the op list literally over numbered slots with the oracle's step functions."""
    L, sizes = spec.L, spec.sizes
    B = d["input_dense"].shape[1]
    inp = d["input_dense"].astype(orc.real)
    local = [None] * n_local          # slot -> (time index of the state, [V per layer])
    remote = [None] * n_remote
    S = [np.zeros((T + 1, B, sizes[l + 1]), orc.real) for l in range(L)]
    dW_ff = [np.zeros((sizes[l], sizes[l + 1])) for l in range(L)]
    dW_rec = [np.zeros((sizes[l + 1], sizes[l + 1])) for l in range(L)]
    delta_next = [np.zeros((B, sizes[l + 1])) for l in range(L)]
    count = dict(fwd=np.zeros(T + 1, int), re1=np.zeros(T + 1, int), re2=np.zeros(T + 1, int),
                 bwd=np.zeros(T + 1, int), d2h=0, h2d=0)
    readout = None
    for op in ops:
        k = op.kind
        if k == sb.SNN_OP_ZERO:
            local[op.keep_slot] = (0, [np.zeros((B, sizes[l + 1]), orc.real) for l in range(L)])
        elif k == sb.SNN_OP_D2H:
            for i in range(max(1, op.buf_len)):
                remote[op.remote_slot + i] = local[op.in_slot + i]
            count["d2h"] += 1
        elif k == sb.SNN_OP_H2D:
            for i in range(max(1, op.buf_len)):
                local[op.keep_slot + i] = remote[op.remote_slot + i]
            count["h2d"] += 1
        elif k in (sb.SNN_OP_FWD, sb.SNN_OP_REFWD1, sb.SNN_OP_REFWD2):
            tcur, V = local[op.in_slot]
            assert tcur == op.t0, "the input slot must hold the state of step t0"
            for t in range(op.t0 + 1, op.t1 + 1):
                Vn = []
                for l in range(L):
                    below = inp[t - 1] if l == 0 else S[l - 1][t]
                    v, s = orc.forward_step(spec, below, S[l][t - 1], V[l], d["W_ff"][l], d["W_rec"][l])
                    if k == sb.SNN_OP_FWD:
                        S[l][t] = s
                    Vn.append(v)
                V = Vn
                count["fwd" if k == sb.SNN_OP_FWD else "re1" if k == sb.SNN_OP_REFWD1 else "re2"][t] += 1
                local[op.buf_slot + (t - op.t0 - 1) % op.buf_len] = (t, V)
                if op.keep_every > 0 and (t - op.t0) % op.keep_every == 0:
                    local[op.keep_slot + (t - op.t0) // op.keep_every - 1] = (t, V)
            if k == sb.SNN_OP_FWD and op.t1 == T:
                c = np.zeros((B, sizes[L]), orc.real)
                for t in range(1, T + 1):
                    c = c + S[-1][t]
                readout = orc.readout(spec, c, d["targets"], d["W_out"])
        elif k == sb.SNN_OP_BWD:
            loss, _, _, g_out, dW_out = readout
            for t in range(op.t1, op.t0, -1):
                tcur, V = local[op.buf_slot + (t - op.t0 - 1)]
                assert tcur == t, "the chunk buffer must hold the state of the step being back-propagated"
                count["bwd"][t] += 1
                new = [None] * L
                for l in range(L - 1, -1, -1):
                    below = inp[t - 1] if l == 0 else S[l - 1][t]
                    new[l] = orc.backward_step(spec, V[l], below, S[l][t - 1], delta_next[l],
                                               new[l + 1] if l < L - 1 else None, g_out if l == L - 1 else None,
                                               d["W_ff"][l + 1] if l < L - 1 else None, d["W_rec"][l],
                                               dW_ff[l], dW_rec[l])
                delta_next = new
    return dict(loss=readout[0], dW_ff=dW_ff, dW_rec=dW_rec, dW_out=readout[4], count=count)


@pytest.mark.parametrize("strategy,K,R", CASES)
def test_plan_reproduces_full_storage_bptt(orc32, strategy, K, R):
    w = wl.small()
    d = wl.make(w)
    T = w.T
    spec = NetSpec(w.sizes, leak_from_tau(w.tau_mem), w.theta, w.beta, w.scale())
    full = orc32.bptt_full(spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"])
    ops, n_local, n_remote = sb.snn_plan(T, _ckpt(strategy, K, R))
    r = _execute_plan(orc32, spec, d, T, ops, n_local, n_remote)
    assert r["loss"] == full["loss"]
    for a, b in zip(r["dW_ff"] + r["dW_rec"] + [r["dW_out"]], full["dW_ff"] + full["dW_rec"] + [full["dW_out"]]):
        assert np.array_equal(a, b)
    c = r["count"]
    # Fig. 1: one forward and one backward pass over every step; one recomputation pass for
    # CHUNK / REMOTE, two for DOUBLE (the first stops at the last local checkpoint of a segment)
    assert np.all(c["fwd"][1:] == 1) and np.all(c["bwd"][1:] == 1)
    Kc = min(K, T) if K else 0
    if strategy == sb.SNN_STANDARD:
        assert n_local == T + 1 and n_remote == 0 and c["re1"].sum() == 0 and c["re2"].sum() == 0   # Eq. 2
    elif strategy == sb.SNN_CHUNK:
        assert n_local == Kc + math.ceil(T / K) and n_remote == 0                                   # Eq. 4
        assert np.all(c["re1"][1:] == 1) and c["re2"].sum() == 0
    elif strategy == sb.SNN_REMOTE:
        assert n_local == Kc + 2 and n_remote == math.ceil(T / K)                                   # Eq. 6 (+1 staging)
        assert c["d2h"] + c["h2d"] == 2 * math.ceil(T / K)                                          # Eq. 7
        assert np.all(c["re1"][1:] == 1)
    elif strategy == sb.SNN_HIERARCHICAL:
        n_ck = math.ceil(T / K)
        P = min(R, n_ck)
        n_b = math.ceil(n_ck / P)
        assert n_local == Kc + P                                                                    # Eq. 9
        assert n_remote == (n_b - 1) * P and c["d2h"] == c["h2d"] == n_b - 1                        # Eq. 10 as read
        assert np.all(c["re1"][1:] == 1) and c["re2"].sum() == 0
    else:
        assert n_local == Kc + math.ceil(min(R, T) / K) + 1 <= K + R // K + 1                       # Eq. 11 (+1 staging)
        assert n_remote == math.ceil(T / R) and c["d2h"] + c["h2d"] == 2 * math.ceil(T / R)         # Eq. 13
        assert np.all(c["re2"][1:] == 1) and np.all(c["re1"][1:] <= 1)


def test_plan_matches_the_traces_of_the_figure():
    """T = 11, chunk_size = 3, remote_chunk_size = 6 as drawn in Fig. 1 (tests/golden/fig1_traces.txt)."""
    rows = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "fig1_traces.txt")):
        if not line.startswith("#") and line.strip():
            row, item, *vals = line.split()
            rows.setdefault(row, {})[item] = [v for v in vals]
    pairs = lambda v: [(int(a), int(b)) for a, b in zip(v[0::2], v[1::2])]
    for row, strat, K, R in (("chunk", sb.SNN_CHUNK, 3, 0), ("remote", sb.SNN_REMOTE, 3, 0),
                             ("double", sb.SNN_DOUBLE, 3, 6)):
        ops, _, _ = sb.snn_plan(11, sb.snn_ckpt(strat, K, R))
        re1 = [(o.t0, o.t1) for o in ops if o.kind == sb.SNN_OP_REFWD1]
        re2 = [(o.t0, o.t1) for o in ops if o.kind == sb.SNN_OP_REFWD2]
        if row == "double":
            assert re1 == pairs(rows[row]["reforward1"])
            drawn, ours = pairs(rows[row]["reforward2"]), re2
            kept = sorted(o.t0 + o.keep_every * (i + 1) for o in ops if o.kind == sb.SNN_OP_FWD and o.keep_every
                          for i in range((o.t1 - o.t0) // o.keep_every))
            assert [0] + kept == [int(x) for x in rows[row]["ckpt_remote"]]
        else:
            drawn, ours = pairs(rows[row]["reforward1"]), re1
            assert not re2
        assert len(drawn) == len(ours)
        for (a, b), (oa, ob) in zip(drawn, ours):
            assert a == oa and b <= ob <= b + 1


def test_long_sequence_plans_stay_small_and_valid():
    for T, ck in ((10000, sb.snn_ckpt(sb.SNN_REMOTE, 64, 0)), (2000, sb.snn_ckpt(sb.SNN_DOUBLE, 16, 256)),
                  (1000, sb.snn_ckpt(sb.SNN_CHUNK, 32, 0)), (200000, sb.snn_ckpt(sb.SNN_DOUBLE, 32, 1024))):
        ops, n_local, n_remote = sb.snn_plan(T, ck)
        covered = np.zeros(T + 1, int)
        for o in ops:
            if o.kind == sb.SNN_OP_BWD:
                covered[o.t0 + 1:o.t1 + 1] += 1
                assert o.t1 - o.t0 <= o.buf_len
            if o.kind in (sb.SNN_OP_FWD, sb.SNN_OP_REFWD1, sb.SNN_OP_REFWD2):
                assert 0 <= o.in_slot < n_local and o.buf_slot + o.buf_len <= n_local
        assert np.all(covered[1:] == 1)
        if ck.strategy == sb.SNN_DOUBLE:
            assert n_local == ck.chunk_size + ck.remote_chunk_size // ck.chunk_size + 1


def test_suggested_intervals_follow_the_papers_rules():
    """Hyperparameter Study: chunk_size = sqrt(T) (64 at T = 4096); Double: remote_chunk_size within
    64 .. 256 at T = 4096 and chunk_size = sqrt(remote_chunk_size); Remote: the largest chunk that fits."""
    c = sb.snn_suggest_ckpt(None, 4096, 1, sb.SNN_CHUNK)
    assert (c.strategy, c.chunk_size) == (sb.SNN_CHUNK, 64)
    c = sb.snn_suggest_ckpt(None, 4096, 1, sb.SNN_DOUBLE)
    assert 64 <= c.remote_chunk_size <= 256 and c.chunk_size ** 2 == c.remote_chunk_size
    for T in (7, 100, 1000, 5000):
        c = sb.snn_suggest_ckpt(None, T, 1, sb.SNN_DOUBLE)
        assert c.remote_chunk_size % c.chunk_size == 0 and c.chunk_size >= 1
        sb.snn_plan(T, c)
        h = sb.snn_suggest_ckpt(None, T, 1, sb.SNN_HIERARCHICAL)
        assert h.chunk_size >= 1 and h.nb_local >= 1
        sb.snn_plan(T, h)
    net = sb.snn_create([8, 16, 4], 20.0, 1.0)
    budget, _ = sb.snn_workspace_query(net, 1000, 2, sb.snn_ckpt(sb.SNN_REMOTE, 37, 0), 0.25)
    c = sb.snn_suggest_ckpt(net, 1000, 2, sb.SNN_REMOTE, budget, 0.25)
    fits = lambda K: sb.snn_workspace_query(net, 1000, 2, sb.snn_ckpt(sb.SNN_REMOTE, K, 0), 0.25)[0] <= budget
    assert c.chunk_size >= 37 and fits(c.chunk_size) and not fits(c.chunk_size + 1)
    with pytest.raises(sb.SnnError):
        sb.snn_suggest_ckpt(net, 1000, 2, sb.SNN_REMOTE, 1024, 0.25)
    sb.snn_destroy(net)
