"""Pins of the CPU oracle against facts that do not come from the oracle itself:
closed forms, library routines (matmul, autograd, cross-entropy), finite differences,
brute force in pure Python, and the traces and cost models the paper prints."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import snn_workloads as wl
from oracle import checkpointing as ck
from oracle.oracle import (CELL_GRADED, CELL_LIF, SURR_FAST_SIGMOID, SURR_SIGMOID, SURR_TRIANGLE, NetSpec, Oracle,
                           leak_from_tau)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def spec_of(w, **kw):
    a = dict(sizes=w.sizes, alpha=leak_from_tau(w.tau_mem), theta=w.theta, beta=w.beta, scale=w.scale(),
             cell=w.cell)
    a.update(kw)
    return NetSpec(**a)


# ---------------------------------------------------------------- leak + integration (closed form)
@pytest.mark.parametrize("kind,tol", [("f64", 1e-13), ("f32", 2e-6)])
def test_constant_input_trace_closed_form(kind, tol):
    """One always-on input of weight w, no recurrence, unreachable threshold:
    V_t = w (1 - alpha^t) / (1 - alpha)  (geometric series of the leaky integrator)."""
    o = Oracle(kind)
    T, w0 = 60, 0.37
    alpha = float(leak_from_tau(20.0)) if kind == "f32" else math.exp(-1 / 20.0)
    spec = NetSpec((1, 1, 2), alpha, theta=1e30)
    inp = np.ones((T, 1, 1))
    r = o.bptt_full(spec, inp, [0], [np.array([[w0]])], [np.zeros((1, 1))], np.zeros((1, 2)),
                    do_backward=False)
    t = np.arange(T + 1)
    wq = float(o.real(w0))
    expect = wq * (1 - alpha ** t) / (1 - alpha)
    assert np.allclose(r["V"][0][:, 0, 0], expect, rtol=tol, atol=0)
    assert r["S"][0].sum() == 0


def test_first_spike_time_and_subtractive_reset(orc64):
    """With threshold theta and w > theta (1 - alpha): the first spike comes at
    t* = ceil(ln(1 - theta (1 - alpha) / w) / ln alpha), and the step after it
    V = alpha V_{t*} + w - theta (reset by subtraction, applied one step later)."""
    alpha, theta, w0, T = math.exp(-1 / 20.0), 1.0, 0.11, 80
    spec = NetSpec((1, 1, 2), alpha, theta=theta)
    r = orc64.bptt_full(spec, np.ones((T, 1, 1)), [0], [np.array([[w0]])], [np.zeros((1, 1))],
                        np.zeros((1, 2)), do_backward=False)
    V, S = r["V"][0][:, 0, 0], r["S"][0][:, 0, 0]
    tstar = math.ceil(math.log(1 - theta * (1 - alpha) / w0) / math.log(alpha))
    assert np.flatnonzero(S)[0] == tstar
    assert V[tstar] > theta and V[tstar - 1] <= theta
    assert abs(V[tstar + 1] - (alpha * V[tstar] + w0 - theta)) < 1e-14


# ---------------------------------------------------------------- compaction (brute force vs library)
@pytest.mark.parametrize("n", [1, 31, 32, 33, 100, 127, 128, 1000])
def test_compaction_matches_flatnonzero(orc32, n):
    rng = np.random.default_rng(n)
    for v in (rng.standard_normal(n).astype(np.float32), np.zeros(n, np.float32),
              np.full(n, 2.0, np.float32), np.full(n, 0.5, np.float32)):
        idx = orc32.compact(v, 0.5)
        assert np.array_equal(idx, np.flatnonzero(v > np.float32(0.5)))
        assert np.all(np.diff(idx) > 0)


# ---------------------------------------------------------------- readout / loss special cases
def test_all_neurons_spike_reduces_to_softmax_regression(orc64):
    """T = 1, one layer, threshold far below zero: every hidden neuron fires once, so the
    readout sees the constant vector of ones and the step is plain soft-max regression."""
    rng = np.random.default_rng(0)
    B, N0, N1, NO = 3, 4, 6, 5
    spec = NetSpec((N0, N1, NO), 0.9, theta=-1e30, scale=0.7)
    W_out = rng.standard_normal((N1, NO))
    targets = np.array([1, 4, 0], np.int32)
    r = orc64.bptt_full(spec, np.zeros((1, B, N0)), targets, [rng.standard_normal((N0, N1))],
                        [rng.standard_normal((N1, N1))], W_out)
    Wt = torch.tensor(W_out, requires_grad=True)
    logits = 0.7 * torch.ones(B, N1, dtype=torch.float64) @ Wt
    loss = torch.nn.functional.cross_entropy(logits, torch.tensor(targets, dtype=torch.long))
    loss.backward()
    assert abs(r["loss"] - loss.item()) < 1e-12
    assert np.allclose(r["logits"], logits.detach().numpy(), atol=1e-12)
    assert np.allclose(r["dW_out"], Wt.grad.numpy(), atol=1e-12)


def test_silent_network_gives_log_nout_and_zero_hidden_gradients(orc32):
    w = wl.small()
    d = wl.make(w)
    spec = spec_of(w, theta=1e30)
    r = orc32.bptt_full(spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"])
    assert r["counts"].sum() == 0
    assert abs(r["loss"] - math.log(w.sizes[-1])) < 1e-12
    assert np.all(r["logits"] == 0)
    # with nothing spiking the recurrent rows and the deeper feed-forward rows see no event
    assert all(np.all(g == 0) for g in r["dW_rec"]) and np.all(r["dW_ff"][1] == 0)


# ---------------------------------------------------------------- backward: autograd and finite differences
def _torch_bptt(spec, inp, targets, W_ff, W_rec, W_out, spike_fn):
    """The same network written with torch tensor ops; gradients come from autograd."""
    T, B, _ = inp.shape
    Ws_ff = [torch.tensor(np.asarray(w, np.float64), requires_grad=True) for w in W_ff]
    Ws_rec = [torch.tensor(np.asarray(w, np.float64), requires_grad=True) for w in W_rec]
    Wo = torch.tensor(np.asarray(W_out, np.float64), requires_grad=True)
    x = torch.tensor(np.asarray(inp, np.float64))
    V = [torch.zeros(B, n, dtype=torch.float64) for n in spec.sizes[1:-1]]
    S = [torch.zeros(B, n, dtype=torch.float64) for n in spec.sizes[1:-1]]
    c = torch.zeros(B, spec.sizes[-2], dtype=torch.float64)
    for t in range(T):
        below = x[t]
        for l in range(spec.L):
            I = below @ Ws_ff[l] + S[l] @ Ws_rec[l]
            V[l] = spec.alpha * V[l] + I - (spec.theta * S[l] if spec.cell == CELL_LIF else 0.0)
            S[l] = spike_fn(V[l])
            below = S[l]
        c = c + S[-1]
    logits = spec.scale * c @ Wo
    loss = torch.nn.functional.cross_entropy(logits, torch.tensor(np.asarray(targets), dtype=torch.long))
    loss.backward()
    return loss.item(), [w.grad.numpy() for w in Ws_ff], [w.grad.numpy() for w in Ws_rec], Wo.grad.numpy()


class _SurrogateSpike(torch.autograd.Function):
    """Heaviside forward; backward multiplies by the derivative of the named smooth function."""

    @staticmethod
    def forward(ctx, v, theta, beta, kind):
        ctx.save_for_backward(v)
        ctx.theta, ctx.beta, ctx.kind = theta, beta, kind
        return (v > theta).to(v.dtype)

    @staticmethod
    def backward(ctx, g):
        (v,) = ctx.saved_tensors
        x = (v - ctx.theta).detach().requires_grad_(True)
        with torch.enable_grad():
            # fast sigmoid x / (1 + beta |x|) (SuperSpike), logistic sigmoid(beta x), or the piecewise
            # quadratic whose derivative is the triangle beta max(0, 1 - beta |x|)
            if ctx.kind == SURR_FAST_SIGMOID:
                f = x / (1 + ctx.beta * x.abs())
            elif ctx.kind == SURR_SIGMOID:
                f = torch.sigmoid(ctx.beta * x)
            else:
                u = (ctx.beta * x).clamp(-1.0, 1.0)
                f = u - 0.5 * u * u.abs()
            (d,) = torch.autograd.grad(f.sum(), x)
        return g * d, None, None, None


def _tiny(seed, sizes=(5, 7, 6, 3), T=6, B=2, **kw):
    w = wl.small(sizes=sizes, T=T, B=B, seed=seed, p_in=0.4, **kw)
    return w, wl.make(w)


@pytest.mark.parametrize("surr", [SURR_FAST_SIGMOID, SURR_SIGMOID, SURR_TRIANGLE])
def test_backward_matches_autograd_with_surrogate(orc64, surr):
    """Heaviside spikes, surrogate derivative in the backward: torch autograd with a custom
    spike function (derivative obtained by differentiating the smooth function itself)."""
    w, d = _tiny(3)
    # the triangle has support |V - theta| < 1 / beta: a wide one here, so that the tiny case has neurons inside it
    spec = spec_of(w, alpha=math.exp(-1 / 20.0), surrogate=surr, beta=1.0 if surr == SURR_TRIANGLE else 4.0)
    r = orc64.bptt_full(spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"])
    assert 0.05 < np.mean([s[1:].mean() for s in r["S"]]) < 0.6       # the case is not degenerate
    fn = lambda v: _SurrogateSpike.apply(v, spec.theta, spec.beta, surr)
    loss, gff, grec, gout = _torch_bptt(spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"],
                                        d["W_out"], fn)
    assert abs(loss - r["loss"]) < 1e-12
    for a, b in zip(r["dW_ff"] + r["dW_rec"] + [r["dW_out"]], gff + grec + [gout]):
        assert np.abs(b).max() > 0
        assert np.allclose(a, b, rtol=1e-9, atol=1e-13)


def test_graded_cell_matches_autograd(orc64):
    """Thresholded-ReLU events a = V [V > theta]; autograd differentiates torch.where."""
    w, d = _tiny(5, cell=CELL_GRADED, g_rec=(0.3, 0.3), theta=0.2)
    spec = spec_of(w, alpha=math.exp(-1 / 20.0))
    r = orc64.bptt_full(spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"])
    frac = np.mean([(s[1:] != 0).mean() for s in r["S"]])
    assert 0.05 < frac < 0.95
    fn = lambda v: torch.where(v > spec.theta, v, torch.zeros_like(v))
    loss, gff, grec, gout = _torch_bptt(spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"],
                                        d["W_out"], fn)
    assert abs(loss - r["loss"]) < 1e-12
    for a, b in zip(r["dW_ff"] + r["dW_rec"] + [r["dW_out"]], gff + grec + [gout]):
        assert np.abs(b).max() > 0
        assert np.allclose(a, b, rtol=1e-9, atol=1e-13)


def test_smooth_mode_finite_differences_every_weight(orc64):
    """Smooth spikes S = sigmoid(beta (V - theta)) in both passes: the backward pass, reset
    path included, is then the exact gradient, checked by central differences on every weight."""
    w, d = _tiny(11, sizes=(3, 4, 3, 2), T=5, B=2)
    spec = spec_of(w, alpha=math.exp(-1 / 20.0), smooth=True, surrogate=SURR_SIGMOID, beta=3.0)
    args = (d["input_dense"], d["targets"])
    Ws = dict(W_ff=[x.astype(np.float64) for x in d["W_ff"]], W_rec=[x.astype(np.float64) for x in d["W_rec"]],
              W_out=d["W_out"].astype(np.float64))
    r = orc64.bptt_full(spec, *args, Ws["W_ff"], Ws["W_rec"], Ws["W_out"])
    loss_of = lambda: orc64.bptt_full(spec, *args, Ws["W_ff"], Ws["W_rec"], Ws["W_out"],
                                      do_backward=False, keep_states=False)["loss"]
    h = 1e-5
    worst = 0.0
    for name, grads in (("W_ff", r["dW_ff"]), ("W_rec", r["dW_rec"]), ("W_out", [r["dW_out"]])):
        mats = Ws[name] if name != "W_out" else [Ws[name]]
        for M, G in zip(mats, grads):
            scale = np.abs(G).max()
            assert scale > 0
            for idx in np.ndindex(M.shape):
                old = M[idx]
                M[idx] = old + h; lp = loss_of()
                M[idx] = old - h; lm = loss_of()
                M[idx] = old
                worst = max(worst, abs((lp - lm) / (2 * h) - G[idx]) / scale)
    assert worst < 1e-6


def test_surrogate_is_derivative_of_fast_sigmoid(orc64):
    """sigma'(x) read off a one-neuron network (dW_ff = g_out sigma'(V - theta), V = w) must be
    the derivative of the fast sigmoid x / (1 + beta |x|); checked by central differences."""
    beta, theta = 10.0, 1.0
    f = lambda x: x / (1 + beta * abs(x))
    for v in (0.2, 0.93, 1.0, 1.04, 1.7, -0.5):
        spec = NetSpec((1, 1, 2), 0.9, theta=theta, beta=beta)
        W_out = np.array([[0.8, -0.3]])
        r = orc64.bptt_full(spec, np.ones((1, 1, 1)), [1], [np.array([[v]])], [np.zeros((1, 1))], W_out)
        c = np.array([[1.0 if v > theta else 0.0]])
        _, _, _, g_out, _ = orc64.readout(spec, c, np.array([1], np.int32), W_out)
        x = v - theta
        h = 1e-6
        fd = (f(x + h) - f(x - h)) / (2 * h) if x != 0 else 1.0
        if g_out[0, 0] != 0:
            assert abs(r["dW_ff"][0][0, 0] / g_out[0, 0] - fd) < 1e-6


def test_triangle_surrogate_closed_form(orc64):
    """The triangular pseudo-derivative read off a one-neuron network: beta at the threshold, half of it
    half-way to the edge of its support, exactly zero from |V - theta| = 1 / beta on."""
    beta, theta = 4.0, 1.0
    for v, want in ((1.0, 4.0), (1.125, 2.0), (0.875, 2.0), (1.25, 0.0), (0.75, 0.0), (1.3, 0.0), (0.2, 0.0), (1.0625, 3.0)):
        spec = NetSpec((1, 1, 2), 0.9, theta=theta, beta=beta, surrogate=SURR_TRIANGLE)
        W_out = np.array([[0.8, -0.3]])
        r = orc64.bptt_full(spec, np.ones((1, 1, 1)), [1], [np.array([[v]])], [np.zeros((1, 1))], W_out)
        c = np.array([[1.0 if v > theta else 0.0]])
        _, _, _, g_out, _ = orc64.readout(spec, c, np.array([1], np.int32), W_out)
        assert g_out[0, 0] != 0
        assert abs(r["dW_ff"][0][0, 0] / g_out[0, 0] - want) < 1e-12, v


# ---------------------------------------------------------------- canonical fp32 order (pure Python)
def test_fp32_forward_order_matches_scalar_python_loops(orc32):
    """Tiny network re-run with numpy float32 scalars in the stated order: feed-forward terms in
    ascending j, then recurrent ones, one accumulator, one fused leak, one subtraction."""
    w = wl.small(sizes=(6, 8, 4), T=7, B=2, seed=2, p_in=0.4)
    d = wl.make(w)
    spec = spec_of(w)
    r = orc32.bptt_full(spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"],
                        do_backward=False)
    f32 = np.float32
    alpha, theta = f32(spec.alpha), f32(spec.theta)
    N = w.sizes[1]
    V = np.zeros((w.B, N), f32); S = np.zeros((w.B, N), f32)
    for t in range(1, w.T + 1):
        Vn = np.zeros_like(V); Sn = np.zeros_like(S)
        for b in range(w.B):
            for i in range(N):
                acc = f32(0)
                for j in range(w.sizes[0]):
                    if d["input_dense"][t - 1, b, j] != 0:
                        acc = f32(acc + d["W_ff"][0][j, i])
                for j in range(N):
                    if S[b, j] != 0:
                        acc = f32(acc + d["W_rec"][0][j, i])
                # fused multiply-add: the product of two fp32 numbers is exact in double
                v = f32(np.float64(alpha) * np.float64(V[b, i]) + np.float64(acc))
                v = f32(v - theta * S[b, i])
                Vn[b, i] = v; Sn[b, i] = f32(1) if v > theta else f32(0)
        V, S = Vn, Sn
        assert np.array_equal(V, r["V"][0][t]) and np.array_equal(S, r["S"][0][t])
    assert r["S"][0].sum() > 0


def test_fp32_graded_forward_order_matches_scalar_python_loops(orc32):
    """The graded cell in the same style: every event contributes one fused multiply-add
    fma(value, w, acc) in list order (feed-forward, then recurrent, ascending j); the leak is one more
    fused multiply-add; there is no reset; the event value is V where V > theta.  The fused multiply-add
    is evaluated exactly in rational arithmetic and rounded once to the nearest fp32 (ties to even)."""
    w = wl.small(sizes=(6, 8, 4), T=9, B=2, seed=5, p_in=0.5, cell=CELL_GRADED, g_ff=(1.5,), g_rec=(0.6,),
                 theta=0.3)
    d = wl.make(w)
    spec = spec_of(w)
    r = orc32.bptt_full(spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"],
                        do_backward=False)
    f32, f64 = np.float32, np.float64
    alpha, theta = f32(spec.alpha), f32(spec.theta)
    N = w.sizes[1]

    def fma(a, b, c):
        exact = Fraction(float(a)) * Fraction(float(b)) + Fraction(float(c))
        near = f32(float(exact))                  # within one ulp of the answer: test it and its neighbours
        cands = [near, np.nextafter(near, f32(np.inf)), np.nextafter(near, f32(-np.inf))]
        dist = [abs(Fraction(float(x)) - exact) for x in cands]
        best = min(dist)
        winners = [x for x, e in zip(cands, dist) if e == best]
        if len(winners) > 1:                      # a tie: the even mantissa wins
            winners = [x for x in winners if (int(np.array(x, f32).view(np.uint32)) & 1) == 0]
        return winners[0]

    V = np.zeros((w.B, N), f32); A = np.zeros((w.B, N), f32)
    n_rec_events = 0
    for t in range(1, w.T + 1):
        Vn = np.zeros_like(V); An = np.zeros_like(A)
        for b in range(w.B):
            for i in range(N):
                acc = f32(0)
                for j in range(w.sizes[0]):
                    x = d["input_dense"][t - 1, b, j]
                    if x != 0:
                        acc = fma(x, d["W_ff"][0][j, i], acc)
                for j in range(N):
                    if A[b, j] != 0:
                        acc = fma(A[b, j], d["W_rec"][0][j, i], acc)
                        n_rec_events += 1
                v = fma(alpha, V[b, i], acc)
                Vn[b, i] = v; An[b, i] = v if v > theta else f32(0)
        V, A = Vn, An
        assert np.array_equal(V, r["V"][0][t]) and np.array_equal(A, r["S"][0][t]), t
    assert n_rec_events > 50 and (r["S"][0] != 0).mean() > 0.05


def test_fp32_and_fp64_forward_agree(orc32, orc64):
    w = wl.small()
    d = wl.make(w)
    r32 = orc32.bptt_full(spec_of(w), d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"])
    r64 = orc64.bptt_full(spec_of(w), d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"])
    for l in range(w.L):
        assert np.array_equal(r32["S"][l], r64["S"][l])
        assert np.abs(r32["V"][l] - r64["V"][l]).max() < 1e-5
    for a, b in zip(r32["dW_ff"] + r32["dW_rec"], r64["dW_ff"] + r64["dW_rec"]):
        assert np.abs(a - b).max() <= 1e-4 * np.abs(b).max()


# ---------------------------------------------------------------- sparsity identities of dW
def test_weight_gradient_sparsity_identities(orc32):
    w = wl.small(p_in=0.05, T=9)
    d = wl.make(w)
    r = orc32.bptt_full(spec_of(w), d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"],
                        keep_delta=True)
    never = d["input_dense"].sum(axis=(0, 1)) == 0
    assert never.any() and np.all(r["dW_ff"][0][never] == 0) and np.abs(r["dW_ff"][0][~never]).max() > 0
    for l in range(w.L):
        S, D = r["S"][l].astype(np.float64), r["delta"][l]
        # column sums of dW_rec = sum_t sum_b (number of own spikes at t-1) * delta_t
        cnt = S[:-1].sum(axis=2)                       # [T][B] spikes at t-1 for t = 1..T
        expect = np.einsum("tb,tbn->n", cnt, D[1:w.T + 1])
        assert np.allclose(r["dW_rec"][l].sum(axis=0), expect, rtol=1e-10, atol=1e-14)
        # and the whole matrix is the sum of outer products (library einsum)
        full = np.einsum("tbj,tbi->ji", S[:-1], D[1:w.T + 1])
        assert np.allclose(r["dW_rec"][l], full, rtol=1e-10, atol=1e-14)


# ---------------------------------------------------------------- checkpointing: exactness, traces, cost models
CASES = [(ck.STANDARD, 0, 0), (ck.CHUNK, 4, 0), (ck.CHUNK, 1, 0), (ck.CHUNK, 13, 0), (ck.CHUNK, 50, 0),
         (ck.REMOTE, 4, 0), (ck.REMOTE, 5, 0), (ck.DOUBLE, 2, 6), (ck.DOUBLE, 3, 3), (ck.DOUBLE, 1, 4),
         (ck.DOUBLE, 2, 26), (ck.HIERARCHICAL, 2, 2), (ck.HIERARCHICAL, 2, 3), (ck.HIERARCHICAL, 3, 1),
         (ck.HIERARCHICAL, 4, 9)]   # third number: remote_chunk_size, or nb_local for HIERARCHICAL


@pytest.mark.parametrize("strategy,K,R", CASES)
def test_every_strategy_equals_full_storage_bit_for_bit(orc32, strategy, K, R):
    """Checkpointing only re-derives dropped states, so the gradient is that of plain BPTT."""
    w = wl.small()
    d = wl.make(w)
    spec = spec_of(w)
    full = orc32.bptt_full(spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"])
    c = ck.bptt_checkpointed(orc32, spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"],
                             strategy, K, 0 if strategy == ck.HIERARCHICAL else R, R)
    assert c["loss"] == full["loss"]
    for a, b in zip(c["dW_ff"] + c["dW_rec"] + [c["dW_out"]], full["dW_ff"] + full["dW_rec"] + [full["dW_out"]]):
        assert np.array_equal(a, b)
    for l in range(w.L):
        assert np.array_equal(c["S"][l], full["S"][l])
    st = c["stats"]
    assert st["fwd_steps"] == w.T and np.all(st["bwd_steps"][1:] == 1)
    T = w.T
    Kc = min(K, T) if K else 0
    # cost models: Eq. 2 (base), Eq. 4 (standard checkpointing), Eq. 6 (remote), Eq. 11 (double),
    # transfers of Eq. 7 (2 nb_checkpoints) and Eq. 13 (2 T / remote_chunk_size), intervals rounded up
    if strategy == ck.STANDARD:
        assert st["local_states_peak"] == T and st["transfers"] == 0 and st["refwd1_steps"] == 0
    elif strategy == ck.CHUNK:
        assert st["local_states_peak"] == Kc + math.ceil(T / K) and st["transfers"] == 0
        assert st["refwd1_steps"] == T and st["refwd2_steps"] == 0
    elif strategy == ck.REMOTE:
        assert st["local_states_peak"] == Kc + 1 and st["transfers"] == 2 * math.ceil(T / K)
        assert st["refwd1_steps"] == T
    elif strategy == ck.HIERARCHICAL:
        n_ck = math.ceil(T / K)
        P = min(R, n_ck)
        # Eq. 9: chunk_size + nb_local states; Eq. 10 read as two communications per batch but the last
        assert st["local_states_peak"] == Kc + P and st["transfers"] == 2 * (math.ceil(n_ck / P) - 1)
        assert st["refwd1_steps"] == T
    else:
        assert st["local_states_peak"] == Kc + math.ceil(min(R, T) / K) <= K + R // K
        assert st["transfers"] == 2 * math.ceil(T / R)
        assert st["refwd2_steps"] == T and st["refwd1_steps"] <= T


def _read_fig1():
    rows = {}
    for line in open(os.path.join(GOLDEN, "fig1_traces.txt")):
        if line.startswith("#") or not line.strip():
            continue
        row, item, *vals = line.split()
        rows.setdefault(row, {})[item] = vals
    return rows


def test_traces_match_the_papers_figure(orc32):
    """Fig. 1 drawn for T = 11, chunk_size = 3, remote_chunk_size = 6."""
    fig = _read_fig1()
    w = wl.small(T=11)
    d = wl.make(w)
    spec = spec_of(w)
    run = lambda s, K=0, R=0: ck.bptt_checkpointed(orc32, spec, d["input_dense"], d["targets"], d["W_ff"],
                                                   d["W_rec"], d["W_out"], s, K, R)
    pairs = lambda v: [(int(a), int(b)) for a, b in zip(v[0::2], v[1::2])]
    for row, strat, K, R in (("chunk", ck.CHUNK, 3, 0), ("remote", ck.REMOTE, 3, 0), ("double", ck.DOUBLE, 3, 6)):
        c = run(strat, K, R)
        f = fig[row]
        fwd_ck = [(tier, t) for tier, t in c["ckpts"]]
        if row == "double":
            assert sorted(t for tier, t in fwd_ck if tier == "remote") == [int(x) for x in f["ckpt_remote"]]
            assert sorted(t for tier, t in fwd_ck if tier == "local") == [int(x) for x in f["ckpt_local"]]
        else:
            tier = "local" if row == "chunk" else "remote"
            assert sorted(t for tr, t in fwd_ck if tr == tier) == [int(x) for x in f["ckpt_" + tier]]
        n_fwd, n_re, n_bwd = (int(x) for x in f["passes"])
        st = c["stats"]
        assert st["fwd_steps"] == n_fwd * 11 and np.all(st["bwd_steps"][1:] == n_bwd)
        assert (st["refwd1_steps"] > 0) + (st["refwd2_steps"] > 0) == n_re
        # re-forward_1 arrows of the Double row are drawn exactly as executed; the arrows that fill a
        # chunk are drawn up to the state before the next checkpoint, the execution recomputes that
        # state too (same value), so the drawn range is contained and at most one state shorter
        ours1 = [(a, b) for k, a, b in c["trace"] if k == "reforward1"]
        ours2 = [(a, b) for k, a, b in c["trace"] if k == "reforward2"]
        if row == "double":
            assert ours1 == pairs(f["reforward1"])
            drawn, ours = pairs(f["reforward2"]), ours2
        else:
            drawn, ours = pairs(f["reforward1"]), ours1
        assert len(drawn) == len(ours)
        for (a, b), (oa, ob) in zip(drawn, ours):
            assert a == oa and b <= ob <= b + 1
    plain = run(ck.STANDARD)
    assert plain["stats"]["local_states_peak"] == 11 and plain["stats"]["transfers"] == 0
