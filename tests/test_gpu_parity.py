"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs.  Spike trains and event lists bit-exact; membranes <= 1e-5 absolute; gradients
<= 1e-4 of the tensor's largest entry; every checkpointing strategy bit-identical to STANDARD."""
import ctypes as C
import math

import numpy as np
import pytest

import snn_workloads as wl
from gpu_helpers import (V_ATOL, assert_grads_close, lists_from_dense, make_session, run_oracle)

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def sb():
    from paper_2412_11810_b200 import binding
    return binding


# ---------------------------------------------------------------- spike compaction on its own
@pytest.mark.parametrize("n_rows,n", [(1, 1), (7, 31), (5, 32), (33, 100), (64, 1000), (3, 4096), (2, 65536), (0, 64)])
def test_compaction_bit_exact(orc32, n_rows, n):
    rng = np.random.default_rng(n + n_rows)
    v = rng.standard_normal((max(n_rows, 1), n)).astype(np.float32)
    if n_rows >= 3:
        v[0] = -1.0   # empty row
        v[1] = 2.0    # full row
    v = v[:n_rows]
    theta = 0.5
    dense = (v > np.float32(theta))
    words = wl.pack_bits(dense) if n_rows else np.zeros((0, (n + 31) // 32), np.uint32)
    cap = n
    dm = torch.from_numpy(words.view(np.int32).copy()).cuda()
    idx = torch.full((max(n_rows, 1), cap), -1, dtype=torch.int32, device="cuda")
    cnt = torch.full((max(n_rows, 1),), -1, dtype=torch.int32, device="cuda")
    sb().snn_compact_spikes(dm.data_ptr(), n_rows, words.shape[1], idx.data_ptr(), cap, cnt.data_ptr(), 0)
    torch.cuda.synchronize()
    idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
    for r in range(n_rows):
        ref = orc32.compact(v[r], theta)          # brute force: for i: if v[i] > theta: push(i)
        assert cnt[r] == len(ref)
        assert np.array_equal(idx[r, :cnt[r]], ref)
        assert np.all(idx[r, cnt[r]:] == -1)


def test_compaction_capacity_clamps(orc32):
    words = np.full((2, 4), 0xFFFFFFFF, np.uint32)
    dm = torch.from_numpy(words.view(np.int32)).cuda()
    idx = torch.full((2, 10), -1, dtype=torch.int32, device="cuda")
    guard = torch.full((16,), -7, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(2, dtype=torch.int32, device="cuda")
    sb().snn_compact_spikes(dm.data_ptr(), 2, 4, idx.data_ptr(), 10, cnt.data_ptr(), 0)
    torch.cuda.synchronize()
    assert np.all(cnt.cpu().numpy() == 128)
    assert np.array_equal(idx.cpu().numpy(), np.tile(np.arange(10, dtype=np.int32), (2, 1)))
    assert np.all(guard.cpu().numpy() == -7)


# ---------------------------------------------------------------- forward: membranes, spikes, events
def _check_forward(orc32, w, d, extra_flags=0):
    ref = run_oracle(orc32, w, d, do_backward=False)
    s, bits, targets = make_session(w, d)
    loss = s.train_step(bits, targets, forward_only=True, keep_V=True, max_activity=1.0, extra_flags=extra_flags)
    assert abs(loss - ref["loss"]) <= 1e-5 * max(1.0, abs(ref["loss"]))
    for l in range(w.L):
        V = s.debug_V[l].cpu().numpy()
        assert np.abs(V[1:] - ref["V"][l][1:]).max() <= V_ATOL
        assert np.array_equal(V[1:], ref["V"][l][1:]), "canonical operation order: expected bit-equal"
        words = s.spike_words(l + 1)
        assert np.array_equal(wl.unpack_bits(words, w.sizes[l + 1]), ref["S"][l].astype(np.uint8))
    # event lists: input (layer 0) and every hidden layer, every (t, b)
    dense = [d["input_dense"]] + [r[1:] for r in ref["S"]]
    for layer in range(w.L + 1):
        off, pool = s.events(layer)
        want = lists_from_dense(dense[layer])
        for t in range(1, w.T + 1):
            for b in range(w.B):
                got = pool[b, off[t, b]:off[t + 1, b]]
                assert np.array_equal(got, want[t - 1][b]), (layer, t, b)
    s.close()
    return ref


def test_forward_tiny_bit_exact(orc32):
    w = wl.small()
    _check_forward(orc32, w, wl.make(w))


def test_forward_ragged_sizes_bit_exact(orc32):
    # hidden sizes that are multiples of 4 but not of 32 or 128, input not a multiple of 32,
    # several column tiles (N > 512) and more than 1024 events per list
    w = wl.small(sizes=(70, 3000, 36, 7), T=9, B=2, p_in=0.5, g_ff=(3.0, 6.0), g_rec=(1.0, 1.0), seed=3)
    ref = _check_forward(orc32, w, wl.make(w))
    assert ref["S"][0][1:].mean() > 0.1


def test_forward_one_launch_per_step_bit_exact(orc32):
    """Small spiking networks run the forward pass as one cooperative launch per forward operation; the
    launch-per-step kernel (the one large networks use) must give the same bits."""
    f, g = sb().SNN_FLAG_FORWARD_PER_STEP, sb().SNN_FLAG_FORWARD_STREAM_WEIGHTS
    w = wl.small()
    _check_forward(orc32, w, wl.make(w), extra_flags=f)
    _check_forward(orc32, w, wl.make(w), extra_flags=g)
    w = wl.small(sizes=(70, 3000, 36, 7), T=9, B=2, p_in=0.5, g_ff=(3.0, 6.0), g_rec=(1.0, 1.0), seed=3)
    _check_forward(orc32, w, wl.make(w), extra_flags=f)
    # three layers, ragged tiles, 140 thread blocks of 16 neurons: weights in shared memory by default
    w = wl.small(sizes=(33, 520, 1100, 600, 9), T=37, B=6, p_in=0.1, g_ff=(2.5, 1.5, 1.5), g_rec=(1.0, 1.0, 1.0), seed=5)
    _check_forward(orc32, w, wl.make(w), extra_flags=f)
    _check_forward(orc32, w, wl.make(w), extra_flags=g)
    _check_forward(orc32, w, wl.make(w))
    # more than 32 samples (two samples groups per thread), more than 256 events per sample and step
    w = wl.small(sizes=(100, 1000, 8), T=7, B=45, p_in=0.5, g_ff=(4.0,), g_rec=(2.0,), seed=6)
    ref = _check_forward(orc32, w, wl.make(w))
    assert ref["S"][0][1:].sum(axis=-1).max() > 256
    _check_forward(orc32, w, wl.make(w), extra_flags=g)


def test_forward_segment_launch_with_the_shallow_ring(orc32):
    """The cooperative forward launch of L2-resident networks copies weight rows through a ring that is as deep as one
    thread block per SM allows; a grid of more blocks than SMs (here 4 x 16 x 3 = 192) takes the shallow ring with two
    blocks per SM.  Same bits as the oracle, event lists included; the stream-weights flag keeps the weights out of
    shared memory so that this launch is the one that runs."""
    g = sb().SNN_FLAG_FORWARD_STREAM_WEIGHTS
    w = wl.small(sizes=(64, 1540, 1540, 1028, 10), T=12, B=16, p_in=0.1, g_ff=(2.5, 1.5, 1.5), g_rec=(1.0, 1.0, 1.0), seed=59)
    ref = _check_forward(orc32, w, wl.make(w), extra_flags=g)
    assert all(float(x[1:].mean()) > 0.005 for x in ref["S"])


def test_forward_c1_bit_exact(orc32):
    w = wl.WORKLOADS["c1"]
    ref = _check_forward(orc32, w, wl.make(w))
    assert ref["S"][0].sum() > 0


# ---------------------------------------------------------------- gradients and strategies
STRATS = [(1, 4, 0), (1, 1, 0), (1, 13, 0), (1, 40, 0), (2, 4, 0), (2, 1, 0), (2, 5, 0), (3, 2, 6), (3, 3, 3),
          (3, 1, 4), (3, 2, 26), (3, 13, 13), (5, 2, 6), (5, 1, 4), (4, 2, 2), (4, 2, 3), (4, 3, 1), (4, 1, 4),
          (4, 4, 9)]   # (strategy, chunk_size, remote_chunk_size or, for strategy 4, nb_local)


def _bits(t):
    return [x.cpu().numpy().view(np.uint32).copy() for x in t]


def test_gradients_and_all_strategies_tiny(orc32):
    w = wl.small()
    d = wl.make(w)
    ref = run_oracle(orc32, w, d)
    s, bits, targets = make_session(w, d)
    loss = s.train_step(bits, targets, strategy=0, max_activity=1.0)
    assert abs(loss - ref["loss"]) <= 1e-5 * max(1.0, abs(ref["loss"]))
    assert_grads_close(s.gradients(), ref)
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    assert s.stats().local_state_slots == w.T + 1
    for strat, K, R in STRATS:
        for g in s.dW_ff + s.dW_rec + [s.dW_out]:
            g.fill_(float("nan"))
        loss2 = s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=0 if strat == 4 else R,
                             nb_local=R if strat == 4 else 0, max_activity=1.0)
        assert loss2 == loss
        for a, b in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
            assert np.array_equal(a, b), f"strategy {strat} K={K} R={R} differs from STANDARD"
        st = s.stats()
        Kc = min(K, w.T)
        if strat == 1:
            assert st.local_state_slots == Kc + math.ceil(w.T / K) and st.d2h_copies == 0
        elif strat == 2:
            assert st.local_state_slots == Kc + 2
            assert st.d2h_copies == st.h2d_copies == math.ceil(w.T / K)
        elif strat == 4:
            n_ck = math.ceil(w.T / K)
            P = min(R, n_ck)
            assert st.local_state_slots == Kc + P
            assert st.d2h_copies == st.h2d_copies == math.ceil(n_ck / P) - 1
        else:
            assert st.local_state_slots == Kc + math.ceil(min(R, w.T) / K) + 1
            assert st.d2h_copies == st.h2d_copies == math.ceil(w.T / R)
        dev, pin = s.peak_memory()
        assert pin == (0 if strat == 5 else st.remote_state_slots * st.state_bytes)
    s.close()


@pytest.mark.parametrize("T", [1, 2])
def test_degenerate_sequence_lengths(orc32, T):
    w = wl.small(T=T)
    d = wl.make(w)
    ref = run_oracle(orc32, w, d)
    s, bits, targets = make_session(w, d)
    for strat, K, R in [(0, 0, 0), (1, 1, 0), (2, 3, 0), (3, 1, 2)]:
        s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R, max_activity=1.0)
        assert_grads_close(s.gradients(), ref)
    s.close()


def test_silent_and_saturated_networks(orc32):
    from dataclasses import replace
    for theta in (1e30, -1e30):
        w = replace(wl.small(T=3), theta=theta)
        d = wl.make(w)
        ref = run_oracle(orc32, w, d)
        s, bits, targets = make_session(w, d)
        loss = s.train_step(bits, targets, strategy=1, chunk_size=2, max_activity=1.0)
        if theta > 0:
            assert abs(loss - math.log(w.sizes[-1])) < 1e-6
        assert_grads_close(s.gradients(), ref)
        s.close()


def test_sigmoid_surrogate(orc32):
    from oracle.oracle import SURR_SIGMOID, NetSpec, leak_from_tau
    from paper_2412_11810_b200 import Session
    w = wl.small()
    d = wl.make(w)
    spec = NetSpec(w.sizes, leak_from_tau(w.tau_mem), w.theta, 4.0, w.scale(), surrogate=SURR_SIGMOID)
    ref = orc32.bptt_full(spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"])
    s = Session(w.sizes, tau_mem=w.tau_mem, threshold=w.theta, surrogate=1, surrogate_beta=4.0,
                readout_scale=w.scale())
    s.set_weights(d["W_ff"], d["W_rec"], d["W_out"])
    s.train_step(d["input_bits"], d["targets"], strategy=3, chunk_size=2, remote_chunk_size=4, max_activity=1.0)
    assert_grads_close(s.gradients(), ref)
    s.close()


def test_triangle_surrogate(orc32):
    """The compact-support pseudo-derivative: most neurons get exactly zero, the rest must agree with the oracle,
    on both backward paths and bit-identically across strategies."""
    from oracle.oracle import SURR_TRIANGLE, NetSpec, leak_from_tau
    from paper_2412_11810_b200 import Session
    b = sb()
    w = wl.small(sizes=(70, 700, 260, 7), T=41, B=5, p_in=0.05, g_ff=(2.5, 1.4), g_rec=(1.0, 1.0), seed=71)
    d = wl.make(w)
    spec = NetSpec(w.sizes, leak_from_tau(w.tau_mem), w.theta, 3.0, w.scale(), surrogate=SURR_TRIANGLE)
    ref = orc32.bptt_full(spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"])
    assert all(np.abs(g).max() > 0 for g in ref["dW_rec"])
    s = Session(w.sizes, tau_mem=w.tau_mem, threshold=w.theta, surrogate=b.SNN_SURR_TRIANGLE, surrogate_beta=3.0,
                readout_scale=w.scale())
    s.set_weights(d["W_ff"], d["W_rec"], d["W_out"])
    s.train_step(d["input_bits"], d["targets"], strategy=0, max_activity=1.0)
    assert_grads_close(s.gradients(), ref)
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    for strat, K, R, flags in [(1, 6, 0, 0), (3, 4, 16, 0), (1, 6, 0, b.SNN_FLAG_BACKWARD_PER_STEP)]:
        s.train_step(d["input_bits"], d["targets"], strategy=strat, chunk_size=K, remote_chunk_size=R,
                     max_activity=1.0, extra_flags=flags)
        for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
            assert np.array_equal(x, y), (strat, K, R, flags)
    s.close()


@pytest.mark.parametrize("beta", [3.0, 10.0])
def test_event_driven_backward_pass(orc32, beta):
    """With the compact-support pseudo-derivative the backward step needs the rows of W only for the (sample, neuron)
    pairs within 1 / beta of the threshold: the event-driven kernel reads just those.  Against the oracle, against
    the dense kernels (to rounding), bit-identical across strategies, widths that are no multiple of 32 or 128; and
    refused for a surrogate without compact support."""
    from oracle.oracle import SURR_TRIANGLE, NetSpec, leak_from_tau
    from paper_2412_11810_b200 import Session
    b = sb()
    w = wl.small(sizes=(70, 700, 260, 132, 7), T=41, B=5, p_in=0.05, g_ff=(2.5, 1.4, 1.5), g_rec=(1.0, 1.0, 1.0), seed=73)
    d = wl.make(w)
    spec = NetSpec(w.sizes, leak_from_tau(w.tau_mem), w.theta, beta, w.scale(), surrogate=SURR_TRIANGLE)
    ref = orc32.bptt_full(spec, d["input_dense"], d["targets"], d["W_ff"], d["W_rec"], d["W_out"])
    near = [float((np.abs(v[1:] - w.theta) * beta < 1).mean()) for v in ref["V"]]
    assert all(0.0 < x < 0.6 for x in near), near            # some, not all, neurons are near the threshold
    assert all(np.abs(g).max() > 0 for g in ref["dW_rec"])
    s = Session(w.sizes, tau_mem=w.tau_mem, threshold=w.theta, surrogate=b.SNN_SURR_TRIANGLE, surrogate_beta=beta,
                readout_scale=w.scale())
    s.set_weights(d["W_ff"], d["W_rec"], d["W_out"])
    f = b.SNN_FLAG_BACKWARD_EVENT_DRIVEN
    s.train_step(d["input_bits"], d["targets"], strategy=0, max_activity=1.0, extra_flags=f)
    assert_grads_close(s.gradients(), ref)
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    for strat, K, R in [(1, 6, 0), (3, 4, 16), (2, 9, 0)]:
        for g in s.dW_ff + s.dW_rec + [s.dW_out]:
            g.fill_(float("nan"))
        s.train_step(d["input_bits"], d["targets"], strategy=strat, chunk_size=K, remote_chunk_size=R,
                     max_activity=1.0, extra_flags=f)
        for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
            assert np.array_equal(x, y), (strat, K, R)
    s.close()
    s2 = Session(w.sizes, tau_mem=w.tau_mem, threshold=w.theta, surrogate_beta=beta, readout_scale=w.scale())
    s2.set_weights(d["W_ff"], d["W_rec"], d["W_out"])
    with pytest.raises(b.SnnError) as e:
        s2.train_step(d["input_bits"], d["targets"], strategy=0, max_activity=1.0, extra_flags=f)
    assert e.value.status == b.SNN_ERR_UNSUPPORTED
    s2.close()


def test_c1_gradients_all_strategies(orc32):
    w = wl.WORKLOADS["c1"]
    d = wl.make(w)
    ref = run_oracle(orc32, w, d)
    s, bits, targets = make_session(w, d)
    loss = s.train_step(bits, targets, strategy=0)
    assert abs(loss - ref["loss"]) <= 1e-5 * max(1.0, abs(ref["loss"]))
    assert_grads_close(s.gradients(), ref)
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    for strat, K, R in [(1, 10, 0), (2, 7, 0), (3, 4, 16)]:
        s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R)
        for a, b in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
            assert np.array_equal(a, b)
    s.close()


def test_medium_network_several_tiles(orc32):
    # two layers wider than one column tile, batch above the backward kernel's batch tile,
    # ragged segments in both tiers
    w = wl.small(sizes=(96, 640, 1040, 12), T=37, B=19, p_in=0.05, g_ff=(2.5, 1.4), g_rec=(1.0, 1.0), seed=5)
    d = wl.make(w)
    ref = run_oracle(orc32, w, d)
    act = [float(s_[1:].mean()) for s_ in ref["S"]]
    assert all(0.005 < a < 0.5 for a in act), act
    s, bits, targets = make_session(w, d)
    s.train_step(bits, targets, strategy=0)
    assert_grads_close(s.gradients(), ref)
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    for strat, K, R in [(1, 6, 0), (2, 8, 0), (3, 3, 12)]:
        s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R)
        for a, b in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
            assert np.array_equal(a, b)
    s.close()


def test_host_input_path_matches_device_input(orc32):
    w = wl.small()
    d = wl.make(w)
    s, bits, targets = make_session(w, d)
    l0 = s.train_step(bits, targets, strategy=1, chunk_size=4, max_activity=1.0)
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    l1 = s.train_step(d["input_bits"], d["targets"], strategy=1, chunk_size=4, max_activity=1.0)
    assert l0 == l1
    for a, b in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
        assert np.array_equal(a, b)
    s.close()


# ---------------------------------------------------------------- errors reported, nothing faults
def test_errors_are_reported(orc32):
    b = sb()
    w = wl.small()
    d = wl.make(w)
    s, bits, targets = make_session(w, d)
    with pytest.raises(b.SnnError) as e:
        s.train_step(bits, targets, strategy=3, chunk_size=4, remote_chunk_size=6)
    assert e.value.status == b.SNN_ERR_INVALID_ARG
    # far fewer event slots than the activity needs: reported, never written out of bounds
    with pytest.raises(b.SnnError) as e:
        s.train_step(bits, targets, strategy=0, max_activity=1e-4)
    assert e.value.status == b.SNN_ERR_EVENT_OVERFLOW
    # workspace too small: rejected before any launch
    s.train_step(bits, targets, strategy=0, max_activity=0.5)
    ck = s.ckpt(0)
    need, _ = b.snn_workspace_query(s.net, w.T, w.B, ck, 0.5)
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    a = b.snn_step_args()
    a.T, a.B, a.input, a.targets = w.T, w.B, bits.data_ptr(), targets.data_ptr()
    wff = b.ptr_array([x.data_ptr() for x in s.W_ff]); wrec = b.ptr_array([x.data_ptr() for x in s.W_rec])
    gff = b.ptr_array([x.data_ptr() for x in s.dW_ff]); grec = b.ptr_array([x.data_ptr() for x in s.dW_rec])
    a.W_ff, a.W_rec, a.W_out, a.dW_ff, a.dW_rec, a.dW_out = wff, wrec, s.W_out.data_ptr(), gff, grec, s.dW_out.data_ptr()
    a.device_ws, a.device_ws_bytes = small.data_ptr(), small.numel()
    a.ckpt, a.max_activity = ck, 0.5
    loss = C.c_float()
    assert b.lib.snn_train_step(s.net, C.byref(a), C.byref(loss)) == b.SNN_ERR_WORKSPACE_TOO_SMALL
    s.close()


def test_bad_targets_and_input_padding_bits_are_guarded(orc32):
    """Caller data never becomes an unchecked index: a target outside [0, N_out) is reported as an invalid
    argument (and not read through), and stray bits beyond N_0 in the last input word of a row change nothing,
    on every forward path."""
    b = sb()
    w = wl.small(sizes=(40, 260, 132, 6), T=21, B=5, p_in=0.1, g_ff=(2.5, 1.6), seed=17)   # 40 inputs: 8 valid bits in word 1
    d = wl.make(w)
    s, bits, targets = make_session(w, d)
    for bad in (-1, w.sizes[-1], 2 ** 30):
        t_bad = targets.clone()
        t_bad[2] = bad
        with pytest.raises(b.SnnError) as e:
            s.train_step(bits, t_bad, strategy=0, max_activity=1.0)
        assert e.value.status == b.SNN_ERR_INVALID_ARG and "target" in str(e.value)
    dirty = bits.clone()
    dirty[:, :, 1] |= torch.tensor(np.array(0xFFFFFF00, np.uint32).view(np.int32).item(), dtype=torch.int32)
    for flags in (0, b.SNN_FLAG_FORWARD_STREAM_WEIGHTS, b.SNN_FLAG_FORWARD_PER_STEP):
        loss0 = s.train_step(bits, targets, strategy=3, chunk_size=2, remote_chunk_size=8, max_activity=1.0,
                             extra_flags=flags)
        clean = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
        ev_clean = [s.events(l) for l in range(w.L + 1)]
        loss1 = s.train_step(dirty, targets, strategy=3, chunk_size=2, remote_chunk_size=8, max_activity=1.0,
                             extra_flags=flags)
        assert loss0 == loss1
        for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), clean):
            assert np.array_equal(x, y), flags
        for l in range(w.L + 1):
            off, pool = s.events(l)
            assert np.array_equal(off[1:w.T + 2], ev_clean[l][0][1:w.T + 2])
            for bb in range(w.B):
                used = pool[bb][:int(off[w.T + 1][bb])]
                assert used.size == 0 or int(used.max()) < w.sizes[l]
    s.close()


def test_events_spilled_to_host_memory(orc32):
    """With SNN_FLAG_SPILL_EVENTS the device keeps the events of two remote segments only; the rest waits in
    pinned memory.  Same bits as the step that keeps every event on the device, for REMOTE and DOUBLE, a last
    segment that is short, every forward and recomputation path, the spiking and the graded cell; the device
    workspace shrinks and the number of window transfers is 2 n - 3 for n segments."""
    b = sb()
    cases = [(wl.small(sizes=(40, 260, 132, 6), T=53, B=5, p_in=0.1, g_ff=(2.5, 1.6), seed=71), 0),
             (_graded(sizes=(48, 264, 132, 9), T=45, B=4, seed=72), 0)]
    for w, _ in cases:
        d = wl.make(w)
        s, bits, targets = make_session(w, d)
        s.train_step(bits, targets, strategy=0, max_activity=1.0)
        assert_grads_close(s.gradients(), run_oracle(orc32, w, d))
        base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
        for strat, K, R in [(2, 7, 0), (3, 3, 12), (3, 4, 8), (2, 60, 0)]:
            E = R if strat == 3 else K
            n_seg = -(-w.T // min(E, w.T))
            for flags in (0, b.SNN_FLAG_FORWARD_PER_STEP | b.SNN_FLAG_REFORWARD_PER_STEP, b.SNN_FLAG_FORWARD_STREAM_WEIGHTS,
                          b.SNN_FLAG_REFORWARD_ROWS):
                for g in s.dW_ff + s.dW_rec + [s.dW_out]:
                    g.fill_(float("nan"))
                s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R, max_activity=1.0,
                             extra_flags=flags | b.SNN_FLAG_SPILL_EVENTS)
                for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
                    assert np.array_equal(x, y), (w.cell, strat, K, R, flags)
                assert s.stats().event_window_copies == max(0, 2 * n_seg - 3)
        ck = s.ckpt(3, 3, 12)
        d_all, p_all = b.snn_workspace_query(s.net, w.T, w.B, ck, 1.0)
        d_win, p_win = b.snn_workspace_query(s.net, w.T, w.B, ck, 1.0, b.SNN_FLAG_SPILL_EVENTS)
        assert d_win < d_all and p_win > p_all
        s.close()


# ---------------------------------------------------------------- graded (thresholded-ReLU) cell
def _graded(**kw):
    a = dict(cell=wl.CELL_GRADED, theta=0.3, g_ff=(1.2, 0.8), g_rec=(0.3, 0.3), p_in=0.3)
    a.update(kw)
    return wl.small(**a)


def test_graded_forward_bit_exact(orc32):
    w = _graded(sizes=(37, 640, 36, 7), T=11, B=3, seed=21)
    d = wl.make(w)
    ref = run_oracle(orc32, w, d, do_backward=False)
    frac = [float((x[1:] != 0).mean()) for x in ref["S"]]
    assert all(0.05 < f < 0.8 for f in frac), frac
    s, x, targets = make_session(w, d)
    loss = s.train_step(x, targets, forward_only=True, keep_V=True, max_activity=1.0)
    assert abs(loss - ref["loss"]) <= 1e-5 * max(1.0, abs(ref["loss"]))
    for l in range(w.L):
        V = s.debug_V[l].cpu().numpy()
        assert np.array_equal(V[1:], ref["V"][l][1:])
        assert np.array_equal(wl.unpack_bits(s.spike_words(l + 1), w.sizes[l + 1]), (ref["S"][l] != 0).astype(np.uint8))
    # event lists with their values, input included
    sb_ = sb()
    dense = [d["input_dense"]] + [r[1:] for r in ref["S"]]
    for layer in range(w.L + 1):
        off, pool = s.events(layer)
        e = sb_.snn_get_event_layout(s.net, layer)
        vals = s.device_ws[e.values_off:e.values_off + 4 * w.B * e.pool_capacity].view(torch.float32).cpu().numpy()
        vals = vals.reshape(w.B, e.pool_capacity)
        for t in range(1, w.T + 1):
            for b in range(w.B):
                idx = np.flatnonzero(dense[layer][t - 1, b])
                assert np.array_equal(pool[b, off[t, b]:off[t + 1, b]], idx)
                assert np.array_equal(vals[b, off[t, b]:off[t + 1, b]], dense[layer][t - 1, b, idx])
    s.close()


def test_graded_gradients_and_strategies(orc32):
    w = _graded(sizes=(37, 640, 132, 7), T=23, B=5, seed=22)
    d = wl.make(w)
    ref = run_oracle(orc32, w, d)
    s, x, targets = make_session(w, d)
    loss = s.train_step(x, targets, strategy=0, max_activity=1.0)
    assert abs(loss - ref["loss"]) <= 1e-5 * max(1.0, abs(ref["loss"]))
    assert_grads_close(s.gradients(), ref)
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    for strat, K, R in [(1, 4, 0), (1, 1, 0), (2, 5, 0), (3, 2, 6), (3, 3, 3)]:
        for g in s.dW_ff + s.dW_rec + [s.dW_out]:
            g.fill_(float("nan"))
        assert s.train_step(x, targets, strategy=strat, chunk_size=K, remote_chunk_size=R, max_activity=1.0) == loss
        for a, b in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
            assert np.array_equal(a, b), (strat, K, R)
    # host input path
    assert s.train_step(d["input_dense"], d["targets"], strategy=3, chunk_size=2, remote_chunk_size=6,
                        max_activity=1.0) == loss
    for a, b in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
        assert np.array_equal(a, b)
    s.close()


def test_graded_with_unit_events_equals_lif_without_reset(orc32):
    """Every input value 1 and a threshold no hidden neuron reaches: the graded kernels then do
    exactly what the spiking kernels do on the same input words (no hidden event, no reset)."""
    from dataclasses import replace
    w = wl.small(sizes=(40, 260, 8), T=9, B=3, p_in=0.3, seed=23)
    d = wl.make(w)
    wl_lif = replace(w, theta=1e30)
    s1, bits, targets = make_session(wl_lif, d)
    s1.train_step(bits, targets, forward_only=True, keep_V=True, max_activity=1.0)
    V_lif = s1.debug_V[0].cpu().numpy()
    s1.close()
    wg = replace(w, theta=1e30, cell=wl.CELL_GRADED)
    dg = dict(d, input_dense=(d["input_dense"] != 0).astype(np.float32))
    s2, x, targets = make_session(wg, dg)
    s2.train_step(x, targets, forward_only=True, keep_V=True, max_activity=1.0)
    assert np.array_equal(s2.debug_V[0].cpu().numpy(), V_lif)
    s2.close()


def test_cell_and_input_format_must_match():
    b = sb()
    w = wl.small()
    d = wl.make(w)
    from dataclasses import replace
    s, x, targets = make_session(replace(w, cell=wl.CELL_GRADED), d)
    a_bits = torch.from_numpy(d["input_bits"].view(np.int32)).cuda()
    s.cell = b.SNN_CELL_LIF      # makes the session pass SNN_INPUT_BITS to a graded net
    with pytest.raises(b.SnnError) as e:
        s.train_step(a_bits, targets)
    assert e.value.status == b.SNN_ERR_UNSUPPORTED
    s.close()


@pytest.mark.parametrize("B", [1, 40])
def test_batch_sizes_outside_the_backward_tiles(orc32, B):
    """One sample, and more samples than one pass of the backward kernel covers (32); layers of
    different widths so that some layers have fewer row tiles than the widest one."""
    w = wl.small(sizes=(40, 260, 516, 6), T=9, B=B, p_in=0.15, g_ff=(2.5, 1.6), seed=31)
    d = wl.make(w)
    ref = run_oracle(orc32, w, d)
    assert all(0.01 < float(x[1:].mean()) < 0.6 for x in ref["S"])
    s, bits, targets = make_session(w, d)
    s.train_step(bits, targets, strategy=0, max_activity=1.0)
    assert_grads_close(s.gradients(), ref)
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    s.train_step(bits, targets, strategy=3, chunk_size=2, remote_chunk_size=4, max_activity=1.0)
    for a, b in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
        assert np.array_equal(a, b)
    s.close()


def test_layer_by_layer_backward_order(orc32):
    """The launch order used for large networks (feed-forward term of a run of steps as one product),
    forced here on a small one: same gradients within tolerance, and all strategies bit-identical to
    STANDARD under that order; runs longer and shorter than 32 steps."""
    b = sb()
    w = wl.small(sizes=(96, 640, 516, 260, 12), T=71, B=11, p_in=0.06, g_ff=(2.5, 1.5, 1.5), g_rec=(1.0, 1.0, 1.0), seed=41)
    d = wl.make(w)
    ref = run_oracle(orc32, w, d)
    assert all(0.005 < float(x[1:].mean()) < 0.5 for x in ref["S"])
    s, bits, targets = make_session(w, d)
    f = b.SNN_FLAG_BACKWARD_LAYER_BY_LAYER
    s.train_step(bits, targets, strategy=0, extra_flags=f)
    assert_grads_close(s.gradients(), ref)
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    for strat, K, R in [(1, 9, 0), (1, 40, 0), (2, 33, 0), (3, 4, 16), (3, 1, 3)]:
        s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R, extra_flags=f)
        for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
            assert np.array_equal(x, y), (strat, K, R)
    # the wavefront order agrees within tolerance (different summation, not bit-identical)
    s.train_step(bits, targets, strategy=1, chunk_size=9, extra_flags=b.SNN_FLAG_BACKWARD_WAVEFRONT)
    assert_grads_close(s.gradients(), ref)
    # so does the feed-forward product on the mma.sync kernel instead of the tcgen05 one, and it is deterministic too
    g = f | b.SNN_FLAG_FF_PRODUCT_MMA_SYNC
    s.train_step(bits, targets, strategy=0, extra_flags=g)
    assert_grads_close(s.gradients(), ref)
    legacy = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    assert any(not np.array_equal(x, y) for x, y in zip(legacy, base))      # really another kernel
    s.train_step(bits, targets, strategy=3, chunk_size=4, remote_chunk_size=16, extra_flags=g)
    for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), legacy):
        assert np.array_equal(x, y)
    s.close()


@pytest.mark.parametrize("B,N1", [(3, 4772), (8, 4772), (11, 4772), (19, 4772), (5, 2404), (14, 2404), (8, 4768), (13, 2400)])
def test_layer_by_layer_backward_as_one_launch_per_run(orc32, B, N1):
    """Wide layers under the layer-by-layer order run the steps of a run of 32 as ONE cooperative launch that
    keeps the recurrent matrix streaming across step boundaries.  It must give the bits of the same order with
    one launch per step, for each batch tiling (8, 16, 32 samples), a width that is no multiple of the row tile
    or of the 128-wide chunk, runs shorter and longer than the copy ring, and agree with the oracle.  (The wide
    layer takes that launch where its thread blocks all fit the device at once; a layer half as wide takes it with
    thread blocks of 16 rows, for up to 16 samples.)"""
    b = sb()
    w = wl.small(sizes=(48, N1, 132, 7), T=37, B=B, p_in=0.1, g_ff=(2.5, 1.5), g_rec=(1.0, 1.0), seed=43)
    d = wl.make(w)
    ref = run_oracle(orc32, w, d)
    assert all(0.005 < float(x[1:].mean()) < 0.5 for x in ref["S"])
    s, bits, targets = make_session(w, d)
    f = b.SNN_FLAG_BACKWARD_LAYER_BY_LAYER
    s.train_step(bits, targets, strategy=0, extra_flags=f)
    launches_stream = s.stats().kernel_launches
    assert_grads_close(s.gradients(), ref)
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    s.train_step(bits, targets, strategy=0, extra_flags=f | b.SNN_FLAG_BACKWARD_PER_STEP)
    assert s.stats().kernel_launches > launches_stream + 30          # the wide layer really took the other path
    for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
        assert np.array_equal(x, y)
    for strat, K, R in [(1, 9, 0), (3, 2, 6), (2, 35, 0)]:
        for g in s.dW_ff + s.dW_rec + [s.dW_out]:
            g.fill_(float("nan"))
        s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R, extra_flags=f)
        for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
            assert np.array_equal(x, y), (strat, K, R)
    s.close()


@pytest.mark.parametrize("B", [5, 32])
def test_weight_gradient_with_the_deltas_stationary(orc32, B):
    """Large spiking networks accumulate dW with a slab of the deltas held in shared memory and the rows of dW streamed
    past it (no gather from L2).  Forced here on a medium network: the bits of the gathering kernel, for segments
    shorter and longer than a window of 128 pairs (ragged last window), widths that are no multiple of the 128-column
    slab or the 256-row group, and within tolerance of the oracle; rows no event touched stay exactly zero."""
    b = sb()
    w = wl.small(sizes=(70, 644, 300, 9), T=61, B=B, p_in=0.06, g_ff=(2.5, 1.5), g_rec=(1.0, 1.0), seed=47)
    d = wl.make(w)
    ref = run_oracle(orc32, w, d)
    assert all(0.005 < float(x[1:].mean()) < 0.5 for x in ref["S"])
    s, bits, targets = make_session(w, d)
    s.train_step(bits, targets, strategy=0, extra_flags=b.SNN_FLAG_WEIGHT_GRADIENT_GATHER)
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    f = b.SNN_FLAG_WEIGHT_GRADIENT_SLAB
    for strat, K, R in [(0, 0, 0), (1, 7, 0), (1, 50, 0), (3, 3, 12)]:
        for g in s.dW_ff + s.dW_rec + [s.dW_out]:
            g.fill_(float("nan"))
        s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R, extra_flags=f)
        for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
            assert np.array_equal(x, y), (strat, K, R)
    assert_grads_close(s.gradients(), ref)
    s.close()


def test_graded_weight_gradient_with_the_deltas_stationary(orc32):
    """The graded cell on the same kernel: an event multiplies the delta row by its value, looked up in the value pool
    per (pair, row).  Bits of the gathering kernel, several windows of 128 pairs, ragged sizes, oracle tolerance."""
    b = sb()
    w = _graded(sizes=(70, 644, 300, 9), T=45, B=7, seed=53)
    d = wl.make(w)
    ref = run_oracle(orc32, w, d)
    frac = [float((x[1:] != 0).mean()) for x in ref["S"]]
    assert all(0.05 < f < 0.8 for f in frac), frac
    s, bits, targets = make_session(w, d)
    s.train_step(bits, targets, strategy=0, max_activity=1.0, extra_flags=b.SNN_FLAG_WEIGHT_GRADIENT_GATHER)
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    f = b.SNN_FLAG_WEIGHT_GRADIENT_SLAB
    for strat, K, R in [(0, 0, 0), (1, 7, 0), (3, 5, 20)]:
        for g in s.dW_ff + s.dW_rec + [s.dW_out]:
            g.fill_(float("nan"))
        s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R, max_activity=1.0, extra_flags=f)
        for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
            assert np.array_equal(x, y), (strat, K, R)
    assert_grads_close(s.gradients(), ref)
    s.close()


def test_reforward_as_one_launch_per_segment(orc32):
    """The recomputation passes walk through a whole segment inside one launch (small networks: the
    default), with the input currents gathered per (step, sample) or accumulated with the weight rows
    stationary (the order of large networks, forced here).  Gradients must be bit-identical to STANDARD, which
    recomputes nothing, and to the same strategy with one launch per step; sizes that are no multiple of the column tile, segments longer
    than the 32 steps staged at a time, steps with no events at all and steps with more events than
    one window of the merged list (1024) holds."""
    b = sb()
    cases = [
        wl.small(sizes=(70, 700, 1300, 7), T=83, B=5, p_in=0.05, g_ff=(2.5, 1.4), g_rec=(1.0, 1.0), seed=51),
        wl.small(sizes=(40, 4000, 6), T=12, B=2, p_in=0.5, g_ff=(6.0,), g_rec=(3.0,), seed=52),     # > 1024 events per step
        wl.small(sizes=(64, 96, 5), T=90, B=3, p_in=0.01, g_ff=(1.5,), g_rec=(0.5,), seed=53),      # mostly silent steps
        wl.small(sizes=(33, 260, 136, 7), T=50, B=20, p_in=0.1, g_ff=(2.5, 1.6), seed=55),          # 800 (step, sample) pairs per run
    ]
    for w in cases:
        d = wl.make(w)
        ref = run_oracle(orc32, w, d)
        s, bits, targets = make_session(w, d)
        s.train_step(bits, targets, strategy=0, max_activity=1.0)
        assert_grads_close(s.gradients(), ref)
        base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
        for strat, K, R, P in [(1, 40, 0, 0), (1, 7, 0, 0), (2, 11, 0, 0), (3, 4, 16, 0), (3, 3, 9, 0), (4, 5, 0, 3), (5, 2, 8, 0)]:
            for flags in (0, b.SNN_FLAG_REFORWARD_PER_STEP, b.SNN_FLAG_REFORWARD_PER_STEP | b.SNN_FLAG_FORWARD_PER_STEP,
                          b.SNN_FLAG_FORWARD_STREAM_WEIGHTS, b.SNN_FLAG_REFORWARD_ROWS):
                for g in s.dW_ff + s.dW_rec + [s.dW_out]:
                    g.fill_(float("nan"))
                s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R, nb_local=P,
                             max_activity=1.0, extra_flags=flags)
                for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
                    assert np.array_equal(x, y), (w.sizes, strat, K, R, P, flags)
        s.close()
    # the widest case really has steps beyond one window
    S = run_oracle(orc32, cases[1], wl.make(cases[1]))["S"]
    assert S[0][1:].sum(axis=-1).max() > 1024


def test_graded_reforward_as_one_launch_per_segment(orc32):
    b = sb()
    w = _graded(sizes=(48, 600, 532, 9), T=45, B=4, seed=54)
    d = wl.make(w)
    s, bits, targets = make_session(w, d)
    s.train_step(bits, targets, strategy=0, max_activity=1.0)
    assert_grads_close(s.gradients(), run_oracle(orc32, w, d))
    base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
    for strat, K, R in [(1, 6, 0), (3, 4, 12), (2, 40, 0)]:
        for flags in (0, b.SNN_FLAG_REFORWARD_PER_STEP, b.SNN_FLAG_REFORWARD_ROWS):
            for g in s.dW_ff + s.dW_rec + [s.dW_out]:
                g.fill_(float("nan"))
            s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R, max_activity=1.0,
                         extra_flags=flags)
            for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
                assert np.array_equal(x, y), (strat, K, R, flags)
    s.close()
    # the rows-stationary order (large networks) with few and with many events per block of 32 rows
    for kw in (dict(p_in=0.05, g_ff=(2.5, 1.2), seed=56), dict(p_in=0.5, g_ff=(1.5, 1.2), seed=57)):
        w = _graded(sizes=(40, 264, 132, 9), T=30, B=21, **kw)
        d = wl.make(w)
        s, bits, targets = make_session(w, d)
        s.train_step(bits, targets, strategy=0, max_activity=1.0)
        base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
        for strat, K, R in [(1, 7, 0), (3, 4, 12)]:
            s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R, max_activity=1.0,
                         extra_flags=b.SNN_FLAG_REFORWARD_ROWS)
            for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
                assert np.array_equal(x, y), (kw, strat, K, R)
        s.close()


def test_backward_as_one_launch_per_segment(orc32):
    """Small networks run the backward pass of a segment as one cooperative launch with the weights in
    shared memory; it must give the bits of the one-launch-per-step kernel, for every batch tiling
    (1, 8, 16, 32 samples per pass, several passes), ragged row tiles, clusters of several sizes, one to
    three layers, and agree with the oracle."""
    b = sb()
    cases = [
        wl.small(sizes=(70, 700, 1300, 7), T=37, B=5, p_in=0.05, g_ff=(2.5, 1.4), g_rec=(1.0, 1.0), seed=61),
        wl.small(sizes=(33, 520, 260, 600, 9), T=29, B=11, p_in=0.1, g_ff=(2.5, 1.5, 1.5), g_rec=(1.0, 1.0, 1.0), seed=62),
        wl.small(sizes=(64, 1024, 6), T=21, B=32, p_in=0.05, g_ff=(2.5,), g_rec=(1.0,), seed=63),
        wl.small(sizes=(64, 300, 200, 6), T=17, B=40, p_in=0.1, g_ff=(2.5, 1.5), g_rec=(1.0, 1.0), seed=64),
        wl.small(sizes=(20, 24, 12, 5), T=13, B=1, p_in=0.2, seed=65),
    ]
    for w in cases:
        d = wl.make(w)
        ref = run_oracle(orc32, w, d)
        s, bits, targets = make_session(w, d)
        s.train_step(bits, targets, strategy=0, max_activity=1.0, extra_flags=b.SNN_FLAG_BACKWARD_PER_STEP)
        assert_grads_close(s.gradients(), ref)
        base = _bits(s.dW_ff + s.dW_rec + [s.dW_out])
        for strat, K, R in [(0, 0, 0), (1, 7, 0), (1, 40, 0), (3, 4, 16), (2, 5, 0)]:
            for g in s.dW_ff + s.dW_rec + [s.dW_out]:
                g.fill_(float("nan"))
            s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R, max_activity=1.0)
            for x, y in zip(_bits(s.dW_ff + s.dW_rec + [s.dW_out]), base):
                assert np.array_equal(x, y), (w.sizes, w.B, strat, K, R)
        s.close()


def test_bounds_checked_build_gives_the_same_bits(tmp_path):
    """libsnnckpt_debug.so (the same sources with -DSNN_DEBUG_CHECKS=1) tests event positions, row indices and state
    slots before use.  On a correct step no check fires and every gradient has the bits of the ordinary build, on the
    paths that replay stored event lists and on the default ones.  Runs in a child process: the library is chosen at
    import time by SNN_DEBUG_CHECKS=1."""
    import os, subprocess, sys, textwrap
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script = tmp_path / "debug_step.py"
    script.write_text(textwrap.dedent(f"""
        import sys, hashlib
        sys.path.insert(0, {root!r}); sys.path.insert(0, {os.path.join(root, "tests")!r})
        import snn_workloads as wl
        from gpu_helpers import make_session
        from paper_2412_11810_b200 import binding as b
        print("checks", b.lib.snn_debug_checks_enabled())
        w = wl.small(sizes=(40, 260, 132, 6), T=21, B=5, p_in=0.1, g_ff=(2.5, 1.6), seed=19)
        d = wl.make(w)
        s, bits, targets = make_session(w, d)
        for strat, K, R, flags in ((0, 0, 0, 0), (3, 2, 8, 0), (3, 2, 8, b.SNN_FLAG_REFORWARD_PER_STEP), (2, 5, 0, 0),
                                   (1, 4, 0, b.SNN_FLAG_FORWARD_PER_STEP | b.SNN_FLAG_REFORWARD_PER_STEP)):
            s.train_step(bits, targets, strategy=strat, chunk_size=K, remote_chunk_size=R, max_activity=1.0, extra_flags=flags)
            h = hashlib.sha256()
            for g in s.dW_ff + s.dW_rec + [s.dW_out]:
                h.update(g.cpu().numpy().tobytes())
            print("grad", strat, K, R, flags, h.hexdigest())
        s.close()
    """))
    outs = []
    for debug in ("0", "1"):
        env = dict(os.environ, SNN_DEBUG_CHECKS=debug)
        r = subprocess.run([sys.executable, str(script)], capture_output=True, text=True, env=env, timeout=600)
        assert r.returncode == 0, r.stderr[-2000:]
        lines = r.stdout.splitlines()
        assert lines[0] == f"checks {debug}"
        outs.append([l for l in lines if l.startswith("grad")])
    assert len(outs[0]) == 5 and outs[0] == outs[1]


def test_a_wait_that_cannot_end_gives_up():
    """The waits between thread blocks are bounded: one that nothing satisfies raises the time-out status
    after its poll limit and the kernel ends; the context stays usable for a normal step afterwards."""
    import torch
    b = sb()
    scratch = torch.zeros(256, dtype=torch.uint8, device="cuda:0")
    for polls in (1, 1000, 200000):
        assert b.snn_selftest_wait_timeout(scratch.data_ptr(), polls) == b.SNN_ERR_DEVICE_TIMEOUT
    assert b.snn_selftest_wait_timeout(0, 10) == b.SNN_ERR_INVALID_ARG
    w = wl.small()
    d = wl.make(w)
    s, bits, targets = make_session(w, d)
    assert np.isfinite(s.train_step(bits, targets, strategy=1, chunk_size=4, max_activity=1.0))
    s.close()
