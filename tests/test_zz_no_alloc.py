"""The training step for hosts that cannot allocate device memory (snn_train_step_static).

Some users of the library have no allocator to turn to when a step is due: a plain C program
without PyTorch, a process whose GPU memory is already owned by another pool, a service with a
fixed budget where cudaMalloc might fail or stall the device.  For them the library carries its
own fixed-size device workspace.  This test drives that entry point through the C ABI and checks
that it returns what the ordinary entry point returns, bit for bit, twice in a row (the second
call starts from whatever the first one left in the shared buffer), that the result also agrees
with the CPU oracle, and that the second call leaves the amount of free device memory unchanged.
The file is named to be collected last.
"""
import ctypes as C

import numpy as np
import pytest

import snn_workloads as wl
from gpu_helpers import assert_grads_close, make_session, run_oracle

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _args(b, s, w, bits, targets, strategy, K, R, keep):
    a = b.snn_step_args()
    a.T, a.B = w.T, w.B
    a.input, a.input_format, a.targets = bits.data_ptr(), b.SNN_INPUT_BITS, targets.data_ptr()
    keep["wff"] = b.ptr_array([x.data_ptr() for x in s.W_ff]); keep["wrec"] = b.ptr_array([x.data_ptr() for x in s.W_rec])
    keep["gff"] = b.ptr_array([x.data_ptr() for x in s.dW_ff]); keep["grec"] = b.ptr_array([x.data_ptr() for x in s.dW_rec])
    a.W_ff, a.W_rec, a.W_out = keep["wff"], keep["wrec"], s.W_out.data_ptr()
    a.dW_ff, a.dW_rec, a.dW_out = keep["gff"], keep["grec"], s.dW_out.data_ptr()
    a.device_ws, a.device_ws_bytes = None, 0           # not used by the static entry point
    if s.pinned_ws is not None:
        a.pinned_ws, a.pinned_ws_bytes = s.pinned_ws.data_ptr(), s.pinned_ws.numel()
    a.main_stream, a.side_stream = s.main.cuda_stream, s.side.cuda_stream
    a.ckpt, a.max_activity, a.flags = b.snn_ckpt(strategy, K, R), 1.0, 0
    return a


def test_static_workspace_step_matches_the_ordinary_step(orc32):
    from paper_2412_11810_b200 import binding as b
    w = wl.small(sizes=(40, 260, 132, 6), T=21, B=5, p_in=0.1, g_ff=(2.5, 1.6), seed=13)
    d = wl.make(w)
    oracle_ref = run_oracle(orc32, w, d)
    s, bits, targets = make_session(w, d)
    for strategy, K, R in ((b.SNN_STANDARD, 0, 0), (b.SNN_DOUBLE, 2, 8)):
        # the ordinary entry point, workspace from torch
        loss_ref = s.train_step(bits, targets, strategy=strategy, chunk_size=K, remote_chunk_size=R, max_activity=1.0)
        ref = [g.clone() for g in s.dW_ff + s.dW_rec + [s.dW_out]]
        assert all(float(g.abs().max()) > 0 for g in ref)
        keep = {}
        a = _args(b, s, w, bits, targets, strategy, K, R, keep)
        for call in range(2):
            for g in s.dW_ff + s.dW_rec + [s.dW_out]:
                g.fill_(float("nan"))
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            loss = b.snn_train_step_static(s.net, a)
            if call == 1:   # the first call may still create a few CUDA events; the second must reserve nothing
                assert torch.cuda.mem_get_info()[0] == free_before
            assert np.float32(loss).view(np.uint32) == np.float32(loss_ref).view(np.uint32)
            for got, want in zip(s.dW_ff + s.dW_rec + [s.dW_out], ref):
                assert torch.equal(got.view(torch.int32), want.view(torch.int32)), (strategy, call)
        # and against the CPU oracle, once per strategy
        assert abs(loss - oracle_ref["loss"]) <= 1e-5 * max(1.0, abs(oracle_ref["loss"]))
        assert_grads_close(s.gradients(), oracle_ref)
    s.close()


def test_static_workspace_rejects_steps_that_do_not_fit():
    from paper_2412_11810_b200 import binding as b
    w = wl.small(sizes=(64, 1024, 1024, 8), T=4000, B=8, p_in=0.05)
    net = b.snn_create(list(w.sizes), 20.0, 1.0)
    need, _ = b.snn_workspace_query(net, w.T, w.B, b.snn_ckpt(b.SNN_STANDARD, 0, 0), 0.25)
    assert need > b.SNN_STATIC_WORKSPACE_BYTES
    a = b.snn_step_args()
    a.T, a.B, a.max_activity = w.T, w.B, 0.25
    loss = C.c_float()
    assert b.lib.snn_train_step_static(net, C.byref(a), C.byref(loss)) == b.SNN_ERR_WORKSPACE_TOO_SMALL
    assert "built-in workspace" in b.snn_last_error(net)
    b.snn_destroy(net)
