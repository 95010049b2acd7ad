"""ctypes binding of libsnnckpt.so: the same names and arguments as include/snn.h.

Argument marshalling only.  PyTorch appears here for device / pinned memory and streams.
Importing this module fails loudly when the CUDA library has not been built: there is no
CPU fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
# SNN_DEBUG_CHECKS=1 in the environment selects the bounds-checked build of the same sources
LIB_PATH = os.path.join(HERE, "libsnnckpt_debug.so" if os.environ.get("SNN_DEBUG_CHECKS") == "1" else "libsnnckpt.so")

SNN_OK, SNN_ERR_INVALID_ARG, SNN_ERR_WORKSPACE_TOO_SMALL, SNN_ERR_EVENT_OVERFLOW = 0, 1, 2, 3
SNN_ERR_DEVICE_TIMEOUT, SNN_ERR_CUDA, SNN_ERR_UNSUPPORTED, SNN_ERR_DEBUG_CHECK = 4, 5, 6, 7
SNN_STANDARD, SNN_CHUNK, SNN_REMOTE, SNN_DOUBLE, SNN_HIERARCHICAL, SNN_DOUBLE_LOCAL = 0, 1, 2, 3, 4, 5
SNN_CELL_LIF, SNN_CELL_GRADED = 0, 1
SNN_SURR_FAST_SIGMOID, SNN_SURR_SIGMOID, SNN_SURR_TRIANGLE = 0, 1, 2
SNN_INPUT_BITS, SNN_INPUT_DENSE = 0, 1
SNN_FLAG_INPUT_ON_HOST, SNN_FLAG_FORWARD_ONLY, SNN_FLAG_TIME_PHASES = 1, 2, 4
SNN_FLAG_BACKWARD_LAYER_BY_LAYER, SNN_FLAG_BACKWARD_WAVEFRONT = 8, 16
SNN_FLAG_REFORWARD_PER_STEP = 32
SNN_FLAG_FORWARD_PER_STEP = 64
SNN_FLAG_FORWARD_STREAM_WEIGHTS = 128
SNN_FLAG_BACKWARD_PER_STEP = 256
SNN_FLAG_REFORWARD_ROWS = 512
SNN_FLAG_FF_PRODUCT_MMA_SYNC = 1024
SNN_FLAG_SPILL_EVENTS = 2048
SNN_FLAG_BACKWARD_EVENT_DRIVEN = 4096
SNN_FLAG_WEIGHT_GRADIENT_GATHER = 8192
SNN_FLAG_WEIGHT_GRADIENT_SLAB = 16384
PHASE_NAMES = ["fwd", "refwd1", "refwd2", "bwd", "dw", "readout", "d2h", "h2d", "ffgemm"]
SNN_OP_FWD, SNN_OP_REFWD1, SNN_OP_REFWD2, SNN_OP_BWD, SNN_OP_D2H, SNN_OP_H2D, SNN_OP_ZERO = range(7)
STRATEGY_NAMES = {SNN_STANDARD: "standard", SNN_CHUNK: "chunk", SNN_REMOTE: "remote", SNN_DOUBLE: "double",
                  SNN_HIERARCHICAL: "hierarchical", SNN_DOUBLE_LOCAL: "double_local"}

EXPORTS = ["snn_create", "snn_destroy", "snn_alpha", "snn_workspace_query", "snn_workspace_query_flags", "snn_train_step", "snn_peak_memory",
           "snn_memory_stats_get", "snn_last_error", "snn_plan", "snn_compact_spikes", "snn_get_event_layout",
           "snn_phase_times_get", "snn_train_step_static", "snn_suggest_ckpt", "snn_selftest_wait_timeout",
           "snn_debug_checks_enabled"]
SNN_STATIC_WORKSPACE_BYTES = 32 << 20


class snn_config(C.Structure):
    _fields_ = [("n_sizes", C.c_int32), ("sizes", C.POINTER(C.c_int32)), ("tau_mem", C.c_float),
                ("threshold", C.c_float), ("surrogate", C.c_int32), ("surrogate_beta", C.c_float),
                ("cell", C.c_int32), ("readout_scale", C.c_float)]


class snn_ckpt(C.Structure):
    _fields_ = [("strategy", C.c_int32), ("chunk_size", C.c_int32), ("remote_chunk_size", C.c_int32),
                ("nb_local", C.c_int32)]


class snn_step_args(C.Structure):
    _fields_ = [("T", C.c_int32), ("B", C.c_int32), ("input", C.c_void_p), ("input_format", C.c_int32),
                ("targets", C.c_void_p), ("W_ff", C.POINTER(C.c_void_p)), ("W_rec", C.POINTER(C.c_void_p)),
                ("W_out", C.c_void_p), ("dW_ff", C.POINTER(C.c_void_p)), ("dW_rec", C.POINTER(C.c_void_p)),
                ("dW_out", C.c_void_p), ("device_ws", C.c_void_p), ("device_ws_bytes", C.c_size_t),
                ("pinned_ws", C.c_void_p), ("pinned_ws_bytes", C.c_size_t), ("main_stream", C.c_void_p),
                ("side_stream", C.c_void_p), ("ckpt", snn_ckpt), ("max_activity", C.c_float),
                ("flags", C.c_uint32), ("debug_V", C.POINTER(C.c_void_p))]


class snn_memory_stats(C.Structure):
    _fields_ = [("state_bytes", C.c_size_t), ("local_state_slots", C.c_int32), ("remote_state_slots", C.c_int32),
                ("d2h_copies", C.c_int32), ("h2d_copies", C.c_int32), ("kernel_launches", C.c_int32),
                ("event_bytes", C.c_size_t), ("event_window_copies", C.c_int32)]


class snn_phase_times(C.Structure):
    _fields_ = [("ms", C.c_float * 9), ("launches", C.c_int32 * 9)]


class snn_op(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("kind", "t0", "t1", "in_slot", "buf_slot", "buf_len", "keep_every",
                                         "keep_slot", "remote_slot")]


class snn_event_layout(C.Structure):
    _fields_ = [("offsets_off", C.c_size_t), ("pool_off", C.c_size_t), ("values_off", C.c_size_t),
                ("pool_capacity", C.c_size_t), ("mask_off", C.c_size_t), ("mask_words", C.c_int32)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python paper_2412_11810_b200/build.py` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    lib.snn_create.argtypes = [C.POINTER(snn_config), C.POINTER(C.c_void_p)]
    lib.snn_destroy.argtypes = [C.c_void_p]
    lib.snn_destroy.restype = None
    lib.snn_alpha.argtypes = [C.c_void_p]
    lib.snn_alpha.restype = C.c_float
    lib.snn_debug_checks_enabled.argtypes = []
    lib.snn_debug_checks_enabled.restype = C.c_int32
    lib.snn_workspace_query.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(snn_ckpt), C.c_float,
                                        C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    lib.snn_workspace_query_flags.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(snn_ckpt), C.c_float,
                                              C.c_uint32, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    lib.snn_train_step.argtypes = [C.c_void_p, C.POINTER(snn_step_args), C.POINTER(C.c_float)]
    lib.snn_train_step_static.argtypes = [C.c_void_p, C.POINTER(snn_step_args), C.POINTER(C.c_float)]
    lib.snn_peak_memory.argtypes = [C.c_void_p, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    lib.snn_memory_stats_get.argtypes = [C.c_void_p, C.POINTER(snn_memory_stats)]
    lib.snn_last_error.argtypes = [C.c_void_p]
    lib.snn_last_error.restype = C.c_char_p
    lib.snn_plan.argtypes = [C.c_int32, C.POINTER(snn_ckpt), C.POINTER(snn_op), C.c_int32, C.POINTER(C.c_int32),
                             C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.snn_compact_spikes.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p,
                                       C.c_void_p]
    lib.snn_phase_times_get.argtypes = [C.c_void_p, C.POINTER(snn_phase_times)]
    lib.snn_suggest_ckpt.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_size_t, C.c_float,
                                     C.POINTER(snn_ckpt)]
    lib.snn_get_event_layout.argtypes = [C.c_void_p, C.c_int32, C.POINTER(snn_event_layout)]
    lib.snn_selftest_wait_timeout.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
    return lib


lib = _load()


class SnnError(RuntimeError):
    def __init__(self, status: int, message: str = ""):
        super().__init__(f"snn status {status}: {message}")
        self.status = status


def _check(st: int, net=None):
    if st != SNN_OK:
        msg = lib.snn_last_error(net).decode() if net else ""
        raise SnnError(st, msg)


def snn_create(sizes: Sequence[int], tau_mem: float, threshold: float, surrogate: int = SNN_SURR_FAST_SIGMOID,
               surrogate_beta: float = 10.0, cell: int = SNN_CELL_LIF, readout_scale: float = 1.0) -> C.c_void_p:
    arr = (C.c_int32 * len(sizes))(*[int(s) for s in sizes])
    cfg = snn_config(len(sizes), arr, tau_mem, threshold, surrogate, surrogate_beta, cell, readout_scale)
    net = C.c_void_p()
    _check(lib.snn_create(C.byref(cfg), C.byref(net)))
    return net


def snn_destroy(net) -> None:
    lib.snn_destroy(net)


def snn_alpha(net) -> float:
    return float(lib.snn_alpha(net))


def snn_workspace_query(net, T: int, B: int, ckpt: snn_ckpt, max_activity: float, flags: int = 0):
    d, p = C.c_size_t(), C.c_size_t()
    _check(lib.snn_workspace_query_flags(net, T, B, C.byref(ckpt), max_activity, flags, C.byref(d), C.byref(p)), net)
    return d.value, p.value


def snn_train_step(net, args: snn_step_args) -> float:
    loss = C.c_float()
    _check(lib.snn_train_step(net, C.byref(args), C.byref(loss)), net)
    return loss.value


def snn_train_step_static(net, args: snn_step_args) -> float:
    """snn_train_step on the library's built-in device workspace: for hosts that cannot allocate
    device memory themselves (args.device_ws is ignored).  See include/snn.h for the limits."""
    loss = C.c_float()
    _check(lib.snn_train_step_static(net, C.byref(args), C.byref(loss)), net)
    return loss.value


def snn_peak_memory(net):
    d, p = C.c_size_t(), C.c_size_t()
    _check(lib.snn_peak_memory(net, C.byref(d), C.byref(p)), net)
    return d.value, p.value


def snn_memory_stats_get(net) -> snn_memory_stats:
    s = snn_memory_stats()
    _check(lib.snn_memory_stats_get(net, C.byref(s)), net)
    return s


def snn_phase_times_get(net) -> dict:
    """{phase name: (milliseconds, kernel launches)} of the last step run with SNN_FLAG_TIME_PHASES."""
    p = snn_phase_times()
    _check(lib.snn_phase_times_get(net, C.byref(p)), net)
    return {n: (float(p.ms[i]), int(p.launches[i])) for i, n in enumerate(PHASE_NAMES)}


def snn_last_error(net) -> str:
    return lib.snn_last_error(net).decode()


def snn_plan(T: int, ckpt: snn_ckpt):
    """Returns (ops, n_local_slots, n_remote_slots); ops is a list of snn_op."""
    n, nl, nr = C.c_int32(), C.c_int32(), C.c_int32()
    _check(lib.snn_plan(T, C.byref(ckpt), None, 0, C.byref(n), C.byref(nl), C.byref(nr)))
    ops = (snn_op * n.value)()
    _check(lib.snn_plan(T, C.byref(ckpt), ops, n.value, C.byref(n), C.byref(nl), C.byref(nr)))
    return list(ops), nl.value, nr.value


def snn_suggest_ckpt(net, T: int, B: int, strategy: int, device_budget_bytes: int = 0,
                     max_activity: float = 0.25) -> snn_ckpt:
    """Checkpoint intervals by the paper's rules of thumb (host only; net may be None except for REMOTE
    with a budget)."""
    c = snn_ckpt()
    _check(lib.snn_suggest_ckpt(net, T, B, strategy, device_budget_bytes, max_activity, C.byref(c)), net)
    return c


def snn_compact_spikes(masks_ptr: int, n_rows: int, n_words: int, idx_out_ptr: int, capacity: int,
                       count_out_ptr: int, stream: int = 0) -> None:
    _check(lib.snn_compact_spikes(masks_ptr, n_rows, n_words, idx_out_ptr, capacity, count_out_ptr, stream))


def snn_selftest_wait_timeout(device_scratch_ptr: int, poll_limit: int, stream: int = 0) -> int:
    """Returns the status itself (SNN_ERR_DEVICE_TIMEOUT is the expected outcome)."""
    return lib.snn_selftest_wait_timeout(device_scratch_ptr, poll_limit, stream)


def snn_get_event_layout(net, layer: int) -> snn_event_layout:
    e = snn_event_layout()
    _check(lib.snn_get_event_layout(net, layer, C.byref(e)), net)
    return e


def ptr_array(ptrs: Sequence[Optional[int]]):
    return (C.c_void_p * len(ptrs))(*ptrs)
