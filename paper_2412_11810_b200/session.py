"""Device buffers, streams and argument marshalling around the C ABI (no arithmetic here).

A Session owns the torch tensors a train step needs (weights, gradients, the two workspaces,
two CUDA streams) and fills `snn_step_args`.  Every step of the method runs inside
libsnnckpt.so.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as sb


class Session:
    def __init__(self, sizes: Sequence[int], tau_mem: float = 20.0, threshold: float = 1.0,
                 surrogate: int = sb.SNN_SURR_FAST_SIGMOID, surrogate_beta: float = 10.0,
                 cell: int = sb.SNN_CELL_LIF, readout_scale: float = 1.0, device: str = "cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: this library has no CPU path")
        self.sizes = [int(s) for s in sizes]
        self.L = len(self.sizes) - 2
        self.cell = cell
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.net = sb.snn_create(self.sizes, tau_mem, threshold, surrogate, surrogate_beta, cell, readout_scale)
        self.main = torch.cuda.Stream(device=self.device)
        self.side = torch.cuda.Stream(device=self.device)
        self.W_ff: List[torch.Tensor] = []
        self.W_rec: List[torch.Tensor] = []
        self.W_out: Optional[torch.Tensor] = None
        self.dW_ff: List[torch.Tensor] = []
        self.dW_rec: List[torch.Tensor] = []
        self.dW_out: Optional[torch.Tensor] = None
        self.device_ws: Optional[torch.Tensor] = None
        self.pinned_ws: Optional[torch.Tensor] = None
        self.debug_V: Optional[List[torch.Tensor]] = None
        self._last = None

    def close(self):
        if self.net is not None:
            torch.cuda.synchronize(self.device)
            sb.snn_destroy(self.net)
            self.net = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- parameters ------------------------------------------------------------------------
    def set_weights(self, W_ff, W_rec, W_out):
        dev = self.device
        self.W_ff = [torch.as_tensor(np.ascontiguousarray(w, np.float32)).to(dev) for w in W_ff]
        self.W_rec = [torch.as_tensor(np.ascontiguousarray(w, np.float32)).to(dev) for w in W_rec]
        self.W_out = torch.as_tensor(np.ascontiguousarray(W_out, np.float32)).to(dev)
        for l in range(self.L):
            assert tuple(self.W_ff[l].shape) == (self.sizes[l], self.sizes[l + 1])
            assert tuple(self.W_rec[l].shape) == (self.sizes[l + 1], self.sizes[l + 1])
        assert tuple(self.W_out.shape) == (self.sizes[-2], self.sizes[-1])
        self.dW_ff = [torch.empty_like(w) for w in self.W_ff]
        self.dW_rec = [torch.empty_like(w) for w in self.W_rec]
        self.dW_out = torch.empty_like(self.W_out)

    def ckpt(self, strategy: int, chunk_size: int = 0, remote_chunk_size: int = 0, nb_local: int = 0) -> sb.snn_ckpt:
        return sb.snn_ckpt(strategy, chunk_size, remote_chunk_size, nb_local)

    def ensure_workspace(self, T: int, B: int, ck: sb.snn_ckpt, max_activity: float, flags: int = 0):
        d, p = sb.snn_workspace_query(self.net, T, B, ck, max_activity, flags)
        if self.device_ws is None or self.device_ws.numel() < d:
            self.device_ws = None
            self.device_ws = torch.empty(d, dtype=torch.uint8, device=self.device)
        if p > 0 and (self.pinned_ws is None or self.pinned_ws.numel() < p):
            self.pinned_ws = None
            self.pinned_ws = torch.empty(p, dtype=torch.uint8, pin_memory=True)
        return d, p

    # ---- the training step -----------------------------------------------------------------
    def train_step(self, input_bits, targets, strategy: int = sb.SNN_STANDARD, chunk_size: int = 0,
                   remote_chunk_size: int = 0, max_activity: float = 0.25, forward_only: bool = False,
                   keep_V: bool = False, time_phases: bool = False, nb_local: int = 0,
                   extra_flags: int = 0) -> float:
        """input_bits: uint32 [T][B][ceil(N_0/32)] spike words (LIF cell; int32 storage) or float32
        [T][B][N_0] dense values (graded cell), as a CUDA tensor or as a pinned host tensor / numpy
        array (then it is copied to the device inside the call); targets alike."""
        on_host = not (isinstance(input_bits, torch.Tensor) and input_bits.is_cuda)
        if on_host:
            if not isinstance(input_bits, torch.Tensor):
                arr = np.ascontiguousarray(input_bits)
                arr = arr.astype(np.float32, copy=False) if self.cell == sb.SNN_CELL_GRADED else arr.view(np.int32)
                input_bits = torch.from_numpy(arr).pin_memory()
            if not isinstance(targets, torch.Tensor):
                targets = torch.from_numpy(np.ascontiguousarray(targets, np.int32)).pin_memory()
        T, B = int(input_bits.shape[0]), int(input_bits.shape[1])
        ck = self.ckpt(strategy, chunk_size, remote_chunk_size, nb_local)
        flags = (sb.SNN_FLAG_INPUT_ON_HOST if on_host else 0) | (sb.SNN_FLAG_FORWARD_ONLY if forward_only else 0) \
            | (sb.SNN_FLAG_TIME_PHASES if time_phases else 0) | extra_flags
        self.ensure_workspace(T, B, ck, max_activity, flags)
        dbg = None
        if keep_V:
            self.debug_V = [torch.zeros((T + 1, B, self.sizes[l + 1]), dtype=torch.float32, device=self.device)
                            for l in range(self.L)]
            dbg = sb.ptr_array([t.data_ptr() for t in self.debug_V])
        a = sb.snn_step_args()
        a.T, a.B = T, B
        fmt = sb.SNN_INPUT_DENSE if self.cell == sb.SNN_CELL_GRADED else sb.SNN_INPUT_BITS
        a.input, a.input_format, a.targets = input_bits.data_ptr(), fmt, targets.data_ptr()
        wff = sb.ptr_array([w.data_ptr() for w in self.W_ff]); wrec = sb.ptr_array([w.data_ptr() for w in self.W_rec])
        gff = sb.ptr_array([w.data_ptr() for w in self.dW_ff]); grec = sb.ptr_array([w.data_ptr() for w in self.dW_rec])
        a.W_ff, a.W_rec, a.W_out = wff, wrec, self.W_out.data_ptr()
        a.dW_ff, a.dW_rec, a.dW_out = gff, grec, self.dW_out.data_ptr()
        a.device_ws, a.device_ws_bytes = self.device_ws.data_ptr(), self.device_ws.numel()
        if self.pinned_ws is not None:
            a.pinned_ws, a.pinned_ws_bytes = self.pinned_ws.data_ptr(), self.pinned_ws.numel()
        a.main_stream, a.side_stream = self.main.cuda_stream, self.side.cuda_stream
        a.ckpt, a.max_activity, a.flags = ck, max_activity, flags
        if dbg is not None:
            a.debug_V = dbg
        self._last = (T, B, input_bits, targets)   # keep inputs alive until the call returns
        torch.cuda.current_stream(self.device).synchronize()
        return sb.snn_train_step(self.net, a)

    # ---- inspection ------------------------------------------------------------------------
    def gradients(self):
        return ([g.cpu().numpy() for g in self.dW_ff], [g.cpu().numpy() for g in self.dW_rec],
                self.dW_out.cpu().numpy())

    def events(self, layer: int):
        """Event lists of the last step for layer 0 (input) .. L: (offsets [T+2][B], pool [B][cap])
        as numpy uint32 arrays."""
        T, B, _, _ = self._last
        e = sb.snn_get_event_layout(self.net, layer)
        ws = self.device_ws
        off = ws[e.offsets_off:e.offsets_off + 4 * (T + 2) * B].view(torch.int32).cpu().numpy().view(np.uint32)
        pool = ws[e.pool_off:e.pool_off + 4 * B * e.pool_capacity].view(torch.int32).cpu().numpy().view(np.uint32)
        return off.reshape(T + 2, B), pool.reshape(B, e.pool_capacity)

    def spike_words(self, layer: int):
        """Spike words of hidden layer 1..L of the last step: uint32 [T+1][B][words]."""
        T, B, _, _ = self._last
        e = sb.snn_get_event_layout(self.net, layer)
        n = 4 * (T + 1) * B * e.mask_words
        m = self.device_ws[e.mask_off:e.mask_off + n].view(torch.int32).cpu().numpy().view(np.uint32)
        return m.reshape(T + 1, B, e.mask_words)

    def peak_memory(self):
        return sb.snn_peak_memory(self.net)

    def phase_times(self) -> dict:
        return sb.snn_phase_times_get(self.net)

    def stats(self) -> sb.snn_memory_stats:
        return sb.snn_memory_stats_get(self.net)
