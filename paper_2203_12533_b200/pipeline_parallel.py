"""Pipeline stages on different GPUs of one NVLink domain (one process per stage).

Section 5.3 of the paper runs the decoder as S pipeline stages with M micro-batches (GPipe
schedule); the output of stage k lands directly in stage k+1's input buffers.  Here a stage is a
process with its own GPU and a run of consecutive layers.  Every stage owns two inbound buffers
that its neighbours map: `x_in[m]` (written by the previous stage's last forward kernel) and
`dy_in[m]` (written by the next stage's last backward kernel).  The hand-off is therefore not a
copy: the producing kernel's stores go straight to the consumer's memory, because the layer calls
take any device pointer as their output.  This module is host plumbing only (buffers, handle
exchange, order of calls and signals); every arithmetic step is a `pw_layer_fwd` / `pw_layer_bwd`.

Signals: after the kernels that fill a neighbour's buffer are enqueued, the producer sends a token
and the consumer receives it before it enqueues the kernels that read the buffer - NCCL send/recv
on the compute stream (no host synchronisation) with the NCCL backend, stream synchronize + a host
send/recv otherwise.  No kernel waits on another kernel.
"""
from __future__ import annotations

import torch

from .data_parallel import _Library


class PipelineStage:
    """Stage `rank` of `world`: `n_layers` consecutive layers, `n_micro` micro-batches, GPipe order.

        st = PipelineStage(layer, n_layers, n_micro, device)
        st.x_in[m].copy_(...)        # stage 0 only: the micro-batch inputs
        st.dy_in[m].copy_(...)       # last stage only: gradient of the loss w.r.t. its output
        st.run(params, grads)        # all forwards, then all backwards
        st.y_out[m], st.dx_out[m]    # last stage's outputs / stage 0's input gradients
    """

    def __init__(self, layer, n_layers, n_micro, device, group=None, library=None):
        import torch.distributed as dist
        self.lib = library or _Library()
        self.layer, self.L, self.M, self.device, self.group = layer, n_layers, n_micro, device, group
        self.dist = dist if dist.is_available() and dist.is_initialized() else None
        self.rank = self.dist.get_rank(group) if self.dist else 0
        self.world = self.dist.get_world_size(group) if self.dist else 1
        T, d = layer.T, layer.d
        self.act_elems = T * d
        act_bytes = self.act_elems * 2
        self._x_ptr, xh = self.lib.shared_alloc(n_micro * act_bytes)
        self._dy_ptr, dyh = self.lib.shared_alloc(n_micro * act_bytes)
        view = lambda ptr: [self.lib.tensor_at(ptr + m * act_bytes, self.act_elems, torch.bfloat16, device).view(T, d)
                            for m in range(n_micro)]
        self.x_in, self.dy_in = view(self._x_ptr), view(self._dy_ptr)
        mine = (self.rank, xh, dyh, self.act_elems, n_micro)
        everyone = [mine]
        if self.world > 1:
            everyone = [None] * self.world
            self.dist.all_gather_object(everyone, mine, group=group)
        for k, info in enumerate(everyone):
            if info[0] != k or info[3:] != mine[3:]:
                raise RuntimeError(f"stage {k} reported {info[0]}, {info[3:]}; expected {k}, {mine[3:]}")
        self._opened = []
        self.is_first, self.is_last = self.rank == 0, self.rank == self.world - 1
        if self.is_last:
            self.y_out = [torch.empty((T, d), dtype=torch.bfloat16, device=device) for _ in range(n_micro)]
            self._y_ptrs = [t.data_ptr() for t in self.y_out]
        else:
            base = self.lib.shared_open(everyone[self.rank + 1][1])          # the next stage's x_in
            self._opened.append(base)
            self.y_out, self._y_ptrs = None, [base + m * act_bytes for m in range(n_micro)]
        if self.is_first:
            self.dx_out = [torch.empty((T, d), dtype=torch.bfloat16, device=device) for _ in range(n_micro)]
            self._dx_ptrs = [t.data_ptr() for t in self.dx_out]
        else:
            base = self.lib.shared_open(everyone[self.rank - 1][2])          # the previous stage's dy_in
            self._opened.append(base)
            self.dx_out, self._dx_ptrs = None, [base + m * act_bytes for m in range(n_micro)]
        # what the stage keeps between its forwards and its backwards
        self.ctx = [[torch.empty(layer.ctx_bytes, dtype=torch.uint8, device=device) for _ in range(n_micro)] for _ in range(n_layers)]
        self.mid = [[torch.empty((T, d), dtype=torch.bfloat16, device=device) for _ in range(n_micro)] for _ in range(n_layers - 1)]
        self.scratch = torch.empty(layer.scratch_bytes, dtype=torch.uint8, device=device)
        self.dtmp = [torch.empty((T, d), dtype=torch.bfloat16, device=device) for _ in range(2)]
        self._nccl = bool(self.dist) and self.world > 1 and self.dist.get_backend(group) == "nccl"
        self._token = torch.zeros(1, device=device) if self._nccl else torch.zeros(1)
        self.signals = []                                                     # (kind, peer) in order: for the tests
        self._closed = False

    # -- ordering between neighbours --
    def _signal(self, peer, stream):
        if peer < 0 or peer >= self.world:
            return
        self.signals.append(("send", peer))
        if self._nccl:
            with torch.cuda.stream(stream):
                self.dist.send(self._token, peer, group=self.group)
        else:
            self.lib.synchronize(self.device, stream)
            self.dist.send(self._token, peer, group=self.group)

    def _wait(self, peer, stream):
        if peer < 0 or peer >= self.world:
            return
        self.signals.append(("recv", peer))
        if self._nccl:
            with torch.cuda.stream(stream):
                self.dist.recv(self._token, peer, group=self.group)
        else:
            self.dist.recv(self._token, peer, group=self.group)

    def run(self, params, grads, stream=None):
        """All M forwards, then all M backwards (GPipe).  grads receive the sum over micro-batches."""
        L, M, layer = self.L, self.M, self.layer
        assert len(params) == L and len(grads) == L
        stream = stream or torch.cuda.current_stream(self.device)
        x_of = lambda l, m: self.x_in[m] if l == 0 else self.mid[l - 1][m]
        for m in range(M):
            self._wait(self.rank - 1, stream)                                 # x_in[m] has landed
            for l in range(L):
                y = self.mid[l][m] if l < L - 1 else self._y_ptrs[m]
                layer.fwd(params[l], x_of(l, m), y, self.ctx[l][m], self.scratch, stream=stream)
            self._signal(self.rank + 1, stream)
        for m in range(M):
            self._wait(self.rank + 1, stream)                                 # dy_in[m] has landed
            dy = self.dy_in[m]
            for l in range(L - 1, -1, -1):
                dx = self.dtmp[l & 1] if l > 0 else self._dx_ptrs[m]
                layer.bwd(params[l], x_of(l, m), dy, dx, grads[l], m > 0, self.ctx[l][m], self.scratch, stream=stream)
                dy = dx
            self._signal(self.rank - 1, stream)

    def close(self):
        if self._closed:
            return
        self._closed = True
        self.lib.synchronize(self.device)
        if self.dist and self.world > 1:
            self.dist.barrier(group=self.group)
        for ptr in self._opened:
            self.lib.shared_close(ptr)
        if self.dist and self.world > 1:
            self.dist.barrier(group=self.group)
        self.x_in = self.dy_in = None
        self.lib.shared_free(self._x_ptr)
        self.lib.shared_free(self._dy_ptr)
