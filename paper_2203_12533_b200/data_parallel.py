"""Data-parallel replicas inside one NVLink domain (one process per GPU).

Section 5.3 of the paper trains a decoder-only model data parallel over two islands: each island
computes gradients, the islands exchange them, each applies them and starts the next step.  Here a
replica is a GPU.  Every replica keeps all parameter gradients in ONE flat fp32 buffer and all bf16
parameters in ONE flat bf16 buffer, both mapped into every other replica, and `reduce_apply` runs
the library's fused kernel: each replica sums its slice of every replica's gradients straight from
peer memory, steps its slice of the fp32 master copy, and stores the new bf16 values into every
replica's parameter buffer.  This module is host plumbing only (buffer layout, handle exchange,
ordering); the arithmetic is in the kernel.

`torch.distributed` carries the 64-byte buffer handles and the ordering: with the NCCL backend the
barrier is a one-element all-reduce on the compute stream (no host synchronisation); with any other
backend it is a stream synchronize followed by a host barrier.
"""
from __future__ import annotations

import torch


def plan_arena(shapes, align: int = 8):
    """Element offsets of tensors laid out back to back, each starting on a multiple of `align`
    elements (16 bytes of bf16).  Returns (offsets, total)."""
    offsets, at = [], 0
    for shp in shapes:
        n = 1
        for s in shp:
            n *= int(s)
        offsets.append(at)
        at += -(-n // align) * align
    return offsets, at


class _DeviceSpan:
    """Exposes a raw device address to torch through the CUDA array interface (zero copy)."""

    def __init__(self, ptr: int, numel: int, typestr: str):
        self.__cuda_array_interface__ = {"shape": (numel,), "typestr": typestr, "data": (ptr, False), "version": 2}


def tensor_at(ptr: int, numel: int, dtype, device):
    if dtype == torch.bfloat16:
        return torch.as_tensor(_DeviceSpan(ptr, numel, "<i2"), device=device).view(torch.bfloat16)
    assert dtype == torch.float32
    return torch.as_tensor(_DeviceSpan(ptr, numel, "<f4"), device=device)


class _Library:
    """The calls this module needs from the binding (replaced by a fake in the CPU tests)."""

    def __init__(self):
        from . import binding
        self.b = binding

    def shared_alloc(self, nbytes): return self.b.shared_alloc(nbytes)
    def shared_free(self, ptr): self.b.shared_free(ptr)
    def shared_open(self, handle): return self.b.shared_open(handle)
    def shared_close(self, ptr): self.b.shared_close(ptr)
    def dp_slice(self, n, world, rank): return self.b.dp_slice(n, world, rank)
    def dp_reduce_apply(self, *a, **k): self.b.dp_reduce_apply(*a, **k)
    def tensor_at(self, ptr, numel, dtype, device): return tensor_at(ptr, numel, dtype, device)
    def empty_master(self, numel, device): return torch.empty(max(numel, 1), dtype=torch.float32, device=device)

    def synchronize(self, device, stream=None):
        if stream is not None:
            stream.synchronize()
        else:
            torch.cuda.synchronize(device)


class Replica:
    """One data-parallel replica: owns the flat gradient / parameter buffers of this process, maps the
    other replicas', and applies the summed gradients.

        rep = Replica(shapes, device)              # after torch.distributed is initialised (or alone)
        rep.params[i].copy_(initial values)        # identical on every replica
        ... backward writes rep.grads[i] ...
        rep.reduce_apply(lr)                       # first call: init_master=True
        rep.close()
    """

    def __init__(self, shapes, device, group=None, library=None):
        import torch.distributed as dist
        self.lib = library or _Library()
        self.device = device
        self.group = group
        self.dist = dist if dist.is_available() and dist.is_initialized() else None
        self.rank = self.dist.get_rank(group) if self.dist else 0
        self.world = self.dist.get_world_size(group) if self.dist else 1
        self.shapes = [tuple(int(s) for s in shp) for shp in shapes]
        self.offsets, self.total = plan_arena(self.shapes)
        self.lo, self.hi = self.lib.dp_slice(self.total, self.world, self.rank)
        self._grad_ptr, grad_handle = self.lib.shared_alloc(self.total * 4)
        self._param_ptr, param_handle = self.lib.shared_alloc(self.total * 2)
        self.flat_grad = self.lib.tensor_at(self._grad_ptr, self.total, torch.float32, device)
        self.flat_param = self.lib.tensor_at(self._param_ptr, self.total, torch.bfloat16, device)
        self.flat_grad.zero_()
        self.flat_param.zero_()
        self.master = self.lib.empty_master(self.hi - self.lo, device)
        numel = lambda shp: int(torch.Size(shp).numel())
        self.grads = [self.flat_grad[o:o + numel(s)].view(s) for o, s in zip(self.offsets, self.shapes)]
        self.params = [self.flat_param[o:o + numel(s)].view(s) for o, s in zip(self.offsets, self.shapes)]
        # every replica learns every other replica's two handles, in rank order
        mine = (self.rank, grad_handle, param_handle, self.total)
        everyone = [mine]
        if self.world > 1:
            everyone = [None] * self.world
            self.dist.all_gather_object(everyone, mine, group=group)
        self.grad_ptrs, self.param_ptrs, self._opened = [], [], []
        for k, (r, gh, ph, total) in enumerate(everyone):
            if r != k or total != self.total:
                raise RuntimeError(f"replica {k} reported rank {r} / {total} elements; expected {k} / {self.total}")
            if k == self.rank:
                self.grad_ptrs.append(self._grad_ptr)
                self.param_ptrs.append(self._param_ptr)
            else:
                g, p = self.lib.shared_open(gh), self.lib.shared_open(ph)
                self._opened += [g, p]
                self.grad_ptrs.append(g)
                self.param_ptrs.append(p)
        self._token = None
        self._nccl = bool(self.dist) and self.world > 1 and self.dist.get_backend(group) == "nccl"
        self._closed = False

    def order(self, stream=None):
        """Everything every replica enqueued before this point happens before anything any replica
        enqueues after it."""
        if self.world == 1:
            return
        if self._nccl:
            if self._token is None:
                self._token = torch.zeros(1, device=self.device)
            if stream is not None:
                with torch.cuda.stream(stream):
                    self.dist.all_reduce(self._token, group=self.group)
            else:
                self.dist.all_reduce(self._token, group=self.group)
        else:
            self.lib.synchronize(self.device, stream)
            self.dist.barrier(group=self.group)

    def reduce_apply(self, lr, grad_scale=None, init_master=False, stream=None):
        """params <- params - lr * grad_scale * (sum of every replica's grads); grad_scale defaults to
        1 / world (the mean over replicas)."""
        if grad_scale is None:
            grad_scale = 1.0 / self.world
        self.order(stream)                         # every replica's gradients are complete
        self.lib.dp_reduce_apply(self.rank, self.grad_ptrs, self.param_ptrs, self.master, self.total, lr, grad_scale,
                                 init_master=init_master, stream=stream)
        self.order(stream)                         # every replica's slice has landed everywhere

    def close(self):
        if self._closed:
            return
        self._closed = True
        self.lib.synchronize(self.device)
        if self.dist and self.world > 1:
            self.dist.barrier(group=self.group)    # nobody still uses a mapping
        for ptr in self._opened:
            self.lib.shared_close(ptr)
        if self.dist and self.world > 1:
            self.dist.barrier(group=self.group)    # every mapping is closed before any owner frees
        self.grads = self.params = None
        self.flat_grad = self.flat_param = None
        self.lib.shared_free(self._grad_ptr)
        self.lib.shared_free(self._param_ptr)
