"""Distributed Lion with one worker per process (one process per GPU).

The deployment the paper describes (Algorithm 1; Section 3.2 "Communication
Cost"): every worker keeps its own momentum, sends only its binary update to
the server, and receives the aggregated update back.  Here the server's work is
spread over the workers, the 1-bit analogue of reduce-scatter + all-gather:

  1. worker side, local             delta_r = sign(...), m_r <- ...      (d bits out)
  2. all-to-all of bit shards       rank r receives coordinate slice r of every worker
  3. vote on the slice, local       the broadcast message for slice r (1 or K bit planes)
  4. all-gather of the message      every rank now holds Delta for all d coordinates
  5. apply, local                   x <- x - eps (Delta + lambda x), the message read
                                    slice by slice where the all-gather put it

Per rank and step this moves d*(world-1)/world/8 bytes out in step 2 and
K*d*(world-1)/world/8 bytes in step 4 (K = 1 for Majority Vote,
ceil(log2(N+1)) for Averaging): Table 1 of the paper, against 4d bytes each way
for an fp32 gradient exchange.

Steps 1, 3 and 5 are three calls of the C ABI (``dlion_worker_step``,
``dlion_aggregate``, ``dlion_apply_delta_sliced``); steps 2 and 4 are
``torch.distributed`` collectives (NCCL on GPUs).  Received shards land in this
rank's own memory and are read with ordinary loads.  This module only
orchestrates; it holds no optimizer arithmetic.  The three local steps are
reached through a small ``kernels`` object so that the orchestration can be
exercised on CPU ranks (``gloo``) with a stand-in for the CUDA library.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist

ALIGN = 128


def padded_length(d_pad: int, world: int) -> int:
    """Arena length that splits into ``world`` equal slices of whole 128-coordinate groups."""
    q = ALIGN * world
    return (d_pad + q - 1) // q * q


class DlionKernels:
    """The three local steps on this rank's GPU through the CUDA library.

    Two contexts: one over the model's segment table with N = world workers (this rank steps
    worker ``rank`` of it, and applies the broadcast update), and a flat one over this rank's
    coordinate slice (the vote on the slice: padding between tensors is voted on too, which
    is harmless because the apply never touches padding)."""

    def __init__(self, segments, d_pad_x: int, world: int, rank: int, beta1: float, beta2: float,
                 lr: float, weight_decay: float, mode: int, gdtype: int):
        from . import dlion
        self.rank = rank
        slice_len = d_pad_x // world
        self.model = dlion.Dlion(segments, d_pad_x, world, beta1, beta2, lr, weight_decay, mode, gdtype)
        self.server = dlion.Dlion([(0, slice_len)], slice_len, world, beta1, beta2, lr, weight_decay,
                                  mode, gdtype)

    def delta_planes(self) -> int:
        return self.model.delta_planes()

    def set_lr(self, lr: float) -> None:
        self.model.set_lr(lr)

    def worker_step(self, g: torch.Tensor, m: torch.Tensor, packed: torch.Tensor) -> None:
        self.model.worker_step(self.rank, g, m, packed)

    def aggregate(self, packed_slices: torch.Tensor, wire_slice: torch.Tensor) -> None:
        self.server.aggregate(packed_slices, wire_slice)

    def apply_delta_sliced(self, gathered: torch.Tensor, slice_words: int, x: torch.Tensor) -> None:
        self.model.apply_delta_sliced(gathered, slice_words, x)

    # per-tensor mode: this rank's gradient / momentum / parameter tensors, stepped in place
    def bind_tensors(self, grads=None, m=None, x=None) -> None:
        """Each a list of this worker's tensors, one per segment (None: keep the binding)."""
        world = self.model.n_workers

        def rows(own):                                  # only worker `rank`'s row of the table is ever read
            return None if own is None else [list(own)] * world
        self.model.bind_tensors(grads=rows(grads), m=rows(m), x=x)

    def worker_step_tensors(self, packed: torch.Tensor) -> None:
        self.model.worker_step_tensors(self.rank, packed)

    def apply_delta_tensors(self, gathered: torch.Tensor, slice_words: int) -> None:
        self.model.apply_delta_tensors(gathered, slice_words)

    # scatter mode: the worker-side kernel stores its sign words into the ranks' receive buffers
    def bind_scatter(self, receive_buffers, slice_words: int, rows: int) -> None:
        self.model.bind_scatter(receive_buffers, slice_words, slot=self.rank, rows=rows)

    def worker_step_scatter(self, g: torch.Tensor, m: torch.Tensor) -> None:
        self.model.worker_step_scatter(self.rank, g, m)


class DistributedLion:
    """One rank of Distributed Lion.  ``g``, ``m``, ``x`` have ``d_pad_x`` elements
    (``padded_length(d_pad, world)``); ``m`` is this worker's own momentum.

    ``host_staged = True`` routes the two collectives through pinned host buffers (for
    process groups that only move host memory, such as gloo); the default hands the device
    buffers to the group's backend (NCCL).

    ``fused_send = True`` replaces the all-to-all: the receive buffer is allocated as
    symmetric memory (every rank's buffer mapped into every process), the worker-side
    kernel stores each sign word straight into the buffer of the rank that votes on it
    (``dlion_worker_step_scatter``: plain stores to peer memory, no multicast), and a
    barrier of the group orders the votes after all the stores.  The next step's stores
    cannot overtake this step's votes: a rank leaves the all-gather only after every rank
    has produced its part of the message, i.e. has finished reading its receive buffer.
    Exercised with one rank and, with the ranks emulated as buffers on one GPU, in the
    tests; it has not run on several GPUs."""

    def __init__(self, segments: Sequence[Tuple[int, int]], d_pad: int, mode: int, kernels=None,
                 beta1: float = 0.9, beta2: float = 0.99, lr: float = 1e-4, weight_decay: float = 0.0,
                 gdtype: int = 0, group: Optional[dist.ProcessGroup] = None,
                 device: Optional[torch.device] = None, host_staged: bool = False,
                 fused_send: bool = False):
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.mode = mode
        self.d_pad_x = padded_length(d_pad, self.world)
        self.words = self.d_pad_x // 32
        self.slice_words = self.words // self.world
        self.kernels = kernels if kernels is not None else DlionKernels(
            segments, self.d_pad_x, self.world, self.rank, beta1, beta2, lr, weight_decay, mode, gdtype)
        self.k = int(self.kernels.delta_planes())       # planes of the broadcast message, from the library
        dev = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        z = dict(dtype=torch.int32, device=dev)
        self.packed = torch.zeros(self.words, **z)                           # my delta, all coordinates
        self.recv = torch.zeros(self.world, self.slice_words, **z)           # everyone's delta, my slice
        self.wire_slice = torch.zeros(self.k, self.slice_words, **z)         # message for my slice
        # every slice's message, in the order the all-gather delivers them: [slice][plane][word]
        self.gathered = torch.zeros(self.world, self.k, self.slice_words, **z)
        self.fused_send = bool(fused_send)
        if self.fused_send:
            if host_staged:
                raise ValueError("fused_send stores into peer device memory: it cannot be host-staged")
            import torch.distributed._symmetric_memory as symm_mem
            self.recv = symm_mem.empty((self.world, self.slice_words), dtype=torch.int32, device=dev)
            self.recv.zero_()
            self._symm = symm_mem.rendezvous(self.recv, group if group is not None else dist.group.WORLD)
            self.kernels.bind_scatter([int(p) for p in self._symm.buffer_ptrs], self.slice_words, rows=self.world)
            dist.barrier(group=self.group)              # every buffer is zeroed before anyone stores into it
        self.host_staged = bool(host_staged) and dev.type == "cuda"
        if self.host_staged:
            h = dict(dtype=torch.int32, pin_memory=True)
            self.h_packed, self.h_recv = torch.zeros(self.words, **h), torch.zeros(self.words, **h)
            self.h_slice = torch.zeros(self.k * self.slice_words, **h)
            self.h_gathered = torch.zeros(self.world * self.k * self.slice_words, **h)

    def wire_bytes_per_step(self) -> Tuple[int, int]:
        """(bytes this rank sends in the all-to-all, bytes it receives in the all-gather)."""
        others = self.world - 1
        return others * self.slice_words * 4, others * self.k * self.slice_words * 4

    def _all_to_all(self) -> None:
        if not self.host_staged:
            dist.all_to_all_single(self.recv.view(-1), self.packed, group=self.group)
            return
        self.h_packed.copy_(self.packed)                 # ordered on the current stream, then waits
        dist.all_to_all_single(self.h_recv, self.h_packed, group=self.group)
        self.recv.view(-1).copy_(self.h_recv, non_blocking=True)

    def _all_gather(self) -> None:
        if not self.host_staged:
            dist.all_gather_into_tensor(self.gathered.view(-1), self.wire_slice.view(-1), group=self.group)
            return
        self.h_slice.copy_(self.wire_slice.view(-1))
        dist.all_gather_into_tensor(self.h_gathered, self.h_slice, group=self.group)
        self.gathered.view(-1).copy_(self.h_gathered, non_blocking=True)

    def step(self, g: torch.Tensor, m: torch.Tensor, x: torch.Tensor) -> None:
        if self.fused_send:
            self.kernels.worker_step_scatter(g, m)      # the send is part of the kernel
            dist.barrier(group=self.group)              # all stores have landed before anyone votes
        else:
            self.kernels.worker_step(g, m, self.packed)
            self._all_to_all()
        self.kernels.aggregate(self.recv, self.wire_slice)
        self._all_gather()
        self.kernels.apply_delta_sliced(self.gathered, self.slice_words, x)   # read where the all-gather put them

    def step_tensors(self) -> None:
        """The same step on the tensors bound with ``kernels.bind_tensors`` (per-tensor mode)."""
        self.kernels.worker_step_tensors(self.packed)
        self._all_to_all()
        self.kernels.aggregate(self.recv, self.wire_slice)
        self._all_gather()
        self.kernels.apply_delta_tensors(self.gathered, self.slice_words)


class LionOptimizer:
    """Distributed Lion for a list of fp32 parameters on this rank's device.

    ``step()`` is one iteration of Algorithm 1 over all of them: one worker-side launch, the
    exchange, one apply launch.  With a one-rank group this is plain Lion (Eq. 1 of the paper).

    Two ways of reaching the parameters:

    * ``in_place=True``: the parameters and their ``.grad`` tensors stay where the framework
      allocated them and are stepped there through the library's per-tensor pointer tables
      (``dlion_bind_tensors``); only the momentum is this object's own.  Gradient addresses
      are re-read every step, so ``zero_grad(set_to_none=True)`` is fine.  Every parameter
      and gradient must be contiguous and start on a 16-byte boundary.
    * ``in_place=False`` (default): the parameters are moved into one flat fp32 arena (each
      tensor starts on a 128-element boundary) and re-pointed at views of it; their ``.grad``
      become views of a second flat arena, so backward() accumulates straight into the
      buffer the worker-side kernel reads.
    """

    def __init__(self, params, lr: float = 1e-4, betas: Tuple[float, float] = (0.9, 0.99),
                 weight_decay: float = 0.0, mode: int = 0, group: Optional[dist.ProcessGroup] = None,
                 kernels=None, in_place: bool = False, host_staged: bool = False):
        self.params: List[torch.nn.Parameter] = [p for p in params]
        if not self.params:
            raise ValueError("no parameters")
        dev = self.params[0].device
        for p in self.params:
            if p.dtype != torch.float32 or p.device != dev:
                raise ValueError("parameters must be fp32 and on one device")
        self.segments, off = [], 0
        for p in self.params:
            self.segments.append((off, p.numel()))
            off += (p.numel() + ALIGN - 1) // ALIGN * ALIGN
        d_pad = max(off, ALIGN)
        self.in_place = bool(in_place)
        self.core = DistributedLion(self.segments, d_pad, mode, kernels=kernels, beta1=betas[0], beta2=betas[1],
                                    lr=lr, weight_decay=weight_decay, gdtype=0, group=group, device=dev,
                                    host_staged=host_staged)
        n = self.core.d_pad_x
        self.m = torch.zeros(n, dtype=torch.float32, device=dev)
        if self.in_place:
            for p in self.params:
                if not p.is_contiguous() or p.data_ptr() % 16 != 0:
                    raise ValueError("in_place needs contiguous parameters that start on a 16-byte boundary")
            self.x = self.g = None
            self.core.kernels.bind_tensors(m=[self.m[o:o + k] for o, k in self.segments],
                                           x=[p.data.view(-1) for p in self.params])
            return
        self.x = torch.zeros(n, dtype=torch.float32, device=dev)
        self.g = torch.zeros(n, dtype=torch.float32, device=dev)
        with torch.no_grad():
            for p, (o, k) in zip(self.params, self.segments):
                self.x[o:o + k].copy_(p.detach().reshape(-1))
                p.data = self.x[o:o + k].view(p.shape)
                p.grad = self.g[o:o + k].view(p.shape)

    def set_lr(self, lr: float) -> None:
        self.core.kernels.set_lr(lr)

    def zero_grad(self, set_to_none: bool = False) -> None:
        if self.in_place:
            for p in self.params:
                if set_to_none:
                    p.grad = None
                elif p.grad is not None:
                    p.grad.zero_()
            return
        self.g.zero_()                      # the views stay bound to the arena

    @torch.no_grad()
    def step(self) -> None:
        if self.in_place:
            grads = []
            for p in self.params:
                g = p.grad
                if g is None or g.dtype != torch.float32 or not g.is_contiguous() or g.data_ptr() % 16 != 0:
                    raise RuntimeError("in_place needs a contiguous fp32 .grad on a 16-byte boundary for every parameter")
                grads.append(g.view(-1))
            self.core.kernels.bind_tensors(grads=grads)
            self.core.step_tensors()
            return
        for p, (o, k) in zip(self.params, self.segments):
            if p.grad is None or p.grad.data_ptr() != self.g[o:o + k].data_ptr():
                raise RuntimeError("a parameter's .grad no longer points into the gradient arena "
                                   "(use this optimizer's zero_grad(), not set_to_none)")
        self.core.step(self.g, self.m, self.x)
