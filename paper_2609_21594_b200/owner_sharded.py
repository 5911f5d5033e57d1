"""Owner-sharded Muon step over several ranks: the host-side orchestration only.

What one rank does per optimizer step when every 2-D parameter is row-sharded over `world` ranks
(Section 6.4 of the paper: fused gather, compute-owner assignment, relay broadcast, slice-and-apply;
Section 6.7 and Algorithm 2: batches in descending size, at most one batch's broadcast in flight, final
drain).  Parameters, momenta and gradients stay sharded; a whole matrix exists only on its compute owner
and only while its batch is being orthogonalised.

This module holds no arithmetic.  Compute goes through an `ops` object (the CUDA library in production:
`CudaOps` below), communication through a `comm` object (`TorchComm`: torch.distributed, NCCL on GPUs, gloo on
CPUs; `SingleComm` for one rank).  Everything that is decided on the host -- which matrices form a batch, who
owns which matrix, where each shard and each update sits in the exchange buffers, in which order collectives are
issued and settled -- is decided here, once, when the object is built (the static plan of Section 6.2), and is
therefore testable on a CPU with two gloo ranks and a stand-in for `ops`.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import torch

from . import workloads as wl

Shape = Tuple[int, int]
REGION_ALIGN = 8          # elements: every matrix in a broadcast region starts on a 16-byte boundary (bf16)


def _up(x: int, a: int) -> int:
    return (x + a - 1) // a * a


@dataclass
class BatchPlan:
    """Static description of one batch: its matrices, their owners and every offset the exchange needs."""
    index: int
    matrices: List[int]                   # indices into the optimizer's shape list, in batch order
    shapes: List[Shape]
    owners: List[int]                     # compute owner of each matrix of the batch
    layout: "wl.Layout"                   # flat-shard layout of the batch: `world` shards, per-parameter row split
    region_len: List[int]                 # per rank: elements of the broadcast region that rank owns
    region_off: List[int]                 # per matrix of the batch: element offset inside its owner's region
    handle: object = None                 # whatever ops.new_batch returned


def build_batches(shapes: Sequence[Shape], world: int, owner_of: Sequence[int], batch_of: Sequence[int], num_batches: int,
                  align: int = wl.ALIGN_ELEMS) -> List[BatchPlan]:
    """Turns an owner/batch assignment into per-batch layouts and exchange offsets (pure bookkeeping)."""
    out: List[BatchPlan] = []
    for b in range(num_batches):
        mats = [i for i in range(len(shapes)) if batch_of[i] == b]
        bshapes = [tuple(shapes[i]) for i in mats]
        owners = [int(owner_of[i]) for i in mats]
        region_len = [0] * world
        region_off = []
        for (m, n), o in zip(bshapes, owners):
            region_off.append(region_len[o])
            region_len[o] = _up(region_len[o] + m * n, REGION_ALIGN)
        out.append(BatchPlan(b, mats, bshapes, owners, wl.layout_per_param(bshapes, world, align), region_len, region_off))
    return out


class SingleComm:
    """world == 1: nothing to exchange."""
    world, rank = 1, 0

    def all_gather(self, local: torch.Tensor) -> torch.Tensor:
        return local

    def broadcast(self, t: torch.Tensor, src: int):
        return None

    def wait(self, handle) -> None:
        return None


class TorchComm:
    """torch.distributed (NCCL on CUDA tensors, gloo on CPU tensors); payloads travel as raw 16-bit or 32-bit words."""

    def __init__(self, group=None):
        import torch.distributed as dist

        self.dist, self.group = dist, group
        self.world, self.rank = dist.get_world_size(group), dist.get_rank(group)

    @staticmethod
    def _raw(t: torch.Tensor) -> torch.Tensor:
        return t.view(torch.int16) if t.element_size() == 2 else t.view(torch.int32)

    def all_gather(self, local: torch.Tensor) -> torch.Tensor:
        full = torch.empty(self.world * local.numel(), dtype=local.dtype, device=local.device)
        self.dist.all_gather_into_tensor(self._raw(full), self._raw(local), group=self.group)
        return full

    def broadcast(self, t: torch.Tensor, src: int):
        return self.dist.broadcast(self._raw(t), src=src, group=self.group, async_op=True)

    def wait(self, handle) -> None:
        if handle is not None:
            handle.wait()


class CudaOps:
    """The compute half, on the CUDA library (marshalling only)."""

    def __init__(self, ctx, grad_dtype=torch.bfloat16, ns_dtype=torch.bfloat16, device="cuda"):
        from . import binding as mb

        self.mb, self.ctx, self.device = mb, ctx, device
        self.grad_dtype, self.ns_dtype = grad_dtype, ns_dtype

    def owner_plan(self, shapes, world, batch_elems):
        return self.mb.muon_owner_plan(shapes, world, batch_elems)

    def new_batch(self, plan: BatchPlan):
        return self.mb.Layout(self.ctx, plan.layout, 2 if self.ns_dtype == torch.bfloat16 else 4)

    def empty(self, n: int, dtype) -> torch.Tensor:
        return torch.empty(max(n, 1), dtype=dtype, device=self.device)

    def prepare(self, shapes) -> None:
        self.ctx.ensure_workspace(shapes)

    def shard_momentum(self, plan, rank, g, m, u, mu) -> None:
        self.ctx.muon_shard_momentum(plan.handle, rank, g, m, u, mu)

    def materialize_owned(self, plan, flat, mats) -> None:
        self.ctx.muon_materialize_owned(flat, plan.handle, mats)

    def orthogonalize(self, shapes, ins, outs, ns_steps, coeffs) -> None:
        if shapes:
            self.ctx.muon_orthogonalize_batched(ins, outs, shapes, ns_steps, coeffs)

    def shard_apply(self, plan, rank, w, updates, lr, wd) -> None:
        self.ctx.muon_shard_apply(plan.handle, rank, w, updates, lr, wd)

    def sync(self) -> None:
        torch.cuda.synchronize()


@dataclass
class _InFlight:
    plan: BatchPlan
    handles: list = field(default_factory=list)


class OwnerShardedStep:
    """One rank of the owner-sharded step.  State lives in per-batch local shard buffers:

        self.params[b], self.momenta[b]   fp32, shard_len(b) elements: this rank's shard of batch b (in/out)
        self.grads[b]                     gradient dtype, same extent: the caller fills it before every step

    `events` records the order of collectives as (kind, batch, ...) tuples, for tests.
    """

    def __init__(self, shapes: Sequence[Shape], ops, comm, batch_elems: int = 0, align: int = wl.ALIGN_ELEMS):
        self.shapes = [tuple(s) for s in shapes]
        self.ops, self.comm = ops, comm
        self.world, self.rank = comm.world, comm.rank
        owner_of, batch_of, nb = ops.owner_plan(self.shapes, self.world, batch_elems)
        self.owner_of, self.batch_of = owner_of, batch_of
        self.batches = build_batches(self.shapes, self.world, owner_of, batch_of, nb, align)
        self.params, self.momenta, self.grads = [], [], []
        self._staged, self._regions, self._owned_in = [], [], []
        for plan in self.batches:
            plan.handle = ops.new_batch(plan)
            n = plan.layout.shard_len
            self.params.append(ops.empty(n, torch.float32))
            self.momenta.append(ops.empty(n, torch.float32))
            self.grads.append(ops.empty(n, ops.grad_dtype))
            self._staged.append(ops.empty(n, ops.ns_dtype))
            # one region per owner rank: this rank fills its own, receives the others
            self._regions.append([ops.empty(plan.region_len[o], ops.ns_dtype) for o in range(self.world)])
            self._owned_in.append([ops.empty(m * n_, ops.ns_dtype)[:m * n_].view(m, n_) if o == self.rank else None
                                   for (m, n_), o in zip(plan.shapes, plan.owners)])
            if hasattr(ops, "prepare"):               # workspace for the matrices this rank orthogonalises in this batch
                ops.prepare([s for s, o in zip(plan.shapes, plan.owners) if o == self.rank])
        self.events: List[tuple] = []

    # ---- views into the exchange buffers
    def update_views(self, b: int) -> List[torch.Tensor]:
        """The whole-matrix update of every matrix of batch b, wherever its owner's region put it."""
        plan = self.batches[b]
        out = []
        for (m, n), o, off in zip(plan.shapes, plan.owners, plan.region_off):
            out.append(self._regions[b][o][off:off + m * n].view(m, n))
        return out

    def shard_rows(self, b: int, k: int) -> Tuple[int, int]:
        """Rows [r0, r1) of matrix k of batch b that this rank's shard holds (the ceil-chunk row split)."""
        m = self.batches[b].shapes[k][0]
        ch = -(-m // self.world)
        return min(m, self.rank * ch), min(m, (self.rank + 1) * ch)

    # ---- one optimizer step
    def step(self, lr: float, mu: float, wd: float, ns_steps: int, coeffs) -> None:
        pending: Optional[_InFlight] = None
        for b, plan in enumerate(self.batches):
            # step 1: local momentum, then the fused gather of the staged shards of the whole batch
            self.ops.shard_momentum(plan, self.rank, self.grads[b], self.momenta[b], self._staged[b], mu)
            self.events.append(("gather", b))
            full = self.comm.all_gather(self._staged[b])
            # step 2: only the owner materialises a matrix and orthogonalises it, straight into its broadcast region
            mine = [k for k, o in enumerate(plan.owners) if o == self.rank]
            ins = self._owned_in[b]
            self.ops.materialize_owned(plan, full, ins)
            views = self.update_views(b)
            self.ops.orthogonalize([plan.shapes[k] for k in mine], [ins[k] for k in mine], [views[k] for k in mine],
                                   ns_steps, coeffs)
            # step 3: relay broadcast, asynchronous; at most one batch in flight: admitting this one settles the oldest
            if pending is not None:
                self._settle(pending, lr, wd)
            pending = _InFlight(plan)
            for o in range(self.world):
                if plan.region_len[o] > 0:
                    self.events.append(("broadcast", b, o))
                    pending.handles.append(self.comm.broadcast(self._regions[b][o], o))
        if pending is not None:                       # final drain
            self._settle(pending, lr, wd)
        self.events.append(("drained",))

    def _settle(self, inflight: _InFlight, lr: float, wd: float) -> None:
        for h in inflight.handles:
            self.comm.wait(h)
        b = inflight.plan.index
        self.events.append(("apply", b))
        # step 4: every rank extracts its own slice of every update and applies it with decay
        self.ops.shard_apply(inflight.plan, self.rank, self.params[b], self.update_views(b), lr, wd)
