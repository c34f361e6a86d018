"""One model's matrices spread over the GPUs of a node (optimizer-state sharding).

Every weight matrix is an independent unit of the Natural GaLore step: its projector, history, Gram matrix and
moments never meet another matrix's.  So a model shards by assigning whole matrices to ranks; the step itself
needs no exchange, and ranks that need the full set of updated weights afterwards (data-parallel replicas) fetch
each shard from its owner.  This module holds the host-side plumbing only: the partition and the exchange of the
updated weights over ``torch.distributed`` (NCCL on GPUs, gloo in the CPU tests).  The arithmetic stays in the
CUDA library.

Two exchanges are offered.  ``exchange_updated`` runs after the step: one broadcast per owner.
``exchange_overlapped`` runs under it: the library updates the weights in groups of matrices and records an event
after each group (``ngalore_set_update_groups``), and the owner broadcasts group g from a side stream as soon as
that event has fired, while the back-projection of group g + 1 is still running; the weights can travel as bf16
(half the bytes; the owner keeps the fp32 master, the other ranks receive its rounding, which is what a bf16
forward pass reads anyway).

Not run on more than one GPU in this repository's own measurements (single-GPU machines); the partition, both
exchanges and the order of their operations are covered by two-process gloo tests.
"""
from __future__ import annotations

import contextlib
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def matrix_cost(M: int, N: int, r: int, s: int, projection: str = "left") -> int:
    """Bytes one step moves for an M x N matrix in the every-datum-once model: G (bf16) and W (fp32, read and
    written), the projector (bf16) and (4 s + 20) bytes per low-rank element (history, new slot, moments)."""
    rp = min(r, M, N)
    right = projection == "short_side" and M >= N
    low_rank = rp * (M if right else N)
    return 10 * M * N + 2 * (N if right else M) * rp + (4 * s + 20) * low_rank


def partition(shapes: Sequence[Tuple[int, int]], r: int, s: int, world: int,
              projection: str = "left") -> List[List[int]]:
    """Matrix indices owned by each of ``world`` ranks: longest-processing-time-first on ``matrix_cost`` (the
    largest matrix goes to the least loaded rank, and so on), each rank's list in ascending order.  Every rank
    computes the same partition from the same arguments; nothing is communicated."""
    if world < 1:
        raise ValueError("world must be positive")
    load = [0] * world
    owned: List[List[int]] = [[] for _ in range(world)]
    order = sorted(range(len(shapes)), key=lambda i: (-matrix_cost(shapes[i][0], shapes[i][1], r, s, projection), i))
    for i in order:
        k = min(range(world), key=lambda j: (load[j], j))
        owned[k].append(i)
        load[k] += matrix_cost(shapes[i][0], shapes[i][1], r, s, projection)
    return [sorted(o) for o in owned]


def owners(parts: Sequence[Sequence[int]], n_matrices: int) -> List[int]:
    """Owner rank of every matrix."""
    out = [-1] * n_matrices
    for rank, idx in enumerate(parts):
        for i in idx:
            out[i] = rank
    if any(o < 0 for o in out):
        raise ValueError("partition does not cover every matrix")
    return out


def exchange_updated(W: Sequence[torch.Tensor], parts: Sequence[Sequence[int]], group=None) -> None:
    """Make every rank's copy of every matrix equal to its owner's: one broadcast per owner of its matrices packed
    into one flat buffer (on NVSwitch a broadcast runs at link speed to all peers at once)."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    if len(parts) != world:
        raise ValueError("one shard per rank")
    for src in range(world):
        idx = parts[src]
        if not idx:
            continue
        numel = sum(W[i].numel() for i in idx)
        flat = torch.empty(numel, dtype=W[idx[0]].dtype, device=W[idx[0]].device)
        if rank == src:
            torch.cat([W[i].reshape(-1) for i in idx], out=flat)
        dist.broadcast(flat, src=dist.get_global_rank(group, src) if group is not None else src, group=group)
        if rank != src:
            off = 0
            for i in idx:
                n = W[i].numel()
                W[i].copy_(flat[off:off + n].view_as(W[i]))
                off += n


def exchange_overlapped(W: Sequence[torch.Tensor], groups_by_owner: Sequence[Sequence[Sequence[int]]], *,
                        wait_update=None, comm_stream=None, wire: str = "fp32", group=None, log=None) -> None:
    """Refresh every rank's copy of every matrix from its owner, group by group, in a fixed order that all ranks
    share: owners in rank order, each owner's update groups in the order the library updates them.

    groups_by_owner[src][g]: the (global) matrix indices of update group g of rank src.
    wait_update(g):          called on the owner before it reads group g: makes ``comm_stream`` wait for the event
                             the library recorded after updating that group (``NGaLore.stream_wait_update``).
    comm_stream:             the stream packing, collectives and unpacking are enqueued on (None: the current one).
                             The caller's stream has to wait for it before it reads the received weights.
    wire:                    "fp32" (bit-exact copies) or "bf16" (half the bytes; the other ranks receive the
                             owner's weights rounded to bf16, widened back to the dtype of their tensors).
    log:                     optional list; every operation appends (op, src, g), for tests of the ordering.
    """
    if wire not in ("fp32", "bf16"):
        raise ValueError(wire)
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    if len(groups_by_owner) != world:
        raise ValueError("one list of groups per rank")
    ctx = torch.cuda.stream(comm_stream) if comm_stream is not None else contextlib.nullcontext()
    with ctx:
        for src in range(world):
            for g, idx in enumerate(groups_by_owner[src]):
                if not idx:
                    continue
                numel = sum(W[i].numel() for i in idx)
                dtype = torch.bfloat16 if wire == "bf16" else W[idx[0]].dtype
                flat = torch.empty(numel, dtype=dtype, device=W[idx[0]].device)
                if rank == src:
                    if wait_update is not None:
                        wait_update(g)
                        if log is not None:
                            log.append(("wait", src, g))
                    off = 0
                    for i in idx:
                        n = W[i].numel()
                        flat[off:off + n].copy_(W[i].reshape(-1))      # rounds when the wire is bf16
                        off += n
                    if log is not None:
                        log.append(("pack", src, g))
                dist.broadcast(flat, src=dist.get_global_rank(group, src) if group is not None else src, group=group)
                if log is not None:
                    log.append(("bcast", src, g))
                if rank != src:
                    off = 0
                    for i in idx:
                        n = W[i].numel()
                        W[i].copy_(flat[off:off + n].view_as(W[i]))
                        off += n
                    if log is not None:
                        log.append(("unpack", src, g))


class ShardedNGaLore:
    """The optimizer of one model split over the ranks of the default process group: rank k holds the state of
    the matrices ``partition(...)[k]`` only (so the state memory divides by the number of ranks) and steps them;
    ``step`` can then refresh every rank's copy of the other matrices from their owners."""

    def __init__(self, shapes, r, s, T, *, group=None, update_groups: int = 0, wire: str = "fp32", **kw):
        """update_groups >= 2: the weight update runs in that many groups and ``step`` exchanges them while the
        update is still running (``exchange_overlapped``); 0: one broadcast per owner after the step.
        wire: "fp32" or "bf16", the format the weights travel in (overlapped exchange only)."""
        from .ngalore import NGaLore

        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.shapes = [(int(M), int(N)) for M, N in shapes]
        self.parts = partition(self.shapes, r, s, self.world, kw.get("projection", "left"))
        self.mine = self.parts[self.rank]
        self.opt = NGaLore([self.shapes[i] for i in self.mine], r, s, T, **kw) if self.mine else None
        self.wire = wire
        self.groups_by_owner = None
        self.comm_stream = None
        if update_groups >= 2:
            mine_groups = []
            if self.opt is not None:
                self.opt.set_update_groups(update_groups)
                mine_groups = [[self.mine[j] for j in range(a, b)] for a, b in self.opt.update_groups()]
            gathered = [None] * self.world
            dist.all_gather_object(gathered, mine_groups, group=group)     # once, at set-up
            self.groups_by_owner = gathered
            self.comm_stream = torch.cuda.Stream()

    def step(self, W: Sequence[torch.Tensor], G: Sequence[torch.Tensor], exchange: bool = True) -> None:
        """W, G: the full lists (every rank holds every W; G is read for the owned matrices only)."""
        overlapped = exchange and self.groups_by_owner is not None
        if overlapped:
            # whatever the stepping stream did with the weights so far (the forward and backward pass that made G)
            # comes before anything the side stream writes into them; the step enqueued next does not
            main = torch.cuda.current_stream()
            before_step = torch.cuda.Event()
            before_step.record(main)
            self.comm_stream.wait_event(before_step)
        if self.opt is not None:
            self.opt.step([W[i] for i in self.mine], [G[i] for i in self.mine])
        if not exchange:
            return
        if not overlapped:
            exchange_updated(W, self.parts, self.group)
            return
        wait = (lambda g: self.opt.stream_wait_update(g, self.comm_stream)) if self.opt is not None else None
        exchange_overlapped(W, self.groups_by_owner, wait_update=wait, comm_stream=self.comm_stream, wire=self.wire,
                            group=self.group)
        main.wait_stream(self.comm_stream)     # the next reader of W on the stepping stream sees every shard
