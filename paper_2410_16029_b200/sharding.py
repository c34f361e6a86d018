"""One model's matrices spread over the GPUs of a node (optimizer-state sharding).

Every weight matrix is an independent unit of the Natural GaLore step: its projector, history, Gram matrix and
moments never meet another matrix's.  So a model shards by assigning whole matrices to ranks; the step itself
needs no exchange, and ranks that need the full set of updated weights afterwards (data-parallel replicas) fetch
each shard from its owner.  This module holds the host-side plumbing only: the partition and the exchange of the
updated weights over ``torch.distributed`` (NCCL on GPUs, gloo in the CPU tests).  The arithmetic stays in the
CUDA library.

Not run on more than one GPU in this repository's own measurements (single-GPU machines); the partition and the
exchange are covered by two-process gloo tests.
"""
from __future__ import annotations

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


class ShardedNGaLore:
    """The optimizer of one model split over the ranks of the default process group: rank k holds the state of
    the matrices ``partition(...)[k]`` only (so the state memory divides by the number of ranks) and steps them;
    ``step`` can then refresh every rank's copy of the other matrices from their owners."""

    def __init__(self, shapes, r, s, T, *, group=None, **kw):
        from .ngalore import NGaLore

        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.shapes = [(int(M), int(N)) for M, N in shapes]
        self.parts = partition(self.shapes, r, s, self.world, kw.get("projection", "left"))
        self.mine = self.parts[self.rank]
        self.opt = NGaLore([self.shapes[i] for i in self.mine], r, s, T, **kw) if self.mine else None

    def step(self, W: Sequence[torch.Tensor], G: Sequence[torch.Tensor], exchange: bool = True) -> None:
        """W, G: the full lists (every rank holds every W; G is read for the owned matrices only)."""
        if self.opt is not None:
            self.opt.step([W[i] for i in self.mine], [G[i] for i in self.mine])
        if exchange:
            exchange_updated(W, self.parts, self.group)
