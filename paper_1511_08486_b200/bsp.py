"""Bulk-synchronous sufficient-factor broadcasting across processes, one process per GPU.

Section 3 ("Sufficient factor broadcasting") and Section 4 (BSP consistency): every worker computes the
SF pairs of its own data against its full local copy of W, sends them to all other workers, and applies
all workers' pairs; under BSP every copy of W sees the same pairs at every clock, so the copies stay equal.

Here the P workers of the descriptor are split evenly over the processes of a torch.distributed group.
The SF buffer's worker streams are contiguous and equally long, so the broadcast of every worker's pairs
to everybody is ONE in-place all-gather over the stream region of the buffer (NCCL over NVLink on GPUs).
The received streams land in this GPU's own memory; the apply kernels read local memory only.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def worker_range(P: int, world: int, rank: int) -> tuple[int, int]:
    """(first_worker, n_workers) owned by `rank`: P must split evenly so that the all-gather is uniform."""
    if world <= 0 or not 0 <= rank < world:
        raise ValueError(f"rank {rank} outside a group of {world}")
    if P % world != 0:
        raise ValueError(f"P = {P} workers do not split evenly over {world} processes")
    n = P // world
    return rank * n, n


def exchange_bytes(P: int, world: int, stream_stride: int) -> dict:
    """Bytes the broadcast moves per clock: each process sends its streams to the world - 1 others.

    The paper counts O(P^2 K (J + D)) values for P workers with K pairs each (Section 3, Figure 1);
    with `world` processes holding P / world workers each the same count is world (world - 1) shards.
    """
    shard = (P // world) * stream_stride
    return {"shard_bytes": shard, "sent_per_process": shard * (world - 1), "total": shard * world * (world - 1)}


def all_gather_streams(sf_buf: torch.Tensor, streams_off: int, stream_stride: int, P: int, group=None) -> None:
    """In place: every process contributes the streams it owns, all processes end with all P streams.

    sf_buf: 1-D uint8 tensor holding the SF buffer (device memory with NCCL, host memory with gloo).
    """
    world = dist.get_world_size(group)
    first, n = worker_range(P, world, dist.get_rank(group))
    streams = sf_buf[streams_off:streams_off + P * stream_stride]
    mine = streams[first * stream_stride:(first + n) * stream_stride]
    if dist.get_backend(group) != "nccl":
        mine = mine.clone()          # only NCCL documents the aliased (in-place) form
    dist.all_gather_into_tensor(streams, mine, group=group)


class BspSfb:
    """One process's side of the BSP step: factors of its shard, exchange, apply of all K pairs."""

    def __init__(self, ctx, desc, sf_buf: torch.Tensor, group=None):
        from . import binding as B
        self.ctx, self.desc, self.sf_buf, self.group = ctx, desc, sf_buf, group
        self.streams_off, self.stream_stride = B.sfb_sf_buffer_layout(desc)
        self.in_group = dist.is_available() and dist.is_initialized()
        if self.in_group:
            self.world, self.rank = dist.get_world_size(group), dist.get_rank(group)
        else:
            self.world, self.rank = 1, 0
        self.first, self.n_workers = worker_range(desc.P, self.world, self.rank)

    def shard_rows(self) -> slice:
        """Rows of the global minibatch this process computes factors for."""
        return slice(self.first * self.desc.B, (self.first + self.n_workers) * self.desc.B)

    def step(self, W, X_shard, aux_shard, eta: float, clock: int = 0) -> None:
        self.ctx.factors_shard(W, X_shard, aux_shard, self.sf_buf, self.first, self.n_workers)
        if self.in_group:       # also with a group of one process: the collective then has nothing to move
            all_gather_streams(self.sf_buf, self.streams_off, self.stream_stride, self.desc.P, self.group)
        self.ctx.commit_header(self.sf_buf, clock)
        self.ctx.apply(W, self.sf_buf, eta)
