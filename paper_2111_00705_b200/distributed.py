"""Distributed deployment of Algorithm 1: one process per GPU, each holding some of the n
workers, the messages moved with ``torch.distributed`` (NCCL between GPUs).

This module is plumbing: which process holds which workers, and which message rows go where.
All arithmetic of the method runs in the library's kernels through ``binding.CDAdamShard``;
the messages are the d sign bits and q scales per worker that Algorithm 1 sends (Section 5),
or the k coordinates and values of top-k, taken from and delivered into the library's own
buffers without a copy.

Two layouts:

* ``server_rank=None`` (default): every process holds n / world workers.  One all-gather
  gives every process all n worker messages and each computes the server stage itself; the
  results are identical everywhere (same operations, same order), so the server's broadcast
  is not needed.  One collective per iteration instead of two sends.
* ``server_rank=r``: the paper's layout.  Process r is the server and holds no worker; the
  other world - 1 processes hold n / (world - 1) workers each.  The worker messages go to r,
  r runs the server stage, and the server message is broadcast; every process (the server
  too, Algorithm 1 keeps gtil there) then runs the update.
"""
import torch
import torch.distributed as dist

from . import binding


def partition(n, world, rank, server_rank=None):
    """(first_worker, n_local) of `rank` among `world` processes.  Workers are dealt in
    contiguous, equal blocks to the processes that hold workers, in rank order."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    if server_rank is None:
        holders = world
        pos = rank
    else:
        if not (0 <= server_rank < world):
            raise ValueError("server_rank out of range")
        if world < 2:
            raise ValueError("a separate server needs at least two processes")
        holders = world - 1
        if rank == server_rank:
            return 0, 0
        pos = rank if rank < server_rank else rank - 1
    if n % holders != 0:
        raise ValueError("n = %d workers do not divide among %d processes" % (n, holders))
    per = n // holders
    return pos * per, per


def exchange_worker_messages(bits, scales, n, group=None, server_rank=None):
    """Deliver the worker messages.  `bits` (n x words, int32) and `scales` (n x q, float32)
    are the full message buffers of this process with its own rows filled in; on return the
    rows of all workers are present on every process (replicated layout) or on the server
    (server layout; the other processes' buffers keep their own rows only).  In place."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    first, per = partition(n, world, rank, server_rank)
    if server_rank is None:
        dist.all_gather_into_tensor(bits, bits[first:first + per], group=group)
        dist.all_gather_into_tensor(scales, scales[first:first + per], group=group)
        return
    ops = []
    if rank == server_rank:
        for r in range(world):
            if r == server_rank:
                continue
            f, p = partition(n, world, r, server_rank)
            peer = dist.get_global_rank(group, r) if group is not None else r
            ops.append(dist.P2POp(dist.irecv, bits[f:f + p], peer, group))
            ops.append(dist.P2POp(dist.irecv, scales[f:f + p], peer, group))
    else:
        peer = dist.get_global_rank(group, server_rank) if group is not None else server_rank
        ops.append(dist.P2POp(dist.isend, bits[first:first + per], peer, group))
        ops.append(dist.P2POp(dist.isend, scales[first:first + per], peer, group))
    for work in dist.batch_isend_irecv(ops):
        work.wait()


def broadcast_server_message(bits, scales, group=None, server_rank=0):
    """The server's message (words int32, q float32) to every process, in place."""
    src = dist.get_global_rank(group, server_rank) if group is not None else server_rank
    dist.broadcast(bits, src=src, group=group)
    dist.broadcast(scales, src=src, group=group)


class DistributedCDAdam:
    """Algorithm 1 across the processes of a ``torch.distributed`` group, scaled sign (the
    default) or top-k (``compressor=binding.TOPK, k=...``).

    Every process calls ``step(grads_local)`` with the gradients of its own workers
    (n_local x d, CUDA float32; ``None`` on a server that holds none); afterwards
    ``params()`` is x_{t+1}, the same on every process.  Kernels and collectives are
    ordered by the current CUDA stream of torch."""

    def __init__(self, d, n, group=None, server_rank=None, **kwargs):
        self.group, self.server_rank, self.n = group, server_rank, int(n)
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        first, per = partition(self.n, self.world, self.rank, server_rank)
        self.shard = binding.CDAdamShard(d, n, first, per, **kwargs)

    def step(self, grads_local):
        s = self.shard
        s.step_workers(grads_local)
        buf = s.exchange_buffers()
        exchange_worker_messages(buf["worker_bits"], buf["worker_scales"], self.n, self.group, self.server_rank)
        if self.server_rank is None:
            s.step_server()
        else:
            if self.rank == self.server_rank:
                s.step_server()
            broadcast_server_message(buf["server_bits"], buf["server_scales"], self.group, self.server_rank)
        s.step_update()

    def params(self):
        return self.shard.params()

    def close(self):
        self.shard.close()
