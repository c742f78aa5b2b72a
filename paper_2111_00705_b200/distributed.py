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
  is not needed.  One grouped collective per iteration instead of two sends.
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


def _all_gather_together(pairs, group=None):
    """In-place all-gathers of several (whole buffer, own rows) pairs.  On NCCL they are queued
    as one grouped call (one launch moves the sign words and the scales of a message, which
    live in two arrays); other backends get one call per pair."""
    if dist.get_backend(group) == "nccl" and hasattr(dist, "_coalescing_manager"):
        with dist._coalescing_manager(group=group):
            for whole, own in pairs:
                dist.all_gather_into_tensor(whole, own, group=group)
        return
    for whole, own in pairs:
        dist.all_gather_into_tensor(whole, own, group=group)


def exchange_worker_messages(bits, scales, n, group=None, server_rank=None):
    """Deliver the worker messages.  `bits` (n x words, int32) and `scales` (n x q, float32)
    are the full message buffers of this process with its own rows filled in; on return the
    rows of all workers are present on every process (replicated layout) or on the server
    (server layout; the other processes' buffers keep their own rows only).  In place."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    first, per = partition(n, world, rank, server_rank)
    if server_rank is None:
        _all_gather_together([(bits, bits[first:first + per]), (scales, scales[first:first + per])], group)
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


# ---------------------------------------------------------------------------------------------
# Coordinate-sharded deployment: every process owns a coordinate range of all n workers' vectors
# and of the server's.  The one thing that crosses ranges is the l1 norm inside the scaled-sign
# compressor (Appendix A): each process reduces its part of every (worker, segment) sum to a
# double-double, the parts are all-gathered and every process adds them in rank order.  An
# all-reduce is NOT used: its order of additions is the library's choice, and the scale has to
# be the same bits everywhere and equal to the one-process value.
# ---------------------------------------------------------------------------------------------

def range_partition(d, world, rank, align=16384):
    """[lo, hi) of `rank`: [0, d) cut into `world` contiguous ranges whose inner boundaries are
    multiples of `align` (the largest tile of the kernels, so that full tiles stay full); the
    last range takes the ragged end.  Ranges may differ by one `align` unit in length."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    units = -(-d // align)
    if units < world:
        raise ValueError("d = %d is too small for %d ranges aligned to %d" % (d, world, align))
    base, extra = divmod(units, world)
    start = rank * base + min(rank, extra)
    stop = start + base + (1 if rank < extra else 0)
    return start * align, min(d, stop * align)


def gather_range_sums(sums, group=None):
    """In-place all-gather of the l1 parts: `sums` is the [ranks, ...] exchange buffer of this
    process with its own slot [rank] filled in; on return every slot holds its owner's parts,
    slot r from the process of rank r.  No arithmetic happens here."""
    rank = dist.get_rank(group)
    flat = sums.view(sums.shape[0], -1)
    dist.all_gather_into_tensor(flat.view(-1), flat[rank].clone(), group=group)


class RangeShardedCDAdam:
    """Algorithm 1 with scaled sign (or top-k: ``compressor=binding.TOPK, k=...``), coordinate-sharded across the processes of a
    ``torch.distributed`` group: process r owns coordinates range_partition(d, world, r) of every
    vector.  ``step(grads_local)`` takes the n x (hi - lo) gradients of the owned coordinates;
    ``params()`` is the owned slice of x_{t+1}.  Two all-gathers of a few hundred bytes per
    iteration (2 n q and 2 q doubles per process); no vector ever crosses a process."""

    def __init__(self, d, n, group=None, align=16384, **kwargs):
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.lo, self.hi = range_partition(d, self.world, self.rank, align)
        self.range = binding.CDAdamRange(d, n, self.lo, self.hi, self.rank, self.world, **kwargs)

    def step(self, grads_local):
        r = self.range
        if r.compressor == binding.TOPK:       # ten stages, a gather of the histograms / tie counts after eight
            for stage in range(r.TOPK_STAGES):
                r.range_topk(stage, grads_local if stage <= 4 else None)
                buf = r.range_topk_buffer(stage)
                if buf is not None:
                    gather_range_sums(buf, self.group)
            return
        r.range_workers(grads_local)
        gather_range_sums(r.range_buffers()["worker_sums"], self.group)
        r.range_server()
        gather_range_sums(r.range_buffers()["server_sums"], self.group)
        r.range_update()

    def params(self):
        return self.range.params()

    def close(self):
        self.range.close()
