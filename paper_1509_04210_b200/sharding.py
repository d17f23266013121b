"""Range sharding of one parameter server over the GPUs of a node (host plumbing only).

The update is element-wise, so the flat weight vector splits into contiguous ranges, one owner
rank per range, with no exchange inside the update.  What keeps this different from the sharded
servers the paper contrasts itself with (Section 3.3) is that every rank replays the same global
arrival order of messages: all shards update on the same group boundaries, so the weights carry
one timestamp, and a learner's pull returns ranges that all belong to the same version.

The only data that crosses ranks is at the boundary: a learner's gradient is scattered to the
owners of its ranges (``torch.distributed`` send / recv: NCCL between GPUs, landing in the owner's
own memory; gloo on CPU) and a pull gathers the ranges (one broadcast per owner; ranges differ in
length, so the equal-size collectives do not apply).  Everything numerical happens in the
per-rank server object (the CUDA library on a GPU).  No arithmetic lives here.
"""
from __future__ import annotations

ALIGN = 256   # floats: every range starts on a 1 KB boundary, where the kernels' 1 KB warp accesses run at full speed


def shard_bounds(nparams, world, align=ALIGN):
    """[lo_0, hi_0), ..., [lo_{world-1}, hi_{world-1}): contiguous, disjoint, covering 0..nparams,
    every lo a multiple of ``align``, sizes as equal as that allows (trailing ranks may be empty
    when the vector is shorter than world * align)."""
    units = -(-int(nparams) // align)
    cuts = [min(int(nparams), (units * r // world) * align) for r in range(world + 1)]
    cuts[-1] = int(nparams)
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


class ShardedServer:
    """One rank's part of a range-sharded server.

    ``make_server(nparams_local)`` builds the local server (``binding.ParameterServer`` with the
    protocol parameters bound); it must offer push / step / pull / timestamp / set_weights.
    ``empty(n, kind)`` allocates a local vector of n elements for gradients (kind "grad") or weights
    (kind "weights") on the rank's device; tensors are torch tensors on that device.
    Every rank must make the same calls in the same order (they come from the same event stream).
    On GPUs the slice copies and the collectives run on torch's current stream while the local
    server enqueues on its own: leave the server on the default stream, or give it torch's current
    stream (``set_stream``), so that a slice is complete before the update reads it and a pulled
    range is complete before it is broadcast.
    """

    def __init__(self, make_server, nparams, c, empty, group=None):
        import torch.distributed as dist

        self.dist, self.group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        self.nparams, self.c = int(nparams), int(c)
        self.bounds = shard_bounds(nparams, self.world)
        self.lo, self.hi = self.bounds[self.rank]
        self.empty = empty
        self.server = make_server(self.hi - self.lo) if self.hi > self.lo else None
        self._borrowed = []   # staging slices stay alive until the update that reads them was issued

    def set_weights(self, theta_full):
        """Every rank holds the same initial vector and keeps its own range."""
        if self.server is not None:
            self.server.set_weights(theta_full[self.lo:self.hi].contiguous())

    def push(self, src_rank, grad_full, pulled_ts):
        """The learner living on rank ``src_rank`` pushes: its gradient (``grad_full`` there, None
        elsewhere) is cut into the owners' ranges and each owner queues its range."""
        mine = self.empty(self.hi - self.lo, "grad")
        if self.rank == src_rank:
            for r, (lo, hi) in enumerate(self.bounds):
                if hi == lo:
                    continue
                if r == self.rank:
                    mine.copy_(grad_full[lo:hi])
                else:
                    self.dist.send(grad_full[lo:hi].contiguous(), dst=r, group=self.group)
        elif self.hi > self.lo:
            self.dist.recv(mine, src=src_rank, group=self.group)
        if self.server is None:
            return 0
        self._borrowed.append(mine)
        return self.server.push(mine, pulled_ts)

    def step(self):
        """One update on every shard; returns what the local server returned (1 = updated)."""
        if self.server is None:
            return 1
        r = self.server.step()
        if r == 1:
            del self._borrowed[: self.c]
        return r

    def pull(self, dst_full):
        """All ranks receive the whole vector (ranges gathered from their owners); returns the timestamp."""
        mine = self.empty(self.hi - self.lo, "weights")
        ts = 0
        if self.server is not None:
            ts = self.server.pull(mine)
        for r, (lo, hi) in enumerate(self.bounds):
            if hi == lo:
                continue
            part = mine if r == self.rank else self.empty(hi - lo, "weights")
            self.dist.broadcast(part, src=r, group=self.group)
            dst_full[lo:hi].copy_(part)
        return ts

    def timestamp(self):
        return 0 if self.server is None else self.server.timestamp()

    def check_single_timestamp(self):
        """Raises unless every non-empty shard carries the same timestamp; returns it."""
        import torch

        ts = self.timestamp()
        big = 2 ** 62
        t = torch.tensor([ts if self.server is not None else -big, -(ts if self.server is not None else big)],
                         dtype=torch.int64)
        dev = self.empty(1, "weights").device
        t = t.to(dev)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX, group=self.group)
        hi, lo = int(t[0]), -int(t[1])
        if hi != lo:
            raise RuntimeError("shards disagree on the weight timestamp: %d .. %d" % (lo, hi))
        return hi
