"""Sharded operation across processes: one rank per GPU, each owning a contiguous block of the K workers
of Algorithm 1 (scaled sign).  torch.distributed is used for plumbing only -- exchanging the 512-byte
descriptions of where each rank's message rows live (once, at start) and the two barriers per step; the
messages themselves are never copied by a collective: every rank's server pass reads them in place from
the owners' memory (CUDA IPC mappings, NVLink between GPUs), inside the aggregation kernel.

The engine is injected so that the rank logic can be exercised without a GPU (tests use a recording fake).
"""
from typing import Callable, List, Optional, Tuple


def worker_range(num_workers: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous split of K workers over `world` ranks: (first worker, how many); the first K mod world
    ranks hold one more.  Every rank must own at least one worker."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank / world size")
    if num_workers < world:
        raise ValueError("fewer workers than ranks: every rank must own at least one worker")
    base, rem = divmod(num_workers, world)
    begin = rank * base + min(rank, rem)
    return begin, base + (1 if rank < rem else 0)


class ShardedRun:
    """One rank of a sharded run.

    make_engine(worker_begin, num_local) -> object with shard_export() -> bytes, shard_attach(bytes),
    step_begin(grads_local, lr), step_end(), close() and optionally shard_detach().  `barrier()` must order
    the device work every rank enqueued before it ahead of the device work any rank enqueues after it.
    Defaults: with the NCCL backend a one-element all-reduce on the current CUDA stream (stream-ordered on
    every rank: its kernel starts after the rank's earlier work and ends only when every rank's has started;
    the host does not wait); otherwise synchronise the device, then torch.distributed.barrier."""

    def __init__(self, num_workers: int, make_engine: Callable, group=None, barrier: Optional[Callable] = None,
                 allreduce_average: bool = False):
        import torch.distributed as dist
        self.dist = dist
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        self.num_workers = num_workers
        self.begin, self.count = worker_range(num_workers, self.world, self.rank)
        self.engine = make_engine(self.begin, self.count)
        self._flag = None
        if barrier is None and dist.get_backend(group) == "nccl":
            import torch
            self._flag = torch.zeros(1, device="cuda")
            barrier = self._stream_barrier
        self._barrier = barrier if barrier is not None else self._default_barrier
        blobs: List[Optional[bytes]] = [None] * self.world
        dist.all_gather_object(blobs, self.engine.shard_export(), group=group)
        for b in blobs:                       # rank order; includes this rank's own rows
            self.engine.shard_attach(b)
        self._readers_pending = False         # peers may still be reading this rank's rows
        self.allreduce_average = allreduce_average
        self._sum = None
        if allreduce_average:
            self.engine.shard_set_avg_mode(True)
        self._barrier()

    def _stream_barrier(self):
        self.dist.all_reduce(self._flag, group=self.group)

    def _default_barrier(self):
        import torch
        if torch.cuda.is_available():
            torch.cuda.synchronize()
        self.dist.barrier(group=self.group)

    def step(self, grads_local, lr: float):
        """Iteration t for this rank's workers.  The barrier that protects the message rows from being
        overwritten while peers still read them is taken lazily, at the start of the next step, so the
        caller's gradient computation overlaps the slowest peer's server pass."""
        if self._readers_pending:
            self._barrier()
        self.engine.step_begin(grads_local, lr)
        self._barrier()                       # every rank's messages are complete
        self.engine.step_end()
        self._readers_pending = True
        if self.allreduce_average and self.engine.avg_due:
            # Section 3.2: the local errors are averaged with an all-reduce (2 d floats per rank instead of
            # reading all K d stored differences in place; the sum order is the collective's)
            self._sum = self.engine.avg_local_sum(self._sum)
            self.dist.all_reduce(self._sum, group=self.group)
            self.engine.avg_set(self._sum)

    def finish(self):
        """Orders everything after it behind every peer's reads of this rank's rows (call before reading
        results or reusing buffers; with the stream-ordered barrier the host still has to synchronise the
        stream before it looks at device memory)."""
        if self._readers_pending:
            self._barrier()
            self._readers_pending = False

    def close(self):
        """Orderly shutdown: every rank unmaps its peers' rows before any rank frees its own."""
        self.finish()
        if hasattr(self.engine, "shard_detach"):
            self.engine.shard_detach()           # waits for this rank's stream, then unmaps
        self._barrier()
        if self._flag is not None:
            import torch
            torch.cuda.synchronize()             # the stream-ordered barrier has actually completed
        self.engine.close()


def sharded_sae(num_workers, tensor_sizes, x0, group=None, barrier=None, allreduce_average=False, **kw) -> ShardedRun:
    """ShardedRun over the CUDA library: every rank passes the same num_workers, tensor_sizes, x0 and options
    (compressor: scaled sign, the default, or Top-K)."""
    from . import binding as sb

    def make(begin, count):
        return sb.Sae(num_workers, tensor_sizes, x0, shard=(begin, count), **kw)

    return ShardedRun(num_workers, make, group=group, barrier=barrier, allreduce_average=allreduce_average)
