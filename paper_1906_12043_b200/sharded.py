"""CoCoD-SGD with the workers spread over several GPUs, one process per GPU (the paper's own
layout: Section 5.1 runs one worker per GPU and averages the models with an all-reduce).

Each process holds a contiguous block of the K_global workers in an engine of its own.  Step II
(local steps) and line 6 (merge) of Algorithm 1 stay local; only Step I's weighted mean spans the
GPUs, and it stays on the side stream so that it still overlaps the local steps.  This module is
plumbing over ``torch.distributed``: which workers live where, what is queued on the side stream in
which order, and the exchange of buffer addresses.  All arithmetic runs in the library's kernels
(or, for the all-reduce form, in the collective library's reduction).

Two ways to complete the mean (``exchange=``):

``"allreduce"``  the engine's kernel leaves this GPU's partial weighted sum in the average buffer
                 and one all-reduce of P floats over the process group finishes it;
``"gather"``     one kernel per GPU reads the K_global stored copies of its share of the columns
                 directly from the GPUs that hold them (peer loads over NVLink), sums them in
                 worker order and stores the finished columns into every GPU's average buffer
                 (peer stores); two barriers on the side stream order it against the other
                 processes.  Its result does not depend on how the workers are spread.

Every process must make the same sequence of calls.
"""
from __future__ import annotations

import contextlib


def shard_workers(K_global: int, G: int, rank: int):
    """(first, count) of the contiguous block of workers that process ``rank`` of ``G`` holds:
    blocks differ in size by at most one, larger blocks first."""
    if not (G >= 1 and 0 <= rank < G and K_global >= G):
        raise ValueError("need 0 <= rank < G <= K_global")
    base, rem = divmod(K_global, G)
    first = rank * base + min(rank, rem)
    return first, base + (1 if rank < rem else 0)


class WorkerShardedEngine:
    """Algorithm 1 over K_global workers, of which this process holds ``shard_workers(...)``.

    ``group``: a ``torch.distributed`` process group (None = the default group).  ``sync`` says
    how the gather form orders itself against the other processes: ``"stream"`` queues a
    one-element all-reduce on the side stream (the host never blocks; needs a backend that works
    on CUDA tensors, i.e. NCCL with one GPU per process), ``"host"`` synchronises the side stream
    and calls the group's host barrier (any backend; blocks the host twice per round).
    ``engine_factory(K, P, lr, mu, wd)`` builds the local engine (default: the CUDA engine).
    """

    def __init__(self, K_global: int, P: int, lr: float, mu: float, wd: float, *, group=None, batch_sizes=None,
                 exchange: str = "allreduce", sync: str = "stream", engine_factory=None):
        import torch.distributed as dist
        if exchange not in ("allreduce", "gather"):
            raise ValueError(exchange)
        if sync not in ("stream", "host"):
            raise ValueError(sync)
        if not dist.is_initialized():
            raise RuntimeError("torch.distributed is not initialised")
        self._dist, self.group = dist, group
        self.rank, self.G = dist.get_rank(group), dist.get_world_size(group)
        self.K_global, self.P = int(K_global), int(P)
        self.first, self.K = shard_workers(self.K_global, self.G, self.rank)
        self.exchange, self.sync_mode = exchange, sync
        if batch_sizes is not None and len(batch_sizes) != self.K_global:
            raise ValueError("need the batch sizes of all K_global workers")
        if engine_factory is None:
            from .engine import Engine as engine_factory
        self.engine = engine_factory(self.K, self.P, lr, mu, wd)
        self.engine.set_shard(self.K_global, self.first, batch_sizes)
        self._mean = self.engine.mean_buffer()
        self._flag = None
        self._attached = False
        if exchange == "gather":
            blobs = [None] * self.G
            dist.all_gather_object(blobs, self.engine.ipc_export(), group=group)
            self.engine.ipc_attach(self.rank, blobs)
            self._attached = True
            if sync == "stream":
                import torch
                self._flag = torch.zeros(1, dtype=torch.float32, device=self._mean.device)
            self._host_barrier()          # nobody starts a round before everybody is attached

    # -- ordering against the other processes
    @staticmethod
    def _on(side):
        if side is None:
            return contextlib.nullcontext()
        import torch
        return torch.cuda.stream(side)

    def _host_barrier(self):
        self._dist.barrier(group=self.group)

    def _side_barrier(self, side):
        """Work queued on the side stream after this runs only after every process's side stream
        has reached the same point."""
        if self.sync_mode == "stream":
            with self._on(side):
                self._dist.all_reduce(self._flag, group=self.group)
        else:
            if side is not None:
                side.synchronize()
            self._host_barrier()

    # -- Algorithm 1
    def local_step(self, grads):
        """Step II for this process's workers.  grads: K x P (this process's rows)."""
        self.engine.local_step(grads)

    def comm_begin(self, side_stream=None):
        """Step I: store x_t^i, then the weighted mean over ALL workers, queued on ``side_stream``."""
        eng = self.engine
        eng.comm_begin(side_stream)
        if self.exchange == "allreduce":
            with self._on(side_stream):
                self._dist.all_reduce(self._mean, group=self.group)       # sum of the partial sums, in place
        else:
            self._side_barrier(side_stream)       # every GPU's stored copies exist
            eng.comm_gather()
            self._side_barrier(side_stream)       # every GPU's columns have arrived everywhere
        eng.comm_exchanged()

    def comm_end(self):
        """Line 6 for this process's workers."""
        self.engine.comm_end()

    def local_step_end(self, grads):
        """The round's last local step and line 6 in one pass (equal to local_step + comm_end)."""
        self.engine.local_step_end(grads)

    # -- around it
    def set_params(self, x0):
        self.engine.set_params(x0)

    def set_lr(self, lr: float):
        self.engine.set_lr(lr)

    def get_params(self, out=None):
        return self.engine.get_params(out)

    def get_momentum(self, out=None):
        return self.engine.get_momentum(out)

    def get_mean(self, out=None):
        return self.engine.get_mean(out)

    def sync(self):
        self.engine.sync()

    def close(self):
        """Collective: every process calls it.  Nobody unmaps or frees a buffer that another
        process's kernels may still address."""
        if self.engine is None:
            return
        self.engine.sync()
        self._host_barrier()
        if self._attached:
            self.engine.ipc_detach()
            self._attached = False
            self._host_barrier()
        self.engine.destroy()
        self.engine = None
