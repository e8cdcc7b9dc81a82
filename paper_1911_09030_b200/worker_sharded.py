"""Algorithm 3 (Local AdaAlter) with the WORKERS spread over ranks, one process per GPU.

This is the layout the paper describes: every rank advances its own replicas locally and,
every H steps, all ranks exchange x and B^2 (Section 4.2).  The arithmetic runs in the CUDA
library; this module only orders the phases of a synchronisation and moves handles:

    export  (local tree sums -> exchange buffer)
    exchange, one of
      "peer":      stream sync + barrier, `combine` (each rank reduces its coordinate slice over
                   all ranks' buffers with peer loads and writes the total back to all), stream
                   sync + barrier
      "allreduce": one all-reduce(SUM) of the exchange buffer by torch.distributed (NCCL)
    import  (total / W_total -> every local replica, stale accumulator; t' = 0)

The engine is anything with the methods used below; the CUDA engine is `CudaEngine`.
"""
from __future__ import annotations

from typing import Optional


class WorkerShardedJob:
    def __init__(self, engine, H: int, exchange: str = "peer", dist=None, group=None):
        if exchange not in ("peer", "allreduce"):
            raise ValueError("exchange must be 'peer' or 'allreduce'")
        self.engine, self.H, self.exchange, self.dist, self.group = engine, int(H), exchange, dist, group
        self.syncs = 0

    def _barrier(self):
        if self.dist is not None and self.dist.is_initialized() and self.dist.get_world_size(self.group) > 1:
            self.dist.barrier(group=self.group)

    def sync(self):
        e = self.engine
        e.export()
        if self.exchange == "peer":
            e.stream_sync()
            self._barrier()            # every rank's sums are in its buffer
            e.combine()
            e.stream_sync()
            self._barrier()            # every slice of every buffer holds the total
        else:
            buf = e.buffer_tensor()
            if self.dist is not None and self.dist.is_initialized() and self.dist.get_world_size(self.group) > 1:
                self.dist.all_reduce(buf, op=self.dist.ReduceOp.SUM, group=self.group)
        e.import_()
        self.syncs += 1

    def run(self, T: int):
        """T iterations of Algorithm 3: local step; if t' == H: synchronise."""
        for _ in range(int(T)):
            self.engine.local_step()
            if self.engine.t_prime() == self.H:
                self.sync()


class _DeviceBuffer:
    """Minimal __cuda_array_interface__ carrier so that torch can alias library-owned memory."""

    def __init__(self, ptr: int, nfloats: int):
        self.__cuda_array_interface__ = {"shape": (nfloats,), "typestr": "<f4", "data": (ptr, False), "version": 2}


class CudaEngine:
    """The CUDA library as the engine of a WorkerShardedJob."""

    def __init__(self, ctx, rank: int, world: int):
        self.ctx, self.rank, self.world = ctx, int(rank), int(world)
        ctx.comm_create(rank, world)
        self._tensor = None

    def attach_peers(self, dist, group=None):
        """Exchange CUDA IPC handles of the exchange buffers and map every peer's buffer."""
        if self.world == 1:
            return
        handles = [None] * self.world
        dist.all_gather_object(handles, self.ctx.comm_ipc_handle(), group=group)
        for r, h in enumerate(handles):
            if r != self.rank:
                self.ctx.comm_open_peer(r, h)

    def local_step(self):
        self.ctx.local_step()

    def t_prime(self):
        return self.ctx.get_counters()[1]

    def export(self):
        self.ctx.comm_export()

    def combine(self):
        self.ctx.comm_combine()

    def import_(self):
        self.ctx.comm_import()

    def stream_sync(self):
        self.ctx.stream_sync()

    def buffer_tensor(self):
        if self._tensor is None:
            import torch
            ptr, nbytes = self.ctx.comm_buffer()
            self._tensor = torch.as_tensor(_DeviceBuffer(ptr, nbytes // 4), device="cuda")
        return self._tensor
