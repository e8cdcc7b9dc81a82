"""Algorithm 3 (Local AdaAlter) with the WORKERS spread over ranks, one process per GPU.

This is the layout the paper describes: every rank advances its own replicas locally and,
every H steps, all ranks exchange x and B^2 (Section 4.2).  The arithmetic runs in the CUDA
library; this module only orders the phases of a synchronisation and moves handles:

    export  (local tree sums -> exchange buffer)
    exchange, one of
      "peer":      stream sync + barrier, `combine` (each rank reduces its coordinate slice over
                   all ranks' buffers with peer loads and writes the total back to all), stream
                   sync + barrier
      "allreduce": stream sync, one all-reduce(SUM) of the exchange buffer by torch.distributed
                   (NCCL), wait for it
    import  (total / W_total -> every local replica, stale accumulator; t' = 0)

The engine is anything with the methods used below; the CUDA engine is `CudaEngine`.
"""
from __future__ import annotations

import time
from typing import Optional


class WorkerShardedJob:
    def __init__(self, engine, H: int, exchange: str = "peer", dist=None, group=None, fused: bool = False):
        """fused=True: the step that completes a period writes only its sums to the exchange buffer
        and the first step of the next period starts from the exchanged totals, so a
        synchronisation adds no pass over the replicas (engine needs step_export/import_step)."""
        if exchange not in ("peer", "allreduce"):
            raise ValueError("exchange must be 'peer' or 'allreduce'")
        self.engine, self.H, self.exchange, self.dist, self.group = engine, int(H), exchange, dist, group
        self.fused = bool(fused) and self.H > 1
        self.syncs = 0
        self.exchange_seconds = 0.0   # host time between "this rank's sums are ready" and "totals are back"

    def _barrier(self):
        if self.dist is not None and self.dist.is_initialized() and self.dist.get_world_size(self.group) > 1:
            self.dist.barrier(group=self.group)

    def sync(self):
        self.engine.export()
        self._exchange()
        self.engine.import_()
        self.syncs += 1

    def _exchange(self):
        e = self.engine
        multi = self.dist is not None and self.dist.is_initialized() and self.dist.get_world_size(self.group) > 1
        if self.exchange == "peer":
            e.stream_sync()
            t0 = time.perf_counter()
            self._barrier()            # every rank's sums are in its buffer
            e.combine()
            e.stream_sync()
            self._barrier()            # every slice of every buffer holds the total
            self.exchange_seconds += time.perf_counter() - t0
        elif multi:
            buf = e.buffer_tensor()
            # The export kernel ran on the context's stream, the collective runs on the process
            # group's: finish the first before the second reads the buffer, and finish the second
            # before the import kernel (context stream again) reads the totals.
            e.stream_sync()
            t0 = time.perf_counter()
            self.dist.all_reduce(buf, op=self.dist.ReduceOp.SUM, group=self.group)
            done = getattr(e, "collective_done", None)
            if done is not None:
                done()
            self.exchange_seconds += time.perf_counter() - t0

    def run(self, T: int):
        """T iterations of Algorithm 3: local step; if t' == H: synchronise."""
        e, k, T = self.engine, 0, int(T)
        while k < T:
            if self.fused and e.t_prime() + 1 == self.H:
                e.step_export()                 # iteration k: the step that completes the period
                self._exchange()
                k += 1
                if k < T:
                    e.import_step()             # iteration k+1 starts from the exchanged means
                    k += 1
                else:
                    e.import_()
                self.syncs += 1
            else:
                e.local_step()
                k += 1
                if e.t_prime() == self.H:
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

    def step_export(self):
        self.ctx.comm_step_export()

    def import_step(self):
        self.ctx.comm_import_step()

    def stream_sync(self):
        self.ctx.stream_sync()

    def collective_done(self):
        """Block until the collective torch enqueued on its current stream has finished."""
        import torch
        torch.cuda.current_stream().synchronize()

    def buffer_tensor(self):
        if self._tensor is None:
            import torch
            ptr, nbytes = self.ctx.comm_buffer()
            self._tensor = torch.as_tensor(_DeviceBuffer(ptr, nbytes // 4), device="cuda")
        return self._tensor
