"""Sharding by worker on the GPU: the three-phase synchronisation (export / combine / import)
against the single-context kernels and the oracle.  Several ranks are emulated as several
contexts of one process on one GPU and one stream (their kernels never wait for each other;
the host orders the phases)."""
import numpy as np
import pytest

from oracle.oracle import Oracle
from paper_1911_09030_b200 import local_adaalter as la
from paper_1911_09030_b200.worker_sharded import CudaEngine, WorkerShardedJob

pytestmark = pytest.mark.gpu


def _arrays(n, seed):
    rng = np.random.default_rng(seed)
    return rng.uniform(0.1, 10, n).astype(np.float32), rng.standard_normal(n).astype(np.float32)


def _single(n, W, H, a, c, T):
    g = la.LocalAdaAlter([n], W, 0.1, 1.0, H)
    g.set_grad_quadratic(9, a, c, 0.3)
    g.run(T)
    return g


@pytest.mark.parametrize("n", [64, 1000, 70001])
def test_world_of_one_equals_la_sync(n):
    W, H, T = 4, 3, 10
    a, c = _arrays(n, n)
    ref = _single(n, W, H, a, c, T)
    g = la.LocalAdaAlter([n], W, 0.1, 1.0, la.LA_H_NEVER)
    g.set_grad_quadratic(9, a, c, 0.3)
    job = WorkerShardedJob(CudaEngine(g, 0, 1), H, exchange="peer")
    job.run(T)
    assert g.get_counters() == ref.get_counters() == (T, T % H, T // H)
    for i in range(W):
        for u, v in zip(g.read_state(i), ref.read_state(i)):
            assert np.array_equal(u.view(np.uint32), v.view(np.uint32))


@pytest.mark.parametrize("world,W_local", [(2, 4), (4, 2), (2, 1), (3, 2), (8, 2)])
def test_emulated_ranks_equal_single_gpu_job_bitwise(world, W_local):
    n, H, T = 5000, 4, 9
    W_total = world * W_local
    a, c = _arrays(n, world * 10 + W_local)
    ref = _single(n, W_total, H, a, c, T)
    o = Oracle(n, W_total, 0.1, 1.0, H)
    o.set_grad_quadratic(9, a, c, 0.3)
    o.run(T)
    ctxs = []
    for r in range(world):
        g = la.LocalAdaAlter([n], W_local, 0.1, 1.0, la.LA_H_NEVER)
        g.set_grad_quadratic(9, a, c, 0.3)
        g.comm_create(r, world)
        ctxs.append(g)
    for r in range(world):
        for q in range(world):
            if q != r:
                ctxs[r].comm_set_peer(q, ctxs[q].comm_buffer()[0])
    for t in range(1, T + 1):
        for g in ctxs:
            g.local_step()
        if t % H == 0:
            for g in ctxs:
                g.comm_export()
            for g in ctxs:
                g.stream_sync()
            for g in ctxs:
                g.comm_combine()
            for g in ctxs:
                g.stream_sync()
            for g in ctxs:
                g.comm_import()
    for r, g in enumerate(ctxs):
        assert g.get_counters() == ref.get_counters()
        for i in range(W_local):
            gw = r * W_local + i
            for name, u, v, w in zip("x b2 bs".split(), g.read_state(i), ref.read_state(gw), o.read(gw)):
                assert np.array_equal(u.view(np.uint32), w.view(np.uint32)), f"{name} vs oracle, rank {r} worker {i}"
                if W_local & (W_local - 1) == 0:
                    assert np.array_equal(u.view(np.uint32), v.view(np.uint32)), f"{name} vs single GPU"


def test_allreduce_mode_with_one_rank_and_buffer_alias():
    n, W, H, T = 3000, 8, 2, 6
    a, c = _arrays(n, 3)
    ref = _single(n, W, H, a, c, T)
    g = la.LocalAdaAlter([n], W, 0.1, 1.0, la.LA_H_NEVER)
    g.set_grad_quadratic(9, a, c, 0.3)
    eng = CudaEngine(g, 0, 1)
    job = WorkerShardedJob(eng, H, exchange="allreduce")
    job.run(T)
    buf = eng.buffer_tensor()
    assert buf.is_cuda and buf.numel() == 2 * ((n + 63) // 64 * 64)
    x0 = g.read_state(0)[0]
    assert np.array_equal(x0, ref.read_state(0)[0])
    # after the last import the buffer still holds the totals: mean = total / W
    np.testing.assert_array_equal((buf[:n].cpu().numpy() / np.float32(W)), x0)


def test_misuse_is_reported():
    g = la.LocalAdaAlter([64], 2, 0.1, 1.0, 2)
    with pytest.raises(la.LocalAdaAlterError):
        g.comm_export()                      # no exchange buffer yet
    g.comm_create(0, 2)
    with pytest.raises(la.LocalAdaAlterError) as e:
        g.comm_combine()                     # peer 1 not attached
    assert "not attached" in str(e.value)
    with pytest.raises(la.LocalAdaAlterError):
        g.comm_create(3, 2)
    with pytest.raises(la.LocalAdaAlterError):
        g.set_worker_range(7, 8)
    # three local workers on each of two ranks would not reproduce the adjacent-pair tree over six
    g3 = la.LocalAdaAlter([64], 3, 0.1, 1.0, 2)
    with pytest.raises(la.LocalAdaAlterError) as e:
        g3.comm_create(0, 2)
    assert e.value.code == la.LA_EINVAL and "power of two" in str(e.value)
    g3.comm_create(0, 1)                     # a single rank may hold any number of workers


TWO_PROCESS = r'''
import os, sys
sys.path.insert(0, os.environ["LA_ROOT"])
import numpy as np, torch, torch.distributed as dist
from paper_1911_09030_b200 import local_adaalter as la
from paper_1911_09030_b200.worker_sharded import CudaEngine, WorkerShardedJob
from oracle.oracle import Oracle
mode = os.environ["LA_MODE"]
dist.init_process_group("gloo")               # host barriers, handle exchange; in the all-reduce mode also the collective
rank, world = dist.get_rank(), dist.get_world_size()
torch.cuda.set_device(0)                      # both ranks share the one GPU; no kernel waits for the other rank
n, W_local, H, T = 40000, 4, 3, 11
rng = np.random.default_rng(0)
a = rng.uniform(0.1, 10, n).astype(np.float32); c = rng.standard_normal(n).astype(np.float32)
o = Oracle(n, W_local * world, 0.1, 1.0, H)
own = torch.cuda.Stream() if mode == "allreduce_fused_own_stream" else None
g = la.LocalAdaAlter([n], W_local, 0.1, 1.0, la.LA_H_NEVER, stream=own.cuda_stream if own else None)
if mode == "supplied":
    # caller-supplied gradients: every rank draws the full [W_total][n] table from the same seed and
    # passes its own rows; the step that completes a period is fused with the export
    eng = CudaEngine(g, rank, world)
    eng.attach_peers(dist)
    job = WorkerShardedJob(eng, H, exchange="peer", dist=dist)
    grng = np.random.default_rng(1)
    for t in range(1, T + 1):
        G = grng.standard_normal((W_local * world, n)).astype(np.float32)
        if rank == 0:
            o.local_step(G)
        Gd = torch.from_numpy(G[rank * W_local:(rank + 1) * W_local].copy()).cuda()
        if t % H == 0:
            g.comm_step_grads_export(Gd.data_ptr(), la.LA_F32)
            job._exchange()
            g.comm_import()
            if rank == 0:
                o.sync()
        else:
            g.local_step_grads(Gd.data_ptr(), la.LA_F32)
        g.stream_sync()                       # Gd is released at the end of the iteration
else:
    g.set_grad_quadratic(9, a, c, 0.3)
    o.set_grad_quadratic(9, a, c, 0.3)
    eng = CudaEngine(g, rank, world)
    eng.attach_peers(dist)                    # CUDA IPC handles through the process group
    job = WorkerShardedJob(eng, H, exchange="allreduce" if mode.startswith("allreduce") else "peer", dist=dist,
                           fused=mode != "peer")
    job.run(5)                                # ends inside a period ...
    job.run(T - 5)                            # ... and the schedule carries on
    assert job.syncs == T // H
    if rank == 0:
        o.run(T)
g.stream_sync()
mine = [g.read_state(i) for i in range(W_local)]
parts = [None] * world
dist.all_gather_object(parts, (rank, mine, g.get_counters(), g.get_stats()))
dist.barrier()
if rank == 0:
    for r, st, cnt, stats in parts:
        assert cnt == o.counters(), (cnt, o.counters())
        if mode != "peer":
            assert stats["launches_fused"] >= T // H          # the exchange-fused kernels ran
        for i in range(W_local):
            for u, v in zip(st[i], o.read(r * W_local + i)):
                assert np.array_equal(u.view(np.uint32), v.view(np.uint32)), (r, i)
    print("IPC_PEER_OK", mode)
g.close()
dist.destroy_process_group()
'''


@pytest.mark.parametrize("mode", ["peer", "peer_fused", "allreduce_fused_own_stream", "supplied"])
def test_two_processes_exchange_through_cuda_ipc(tmp_path, mode):
    """Two OS processes (gloo for the host-side barriers and the handle exchange) map each other's
    exchange buffer with CUDA IPC and synchronise across the process boundary; the result is the
    oracle's with W_total workers, bitwise.  Both processes use the same GPU here.
      peer                        export, peer-load combine kernel, import
      peer_fused                  the steps next to a synchronisation fused with the exchange
                                  (step+export, combine, import+step)
      allreduce_fused_own_stream  the same with the buffer all-reduced by torch.distributed (two ranks:
                                  one addition per element, so still bitwise) and the context on a
                                  stream of its own, so the ordering between the context's stream
                                  and the collective is what makes it pass
      supplied                    caller-supplied gradient tables, the closing step fused with the export"""
    import os, socket, subprocess, sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script = tmp_path / "ipc_worker.py"
    script.write_text(TWO_PROCESS)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ, LA_ROOT=root, MASTER_ADDR="127.0.0.1", LA_MODE=mode)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", str(port), str(script)]
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "IPC_PEER_OK " + mode in r.stdout


@pytest.mark.parametrize("H,T", [(2, 9), (3, 10), (4, 8), (5, 5), (1, 4)])
def test_fused_exchange_steps_with_one_rank(H, T):
    n, W = 30001, 8
    a, c = _arrays(n, H)
    ref = _single(n, W, H, a, c, T)
    g = la.LocalAdaAlter([n], W, 0.1, 1.0, la.LA_H_NEVER)
    g.set_grad_quadratic(9, a, c, 0.3)
    job = WorkerShardedJob(CudaEngine(g, 0, 1), H, exchange="peer", fused=True)
    job.run(3)
    job.run(T - 3)
    assert g.get_counters() == ref.get_counters()
    assert job.syncs == T // H
    for i in range(W):
        for u, v in zip(g.read_state(i), ref.read_state(i)):
            assert np.array_equal(u.view(np.uint32), v.view(np.uint32))
    if H > 1:
        st = g.get_stats()
        assert st["launches_fused"] >= T // H          # step+export / import+step kernels were used


@pytest.mark.parametrize("world,W_local,grad", [(2, 4, "quadratic"), (4, 2, "noise"), (2, 8, "supplied")])
def test_fused_exchange_steps_with_emulated_ranks(world, W_local, grad):
    import torch
    n, H, T = 6002, 3, 8
    W_total = world * W_local
    a, c = _arrays(n, 5)
    o = Oracle(n, W_total, 0.1, 1.0, H)
    ctxs = []
    for r in range(world):
        g = la.LocalAdaAlter([n], W_local, 0.1, 1.0, la.LA_H_NEVER)
        g.comm_create(r, world)
        ctxs.append(g)
    if grad == "quadratic":
        o.set_grad_quadratic(9, a, c, 0.3)
        for g in ctxs:
            g.set_grad_quadratic(9, a, c, 0.3)
    elif grad == "noise":
        o.set_grad_noise(9, None)
        for g in ctxs:
            g.set_grad_noise(9, None)
    for r in range(world):
        for q in range(world):
            if q != r:
                ctxs[r].comm_set_peer(q, ctxs[q].comm_buffer()[0])
    rng = np.random.default_rng(1)

    def exchange():
        for g in ctxs:
            g.stream_sync()
        for g in ctxs:
            g.comm_combine()
        for g in ctxs:
            g.stream_sync()

    t = 0
    while t < T:
        closes = (ctxs[0].get_counters()[1] + 1 == H)
        if grad == "supplied":
            G = rng.standard_normal((W_total, n)).astype(np.float32)
            o.local_step(G)
            for r, g in enumerate(ctxs):
                Gd = torch.from_numpy(G[r * W_local:(r + 1) * W_local].copy()).cuda()
                if closes:
                    g.comm_step_grads_export(Gd.data_ptr(), la.LA_F32)
                else:
                    g.local_step_grads(Gd.data_ptr(), la.LA_F32)
                g.stream_sync()
            t += 1
            if closes:
                exchange()
                o.sync()
                if t < T:                         # the next iteration starts from the exchanged totals, in one pass
                    G = rng.standard_normal((W_total, n)).astype(np.float32)
                    o.local_step(G)
                    for r, g in enumerate(ctxs):
                        Gd = torch.from_numpy(G[r * W_local:(r + 1) * W_local].copy()).cuda()
                        g.comm_import_step_grads(Gd.data_ptr(), la.LA_F32)
                        g.stream_sync()
                    t += 1
                else:
                    for g in ctxs:
                        g.comm_import()
            continue
        if closes:
            for g in ctxs:
                g.comm_step_export()
            exchange()
            t += 1
            if t < T:
                for g in ctxs:
                    g.comm_import_step()
                t += 1
            else:
                for g in ctxs:
                    g.comm_import()
        else:
            for g in ctxs:
                g.local_step()
            t += 1
    if grad != "supplied":
        o.run(T)
    for r, g in enumerate(ctxs):
        assert g.get_counters() == o.counters()
        for i in range(W_local):
            for name, u, w in zip("x b2 bs".split(), g.read_state(i), o.read(r * W_local + i)):
                assert np.array_equal(u.view(np.uint32), w.view(np.uint32)), f"{name} rank {r} worker {i}"
