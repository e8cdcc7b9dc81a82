"""The multi-rank path on CPU: two gloo ranks each take their coordinate shard, run the oracle
on it, and the gathered result equals the single-process run; timings reduce with MAX."""
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

from paper_1911_09030_b200 import sharding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import os, sys
sys.path.insert(0, os.environ["LA_ROOT"])
import numpy as np, torch, torch.distributed as dist
from paper_1911_09030_b200 import sharding, workloads
from oracle.oracle import Oracle
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
N, W, T = 1000, 4, 13
wl = workloads.config("c1")
lo, hi = sharding.coordinate_shard(N, rank, world)
arr = wl.arrays(lo, hi - lo)
o = Oracle(hi - lo, W, wl.eta, wl.eps, wl.H, j_base=lo)
o.set_grad_quadratic(wl.noise_seed, arr["a"], arr["c"], wl.sigma)
o.run(T)
x = np.stack([o.read(i)[0] for i in range(W)])
pieces = [None] * world
dist.all_gather_object(pieces, (lo, hi, x, o.counters()))
slow = sharding.max_over_ranks(1.0 + rank, dist)
# weak-scaling bases are disjoint
bases = [None] * world
dist.all_gather_object(bases, sharding.weak_scaling_base(N, rank))
if rank == 0:
    full = Oracle(N, W, wl.eta, wl.eps, wl.H)
    a = wl.arrays(0, N)
    full.set_grad_quadratic(wl.noise_seed, a["a"], a["c"], wl.sigma)
    full.run(T)
    ref = np.stack([full.read(i)[0] for i in range(W)])
    pieces.sort(key=lambda p: p[0])
    got = np.concatenate([p[2] for p in pieces], axis=1)
    assert pieces[0][0] == 0 and pieces[-1][1] == N
    assert all(p[1] == q[0] for p, q in zip(pieces, pieces[1:]))
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))
    assert all(p[3] == full.counters() for p in pieces)
    assert slow == float(world)
    assert bases == [r * 1000 for r in range(world)]
    print("SHARDING_OK")
dist.destroy_process_group()
'''


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_coordinate_shards_cover_and_align():
    for N in (1, 3, 4, 5, 1000, 1001, 65536, 400007886):
        for world in (1, 2, 3, 4, 8):
            sh = sharding.all_shards(N, world)
            assert sh[0][0] == 0 and sh[-1][1] == N
            assert all(a[1] == b[0] for a, b in zip(sh, sh[1:]))
            assert all(lo % 4 == 0 for lo, _ in sh)
            sizes = [hi - lo for lo, hi in sh]
            assert max(sizes) - min(sizes) <= 4 + 3
    with pytest.raises(ValueError):
        sharding.coordinate_shard(10, 2, 2)


def test_two_gloo_ranks_reproduce_the_single_process_job(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, LA_ROOT=ROOT, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), str(script)]
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "SHARDING_OK" in r.stdout


def test_reference_arm_runs_on_rank0_only(tmp_path):
    """`bench.py --impl reference` under torchrun: rank 0 prints the line, the others exit 0."""
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()),
           os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
           "--workload", "c1"]
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-3000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    import json
    doc = json.loads(lines[0])
    assert doc["impl"] == "reference" and doc["cpu_baseline"]["kind"] == "oracle" and doc["value"] > 0


WORKER_BY_WORKER = r'''
import os, sys
sys.path.insert(0, os.environ["LA_ROOT"])
import numpy as np, torch, torch.distributed as dist
from paper_1911_09030_b200.worker_sharded import WorkerShardedJob
from oracle.oracle import Oracle

class OracleEngine:
    """CPU stand-in for the CUDA engine (test infrastructure): the local replicas live in an
    oracle instance; export/import are written out with numpy."""
    def __init__(self, o, W_local, W_total, n):
        self.o, self.W, self.W_total, self.n = o, W_local, W_total, n
        self.buf = torch.zeros(2 * n, dtype=torch.float32)
    def local_step(self): self.o.local_step()
    def t_prime(self): return self.o.counters()[1]
    def stream_sync(self): pass
    def _tree(self, rows):
        rows = list(rows)
        while len(rows) > 1:
            nxt = [rows[k] + rows[k + 1] for k in range(0, len(rows) - 1, 2)]
            if len(rows) % 2: nxt.append(rows[-1])
            rows = nxt
        return rows[0]
    def export(self):
        xs, bs = zip(*[self.o.read(i)[:2] for i in range(self.W)])
        self.buf[:self.n] = torch.from_numpy(self._tree(xs))
        self.buf[self.n:] = torch.from_numpy(self._tree(bs))
    def combine(self): raise AssertionError("peer exchange needs device memory")
    def buffer_tensor(self): return self.buf
    def step_export(self):          # the closing step, then its sums (the CUDA engine never stores y, A^2)
        self.o.local_step(); self.export()
    def import_step(self):          # the means, then the first step of the next period
        self.import_(); self.o.local_step()
    def import_(self):
        w = np.float32(self.W_total)
        xm = self.buf[:self.n].numpy() / w
        bm = self.buf[self.n:].numpy() / w
        for i in range(self.W):
            self.o.write(i, xm, bm, bm)
        t, tp, ns = self.o.counters()
        self.o.set_counters(t, 0, ns + 1)

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
n, W_local, H, T = 257, 4, 3, 10
W_total = W_local * world
rng = np.random.default_rng(0)
a = rng.uniform(0.1, 10, n).astype(np.float32); c = rng.standard_normal(n).astype(np.float32)
o = Oracle(n, W_local, 0.1, 1.0, 0xFFFFFFFF)
o.set_grad_quadratic(9, a, c, 0.3)
o.set_worker_base(rank * W_local)
job = WorkerShardedJob(OracleEngine(o, W_local, W_total, n), H, exchange="allreduce", dist=dist,
                       fused=os.environ.get("LA_FUSED") == "1")
job.run(4)                      # ends inside a period; the schedule carries on in the next call
job.run(T - 4)
assert job.exchange_seconds > 0.0
mine = np.stack([o.read(i)[0] for i in range(W_local)])
parts = [None] * world
dist.all_gather_object(parts, (rank, mine, o.counters(), job.syncs))
if rank == 0:
    full = Oracle(n, W_total, 0.1, 1.0, H)
    full.set_grad_quadratic(9, a, c, 0.3)
    full.run(T)
    for r, xs, cnt, syncs in parts:
        assert cnt == full.counters() and syncs == T // H
        for i in range(W_local):
            ref = full.read(r * W_local + i)[0]
            assert np.array_equal(xs[i].view(np.uint32), ref.view(np.uint32)), (r, i)
    print("BY_WORKER_OK")
dist.destroy_process_group()
'''


@pytest.mark.parametrize("fused", [False, True])
def test_two_gloo_ranks_sharded_by_worker(tmp_path, fused):
    """The by-worker choreography (export, all-reduce, import, counters; also with the steps next to
    a synchronisation fused into the exchange) on two CPU ranks with an oracle-backed engine equals
    the single-process oracle with W_total workers, bitwise."""
    script = tmp_path / "by_worker.py"
    script.write_text(WORKER_BY_WORKER)
    env = dict(os.environ, LA_ROOT=ROOT, MASTER_ADDR="127.0.0.1", LA_FUSED="1" if fused else "0")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), str(script)]
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "BY_WORKER_OK" in r.stdout
