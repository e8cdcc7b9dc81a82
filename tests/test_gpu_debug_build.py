"""The checked build (liblocal_adaalter_debug.so, the library compiled with -DLA_DEBUG): its kernels
range-check every address they form.  It stands in for compute-sanitizer: on the shapes below no
kernel of any fusion mode, worker count or gradient source forms an address outside its ranges or
off its row, the results stay bitwise those of the oracle, and the report path works (shown with
the narrowing knob, which flags in-bounds accesses — no bad address is ever formed)."""
import os
import subprocess
import sys

import pytest

from paper_1911_09030_b200 import local_adaalter as la

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import os, sys
sys.path.insert(0, os.environ["LA_ROOT"])
import numpy as np, torch
from paper_1911_09030_b200 import local_adaalter as la
from paper_1911_09030_b200.worker_sharded import CudaEngine, WorkerShardedJob
from oracle.oracle import Oracle
assert la.debug_build(), "the checked library was not loaded"
rng = np.random.default_rng(3)
launches = 0
for W in (1, 3, 4, 5, 8, 16, 33, 48):
    for n in (4, 1001, 70002):
        a = rng.uniform(0.1, 10, n).astype(np.float32); c = rng.standard_normal(n).astype(np.float32)
        for fusion in (0, 1, 2, 3, 4):
            for bf16 in (False, True):
                if bf16 and fusion in (0, 2):
                    continue
                H, T = 3, 8
                g = la.LocalAdaAlter([n], W, 0.1, 1.0, H)
                o = Oracle(n, W, 0.1, 1.0, H)
                g.set_grad_quadratic(9, a, c, 0.3); o.set_grad_quadratic(9, a, c, 0.3)
                if bf16:
                    g.set_grad_dtype(la.LA_BF16); o.set_grad_bf16(True)
                g.set_fusion(fusion)
                g.run(T); o.run(T)
                g.stream_sync()                       # LA_EBOUNDS here if any kernel left its ranges
                for i in (0, W - 1):
                    for u, v in zip(g.read_state(i), o.read(i)):
                        assert np.array_equal(u.view(np.uint32), v.view(np.uint32)), (W, n, fusion, bf16, i)
                st = g.get_stats()
                launches += st["launches_local"] + st["launches_sync"] + st["launches_fused"]
                g.close()
# supplied gradient tables (vector and scalar paths), both rules that take them, bf16 and fp32
for W, n in ((4, 4096), (8, 1001), (5, 70002)):
    for dtype, tdt in ((la.LA_F32, torch.float32), (la.LA_BF16, torch.bfloat16)):
        for rule in (la.LA_RULE_ADAALTER, la.LA_RULE_ADAGRAD):
            g = la.LocalAdaAlter([n], W, 0.1, 1.0, 2)
            g.set_rule(rule)
            g.set_fusion(1 if W == 8 else 4)
            for t in range(5):
                G = torch.randn(W, n, device="cuda").to(tdt)
                g.step_grads(G.data_ptr(), dtype)
                g.stream_sync()
            g.close()
# the two baseline rules with generated gradients, and the hand-over between rules
g = la.LocalAdaAlter([70002], 6, 0.1, 1.0, 4)
g.set_grad_noise(5, None)
for rule in (la.LA_RULE_LOCAL_SGD, la.LA_RULE_ADAGRAD, la.LA_RULE_ADAALTER):
    g.set_rule(rule)
    g.run(8)
    g.stream_sync()
g.close()
# by-worker passes (export / import, exchange-fused steps) with one rank
g = la.LocalAdaAlter([70002], 4, 0.1, 1.0, la.LA_H_NEVER)
g.set_grad_noise(5, None)
job = WorkerShardedJob(CudaEngine(g, 0, 1), 3, exchange="peer", fused=True)
job.run(10)
g.stream_sync()
job = WorkerShardedJob(CudaEngine(g, 0, 1), 2, exchange="peer", fused=False)
job.run(5)
g.stream_sync()
g.close()
print("CHECKED_CLEAN", launches)

# The report path.  The last row of the arena is declared foreign: the accesses that (legitimately)
# go there are skipped and counted, and the next synchronising call says so.
n, W = 1001, 4
g = la.LocalAdaAlter([n], W, 0.1, 1.0, 2)
g.set_grad_constant(np.ones(n, np.float32))           # reads the last array of the arena (s)
g.debug_narrow(4 * 1024)
g.run(2)
try:
    g.stream_sync()
    raise SystemExit("the narrowed range was not reported")
except la.LocalAdaAlterError as e:
    assert e.code == la.LA_EBOUNDS and "outside every range" in str(e), str(e)
g.debug_narrow(0)
g.set_init(None, 0.0)
g.run(2)
g.stream_sync()                                       # clean again, and the count was cleared
x = g.read_state(0)[0]
o = Oracle(n, W, 0.1, 1.0, 2); o.set_grad_constant(np.ones(n, np.float32)); o.run(2)
assert np.array_equal(x.view(np.uint32), o.read(0)[0].view(np.uint32))
g.close()
print("CHECKED_REPORTS")
'''


def test_checked_build_is_clean_and_reports(tmp_path):
    script = tmp_path / "checked.py"
    script.write_text(CHILD)
    env = dict(os.environ, LA_ROOT=ROOT, LA_LIBRARY="debug")
    r = subprocess.run([sys.executable, str(script)], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "CHECKED_CLEAN" in r.stdout and "CHECKED_REPORTS" in r.stdout


def test_normal_library_is_not_the_checked_build():
    assert not la.debug_build()
    g = la.LocalAdaAlter([64], 2, 0.1, 1.0, 2)
    with pytest.raises(la.LocalAdaAlterError) as e:
        g.debug_narrow(256)
    assert e.value.code == la.LA_ESTATE
    g.close()
