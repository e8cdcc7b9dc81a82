"""GPU parity at the full sizes of configurations 2-5, in the launch configuration the
benchmark times, checked on sampled coordinate ranges (both ends of the vector, every
tensor boundary, seeded random windows).  Sampling is exact: coordinates never interact in
Algorithm 3, and the oracle is keyed on global coordinate indices."""
import numpy as np
import pytest

from oracle.oracle import Oracle
from paper_1911_09030_b200 import local_adaalter as la
from paper_1911_09030_b200 import workloads
from parity_util import max_scaled_err

pytestmark = pytest.mark.gpu

TOL_STEP, TOL_RUN = 1e-6, 1e-5


def _make_gpu(wl, arr, H, fusion):
    g = la.LocalAdaAlter.with_torch_arena(wl.sizes, wl.W, wl.eta, wl.eps, H, b0sq=wl.b0sq)
    if wl.grad == "quadratic":
        g.set_grad_quadratic(wl.noise_seed, arr["a"], arr["c"], wl.sigma)
    elif wl.grad == "noise_scaled":
        g.set_grad_noise(wl.noise_seed, arr["s"])
    else:
        g.set_grad_noise(wl.noise_seed, None)
    if wl.bf16_grads:
        g.set_grad_dtype(la.LA_BF16)
    g.set_fusion(fusion)
    return g


def _make_oracle(wl, arr, H, lo, hi):
    o = Oracle(hi - lo, wl.W, wl.eta, wl.eps, H, wl.b0sq, j_base=lo)
    if wl.grad == "quadratic":
        o.set_grad_quadratic(wl.noise_seed, arr["a"][lo:hi], arr["c"][lo:hi], wl.sigma)
    elif wl.grad == "noise_scaled":
        o.set_grad_noise(wl.noise_seed, arr["s"][lo:hi])
    else:
        o.set_grad_noise(wl.noise_seed, None)
    if wl.bf16_grads:
        o.set_grad_bf16(True)
    return o


def _check(g, oracles, ranges, W, tol):
    for (lo, hi), o in zip(ranges, oracles):
        for i in range(W):
            gx, gb, gs = g.read_range(i, lo, hi - lo)
            ox, ob, os_ = o.read(i)
            for name, a, b in (("x", gx, ox), ("B2", gb, ob), ("Bs", gs, os_)):
                assert np.all(np.isfinite(a))
                e = max_scaled_err(a, b)
                assert e <= tol, f"{name} worker {i} range {lo}:{hi}: {e:.3e}"
                bad = np.flatnonzero(a.view(np.uint32) != b.view(np.uint32))
                assert bad.size == 0, f"{name} worker {i} range {lo}:{hi}: {bad.size} bitwise mismatches"
        assert g.get_counters() == o.counters()


def _run_config(name, H=None, fusion=la.LA_FUSE_STEP_SYNC, span=2048, extra=3):
    wl = workloads.config(name)
    H = wl.H if H is None else H
    arr = wl.arrays()
    ranges = workloads.sample_ranges(wl, span=span, extra=extra)
    g = _make_gpu(wl, arr, H, fusion)
    oracles = [_make_oracle(wl, arr, H, lo, hi) for lo, hi in ranges]
    g.run(1)
    for o in oracles:
        o.run(1)
    _check(g, oracles, ranges, wl.W, TOL_STEP)
    g.run(wl.T - 1)
    for o in oracles:
        o.run(wl.T - 1)
    _check(g, oracles, ranges, wl.W, TOL_RUN)
    assert g.get_counters() == (wl.T, wl.T % H, wl.T // H)
    g.close()


def test_config2_flat_scaled_noise():
    _run_config("c2", span=1024, extra=2)


def test_config2_period_fusion():
    _run_config("c2", fusion=la.LA_FUSE_PERIOD, span=1024, extra=2)


def test_config3_six_tensors_quadratic():
    _run_config("c3", span=2048, extra=3)


@pytest.mark.parametrize("H,fusion", [(1, 2), (4, 0), (16, 1), (64, 2), (16, 3)])
def test_config4_sync_period_sweep(H, fusion):
    _run_config("c4", H=H, fusion=fusion, span=512, extra=2)


def test_config5_ragged_bf16():
    wl = workloads.config("c5")
    assert len(wl.sizes) == 200 and min(wl.sizes) >= 1024 and abs(wl.N - 4e8) < 4e6
    _run_config("c5", span=1024, extra=2)
    _run_config("c5", fusion=la.LA_FUSE_PERIOD, span=512, extra=1)


def test_beyond_32_bit_indexing():
    """W x N above 2^32 elements (17 GiB per state array): every offset computation is 64-bit.
    Checked on windows at both ends of the vector and around the 2^32-byte and 2^32-element
    marks of replica rows."""
    N, W, H, T = (1 << 30) + 6, 4, 3, 4
    g = la.LocalAdaAlter.with_torch_arena([N], W, 0.05, 0.5, H, b0sq=0.0)
    g.set_grad_noise(11, None)
    g.set_fusion(la.LA_FUSE_STEP_SYNC)
    g.run(2)
    g.set_fusion(la.LA_FUSE_PERIOD)
    g.run(T - 2)
    ranges = [(0, 256), ((1 << 29) - 128, (1 << 29) + 128), (N - 262, N), (123456788, 123456788 + 200)]
    for lo, hi in ranges:
        o = Oracle(hi - lo, W, 0.05, 0.5, H, 0.0, j_base=lo)
        o.set_grad_noise(11, None)
        o.run(T)
        for i in range(W):
            for a, b in zip(g.read_range(i, lo, hi - lo), o.read(i)):
                assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), (lo, i)
        assert g.get_counters() == o.counters()
    g.close()


def _deep_ranges(wl, nblocks=64, block=1 << 16, ends=4096, around=8):
    """At least 2^22 coordinates of the full-size vector: `nblocks` blocks spread evenly (so that
    every part of the grid is hit), both ends, and a window around every tensor boundary."""
    N = wl.N
    want = [(0, min(ends, N)), (max(0, (N - ends) // 4 * 4), N)]
    step = N // nblocks
    for k in range(nblocks):
        lo = (k * step) // 4 * 4
        want.append((lo, min(N, lo + block)))
    off = 0
    for sz in wl.sizes[:-1]:
        off += sz
        lo = max(0, (off - around) // 4 * 4)
        want.append((lo, min(N, lo + 2 * around + 4)))
    want.sort()
    merged = []
    for lo, hi in want:
        if merged and lo <= merged[-1][1]:
            merged[-1] = (merged[-1][0], max(merged[-1][1], hi))
        else:
            merged.append((lo, hi))
    return merged


DEEP_CASES = [("c2", None, (1, 3, 4)), ("c3", None, (1, 3, 4)), ("c5", None, (1, 3, 4)),
              ("c4", 1, (2,)), ("c4", 4, (0, 4)), ("c4", 16, (1, 3)), ("c4", 64, (2,))]


@pytest.mark.parametrize("name,H,fusions", DEEP_CASES, ids=[f"{n}-H{h}-f{''.join(map(str, f))}" for n, h, f in DEEP_CASES])
def test_full_size_run_on_four_million_coordinates(name, H, fusions):
    """Each configuration at full size, full W and T, in the launch configuration the benchmark
    times; the oracle re-computes >= 2^22 coordinates (blocks spread over the whole vector, both
    ends, every tensor boundary), one block per host thread; every x, B^2 and stale B^2 of every
    worker must agree bit for bit.  One oracle pass serves all fusion modes of a case."""
    import os
    import threading
    from concurrent.futures import ThreadPoolExecutor
    wl = workloads.config(name)
    H = wl.H if H is None else H
    arr = wl.arrays()
    gpus = []
    for fusion in fusions:
        g = _make_gpu(wl, arr, H, fusion)
        g.run(wl.T)
        assert g.get_counters() == (wl.T, wl.T % H, wl.T // H)
        gpus.append(g)
    ranges = _deep_ranges(wl)
    assert sum(hi - lo for lo, hi in ranges) >= 1 << 22
    ctx_lock = threading.Lock()                      # a context serves one caller thread at a time

    def check(rng):
        lo, hi = rng
        o = _make_oracle(wl, arr, H, lo, hi)
        o.run(wl.T)
        bad = 0
        for i in range(wl.W):
            ref = o.read(i)
            for g in gpus:
                with ctx_lock:
                    got = g.read_range(i, lo, hi - lo)
                for a, b in zip(got, ref):
                    bad += int(np.count_nonzero(a.view(np.uint32) != b.view(np.uint32)))
        o.close()
        return bad

    with ThreadPoolExecutor(max_workers=min(32, os.cpu_count() or 1)) as ex:
        mismatches = sum(ex.map(check, ranges))
    assert mismatches == 0
    for g in gpus:
        g.close()
