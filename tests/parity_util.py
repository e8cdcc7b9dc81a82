"""Helpers shared by the GPU parity tests: build the CUDA context and the CPU oracle from
the same seeded inputs and compare them."""
import numpy as np

from oracle.oracle import Oracle
from paper_1911_09030_b200 import local_adaalter as la


def make_pair(n, W, eta, eps, H, grad, *, b0sq=0.0, x0=None, seed=1, arrays=None, sigma=0.0,
              bf16=False, identical=False, warmup=0, fusion=0, sizes=None, j_base=0, oracle_range=None):
    """Returns (gpu_ctx, oracle).  `oracle_range=(lo, hi)` restricts the oracle to a coordinate
    range of the job (coordinates are independent)."""
    arrays = arrays or {}
    g = la.LocalAdaAlter(sizes if sizes is not None else [n], W, eta, eps, H, b0sq=b0sq, j_base=j_base)
    lo, hi = oracle_range if oracle_range else (0, n)
    sl = slice(lo, hi)
    o = Oracle(hi - lo, W, eta, eps, H, b0sq, None if x0 is None else x0[sl], j_base=j_base + lo)
    if x0 is not None or b0sq != 0.0:
        g.set_init(x0, b0sq)
    if grad == "noise":
        g.set_grad_noise(seed, None)
        o.set_grad_noise(seed, None)
    elif grad == "noise_scaled":
        g.set_grad_noise(seed, arrays["s"])
        o.set_grad_noise(seed, arrays["s"][sl])
    elif grad == "quadratic":
        g.set_grad_quadratic(seed, arrays["a"], arrays["c"], sigma)
        o.set_grad_quadratic(seed, arrays["a"][sl], arrays["c"][sl], sigma)
    elif grad == "constant":
        s = arrays.get("s")
        g.set_grad_constant(s)
        o.set_grad_constant(None if s is None else s[sl])
    else:
        raise ValueError(grad)
    if bf16:
        g.set_grad_dtype(la.LA_BF16)
        o.set_grad_bf16(True)
    if identical:
        g.set_identical_workers(True)
        o.set_identical_workers(True)
    if warmup:
        g.set_warmup(warmup)
        o.set_warmup(warmup)
    g.set_fusion(fusion)
    return g, o


def max_scaled_err(got, ref):
    """max |got - ref| / max(1, |ref|) — the tolerance form of the parity contract."""
    got = got.astype(np.float64)
    ref = ref.astype(np.float64)
    return float(np.max(np.abs(got - ref) / np.maximum(1.0, np.abs(ref)))) if got.size else 0.0


def compare(g, o, W, tol, rng=None, bitwise=True):
    """Compare every worker's x, B^2 and the stale accumulator.  Returns the worst scaled error."""
    worst = 0.0
    for i in range(W):
        ox, ob, os_ = o.read(i)
        if rng is None:
            gx, gb, gs = g.read_state(i)
        else:
            gx, gb, gs = g.read_range(i, rng[0], rng[1] - rng[0])
        for name, a, b in (("x", gx, ox), ("B2", gb, ob), ("Bs", gs, os_)):
            assert np.all(np.isfinite(a)), f"{name}: non-finite values on the GPU (worker {i})"
            e = max_scaled_err(a, b)
            worst = max(worst, e)
            assert e <= tol, f"{name} worker {i}: scaled error {e:.3e} > {tol:.1e}"
            if bitwise:
                bad = np.flatnonzero(a.view(np.uint32) != b.view(np.uint32))
                assert bad.size == 0, (f"{name} worker {i}: {bad.size} elements differ bitwise, "
                                       f"first at {bad[0]}: {a[bad[0]]!r} vs {b[bad[0]]!r}")
    assert g.get_counters() == o.counters(), "step / sync counters differ"
    return worst
