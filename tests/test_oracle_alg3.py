"""Pins for the CPU oracle's Algorithm 3 (Local AdaAlter) arithmetic.

Each test checks the oracle against something fixed by the paper or by
mathematics, not against itself: a hand-worked case, an independent
brute-force evaluation with every iterate stored separately, closed forms, and
reductions to simpler recursions.  CPU only.
"""
import math
import os

import numpy as np
import pytest

from oracle.oracle import Oracle, noise_fill

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------- helpers
def brute_force(x0, G, eta, eps, H, b0sq, W, grad_fn=None, T=None):
    """Algorithm 3 written literally in Python floats (fp64), with x, y, A^2, B^2 kept
    as separate per-iteration tables so that no in-place update can hide an aliasing
    mistake.  `G[t-1][i][j]` prescribes gradients unless `grad_fn(i, t, j, x)` is given."""
    n = len(x0)
    T = len(G) if T is None else T
    x = [[[x0[j] for j in range(n)] for _ in range(W)]]
    B2 = [[[b0sq for _ in range(n)] for _ in range(W)]]
    for t in range(1, T + 1):
        tp = (t - 1) % H + 1
        y = [[0.0] * n for _ in range(W)]
        A2 = [[0.0] * n for _ in range(W)]
        for i in range(W):
            for j in range(n):
                g = grad_fn(i, t, j, x[t - 1][i][j]) if grad_fn else G[t - 1][i][j]
                den = math.sqrt(B2[t - tp][i][j] + tp * eps * eps)
                y[i][j] = x[t - 1][i][j] - eta * g / den
                A2[i][j] = B2[t - 1][i][j] + g * g
        if t % H != 0:
            x.append(y)
            B2.append(A2)
        else:
            xm = [sum(y[k][j] for k in range(W)) / W for j in range(n)]
            bm = [sum(A2[k][j] for k in range(W)) / W for j in range(n)]
            x.append([list(xm) for _ in range(W)])
            B2.append([list(bm) for _ in range(W)])
    return x, B2


def read_golden():
    rows = []
    with open(os.path.join(GOLDEN, "alg3_hand_case.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            rows.append([float(v) for v in line.split()])
    return rows


# --------------------------------------------------------------------------- I1
def test_hand_worked_case():
    """Hand-derived trajectory (Algorithm 3): fixes the stale-denominator timing, the t'
    schedule, accumulate-then-average, and that the stale B^2 moves only at a sync."""
    o = Oracle(n=1, W=2, eta=1.0, eps=1.0, H=2, b0sq=0.0)
    for t, g0, g1, x0, x1, b0, b1, bs in read_golden():
        o.local_step(np.array([[g0], [g1]], np.float32))
        if o.counters()[1] == 2:
            o.sync()
        xa, ba, s = o.read_all()
        xs = [o.read_shadow(i)[0][0] for i in range(2)]
        assert xs[0] == pytest.approx(x0, abs=1e-14) and xs[1] == pytest.approx(x1, abs=1e-14)
        assert xa[0, 0] == pytest.approx(x0, abs=5e-7) and xa[1, 0] == pytest.approx(x1, abs=5e-7)
        assert (ba[0, 0], ba[1, 0], s[0]) == (b0, b1, bs)
        assert o.counters()[0] == t
    assert o.counters() == (4, 0, 2)


# --------------------------------------------------------------------------- I13
@pytest.mark.parametrize("W,n,H,T", [(1, 3, 2, 5), (2, 5, 3, 6), (3, 4, 1, 4), (3, 2, 4, 6), (2, 1, 7, 6)])
def test_brute_force_prescribed(W, n, H, T):
    rng = np.random.default_rng(100 * W + 10 * n + H)
    G = rng.standard_normal((T, W, n)).astype(np.float32)
    x0 = rng.standard_normal(n).astype(np.float32)
    eta, eps, b0sq = 0.3, 0.5, 0.25
    o = Oracle(n, W, eta, eps, H, b0sq, x0)
    xs, B2s = brute_force([float(v) for v in x0], G.astype(np.float64).tolist(),
                          float(np.float32(eta)), float(np.float32(eps)), H, b0sq, W)
    for t in range(1, T + 1):
        o.local_step(G[t - 1])
        if o.counters()[1] == H:
            o.sync()
        for i in range(W):
            xd, bd, _ = o.read_shadow(i)
            xf, bf, _ = o.read(i)
            np.testing.assert_allclose(xd, xs[t][i], rtol=0, atol=1e-13)
            np.testing.assert_allclose(bd, B2s[t][i], rtol=1e-14)
            np.testing.assert_allclose(xf, xs[t][i], rtol=0, atol=2e-6)
            np.testing.assert_allclose(bf, B2s[t][i], rtol=1e-6)


def test_brute_force_state_dependent_gradient():
    """Quadratic source: the gradient is evaluated at the worker's OWN iterate."""
    W, n, H, T, seed = 3, 4, 3, 7, 11
    rng = np.random.default_rng(5)
    a = rng.uniform(0.1, 2.0, n).astype(np.float32)
    c = rng.standard_normal(n).astype(np.float32)
    sigma, eta, eps, b0sq = np.float32(0.3), np.float32(0.2), np.float32(1.0), 1.0
    xi = np.stack([np.stack([noise_fill(seed, t, i, 0, n) for i in range(W)]) for t in range(1, T + 1)])

    def grad(i, t, j, x):
        return float(a[j]) * (x - float(c[j])) + float(sigma) * float(xi[t - 1, i, j])

    xs, B2s = brute_force([0.0] * n, None, float(eta), float(eps), H, b0sq, W, grad_fn=grad, T=T)
    o = Oracle(n, W, eta, eps, H, b0sq)
    o.set_grad_quadratic(seed, a, c, sigma)
    o.run(T)
    for i in range(W):
        np.testing.assert_allclose(o.read_shadow(i)[0], xs[T][i], rtol=0, atol=1e-13)
        np.testing.assert_allclose(o.read(i)[0], xs[T][i], rtol=0, atol=3e-6)
        np.testing.assert_allclose(o.read(i)[1], B2s[T][i], rtol=2e-6)
    assert o.counters() == (T, T % H, T // H)


# --------------------------------------------------------------------------- I8 / I9
@pytest.mark.parametrize("H", [1, 3, 4, 16, 100])
def test_constant_gradient_closed_form(H):
    """g constant: B^2 after k steps = b0^2 + k g^2, and
    x_T = x_0 - eta g sum_t (b0^2 + (t-t') g^2 + t' eps^2)^(-1/2)."""
    n, W, T = 6, 4, 23
    g = np.array([0.5, -1.5, 2.0, 1.0, -0.25, 3.0], np.float32)
    eta, eps, b0sq = 0.5, 0.75, 1.0
    o = Oracle(n, W, eta, eps, H, b0sq)
    o.set_grad_constant(g)
    o.run(T)
    exp_x = np.zeros(n)
    for t in range(1, T + 1):
        tp = (t - 1) % H + 1
        exp_x -= eta * g.astype(np.float64) / np.sqrt(b0sq + (t - tp) * g.astype(np.float64) ** 2 + tp * eps * eps)
    for i in range(W):
        x, b2, _ = o.read(i)
        xd, b2d, bsd = o.read_shadow(i)
        np.testing.assert_allclose(b2d, b0sq + T * g.astype(np.float64) ** 2, rtol=1e-14)
        np.testing.assert_allclose(b2, b0sq + T * g.astype(np.float64) ** 2, rtol=1e-6)
        np.testing.assert_allclose(xd, exp_x, rtol=1e-13)
        np.testing.assert_allclose(x, exp_x, rtol=5e-6)
        np.testing.assert_allclose(bsd, b0sq + (T - T % H) * g.astype(np.float64) ** 2, rtol=1e-14)


def test_placeholder_exactness_h_independent():
    """|g| = eps: the placeholder t' eps^2 equals the gradient mass it stands in for, so the
    trajectory does not depend on H.  With g = eps = 1 and integer b0^2 every accumulator is an
    exact fp32 integer and the fp32 runs agree bit for bit; x_T = -eta sum_t (b0^2+t)^(-1/2)."""
    T, eta, b0sq = 16, 0.5, 1.0
    ref = None
    for H in (1, 4, 16):
        o = Oracle(3, 2, eta, 1.0, H, b0sq)
        o.set_grad_constant(None)
        o.run(T)
        x, b2, _ = o.read(1)
        assert np.all(b2 == b0sq + T)
        if ref is None:
            ref = x
        assert np.array_equal(x.view(np.uint32), ref.view(np.uint32))
    closed = -eta * sum((b0sq + t) ** -0.5 for t in range(1, T + 1))
    assert closed == pytest.approx(-2.953265116, abs=1e-9)
    np.testing.assert_allclose(ref, closed, rtol=1e-6)


# --------------------------------------------------------------------------- I4
def test_h1_is_synchronous_adaalter():
    """H = 1: x <- x - eta mean_i(g_i)/sqrt(B^2 + eps^2) with the PRE-update B^2, then
    B^2 <- B^2 + mean_i(g_i^2) (mean of squares)."""
    W, n, T = 4, 5, 9
    rng = np.random.default_rng(3)
    G = rng.standard_normal((T, W, n)).astype(np.float32)
    eta, eps, b0sq = 0.1, 0.3, 0.5
    o = Oracle(n, W, eta, eps, 1, b0sq)
    x = np.zeros(n)
    B = np.full(n, b0sq)
    e32, p32 = float(np.float32(eta)), float(np.float32(eps))
    for t in range(T):
        o.local_step(G[t])
        o.sync()
        g = G[t].astype(np.float64)
        x = x - e32 * g.mean(0) / np.sqrt(B + p32 * p32)
        B = B + (g * g).mean(0)
    for i in range(W):
        xd, bd, bsd = o.read_shadow(i)
        np.testing.assert_allclose(xd, x, atol=1e-13)
        np.testing.assert_allclose(bd, B, rtol=1e-14)
        np.testing.assert_allclose(bsd, B, rtol=1e-14)
        np.testing.assert_allclose(o.read(i)[0], x, atol=2e-6)


def test_h1_differs_from_adagrad():
    """Section 4.2 remark: even H = 1 is not AdaGrad (AdaGrad divides by the UPDATED B^2)."""
    o = Oracle(1, 1, 1.0, 1.0, 1, 0.0)
    o.local_step(np.array([[2.0]], np.float32))
    o.sync()
    assert o.read_shadow(0)[0][0] == pytest.approx(-2.0)            # AdaAlter: 2/sqrt(0+1)
    assert -2.0 / math.sqrt(4.0 + 1.0) != pytest.approx(-2.0)       # AdaGrad would give -0.894


# --------------------------------------------------------------------------- I5
def test_single_worker_serial_recursion():
    n, H, T = 7, 3, 11
    rng = np.random.default_rng(8)
    G = rng.standard_normal((T, 1, n)).astype(np.float32)
    eta, eps, b0sq = np.float32(0.25), np.float32(0.5), 0.0
    o = Oracle(n, 1, eta, eps, H, b0sq)
    x = np.zeros(n)
    B = np.full(n, b0sq)
    snap = B.copy()
    for t in range(1, T + 1):
        o.local_step(G[t - 1])
        before = [v.copy() for v in o.read(0)]
        if o.counters()[1] == H:
            o.sync()
            after = o.read(0)
            assert np.array_equal(before[0], after[0]) and np.array_equal(before[1], after[1])
        tp = (t - 1) % H + 1
        g = G[t - 1, 0].astype(np.float64)
        x = x - float(eta) * g / np.sqrt(snap + tp * float(eps) ** 2)
        B = B + g * g
        if t % H == 0:
            snap = B.copy()
    np.testing.assert_allclose(o.read_shadow(0)[0], x, atol=1e-13)
    np.testing.assert_allclose(o.read_shadow(0)[2], snap, rtol=1e-14)


# --------------------------------------------------------------------------- I6
@pytest.mark.parametrize("W", [2, 4, 8, 16])
def test_identical_workers_sync_is_identity(W):
    n, H, T = 64, 4, 13
    rng = np.random.default_rng(W)
    a = rng.uniform(0.1, 10, n).astype(np.float32)
    c = rng.standard_normal(n).astype(np.float32)
    multi = Oracle(n, W, 0.1, 1.0, H)
    multi.set_grad_quadratic(9, a, c, 0.1)
    multi.set_identical_workers(True)
    single = Oracle(n, 1, 0.1, 1.0, H)
    single.set_grad_quadratic(9, a, c, 0.1)
    multi.run(T)
    single.run(T)
    xs, b2s, bss = single.read(0)
    for i in range(W):
        x, b2, bs = multi.read(i)
        assert np.array_equal(x, xs) and np.array_equal(b2, b2s) and np.array_equal(bs, bss)


# --------------------------------------------------------------------------- I7
def test_no_sync_when_h_exceeds_t():
    n, W, T = 16, 3, 9
    o = Oracle(n, W, 0.1, 0.5, 0xFFFFFFFF, 2.0)
    o.set_grad_noise(4)
    xi = np.stack([np.stack([noise_fill(4, t, i, 0, n) for i in range(W)]) for t in range(1, T + 1)])
    o.run(T)
    assert o.counters() == (T, T, 0)
    den = np.sqrt(2.0 + np.arange(1, T + 1, dtype=np.float64) * float(np.float32(0.5)) ** 2)
    for i in range(W):
        xd, b2d, bsd = o.read_shadow(i)
        assert np.all(bsd == 2.0)
        np.testing.assert_allclose(xd, -float(np.float32(0.1)) * (xi[:, i].astype(np.float64) / den[:, None]).sum(0),
                                   atol=1e-13)
        np.testing.assert_allclose(b2d, 2.0 + (xi[:, i].astype(np.float64) ** 2).sum(0), rtol=1e-14)


# --------------------------------------------------------------------------- I2 / I3 / I10
def test_accumulator_identity_and_mean_iterate():
    """B-bar^2_t = b0^2 + sum_s mean_i g^2 at sync points (Table 1 / Appendix A); the worker
    mean follows x-bar_t = x-bar_{t-1} - eta mean_i(g)/sqrt(stale + t' eps^2) and a sync
    leaves it unchanged; after a sync all replicas coincide and B^2_i equals the stale B^2."""
    W, n, H, T = 4, 9, 3, 12
    rng = np.random.default_rng(21)
    G = rng.standard_normal((T, W, n)).astype(np.float32)
    eta, eps, b0sq = np.float32(0.2), np.float32(0.7), 1.0
    o = Oracle(n, W, eta, eps, H, b0sq)
    xbar = np.zeros(n)
    acc = np.full(n, b0sq)
    stale = np.full(n, b0sq)
    for t in range(1, T + 1):
        tp = (t - 1) % H + 1
        prev_b2 = np.stack([o.read(i)[1] for i in range(W)])
        o.local_step(G[t - 1])
        g = G[t - 1].astype(np.float64)
        xbar = xbar - float(eta) * g.mean(0) / np.sqrt(stale + tp * float(eps) ** 2)
        acc = acc + (g * g).mean(0)
        now_b2 = np.stack([o.read(i)[1] for i in range(W)])
        assert np.all(now_b2 >= prev_b2)                      # non-decreasing within a period
        if o.counters()[1] == H:
            o.sync()
            stale = acc.copy()
            xa, ba, bs = o.read_all()
            assert all(np.array_equal(xa[0], xa[i]) and np.array_equal(ba[0], ba[i]) for i in range(W))
            assert np.array_equal(ba[0], bs)
            np.testing.assert_allclose(o.read_shadow(0)[1], acc, rtol=1e-14)
        mean_now = np.mean([o.read_shadow(i)[0] for i in range(W)], axis=0)
        np.testing.assert_allclose(mean_now, xbar, atol=1e-13)


# --------------------------------------------------------------------------- I11 / I12
def test_coordinate_independence_and_slices():
    n, W = 1000, 4
    rng = np.random.default_rng(2)
    s = rng.uniform(0.1, 1, n).astype(np.float32)
    full = Oracle(n, W, 0.01, 1e-3, 8)
    full.set_grad_noise(2, s)
    full.run(20)
    lo, hi = 368, 492
    part = Oracle(hi - lo, W, 0.01, 1e-3, 8, j_base=lo)
    part.set_grad_noise(2, s[lo:hi])
    part.run(20)
    for i in range(W):
        for u, v in zip(full.read(i), part.read(i)):
            assert np.array_equal(u[lo:hi], v)


def test_checkpoint_resume_bitwise():
    n, W, H = 50, 3, 4
    rng = np.random.default_rng(6)
    a = rng.uniform(0.1, 10, n).astype(np.float32)
    c = rng.standard_normal(n).astype(np.float32)

    def make():
        o = Oracle(n, W, 0.1, 1.0, H)
        o.set_grad_quadratic(7, a, c, 0.1)
        return o

    whole = make()
    whole.run(11)
    first = make()
    first.run(6)
    second = make()
    for i in range(W):
        x, b2, bs = first.read(i)
        second.write(i, x, b2, bs)
    second.set_counters(*first.counters())
    second.run(5)
    assert whole.counters() == second.counters() == (11, 3, 2)
    for i in range(W):
        for u, v in zip(whole.read(i), second.read(i)):
            assert np.array_equal(u, v)


# --------------------------------------------------------------------------- schedule / misc
@pytest.mark.parametrize("H,T", [(1, 5), (2, 5), (3, 9), (5, 5), (6, 5)])
def test_schedule_counters(H, T):
    o = Oracle(2, 2, 0.1, 1.0, H)
    o.set_grad_noise(1)
    for t in range(1, T + 1):
        o.run(1)
        tt, tp, ns = o.counters()
        assert tt == t and ns == t // H and tp == t % H       # t' of the NEXT step is tp + 1


def test_manual_sync_resets_step_count():
    o = Oracle(2, 2, 1.0, 1.0, 10, 0.0)
    g = np.ones((2, 2), np.float32)
    o.local_step(g); o.local_step(g)
    o.sync()
    assert o.counters() == (2, 0, 1)
    o.local_step(g)                                           # t' = 1 again, stale B^2 = 2
    assert o.read_shadow(0)[0][0] == pytest.approx(-1 - 1 / math.sqrt(2) - 1 / math.sqrt(3), abs=1e-14)


def test_tree_order_of_worker_sum():
    """The fp32 mean is the adjacent-pair tree ((v0+v1)+(v2+v3))+... divided by W."""
    for W in (3, 5, 6, 7, 8, 11):
        rng = np.random.default_rng(W)
        v = (rng.standard_normal(W) * 10.0 ** rng.integers(-3, 4, W)).astype(np.float32)
        o = Oracle(1, W, 0.1, 1.0, 1)
        for i in range(W):
            o.write(i, x=v[i:i + 1], b2=np.abs(v[i:i + 1]))
        o.sync()
        level = list(v)
        while len(level) > 1:
            nxt = [np.float32(level[k] + level[k + 1]) for k in range(0, len(level) - 1, 2)]
            if len(level) % 2:
                nxt.append(level[-1])
            level = nxt
        assert o.read(0)[0][0] == np.float32(level[0] / np.float32(W))


def test_warmup_learning_rate():
    """Section 6.2: eta_t = eta min(1, t / warm_up_steps)."""
    o = Oracle(1, 1, 0.5, 1.0, 0xFFFFFFFF, 1.0)
    o.set_warmup(4)
    o.set_grad_constant(None)
    x = 0.0
    for t in range(1, 8):
        o.run(1)
        x -= 0.5 * min(1.0, t / 4) / math.sqrt(1.0 + t)
        assert o.read_shadow(0)[0][0] == pytest.approx(x, abs=1e-14)
        assert o.read(0)[0][0] == pytest.approx(x, abs=1e-6)


def test_fp32_tracks_fp64_shadow_on_config1():
    from paper_1911_09030_b200 import workloads
    wl = workloads.config("c1")
    n = 4096
    arr = wl.arrays(0, n)
    o = Oracle(n, wl.W, wl.eta, wl.eps, wl.H, wl.b0sq)
    o.set_grad_quadratic(wl.noise_seed, arr["a"], arr["c"], wl.sigma)
    o.run(wl.T)
    for i in range(wl.W):
        x, b2, _ = o.read(i)
        xd, b2d, _ = o.read_shadow(i)
        assert np.all(np.isfinite(x))
        np.testing.assert_allclose(x, xd, rtol=0, atol=2e-5)
        np.testing.assert_allclose(b2, b2d, rtol=2e-5)
