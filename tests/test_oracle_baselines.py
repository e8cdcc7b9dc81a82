"""Pins for the oracle's baseline update rules: Distributed AdaGrad (Algorithm 1) and Local SGD
(Algorithm 2).  Closed forms, literal brute force with stored iterates, and reductions; CPU only."""
import math

import numpy as np
import pytest

from oracle.oracle import Oracle, noise_fill

ADAALTER, LOCAL_SGD, ADAGRAD = 0, 1, 2


# ------------------------------------------------------------------ Algorithm 1: Distributed AdaGrad
def brute_adagrad(x0, G, eta, eps, T, grad_fn=None):
    """x_t, B2_t stored per iteration; G[t-1][i][j] prescribed or grad_fn(i, t, j, x)."""
    n = len(x0)
    x, B2 = [list(x0)], [[0.0] * n]
    for t in range(1, T + 1):
        W = len(G[t - 1]) if G is not None else grad_fn.W
        gbar = [sum((grad_fn(i, t, j, x[t - 1][j]) if grad_fn else G[t - 1][i][j]) for i in range(W)) / W
                for j in range(n)]
        B2.append([B2[t - 1][j] + gbar[j] ** 2 for j in range(n)])
        x.append([x[t - 1][j] - eta * gbar[j] / math.sqrt(B2[t][j] + eps * eps) for j in range(n)])
    return x, B2


def test_adagrad_hand_case():
    """n=2, d=1, eta=1, eps=1, B0^2=0: gradients (1,3) then (2,2).
    t=1: G=2, B^2=4, x=-2/sqrt5.  t=2: G=2, B^2=8, x=-2/sqrt5-2/3."""
    o = Oracle(1, 2, 1.0, 1.0, 1)
    o.set_rule(ADAGRAD)
    o.local_step(np.array([[1.0], [3.0]], np.float32))
    assert o.read_shadow(0)[0][0] == pytest.approx(-2 / math.sqrt(5), abs=1e-15)
    assert o.read(1)[1][0] == 4.0
    o.local_step(np.array([[2.0], [2.0]], np.float32))
    for i in (0, 1):
        assert o.read_shadow(i)[0][0] == pytest.approx(-2 / math.sqrt(5) - 2 / 3, abs=1e-15)
        assert o.read(i)[0][0] == pytest.approx(-2 / math.sqrt(5) - 2 / 3, abs=3e-7)
        assert o.read(i)[1][0] == 8.0
    assert o.counters() == (2, 0, 2)          # one gradient exchange per iteration


@pytest.mark.parametrize("W,n,T", [(1, 3, 5), (3, 4, 6), (4, 2, 7)])
def test_adagrad_brute_force(W, n, T):
    rng = np.random.default_rng(W * 10 + n)
    G = rng.standard_normal((T, W, n)).astype(np.float32)
    x0 = rng.standard_normal(n).astype(np.float32)
    eta, eps = np.float32(0.3), np.float32(0.5)
    o = Oracle(n, W, eta, eps, 1, 0.0, x0)
    o.set_rule(ADAGRAD)
    xs, Bs = brute_adagrad([float(v) for v in x0], G.astype(np.float64).tolist(), float(eta), float(eps), T)
    for t in range(1, T + 1):
        o.local_step(G[t - 1])
        for i in range(W):
            np.testing.assert_allclose(o.read_shadow(i)[0], xs[t], atol=1e-13)
            np.testing.assert_allclose(o.read_shadow(i)[1], Bs[t], rtol=1e-13)
            np.testing.assert_allclose(o.read(i)[0], xs[t], atol=2e-6)
            np.testing.assert_allclose(o.read(i)[1], Bs[t], rtol=2e-6, atol=1e-7)


def test_adagrad_constant_gradient_closed_form():
    """g constant: B^2_t = t g^2, x_T = -eta sum_t g / sqrt(t g^2 + eps^2)."""
    g = np.array([0.5, -2.0, 1.0], np.float32)
    eta, eps, T = 0.5, 0.25, 17
    o = Oracle(3, 4, eta, eps, 1)
    o.set_rule(ADAGRAD)
    o.set_grad_constant(g)
    o.run(T)
    gd = g.astype(np.float64)
    want = -eta * sum(gd / np.sqrt(t * gd * gd + eps * eps) for t in range(1, T + 1))
    np.testing.assert_allclose(o.read_shadow(2)[0], want, rtol=1e-13)
    np.testing.assert_allclose(o.read(2)[0], want, rtol=3e-6)
    np.testing.assert_allclose(o.read(2)[1], T * gd * gd, rtol=1e-6)


def test_adagrad_uses_square_of_mean_and_updated_accumulator():
    """Algorithm 1 squares the AVERAGED gradient (AdaAlter averages the squares) and divides by
    the accumulator that already contains it (AdaAlter's is stale)."""
    o = Oracle(1, 2, 1.0, 1.0, 1)
    o.set_rule(ADAGRAD)
    o.local_step(np.array([[3.0], [-1.0]], np.float32))      # mean 1, mean of squares 5
    assert o.read(0)[1][0] == 1.0
    assert o.read_shadow(0)[0][0] == pytest.approx(-1 / math.sqrt(2.0), abs=1e-15)
    a = Oracle(1, 2, 1.0, 1.0, 1)
    a.local_step(np.array([[3.0], [-1.0]], np.float32)); a.sync()
    assert a.read(0)[1][0] == 5.0
    assert a.read_shadow(0)[0][0] == pytest.approx(-1.0, abs=1e-15)


def test_adagrad_state_dependent_gradient_and_replicas_equal():
    W, n, T, seed = 3, 5, 6, 4
    rng = np.random.default_rng(1)
    a = rng.uniform(0.1, 2, n).astype(np.float32)
    c = rng.standard_normal(n).astype(np.float32)
    sigma, eta, eps = np.float32(0.5), np.float32(0.4), np.float32(1.0)
    xi = np.stack([np.stack([noise_fill(seed, t, i, 0, n) for i in range(W)]) for t in range(1, T + 1)])

    def grad(i, t, j, x):
        return float(a[j]) * (x - float(c[j])) + float(sigma) * float(xi[t - 1, i, j])
    grad.W = W
    xs, Bs = brute_adagrad([0.0] * n, None, float(eta), float(eps), T, grad_fn=grad)
    o = Oracle(n, W, eta, eps, 5)
    o.set_rule(ADAGRAD)
    o.set_grad_quadratic(seed, a, c, sigma)
    o.run(T)
    np.testing.assert_allclose(o.read_shadow(0)[0], xs[T], atol=1e-13)
    np.testing.assert_allclose(o.read(0)[0], xs[T], atol=3e-6)
    for i in range(1, W):
        assert np.array_equal(o.read(i)[0], o.read(0)[0]) and np.array_equal(o.read(i)[1], o.read(0)[1])
    assert o.counters() == (T, 0, T)


# ------------------------------------------------------------------ Algorithm 2: Local SGD
def brute_local_sgd(x0, G, eta, H, W, T, grad_fn=None):
    n = len(x0)
    x = [[list(x0) for _ in range(W)]]
    for t in range(1, T + 1):
        y = [[x[t - 1][i][j] - eta * (grad_fn(i, t, j, x[t - 1][i][j]) if grad_fn else G[t - 1][i][j])
              for j in range(n)] for i in range(W)]
        if t % H != 0:
            x.append(y)
        else:
            m = [sum(y[k][j] for k in range(W)) / W for j in range(n)]
            x.append([list(m) for _ in range(W)])
    return x


@pytest.mark.parametrize("W,n,H,T", [(1, 3, 2, 5), (2, 4, 3, 7), (3, 2, 1, 4), (4, 3, 5, 9)])
def test_local_sgd_brute_force(W, n, H, T):
    rng = np.random.default_rng(W + 7 * H)
    G = rng.standard_normal((T, W, n)).astype(np.float32)
    x0 = rng.standard_normal(n).astype(np.float32)
    eta = np.float32(0.1)
    o = Oracle(n, W, eta, 1.0, H, 0.0, x0)
    o.set_rule(LOCAL_SGD)
    xs = brute_local_sgd([float(v) for v in x0], G.astype(np.float64).tolist(), float(eta), H, W, T)
    for t in range(1, T + 1):
        o.local_step(G[t - 1])
        if o.counters()[1] == H:
            o.sync()
        for i in range(W):
            np.testing.assert_allclose(o.read_shadow(i)[0], xs[t][i], atol=1e-14)
            np.testing.assert_allclose(o.read(i)[0], xs[t][i], atol=1e-6)
    assert o.counters() == (T, T % H, T // H)
    assert np.all(o.read(0)[1] == 0.0)          # no accumulator in Algorithm 2


def test_local_sgd_noise_free_quadratic_contracts_geometrically():
    """g = a (x - c): x_T - c = (1 - eta a)^T (x_0 - c), for any H (workers stay identical)."""
    a = np.array([0.5, 1.0, 3.0], np.float32)
    c = np.array([1.0, -2.0, 0.25], np.float32)
    eta, T = 0.25, 12
    for H in (1, 4, 100):
        o = Oracle(3, 4, eta, 1.0, H)
        o.set_rule(LOCAL_SGD)
        o.set_grad_quadratic(1, a, c, 0.0)
        o.run(T)
        want = c.astype(np.float64) + (1 - eta * a.astype(np.float64)) ** T * (0 - c.astype(np.float64))
        for i in range(4):
            np.testing.assert_allclose(o.read_shadow(i)[0], want, rtol=1e-12, atol=1e-14)
            np.testing.assert_allclose(o.read(i)[0], want, rtol=2e-6, atol=1e-6)


def test_local_sgd_mean_iterate_is_h_independent_for_linear_gradients():
    """For a gradient linear in x, averaging commutes with the step: the worker mean follows
    x-bar <- x-bar - eta (a (x-bar - c) + sigma mean_i xi_i) whatever H is."""
    n, W, T, seed = 6, 4, 10, 3
    rng = np.random.default_rng(2)
    a = rng.uniform(0.1, 2, n).astype(np.float32)
    c = rng.standard_normal(n).astype(np.float32)
    sigma, eta = np.float32(0.7), np.float32(0.2)
    xi = np.stack([np.stack([noise_fill(seed, t, i, 0, n) for i in range(W)]) for t in range(1, T + 1)]).astype(np.float64)
    xbar = np.zeros(n)
    for t in range(T):
        xbar = xbar - float(eta) * (a.astype(np.float64) * (xbar - c) + float(sigma) * xi[t].mean(0))
    for H in (1, 3, 100):
        o = Oracle(n, W, eta, 1.0, H)
        o.set_rule(LOCAL_SGD)
        o.set_grad_quadratic(seed, a, c, sigma)
        o.run(T)
        mean = np.mean([o.read_shadow(i)[0] for i in range(W)], axis=0)
        np.testing.assert_allclose(mean, xbar, atol=1e-13)
