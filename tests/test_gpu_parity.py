"""GPU parity: the CUDA library (through its C-ABI) against the CPU oracle, element by
element on the same seeded inputs.  Contract: |gpu - ref| <= 1e-6 max(1,|ref|) after one
step and <= 1e-5 max(1,|ref|) after a full run; counters bit-exact.  Because both sides
perform the same sequence of correctly rounded fp32 operations the tests also demand
bitwise equality."""
import itertools

import numpy as np
import pytest

from oracle.oracle import Oracle
from paper_1911_09030_b200 import local_adaalter as la
from paper_1911_09030_b200 import workloads
from parity_util import compare, make_pair

pytestmark = pytest.mark.gpu

TOL_STEP, TOL_RUN = 1e-6, 1e-5


def _arrays(n, seed):
    rng = np.random.default_rng(seed)
    return dict(a=rng.uniform(0.1, 10, n).astype(np.float32), c=rng.standard_normal(n).astype(np.float32),
                s=np.exp(rng.uniform(np.log(1e-3), 0, n)).astype(np.float32))


# ----------------------------------------------------------------------------- configuration 1
@pytest.mark.parametrize("fusion", [0, 1, 2, 3, 4])
def test_config1_full(fusion):
    wl = workloads.config("c1")
    arr = wl.arrays()
    g, o = make_pair(wl.N, wl.W, wl.eta, wl.eps, wl.H, "quadratic", seed=wl.noise_seed, arrays=arr,
                     sigma=wl.sigma, fusion=fusion)
    g.run(1)
    o.run(1)
    compare(g, o, wl.W, TOL_STEP)
    g.run(wl.T - 1)
    o.run(wl.T - 1)
    compare(g, o, wl.W, TOL_RUN)
    assert g.get_counters() == (wl.T, 0, wl.T // wl.H)


# ----------------------------------------------------------------------------- shape sweep
@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 31, 32, 33, 1023, 1025])
@pytest.mark.parametrize("W", [1, 2, 3, 4, 8, 16])
def test_tails_and_worker_counts(n, W):
    T = 7
    arr = _arrays(n, 10 * n + W)
    for H, grad, fusion in [(1, "quadratic", 0), (2, "noise_scaled", 1), (3, "quadratic", 2), (T, "noise", 1),
                            (T + 1, "quadratic", 2), (3, "quadratic", 3), (T + 1, "noise_scaled", 3)]:
        g, o = make_pair(n, W, 0.1, 0.5, H, grad, seed=n + W, arrays=arr, sigma=0.3, fusion=fusion, b0sq=0.25)
        g.run(T)
        o.run(T)
        compare(g, o, W, TOL_RUN)
        g.close()


@pytest.mark.parametrize("W", [5, 6, 7, 9, 10, 11, 13, 14, 15, 17, 20, 23, 24, 29, 32, 40, 48, 63, 64])
def test_generic_worker_counts(W):
    n, T = 257, 9
    arr = _arrays(n, W)
    for H, fusion in [(2, 0), (3, 1), (4, 2), (4, 3), (2, 4), (5, 4)]:
        g, o = make_pair(n, W, 0.05, 1.0, H, "quadratic", seed=W, arrays=arr, sigma=1.0, fusion=fusion)
        g.run(T)
        o.run(T)
        compare(g, o, W, TOL_RUN)


@pytest.mark.parametrize("grad,bf16", [("noise", False), ("noise_scaled", False), ("noise_scaled", True),
                                       ("quadratic", True), ("constant", False)])
@pytest.mark.parametrize("W", [5, 6])
def test_gradient_kinds_with_their_own_register_budget(W, grad, bf16):
    """W = 5 and 6 compile each gradient kind with the number of resident blocks that suits it;
    every kind, every fusion mode, several blocks and a ragged tail."""
    n, H, T = 70003, 3, 8
    arr = _arrays(n, W)
    for fusion in (0, 1, 2, 3, 4):
        g, o = make_pair(n, W, 0.05, 0.7, H, grad, seed=40 + W, arrays=arr, sigma=0.5, bf16=bf16, fusion=fusion)
        g.run(T)
        o.run(T)
        compare(g, o, W, TOL_RUN)


@pytest.mark.parametrize("grad,bf16", [("noise", False), ("noise", True), ("noise_scaled", False),
                                       ("noise_scaled", True), ("quadratic", False), ("quadratic", True),
                                       ("constant", False)])
@pytest.mark.parametrize("fusion", [0, 1, 2, 3, 4])
def test_gradient_modes(grad, bf16, fusion):
    n, W, H, T = 70001, 4, 3, 10      # several blocks and a ragged tail
    arr = _arrays(n, 3)
    g, o = make_pair(n, W, 0.05, 0.7, H, grad, seed=21, arrays=arr, sigma=0.5, bf16=bf16, fusion=fusion)
    g.run(1)
    o.run(1)
    compare(g, o, W, TOL_STEP)
    g.run(T - 1)
    o.run(T - 1)
    compare(g, o, W, TOL_RUN)


# ----------------------------------------------------------------------------- fused == unfused
@pytest.mark.parametrize("W,H", [(2, 1), (4, 4), (8, 3), (16, 2), (3, 2)])
def test_fused_kernels_equal_unfused_bitwise(W, H):
    n, T = 12345, 11
    arr = _arrays(n, 77)
    states = []
    for fusion in (0, 1, 2, 3, 4):
        g = la.LocalAdaAlter([n], W, 0.1, 1.0, H)
        g.set_grad_quadratic(5, arr["a"], arr["c"], 0.2)
        g.set_fusion(fusion)
        g.run(4)
        g.run(T - 4)                   # a run boundary in the middle of a period
        states.append(([g.read_state(i) for i in range(W)], g.get_counters(), g.get_stats()))
        g.close()
    for st, cnt, stats in states[1:]:
        assert cnt == states[0][1]
        for i in range(W):
            for u, v in zip(st[i], states[0][0][i]):
                assert np.array_equal(u.view(np.uint32), v.view(np.uint32))
    assert states[0][2]["launches_fused"] == 0 and states[0][2]["launches_sync"] == T // H
    assert states[1][2]["launches_fused"] == T // H and states[1][2]["launches_sync"] == 0
    assert states[2][2]["launches_fused"] > 0
    # temporal blocking: one pass per (piece of a) period, nothing else
    # (a piece of a single step runs as an ordinary step kernel), never a stand-alone sync
    assert states[3][2]["launches_sync"] == 0
    assert states[3][2]["launches_fused"] + states[3][2]["launches_local"] <= \
        -(-4 // min(H, 8)) + -(-(T - 4) // min(H, 8)) + 2


# ----------------------------------------------------------------------------- schedule
@pytest.mark.parametrize("H,T", [(1, 5), (2, 5), (3, 9), (5, 5), (6, 5), (la.LA_H_NEVER, 6)])
@pytest.mark.parametrize("fusion", [0, 1, 2, 3, 4])
def test_schedule_counters_match_oracle(H, T, fusion):
    g, o = make_pair(64, 2, 0.1, 1.0, H, "noise", seed=1, fusion=fusion)
    for _ in range(T):
        g.run(1)
        o.run(1)
        assert g.get_counters() == o.counters()
    compare(g, o, 2, TOL_RUN)


def test_zero_length_run_and_repeated_sync_are_harmless():
    g, o = make_pair(33, 4, 0.2, 1.0, 2, "noise", seed=3)
    g.run(0); o.run(0)
    assert g.get_counters() == (0, 0, 0)
    g.sync(); o.sync()                      # averaging identical replicas: the identity
    x, b2, bs = g.read_state(3)
    assert np.all(x == 0) and np.all(b2 == 0) and np.all(bs == 0)
    g.run(5); o.run(5)
    compare(g, o, 4, TOL_RUN)


def test_manual_steps_and_sync():
    g, o = make_pair(100, 4, 0.2, 1.0, 10, "noise", seed=3)
    for k in range(3):
        g.local_step(); o.local_step()
    g.sync(); o.sync()
    g.local_step(); o.local_step()
    g.sync(); o.sync()
    g.sync(); o.sync()
    compare(g, o, 4, TOL_RUN)
    assert g.get_counters() == (4, 0, 3)


@pytest.mark.parametrize("fusion", [1, 3, 4])
def test_warmup_matches_oracle(fusion):
    g, o = make_pair(513, 4, 0.5, 1.0, 4, "noise", seed=8, warmup=6, b0sq=1.0, fusion=fusion)
    g.run(11); o.run(11)
    compare(g, o, 4, TOL_RUN)


@pytest.mark.parametrize("H,T,W", [(20, 50, 4), (8, 64, 8), (64, 70, 16), (5, 23, 2), (9, 9, 3)])
def test_period_fusion_long_periods(H, T, W):
    """Periods longer than one pass (8 steps) are cut into pieces; run boundaries fall anywhere."""
    n = 3001
    arr = _arrays(n, H)
    g, o = make_pair(n, W, 0.05, 0.5, H, "quadratic", seed=H, arrays=arr, sigma=0.4, fusion=3)
    g.run(3); g.run(T - 3)
    o.run(T)
    compare(g, o, W, TOL_RUN)


def test_initial_iterate_and_b0():
    n = 777
    x0 = np.random.default_rng(0).standard_normal(n).astype(np.float32)
    arr = _arrays(n, 1)
    g, o = make_pair(n, 8, 0.5, 1.0, 4, "quadratic", seed=2, arrays=arr, sigma=1.0, x0=x0, b0sq=1.0, fusion=2)
    g.run(9); o.run(9)
    compare(g, o, 8, TOL_RUN)


# ----------------------------------------------------------------------------- invariants on the GPU
def test_identical_workers_stay_bitwise_equal():
    n, W = 4099, 8
    arr = _arrays(n, 5)
    g, o = make_pair(n, W, 0.1, 1.0, 4, "quadratic", seed=9, arrays=arr, sigma=0.1, identical=True, fusion=1)
    g.run(10); o.run(10)
    compare(g, o, W, TOL_RUN)
    x0, b0, _ = g.read_state(0)
    for i in range(1, W):
        x, b, _ = g.read_state(i)
        assert np.array_equal(x, x0) and np.array_equal(b, b0)


def test_constant_gradient_closed_form_on_gpu():
    """B^2 = b0^2 + k g^2 and x_T from the closed form, independent of the oracle."""
    n, W, H, T = 6, 4, 3, 23
    gvec = np.array([0.5, -1.5, 2.0, 1.0, -0.25, 3.0], np.float32)
    eta, eps, b0sq = 0.5, 0.75, 1.0
    g = la.LocalAdaAlter([n], W, eta, eps, H, b0sq=b0sq)
    g.set_init(None, b0sq)
    g.set_grad_constant(gvec)
    g.run(T)
    exp_x = np.zeros(n)
    for t in range(1, T + 1):
        tp = (t - 1) % H + 1
        exp_x -= eta * gvec.astype(np.float64) / np.sqrt(b0sq + (t - tp) * gvec.astype(np.float64) ** 2 + tp * eps * eps)
    for i in range(W):
        x, b2, bs = g.read_state(i)
        np.testing.assert_allclose(b2, b0sq + T * gvec.astype(np.float64) ** 2, rtol=1e-6)
        np.testing.assert_allclose(x, exp_x, rtol=5e-6)
        np.testing.assert_allclose(bs, b0sq + (T - T % H) * gvec.astype(np.float64) ** 2, rtol=1e-6)


def test_hand_worked_case_with_supplied_gradients():
    """The hand-derived Algorithm-3 trajectory, driven through la_local_step_grads."""
    import os
    import torch
    rows = [[float(v) for v in l.split()] for l in
            open(os.path.join(os.path.dirname(__file__), "golden", "alg3_hand_case.txt"))
            if l.strip() and not l.startswith("#")]
    g = la.LocalAdaAlter([1], 2, 1.0, 1.0, 2)
    for t, g0, g1, x0, x1, b0, b1, bs in rows:
        grads = torch.tensor([[g0], [g1]], dtype=torch.float32, device="cuda")
        g.local_step_grads(grads.data_ptr(), la.LA_F32)
        if g.get_counters()[1] == 2:
            g.sync()
        xa, ba, sa = g.read_state(0)
        xb, bb, _ = g.read_state(1)
        assert xa[0] == pytest.approx(x0, abs=5e-7) and xb[0] == pytest.approx(x1, abs=5e-7)
        assert (ba[0], bb[0], sa[0]) == (b0, b1, bs)
    assert g.get_counters() == (4, 0, 2)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n", [5, 64, 1001])
def test_supplied_gradients_match_oracle(dtype, n):
    import torch
    W, H, T = 3, 2, 5
    rng = np.random.default_rng(n)
    g = la.LocalAdaAlter([n], W, 0.3, 0.5, H, b0sq=0.25)
    g.set_init(None, 0.25)
    o = Oracle(n, W, 0.3, 0.5, H, 0.25)
    for t in range(T):
        G = torch.from_numpy(rng.standard_normal((W, n)).astype(np.float32))
        if dtype == "bf16":
            Gd = G.to(torch.bfloat16).cuda()
            g.local_step_grads(Gd.data_ptr(), la.LA_BF16)
            o.local_step(Gd.float().cpu().numpy())
        else:
            Gd = G.cuda()
            g.local_step_grads(Gd.data_ptr(), la.LA_F32)
            o.local_step(G.numpy())
        if g.get_counters()[1] == H:
            g.sync(); o.sync()
        g.sync_stream()
    compare(g, o, W, TOL_RUN)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("W,n,H,fusion", [(4, 70002, 3, 1), (8, 4098, 2, 0), (16, 1000, 4, 1), (3, 777, 2, 1),
                                           (2, 12, 1, 1), (5, 4100, 3, 2), (4, 70002, 3, 4), (8, 4098, 2, 4),
                                           (3, 777, 5, 4), (1, 2052, 2, 4), (33, 260, 3, 4), (2, 12, 1, 4),
                                           (5, 4100, 3, 4), (6, 4100, 2, 1), (6, 4102, 3, 4), (6, 777, 2, 0)])
def test_step_grads_full_iteration(dtype, W, n, H, fusion):
    """la_step_grads = local step + the synchronisation when it is due (fused or not); even n takes
    the vector loads, odd n the scalar ones; a table offset by one element is mis-aligned."""
    import torch
    T = 7
    rng = np.random.default_rng(n + W)
    g = la.LocalAdaAlter([n], W, 0.3, 0.5, H, b0sq=0.25)
    g.set_init(None, 0.25)
    g.set_fusion(fusion)
    o = Oracle(n, W, 0.3, 0.5, H, 0.25)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    code = la.LA_F32 if dtype == "f32" else la.LA_BF16
    for t in range(T):
        G = torch.from_numpy(rng.standard_normal((W, n)).astype(np.float32)).to(tdt)
        pad = 1 if t == 2 else 0                                   # once: a mis-aligned table
        buf = torch.empty(W * n + pad, dtype=tdt, device="cuda")
        buf[pad:] = G.reshape(-1).cuda()
        g.step_grads(buf[pad:].data_ptr(), code)
        o.local_step(G.float().numpy())
        if o.counters()[1] == H:
            o.sync()
        g.sync_stream()
        assert g.get_counters() == o.counters()
    compare(g, o, W, TOL_RUN)
    st = g.get_stats()
    if fusion == 0:
        assert st["launches_fused"] == 0 and st["launches_sync"] == T // H
    elif fusion == 4 and H >= 2:
        # sums out at every t' = H, one copy in at every following t' = 1; the final read completed pending sums
        assert st["launches_step_sync"] == T // H and st["launches_sync_step"] == (T - 1) // H
    else:
        assert st["launches_fused"] == T // H and st["launches_sync"] == 0


def test_checkpoint_resume_bitwise():
    n, W, H = 3001, 4, 4
    arr = _arrays(n, 6)

    def make():
        c = la.LocalAdaAlter([n], W, 0.1, 1.0, H)
        c.set_grad_quadratic(7, arr["a"], arr["c"], 0.1)
        c.set_fusion(2)
        return c

    whole = make(); whole.run(11)
    first = make(); first.run(6)
    second = make()
    for i in range(W):
        x, b2, bs = first.read_state(i)
        second.write_state(i, x, b2, bs)
    second.set_counters(*first.get_counters())
    second.run(5)
    assert whole.get_counters() == second.get_counters() == (11, 3, 2)
    for i in range(W):
        for u, v in zip(whole.read_state(i), second.read_state(i)):
            assert np.array_equal(u.view(np.uint32), v.view(np.uint32))


def test_coordinate_sharding_is_exact():
    """Two contexts that own the halves of the coordinate range reproduce the whole job."""
    n, W = 4096 + 512, 4
    arr = _arrays(n, 12)
    whole = la.LocalAdaAlter([n], W, 0.01, 1e-3, 8)
    whole.set_grad_noise(2, arr["s"]); whole.run(20)
    cut = 2048
    parts = []
    for lo, hi in ((0, cut), (cut, n)):
        p = la.LocalAdaAlter([hi - lo], W, 0.01, 1e-3, 8, j_base=lo)
        p.set_grad_noise(2, arr["s"][lo:hi]); p.run(20)
        parts.append(p)
    for i in range(W):
        full = whole.read_state(i)
        for k in range(3):
            joined = np.concatenate([parts[0].read_state(i)[k], parts[1].read_state(i)[k]])
            assert np.array_equal(joined.view(np.uint32), full[k].view(np.uint32))


def test_multi_tensor_views_and_torch_arena():
    import torch
    sizes = [1000, 3, 4096, 77]
    n = sum(sizes)
    arr = _arrays(n, 4)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        g = la.LocalAdaAlter.with_torch_arena(sizes, 4, 0.1, 1.0, 4)
        g.set_grad_quadratic(3, arr["a"], arr["c"], 0.5)
        g.run(9)
    o = Oracle(n, 4, 0.1, 1.0, 4)
    o.set_grad_quadratic(3, arr["a"], arr["c"], 0.5)
    o.run(9)
    compare(g, o, 4, TOL_RUN)
    off = 0
    for k, sz in enumerate(sizes):
        assert g.tensor_range(k) == (off, sz)
        off += sz


def test_runtime_errors_are_reported_not_fatal():
    g = la.LocalAdaAlter([64], 2, 0.1, 1.0, 2)
    with pytest.raises(la.LocalAdaAlterError) as e:
        g.read_state(5)
    assert e.value.code == la.LA_EINVAL and "worker" in str(e.value)
    with pytest.raises(la.LocalAdaAlterError):
        g.read_range(0, 60, 10)
    with pytest.raises(la.LocalAdaAlterError):
        g.set_fusion(9)
    with pytest.raises(la.LocalAdaAlterError):
        g.local_step_grads(0)
    g.run(3)                                   # the context is still usable
    assert g.get_counters() == (3, 1, 1)
    import torch
    too_small = torch.empty(16, device="cuda")
    with pytest.raises(la.LocalAdaAlterError) as e:
        la.LocalAdaAlter([64], 2, 0.1, 1.0, 2, arena=too_small)
    assert e.value.code == la.LA_ENOMEM


def test_profiling_stats():
    g = la.LocalAdaAlter([1 << 16], 4, 0.1, 1.0, 4)
    g.set_grad_noise(1)
    g.set_profiling(True)
    g.run(8)
    st = g.get_stats()
    assert st["launches_local"] == 8 and st["launches_sync"] == 2
    assert st["ms_local"] > 0 and st["ms_sync"] > 0
    assert st["bytes_local"] == 8 * (16 * 4 + 4) * (1 << 16)
    assert st["bytes_sync"] == 2 * (16 * 4 + 4) * (1 << 16)


@pytest.mark.parametrize("W,n", [(4, 1000), (16, 65), (3, 4097), (8, 1)])
def test_no_write_outside_the_arena(W, n):
    """Guard bands around a caller-provided arena stay untouched by every kernel of the path
    (the stand-in for a memory checker: the kernels index only inside la_arena_bytes)."""
    import torch
    need = la.LocalAdaAlter.arena_bytes([n], W) // 4
    guard = 4096                                                   # floats on each side (256-byte multiple)
    buf = torch.full((need + 2 * guard,), -777.0, dtype=torch.float32, device="cuda")
    assert buf.data_ptr() % 256 == 0
    arena = buf[guard:guard + need]
    arr = _arrays(n, 9)
    g = la.LocalAdaAlter([n], W, 0.1, 1.0, 3, arena=arena, device=torch.cuda.current_device())
    g.set_grad_quadratic(4, arr["a"], arr["c"], 0.5)
    for fusion in (0, 1, 2, 3, 4):
        g.set_fusion(fusion)
        g.run(7)
    g.set_grad_noise(4, arr["s"]); g.run(4)
    g.set_grad_dtype(la.LA_BF16); g.run(3); g.set_grad_dtype(la.LA_F32)
    G = torch.randn(W * n, device="cuda")
    g.step_grads(G.data_ptr(), la.LA_F32)
    g.step_grads(G.to(torch.bfloat16).data_ptr(), la.LA_BF16)
    g.sync()
    g.set_rule(la.LA_RULE_LOCAL_SGD); g.run(6)
    g.set_rule(la.LA_RULE_ADAGRAD); g.run(3)
    g.set_rule(la.LA_RULE_ADAALTER)
    g.set_init(None, 0.5)
    g.sync_stream()
    torch.cuda.synchronize()
    assert bool((buf[:guard] == -777.0).all()) and bool((buf[guard + need:] == -777.0).all())
    g.close()


def test_diagnostics_objective_and_replica_spread():
    n, W, H = 5003, 8, 4
    arr = _arrays(n, 31)
    g = la.LocalAdaAlter([n], W, 0.1, 1.0, H, b0sq=1.0)
    g.set_init(None, 1.0)
    g.set_grad_quadratic(3, arr["a"], arr["c"], 0.5)
    a, c = arr["a"].astype(np.float64), arr["c"].astype(np.float64)
    f0, d0 = g.diagnostics()
    assert f0 == pytest.approx(0.5 * np.sum(a * c * c), rel=1e-12) and d0 == 0.0
    g.run(6)                                        # two steps into the second period
    X = np.stack([g.read_state(i)[0] for i in range(W)]).astype(np.float64)
    xbar = X.mean(0)
    f, d = g.diagnostics()
    assert f == pytest.approx(0.5 * np.sum(a * (xbar - c) ** 2), rel=1e-11)
    assert d == pytest.approx(np.sum((X - xbar) ** 2) / W, rel=1e-11) and d > 0
    assert f < f0
    g.run(2)                                        # closes the period: replicas coincide again
    assert g.diagnostics()[1] == 0.0
    g.set_grad_noise(1, None)
    assert np.isnan(g.diagnostics()[0])


@pytest.mark.parametrize("fusion", [0, 1, 3])
@pytest.mark.parametrize("rule", [0, 1])
def test_graph_replay_is_bitwise_and_counts_the_same(fusion, rule):
    """la_set_graph: whole periods replayed from a captured CUDA graph (launch-bound sizes)."""
    import torch
    n, W, H = 6000, 4, 4
    arr = _arrays(n, 17)
    with torch.cuda.stream(torch.cuda.Stream()):
        g = la.LocalAdaAlter.with_torch_arena([n], W, 0.1, 1.0, H)
        p = la.LocalAdaAlter.with_torch_arena([n], W, 0.1, 1.0, H)          # same, launched plainly
        o = Oracle(n, W, 0.1, 1.0, H)
        for ctx in (g, p):
            ctx.set_grad_quadratic(5, arr["a"], arr["c"], 0.3)
            ctx.set_warmup(7)
            ctx.set_rule(rule)
            ctx.set_fusion(fusion)
        o.set_grad_quadratic(5, arr["a"], arr["c"], 0.3)
        o.set_warmup(7)
        o.set_rule(rule)
        g.set_graph(True)
        for T in (9, 3, 12, 2):                     # 9 = two periods + one step; then starts inside a period
            g.run(T); p.run(T); o.run(T)
            assert g.get_counters() == o.counters() == p.get_counters()
        compare(g, o, W, TOL_RUN)
        sg, sp = g.get_stats(), p.get_stats()
        for k in ("launches_local", "launches_sync", "launches_fused", "bytes_local", "bytes_sync", "bytes_fused"):
            assert sg[k] == sp[k], k
        # a changed configuration rebuilds the graph
        g.set_grad_noise(9, arr["s"]); o.set_grad_noise(9, arr["s"])
        g.run(2); o.run(2)                          # finish the open period (t' = 2 -> 0)
        g.run(8); o.run(8)
        compare(g, o, W, TOL_RUN)
        g.close(); p.close()


def test_graph_replay_needs_a_capturable_stream():
    g = la.LocalAdaAlter([64], 2, 0.1, 1.0, 2)      # legacy default stream
    with pytest.raises(la.LocalAdaAlterError) as e:
        g.set_graph(True)
    assert e.value.code == la.LA_ESTATE
    g.run(4)


@pytest.mark.parametrize("seed", range(12))
def test_random_call_sequences_match_oracle(seed):
    """Random interleavings of la_run / la_local_step / la_sync / fusion and launch-shape changes,
    state round trips and rule changes at period boundaries, mirrored on the oracle."""
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 5000))
    W = int(rng.choice([1, 2, 3, 4, 8, 16, 6, 5, 12, 32, 17, 20]))
    H = int(rng.integers(1, 7))
    arr = _arrays(n, seed)
    grad = ["noise", "noise_scaled", "quadratic"][seed % 3]
    g, o = make_pair(n, W, 0.05, 0.7, H, grad, seed=seed, arrays=arr, sigma=0.4, b0sq=0.5)
    rule = 0
    import torch
    for _ in range(40):
        op = rng.integers(0, 9)
        if op <= 2:
            T = int(rng.integers(0, 3 * H + 2))
            g.run(T); o.run(T)
        elif op == 3:
            g.local_step(); o.local_step()
            if rule == 0 and o.counters()[1] >= H and rng.random() < 0.5:
                g.sync(); o.sync()
        elif op == 4 and rule != 2:                              # AdaGrad has nothing to synchronise
            g.sync(); o.sync()
        elif op == 5:
            g.set_fusion(int(rng.integers(0, 5)))
            g.set_launch_shape(int(rng.choice([0, 1, 7, 4096])))
        elif op == 6 and o.counters()[1] == 0:
            rule = int(rng.integers(0, 3))                       # Local AdaAlter, Local SGD, AdaGrad
            g.set_rule(rule); o.set_rule(rule)
        elif op == 7:
            i = int(rng.integers(0, W))
            x, b2, bs = g.read_state(i)
            g.write_state(i, x, b2, bs)                          # a checkpoint round trip changes nothing
        elif op == 8:                                            # a complete iteration with a supplied gradient table
            bf16 = bool(rng.integers(0, 2))
            G = torch.from_numpy(rng.standard_normal((W, n)).astype(np.float32))
            G = G.to(torch.bfloat16) if bf16 else G
            Gd = G.cuda()
            g.step_grads(Gd.data_ptr(), la.LA_BF16 if bf16 else la.LA_F32)
            o.local_step(G.float().numpy())
            if rule != 2 and o.counters()[1] == H:
                o.sync()
            g.sync_stream()
        assert g.get_counters() == o.counters()
    compare(g, o, W, TOL_RUN)


def test_two_contexts_on_two_streams_do_not_interfere():
    import torch
    n, W = 200003, 4
    arr = _arrays(n, 2)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    with torch.cuda.stream(s1):
        g1 = la.LocalAdaAlter.with_torch_arena([n], W, 0.1, 1.0, 3)
    with torch.cuda.stream(s2):
        g2 = la.LocalAdaAlter.with_torch_arena([n], W, 0.2, 0.5, 2)
    g1.set_grad_quadratic(1, arr["a"], arr["c"], 0.3)
    g2.set_grad_noise(2, arr["s"])
    for _ in range(5):                                           # interleaved enqueueing
        g1.run(3); g2.run(4)
    o1 = Oracle(n, W, 0.1, 1.0, 3); o1.set_grad_quadratic(1, arr["a"], arr["c"], 0.3); o1.run(15)
    o2 = Oracle(n, W, 0.2, 0.5, 2); o2.set_grad_noise(2, arr["s"]); o2.run(20)
    compare(g1, o1, W, TOL_RUN)
    compare(g2, o2, W, TOL_RUN)


@pytest.mark.parametrize("fusion", [1, 3])
def test_paper_hyperparameters(fusion):
    """The settings of the paper's experiments (Section 6): eps = 1, b0 = 1, eta = 0.5 with 600
    warm-up steps, 8 workers, H = 4 (the period the paper recommends)."""
    n, W, H, T = 20000, 8, 4, 24
    arr = _arrays(n, 44)
    g, o = make_pair(n, W, 0.5, 1.0, H, "quadratic", seed=6, arrays=arr, sigma=1.0, b0sq=1.0, warmup=600,
                     fusion=fusion)
    g.run(1); o.run(1)
    compare(g, o, W, TOL_STEP)
    g.run(T - 1); o.run(T - 1)
    compare(g, o, W, TOL_RUN)
    x, _, _ = o.read(0)
    xd, _, _ = o.read_shadow(0)
    assert np.max(np.abs(x - xd)) < 1e-5          # fp32 path tracks the literal fp64 formulas


@pytest.mark.parametrize("W", [24, 48])
def test_run_time_worker_counts_over_many_blocks(W):
    """Worker counts without a dedicated kernel, on enough coordinates for several blocks per SM
    and a ragged tail, through every fusion mode."""
    n, H, T = 150001, 3, 7
    arr = _arrays(n, W)
    for fusion in (0, 1, 2, 3, 4):
        g, o = make_pair(n, W, 0.05, 1.0, H, "noise_scaled", seed=W, arrays=arr, fusion=fusion)
        g.run(T); o.run(T)
        compare(g, o, W, TOL_RUN)
        g.close()


def test_noise_building_blocks_over_their_whole_domain():
    """Every one of the 2^24 radii and 2^24 (cos, sin) pairs the kernels can produce, against the
    oracle's recipe, bit for bit.  The radius is sqrt(L) with L from the oracle's table and the
    correctly rounded fp32 square root (numpy's), which is what the oracle's noise draw applies."""
    import torch
    from oracle import oracle as O
    r = torch.empty(1 << 24, dtype=torch.float32, device="cuda")
    c = torch.empty_like(r)
    s = torch.empty_like(r)
    assert la.noise_tables(r.data_ptr(), c.data_ptr(), s.data_ptr()) == la.LA_OK
    torch.cuda.synchronize()
    L = O.table_neg2ln()
    assert L.min() >= 0.0 and L[-1] == 0.0
    want_r = np.sqrt(L, dtype=np.float32)
    assert np.array_equal(r.cpu().numpy().view(np.uint32), want_r.view(np.uint32))
    oc, os_ = O.table_cossin()
    assert np.array_equal(c.cpu().numpy().view(np.uint32), oc.view(np.uint32))
    assert np.array_equal(s.cpu().numpy().view(np.uint32), os_.view(np.uint32))
    assert la.noise_tables(None, None, None) == la.LA_OK


@pytest.mark.parametrize("W,n,H", [(4, 70002, 3), (8, 4099, 2), (16, 1000, 4), (3, 777, 5), (5, 3001, 2), (1, 513, 3), (33, 260, 2)])
def test_mean_once_fusion_pending_sums_are_completed_on_demand(W, n, H):
    """LA_FUSE_MEAN_ONCE keeps the result of a synchronisation as ONE copy (the sums over the workers in
    replica 0's rows) until the next step consumes it.  Runs that end exactly on a period boundary leave
    those sums pending; every way of looking at or touching the state must complete them first, and
    the run must carry on from the pending state in the next call — all bitwise against the oracle."""
    import torch
    arr = _arrays(n, W + H)
    g, o = make_pair(n, W, 0.05, 0.7, H, "quadratic", seed=5, arrays=arr, sigma=0.4, b0sq=0.25, fusion=4)
    g.run(H); o.run(H)                       # ends on the boundary: sums pending
    compare(g, o, W, TOL_RUN)                # a read completes them
    g.run(2 * H); o.run(2 * H)               # pending again ...
    g.run(H + 1); o.run(H + 1)               # ... and consumed by the first step of this call
    compare(g, o, W, TOL_RUN)
    g.run(H - 1); o.run(H - 1)               # pending
    g.local_step(); o.local_step()           # a manual step completes them first
    g.sync(); o.sync()
    compare(g, o, W, TOL_RUN)
    g.run(H); o.run(H)                       # pending
    i = W - 1
    x, b2, bs = g.read_state(i)
    g.write_state(i, x, b2, bs)              # a per-worker write
    g.run(H); o.run(H)                       # pending
    g.set_fusion(2)                          # another fusion mode takes over from the pending state
    g.run(2 * H + 1); o.run(2 * H + 1)
    compare(g, o, W, TOL_RUN)
    g.sync(); o.sync()
    g.set_fusion(4)
    g.run(H); o.run(H)                       # pending
    G = np.random.default_rng(0).standard_normal((W, n)).astype(np.float32)
    Gd = torch.from_numpy(G).cuda()
    g.step_grads(Gd.data_ptr(), la.LA_F32); o.local_step(G)   # supplied gradients after pending sums
    if o.counters()[1] == H:
        o.sync()
    compare(g, o, W, TOL_RUN)
    st = g.get_stats()
    assert st["launches_step_sync"] > 0 and st["launches_sync_step"] > 0


@pytest.mark.parametrize("W,n,H,T,grad,fusion,chunks,bf16", [
    (4, 70001, 3, 10, "quadratic", 4, 3, True), (8, 5000, 2, 7, "noise_scaled", 1, 16, False),
    (3, 1025, 4, 8, "noise", 3, 5, False), (16, 300, 1, 3, "quadratic", 2, 1, False),
    (5, 40000, 5, 11, "quadratic", 0, 7, False), (1, 2049, 2, 4, "noise_scaled", 4, 2, False)])
def test_streamed_run_equals_upload_run_download(W, n, H, T, grad, fusion, chunks, bf16):
    """la_run_streamed pipelines [upload, T iterations, download] over coordinate ranges; outputs,
    device state and counters must be those of la_set_init + la_set_grad_* + la_run + la_read_state,
    i.e. the oracle's, bitwise — also when it is called again on a used context, and for a worker
    other than 0."""
    import torch
    rng = np.random.default_rng(n)
    arr = _arrays(n, W)
    x0 = rng.standard_normal(n).astype(np.float32)
    g, o = make_pair(n, W, 0.05, 0.7, H, grad, seed=4, arrays=arr, sigma=0.4, bf16=bf16, fusion=fusion, b0sq=0.5, x0=x0)
    o.run(T)
    g.run(3)                                                    # a used context: the call re-initialises it
    pin = lambda a: torch.from_numpy(a).pin_memory()
    outs = {k: torch.empty(n, dtype=torch.float32).pin_memory() for k in ("x", "b2", "bs")}
    w = W - 1
    kw = {"a": pin(arr["a"]), "c": pin(arr["c"])} if grad == "quadratic" else ({"s": pin(arr["s"])} if grad == "noise_scaled" else {})
    for rep in range(2):
        g.run_streamed(T, worker=w, x0=pin(x0), x_out=outs["x"], b2_out=outs["b2"], bs_out=outs["bs"], chunks=chunks, **kw)
        assert g.get_counters() == o.counters()
        for got, ref in zip((outs["x"], outs["b2"], outs["bs"]), o.read(w)):
            assert np.array_equal(got.numpy().view(np.uint32), ref.view(np.uint32))
    compare(g, o, W, TOL_RUN)                                   # the resident state as well
    g.run(H + 1); o.run(H + 1)                                  # and the run carries on from it
    compare(g, o, W, TOL_RUN)
    x_np = np.empty(n, np.float32)                              # pageable memory works too (without overlap)
    g.run_streamed(T, worker=0, x0=x0, x_out=x_np, chunks=chunks,
                   **{k: v.numpy() for k, v in kw.items()})
    o2 = make_pair(n, W, 0.05, 0.7, H, grad, seed=4, arrays=arr, sigma=0.4, bf16=bf16, fusion=fusion, b0sq=0.5, x0=x0)[1]
    o2.run(T)
    assert np.array_equal(x_np.view(np.uint32), o2.read(0)[0].view(np.uint32))


@pytest.mark.parametrize("W", [32, 48, 64])
def test_worker_counts_of_whole_tiles(W):
    """Large worker counts — 32 and 64 with their own instantiation, 48 through the run-time path,
    where whole tiles of 16 replicas are summed by the constant-index tree and pushed into the
    run-time counter as aligned blocks: the result is the adjacent-pair tree over all W workers,
    bitwise, for the stand-alone synchronisation, both fusions, supplied gradient tables and
    manual call sequences."""
    import torch
    n, H = 1537, 3
    arr = _arrays(n, W)
    for fusion in (0, 1, 2):
        g, o = make_pair(n, W, 0.05, 0.7, H, "noise_scaled", seed=W, arrays=arr, fusion=fusion, b0sq=0.5)
        g.run(2 * H + 1); o.run(2 * H + 1)
        g.sync(); o.sync()                                         # a manual synchronisation inside a period
        g.run(H); o.run(H)
        compare(g, o, W, TOL_RUN)
        st = g.get_stats()
        assert st["launches_sync"] + st["launches_fused"] >= 3
    g, o = make_pair(n, W, 0.05, 0.7, H, "noise", seed=1, fusion=1)
    rng = np.random.default_rng(W)
    for dtype, tdt in ((la.LA_F32, torch.float32), (la.LA_BF16, torch.bfloat16)):
        for t in range(H + 1):
            G = torch.from_numpy(rng.standard_normal((W, n)).astype(np.float32)).to(tdt)
            Gd = G.cuda()
            g.step_grads(Gd.data_ptr(), dtype); o.local_step(G.float().numpy())
            if o.counters()[1] == H:
                o.sync()
            g.sync_stream()
    compare(g, o, W, TOL_RUN)
