"""GPU parity for the paper's baseline update rules run through the same sweep: Local SGD
(Algorithm 2) and Distributed AdaGrad (Algorithm 1), against the oracle, bitwise."""
import numpy as np
import pytest

from oracle.oracle import Oracle
from paper_1911_09030_b200 import local_adaalter as la
from parity_util import compare, make_pair

pytestmark = pytest.mark.gpu


def _arrays(n, seed):
    rng = np.random.default_rng(seed)
    return dict(a=rng.uniform(0.1, 3, n).astype(np.float32), c=rng.standard_normal(n).astype(np.float32),
                s=rng.uniform(0.1, 1, n).astype(np.float32))


@pytest.mark.parametrize("W", [1, 2, 3, 4, 8, 16, 5])
@pytest.mark.parametrize("grad", ["noise", "noise_scaled", "quadratic", "constant"])
def test_local_sgd_matches_oracle(W, grad):
    n, T = 1027, 11
    arr = _arrays(n, W)
    for H, fusion in [(1, 1), (3, 0), (4, 2), (T + 1, 1)]:
        g, o = make_pair(n, W, 0.05, 1.0, H, grad, seed=3, arrays=arr, sigma=0.5, fusion=fusion)
        g.set_rule(la.LA_RULE_LOCAL_SGD)
        o.set_rule(1)
        g.run(T)
        o.run(T)
        compare(g, o, W, 1e-5)
        g.close()


@pytest.mark.parametrize("W", [1, 2, 3, 4, 8, 16, 6])
@pytest.mark.parametrize("grad", ["noise", "noise_scaled", "quadratic", "constant"])
def test_adagrad_matches_oracle(W, grad):
    n, T = 2050, 9
    arr = _arrays(n, 10 + W)
    g, o = make_pair(n, W, 0.3, 0.5, 4, grad, seed=5, arrays=arr, sigma=1.0, warmup=4)
    g.set_rule(la.LA_RULE_ADAGRAD)
    o.set_rule(2)
    g.run(1)
    o.run(1)
    compare(g, o, W, 1e-6)
    g.run(T - 1)
    o.run(T - 1)
    compare(g, o, W, 1e-5)
    assert g.get_counters() == (T, 0, T)
    with pytest.raises(la.LocalAdaAlterError):
        g.sync()


@pytest.mark.parametrize("W", [3, 8])
@pytest.mark.parametrize("next_rule", [la.LA_RULE_ADAALTER, la.LA_RULE_LOCAL_SGD])
def test_leaving_adagrad_continues_from_the_common_iterate(W, next_rule):
    """Algorithm 1 keeps one iterate that every worker holds.  When another rule takes over, every
    replica must start from it (and from the common accumulator), as in the oracle."""
    n, H = 3001, 4
    arr = _arrays(n, 40 + W)
    g, o = make_pair(n, W, 0.2, 0.5, H, "quadratic", seed=8, arrays=arr, sigma=0.7)
    g.run(H); o.run(H)                                    # replicas have a history of their own first
    g.set_rule(la.LA_RULE_ADAGRAD); o.set_rule(2)
    g.run(3); o.run(3)
    compare(g, o, W, 1e-5)
    g.set_rule(next_rule); o.set_rule(next_rule)
    compare(g, o, W, 1e-5)                                # every worker reads the common iterate
    g.run(H + 1); o.run(H + 1)
    compare(g, o, W, 1e-5)
    g.run(H - 1); o.run(H - 1)
    g.set_rule(la.LA_RULE_ADAGRAD); o.set_rule(2)         # and back again
    g.run(2); o.run(2)
    compare(g, o, W, 1e-5)
    g.close()


def test_state_written_per_worker_under_adagrad_is_kept():
    """A per-worker write after AdaGrad steps makes the replicas individual again."""
    n, W = 515, 4
    arr = _arrays(n, 3)
    g, o = make_pair(n, W, 0.2, 0.5, 2, "noise_scaled", seed=4, arrays=arr)
    g.set_rule(la.LA_RULE_ADAGRAD); o.set_rule(2)
    g.run(2); o.run(2)
    x = np.linspace(-1, 1, n).astype(np.float32)
    b = np.full(n, 2.5, np.float32)
    g.write_state(2, x, b, None); o.write(2, x, b, None)
    compare(g, o, W, 0.0)
    g.set_rule(la.LA_RULE_ADAALTER); o.set_rule(0)
    g.run(3); o.run(3)
    compare(g, o, W, 1e-5)
    g.close()


def test_rule_changes_only_at_a_period_boundary():
    g = la.LocalAdaAlter([64], 2, 0.1, 1.0, 4)
    g.set_grad_noise(1)
    g.run(1)
    with pytest.raises(la.LocalAdaAlterError) as e:
        g.set_rule(la.LA_RULE_LOCAL_SGD)
    assert e.value.code == la.LA_ESTATE
    g.run(3)
    g.set_rule(la.LA_RULE_LOCAL_SGD)
    g.run(4)
    with pytest.raises(la.LocalAdaAlterError):
        g.set_rule(7)
    g.set_grad_dtype(la.LA_BF16)
    with pytest.raises(la.LocalAdaAlterError) as e:
        g.run(1)                                # baselines exist for fp32 gradients only
    assert e.value.code == la.LA_ESTATE


def test_three_rules_on_one_problem_behave_as_the_paper_describes():
    """Noise-free quadratic: all rules descend; with identical workers Local SGD is plain SGD."""
    n, W, T = 512, 4, 40
    arr = _arrays(n, 2)
    f = lambda x: 0.5 * np.sum(arr["a"].astype(np.float64) * (x.astype(np.float64) - arr["c"]) ** 2)
    f0 = f(np.zeros(n, np.float32))
    for rule in (la.LA_RULE_ADAALTER, la.LA_RULE_LOCAL_SGD, la.LA_RULE_ADAGRAD):
        g = la.LocalAdaAlter([n], W, 0.2, 1.0, 4, b0sq=1.0)
        g.set_init(None, 1.0)
        g.set_grad_quadratic(1, arr["a"], arr["c"], 0.0)
        g.set_rule(rule)
        g.run(T)
        assert f(g.read_state(0)[0]) < 0.2 * f0


@pytest.mark.parametrize("rule", [la.LA_RULE_LOCAL_SGD, la.LA_RULE_ADAGRAD])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("W,n", [(4, 4098), (3, 777), (8, 70000)])
def test_baselines_with_supplied_gradients(rule, dtype, W, n):
    """The trainer-facing call (la_step_grads) under the two baseline rules."""
    import torch
    H, T = 3, 7
    rng = np.random.default_rng(n + W)
    g = la.LocalAdaAlter([n], W, 0.2, 0.5, H)
    g.set_rule(rule)
    g.set_fusion(la.LA_FUSE_STEP_SYNC)
    o = Oracle(n, W, 0.2, 0.5, H)
    o.set_rule(rule)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    code = la.LA_F32 if dtype == "f32" else la.LA_BF16
    for t in range(T):
        G = torch.from_numpy(rng.standard_normal((W, n)).astype(np.float32)).to(tdt)
        Gd = G.cuda()
        g.step_grads(Gd.data_ptr(), code)
        o.local_step(G.float().numpy())
        if rule == la.LA_RULE_LOCAL_SGD and o.counters()[1] == H:
            o.sync()
        g.sync_stream()
        assert g.get_counters() == o.counters()
    compare(g, o, W, 1e-5)
