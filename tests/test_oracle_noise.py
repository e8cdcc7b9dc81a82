"""Pins for the oracle's synthetic gradient source (hash, uniforms, Box-Muller recipes,
bf16 rounding).  The source is not from the paper; it is pinned against the published
splitmix64 sequence, against libm in double (exhaustively), against torch's bfloat16
conversion and against the N(0,1) law.  CPU only."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle as O

M64 = (1 << 64) - 1
GAMMA = 0x9E3779B97F4A7C15


def test_splitmix64_published_sequence():
    """First three outputs of the splitmix64 generator seeded with 0 (the sequence commonly
    quoted for seeding xoshiro/xoroshiro): state advances by the golden-ratio increment and
    the output is the finaliser of the state."""
    assert [O.mix64((GAMMA * k) & M64) for k in (1, 2, 3)] == [
        0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_mix64_is_a_bijection_on_a_sample_and_avalanches():
    rng = np.random.default_rng(0)
    zs = [int(v) for v in rng.integers(0, 1 << 63, 2000)]
    outs = {O.mix64(z) for z in zs}
    assert len(outs) == len(set(zs))
    flips = []
    for z in zs[:300]:
        for b in (0, 17, 40, 63):
            flips.append(bin(O.mix64(z) ^ O.mix64(z ^ (1 << b))).count("1"))
    assert 30.0 < np.mean(flips) < 34.0


def test_stream_key_definition():
    seed, t, i = 12345, 77, 5
    kt = O.mix64((seed + GAMMA * t) & M64)
    assert O.stream_key(seed, t, i) == O.mix64((kt + GAMMA * (i + 1)) & M64)
    keys = {O.stream_key(seed, tt, ii) for tt in range(1, 65) for ii in range(16)}
    assert len(keys) == 64 * 16


def test_uniform_bit_fields():
    """u1 numerator = top 24 bits + 1 in [1, 2^24]; u2 numerator = bits 8..31."""
    seed, t, i = 3, 9, 2
    key = O.stream_key(seed, t, i)
    for p in (0, 1, 5, 10**6, (1 << 40) + 3):
        z = O.mix64((key + GAMMA * (p + 1)) & M64)
        assert O.uniform_bits(seed, t, i, p) == ((z >> 40) + 1, (z >> 8) & 0xFFFFFF)


def test_neg2ln_recipe_exhaustive_against_libm():
    """All 2^24 inputs: |L - (-2 ln u1)| and relative error are a few fp32 ulp, L >= 0, and
    u1 = 1 gives exactly 0."""
    r = O.scan_neg2ln()
    assert r["max_abs"] < 2.5e-6          # values reach 33.3, ulp there is 3.8e-6
    assert r["max_rel"] < 3e-7
    assert r["min_L"] == 0.0 and r["L_at_one"] == 0.0
    assert O.neg2ln_u24(1) == pytest.approx(48 * math.log(2), rel=1e-7)


def test_cossin_recipe_exhaustive_against_libm():
    r = O.scan_cossin()
    assert r["max_cos"] < 2e-7 and r["max_sin"] < 2e-7 and r["max_norm"] < 3e-7


def test_cossin_octants_exact_points():
    for o, (c, s) in enumerate([(1, 0), (0, 1), (-1, 0), (0, -1)]):
        cc, ss = O.cossin_u24(o * (1 << 22))
        assert (cc, ss) == (c, s)
    h = math.sqrt(0.5)
    for o, (c, s) in enumerate([(h, h), (-h, h), (-h, -h), (h, -h)]):
        cc, ss = O.cossin_u24(o * (1 << 22) + (1 << 21))
        assert cc == pytest.approx(c, abs=2e-7) and ss == pytest.approx(s, abs=2e-7)


def test_box_muller_pair_structure():
    """Even/odd coordinates of a pair share (u1,u2): xi_even^2 + xi_odd^2 = -2 ln u1 and
    atan2(xi_odd, xi_even) = 2 pi u2."""
    seed, t, i = 5, 3, 1
    xi = O.noise_fill(seed, t, i, 0, 4096).astype(np.float64)
    for p in range(0, 2048, 37):
        k, q = O.uniform_bits(seed, t, i, p)
        r2 = xi[2 * p] ** 2 + xi[2 * p + 1] ** 2
        assert r2 == pytest.approx(-2 * math.log(k / 2 ** 24), rel=2e-6, abs=1e-6)
        if r2 > 1e-3:
            ang = math.atan2(xi[2 * p + 1], xi[2 * p]) % (2 * math.pi)
            d = abs(ang - 2 * math.pi * q / 2 ** 24)
            assert min(d, 2 * math.pi - d) < 1e-6


def test_noise_is_keyed_on_seed_worker_step_coordinate():
    base = O.noise_fill(1, 1, 0, 0, 64)
    assert not np.array_equal(base, O.noise_fill(2, 1, 0, 0, 64))
    assert not np.array_equal(base, O.noise_fill(1, 2, 0, 0, 64))
    assert not np.array_equal(base, O.noise_fill(1, 1, 1, 0, 64))
    assert np.array_equal(base[10:20], O.noise_fill(1, 1, 0, 10, 10))      # counter-based
    assert np.array_equal(base[11:20], O.noise_fill(1, 1, 0, 11, 9))       # odd start


def test_noise_distribution_is_standard_normal():
    from scipy import stats
    x = np.concatenate([O.noise_fill(7, t, i, 0, 1 << 20) for t in (1, 2) for i in (0, 1)]).astype(np.float64)
    n = x.size
    assert abs(x.mean()) < 5 / math.sqrt(n)
    assert abs(x.var() - 1) < 5 * math.sqrt(2 / n)
    assert abs((x ** 3).mean()) < 5 * math.sqrt(15 / n)
    assert abs((x ** 4).mean() - 3) < 5 * math.sqrt(96 / n)
    assert stats.kstest(x[: 1 << 20], "norm").pvalue > 1e-3
    assert np.abs(x).max() <= math.sqrt(48 * math.log(2)) + 1e-5
    # workers and steps are uncorrelated; so are the two members of a pair
    a, b = O.noise_fill(7, 1, 0, 0, 1 << 18), O.noise_fill(7, 1, 1, 0, 1 << 18)
    assert abs(np.corrcoef(a, b)[0, 1]) < 0.01
    assert abs(np.corrcoef(a[0::2], a[1::2])[0, 1]) < 0.01


def test_bf16_round_matches_torch_conversion():
    rng = np.random.default_rng(1)
    vals = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * 10.0 ** rng.integers(-6, 6, 20000),
        np.array([0.0, -0.0, 1.0, 1.00390625, 1.005859375, 1.01171875, 3.4e38, 1e-40, -2.5], np.float32),
    ]).astype(np.float32)
    want = torch.from_numpy(vals).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([O.bf16_round(float(v)) for v in vals], np.float32)
    keep = np.isfinite(want)
    assert np.array_equal(got[keep].view(np.uint32), want[keep].view(np.uint32))
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert O.bf16_round(1.00390625) == 1.0 and O.bf16_round(1.01171875) == 1.015625


def test_gradient_modes_against_their_definitions():
    """g = s xi (noise), g = a (x - c) + sigma xi (quadratic, at the worker's own x),
    bf16 mode rounds g to bfloat16; checked after one step from a known state."""
    n, W, seed = 32, 2, 13
    rng = np.random.default_rng(4)
    s = rng.uniform(0.1, 1, n).astype(np.float32)
    a = rng.uniform(0.1, 10, n).astype(np.float32)
    c = rng.standard_normal(n).astype(np.float32)
    x0 = rng.standard_normal(n).astype(np.float32)
    xi = np.stack([O.noise_fill(seed, 1, i, 0, n) for i in range(W)]).astype(np.float64)
    eta, eps, b0sq = 0.5, 2.0, 3.0
    den = math.sqrt(b0sq + eps * eps)
    for mode in ("noise", "quadratic", "quadratic_bf16"):
        o = O.Oracle(n, W, eta, eps, 5, b0sq, x0)
        if mode == "noise":
            o.set_grad_noise(seed, s)
            g = s.astype(np.float64) * xi
        else:
            o.set_grad_quadratic(seed, a, c, 0.25)
            g = a.astype(np.float64) * (x0.astype(np.float64) - c) + 0.25 * xi
            if mode.endswith("bf16"):
                o.set_grad_bf16(True)
                g = torch.from_numpy(g.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
        o.run(1)
        for i in range(W):
            x, b2, _ = o.read(i)
            tol = 1e-2 if mode.endswith("bf16") else 1e-5     # a bf16 rounding flip costs 2^-8 |g|
            np.testing.assert_allclose(x, x0 - eta * g[i] / den, rtol=tol, atol=tol)
            np.testing.assert_allclose(b2, b0sq + g[i] ** 2, rtol=tol)
            if mode.endswith("bf16"):
                gg = np.sqrt(np.maximum(b2.astype(np.float64) - b0sq, 0))
                # accumulated g^2 is the square of a bf16-representable number
                back = torch.from_numpy(gg.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
                np.testing.assert_allclose(gg, back, rtol=1e-5, atol=1e-4)


def test_whole_domain_tables_are_the_scalar_recipes():
    """The table accessors only loop over the pinned scalar functions."""
    L = O.table_neg2ln()
    c, s = O.table_cossin()
    rng = np.random.default_rng(5)
    for k in [1, 2, 3, (1 << 24) - 1, 1 << 24] + [int(v) for v in rng.integers(1, 1 << 24, 200)]:
        assert L[k - 1] == np.float32(O.neg2ln_u24(k))
    for q in [0, 1, (1 << 21) - 1, 1 << 21, (1 << 24) - 1] + [int(v) for v in rng.integers(0, 1 << 24, 200)]:
        cc, ss = O.cossin_u24(q)
        assert c[q] == np.float32(cc) and s[q] == np.float32(ss)
    assert L[-1] == 0.0 and np.all(L[:-1] > 0) and np.all(np.diff(L.astype(np.float64)) <= 0)
