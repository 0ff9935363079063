"""Pins for oracle/denoisers.py.  The closed-form posterior means are checked
against the defining conditional expectation m(t, y) = E[x* | t x* + sqrt(t) xi = y]
(Eq. 4) evaluated by brute-force quadrature, so a wrong sign, a dropped factor of t
or a transposed eigenvector matrix fails."""
import math

import numpy as np
import pytest
import torch

import workloads
from oracle import denoisers as den


def _posterior_mean_quadrature_1d(prior_pdf, t, y, lo=-12.0, hi=12.0, n=200_001):
    x = np.linspace(lo, hi, n)
    logw = np.log(prior_pdf(x) + 1e-300)
    if t > 0:
        logw = logw - (y - t * x) ** 2 / (2 * t)
    w = np.exp(logw - logw.max())
    return float(np.sum(x * w) / np.sum(w))


@pytest.mark.parametrize("t,y", [(0.0, 0.0), (0.5, -1.2), (3.0, 7.0), (40.0, -95.0)])
def test_gmm_closed_form_vs_quadrature_1d(t, y):
    c = np.array([[-2.0], [0.5], [3.0]])
    pi = np.array([0.2, 0.5, 0.3])
    s = 0.4
    prior = lambda x: sum(p * np.exp(-(x - m) ** 2 / (2 * s * s)) / (s * math.sqrt(2 * math.pi))
                          for p, m in zip(pi, c[:, 0]))
    g = den.GmmPosteriorMean(np.array([t]), c, pi, s)
    ref = _posterior_mean_quadrature_1d(prior, float(np.float32(t)), y)
    assert g(0, np.array([y]))[0] == pytest.approx(ref, abs=2e-6)


def test_gmm_closed_form_vs_quadrature_2d():
    wl = workloads.make("cfg1_gmm2d")
    g = den.from_workload(wl)
    c = wl.means.astype(np.float64)
    s = float(np.float32(wl.sigma))
    ax = np.linspace(-6.5, 6.5, 1301)
    X0, X1 = np.meshgrid(ax, ax, indexing="ij")
    prior = np.zeros_like(X0)
    for j in range(len(c)):
        prior += np.exp(-((X0 - c[j, 0]) ** 2 + (X1 - c[j, 1]) ** 2) / (2 * s * s))
    rng = np.random.default_rng(0)
    for i in (1, 3, 17, 60):
        t = float(np.float32(wl.t[i]))
        xstar = c[rng.integers(len(c))] + s * rng.standard_normal(2)
        y = t * xstar + math.sqrt(t) * rng.standard_normal(2)
        logw = np.log(prior + 1e-300) - ((y[0] - t * X0) ** 2 + (y[1] - t * X1) ** 2) / (2 * t)
        w = np.exp(logw - logw.max())
        ref = np.array([np.sum(X0 * w), np.sum(X1 * w)]) / np.sum(w)
        assert np.allclose(g(i, y), ref, atol=5e-5), (i, g(i, y), ref)


def test_gmm_special_cases():
    c = np.array([[1.0, -2.0, 0.5], [0.0, 3.0, 1.0]])
    pi = np.array([0.25, 0.75])
    g = den.GmmPosteriorMean(np.array([0.0, 2.0]), c, pi, 0.7)
    # t = 0 (where the chain starts, y_0 = 0): posterior mean = prior mean
    assert np.allclose(g(0, np.zeros(3)), pi @ c)
    # one component N(c, s^2 I) is the Gaussian case with Sigma = s^2 I
    g1 = den.GmmPosteriorMean(np.array([0.0, 2.0]), c[:1], np.array([1.0]), 0.7)
    s2 = float(np.float32(0.7)) ** 2
    gg = den.GaussPosteriorMean(np.array([0.0, 2.0]), c[0], np.eye(3), np.full(3, s2))
    y = np.array([0.3, -4.0, 2.0])
    assert np.allclose(g1(1, y), gg(1, y), atol=1e-7)


def test_gauss_closed_form_vs_solve_and_quadrature():
    wl = workloads.make("gauss_small")
    g = den.from_workload(wl)
    Q, lam, mu0 = wl.Q.astype(np.float64), wl.lam.astype(np.float64), wl.mu0.astype(np.float64)
    Sigma = Q @ np.diag(lam) @ Q.T
    rng = np.random.default_rng(1)
    for i in (0, 1, 7, 50):
        t = float(np.float32(wl.t[i]))
        y = rng.standard_normal(wl.d) * (1 + t)
        # Bayes: precision Sigma^-1 + t I, mean (Sigma^-1 + t I)^-1 (Sigma^-1 mu0 + y)
        P = np.linalg.inv(Sigma)
        ref = np.linalg.solve(P + t * np.eye(wl.d), P @ mu0 + y)
        assert np.allclose(g(i, y), ref, rtol=0, atol=1e-5 * (1 + np.abs(ref).max()))
    # d = 1 against quadrature of the definition
    g1 = den.GaussPosteriorMean(np.array([1.5]), np.array([0.7]), np.array([[1.0]]), np.array([2.0]))
    prior = lambda x: np.exp(-(x - 0.7) ** 2 / (2 * 2.0))
    ref = _posterior_mean_quadrature_1d(prior, 1.5, 4.0, lo=-30, hi=30)
    assert g1(0, np.array([4.0]))[0] == pytest.approx(ref, abs=1e-6)


def test_round_bf16_matches_torch_cast():
    rng = np.random.default_rng(2)
    x = np.concatenate([rng.standard_normal(20000) * 10 ** rng.uniform(-6, 6, 20000),
                        # exact ties between two bf16 neighbours (round to even)
                        np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(2.0 + 2.0 ** -7), 0.0, -0.0])])
    ours = den.round_bf16(x)
    ref = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(ours, ref)
    assert den.round_bf16(1.0 + 2.0 ** -8) == 1.0                 # tie -> even mantissa
    assert den.round_bf16(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6


def test_time_embedding_values():
    e = den.time_embedding(0, 100, 8)
    assert np.array_equal(e, np.array([0, 0, 0, 0, 1, 1, 1, 1], dtype=float))
    e = den.time_embedding(25, 100, 4)        # tau = 250, w = [1, 1e-2]
    assert np.allclose(e, [math.sin(250.0), math.sin(2.5), math.cos(250.0), math.cos(2.5)], atol=1e-12)


def test_resmlp_matches_plain_loops():
    wl = workloads.make("mlp_tiny")
    g = den.from_workload(wl)
    rng = np.random.default_rng(3)
    f = lambda bits: workloads.bf16_bits_to_f32(bits).astype(np.float64)
    W_in, W_hid, W_out = f(wl.W_in), f(wl.W_hid), f(wl.W_out)
    bf = lambda v: float(torch.tensor(v, dtype=torch.float32).to(torch.bfloat16))
    for i, chain in ((0, 0), (7, 3), (39, 4)):
        y = rng.standard_normal(wl.d) * (1 + wl.t[i])
        x = [bf(float(wl.c_in[i]) * yy) for yy in y] + [bf(float(c)) for c in wl.cond[chain]]
        tau = 1000.0 * i / wl.K
        half = wl.d_temb // 2
        x += [bf(math.sin(tau * math.exp(-math.log(1e4) * k / half))) for k in range(half)]
        x += [bf(math.cos(tau * math.exp(-math.log(1e4) * k / half))) for k in range(half)]
        h = []
        for o in range(wl.width):
            acc = float(wl.b_in[o])
            for k in range(wl.in_dim):
                acc += W_in[o, k] * x[k]
            h.append(bf(acc))
        for l in range(wl.n_layers):
            hn = []
            for o in range(wl.width):
                acc = float(wl.b_hid[l, o])
                for k in range(wl.width):
                    acc += W_hid[l, o, k] * h[k]
                hn.append(bf(h[o] + acc / (1.0 + math.exp(-acc))))
            h = hn
        out = []
        for o in range(wl.d):
            acc = float(wl.b_out[o])
            for k in range(wl.width):
                acc += W_out[o, k] * h[k]
            out.append(float(wl.c_skip[i]) * y[o] + float(wl.c_out[i]) * acc)
        got = g(i, y, chain)
        # identical rounding points; a bf16 flip from summation order would show as ~4e-3 relative
        assert np.allclose(got, out, rtol=1e-9, atol=1e-9), np.abs(got - np.array(out)).max()
        assert np.allclose(g.batch([i], y[None], chain)[0], got, rtol=1e-9, atol=1e-9)


@pytest.mark.parametrize("name", ["mlp_tiny", "mlp_ragged"])
def test_resmlp_batch_rows_match_single_calls_mixed_steps(name):
    """`batch` (one matrix product per layer over several points) against `__call__` row by row, with a
    different step in every row: a row must get its own step's c_in, time embedding, c_skip and c_out, and
    the conditioning of the chain it is called for."""
    wl = workloads.make(name)
    g = den.from_workload(wl)
    rng = np.random.default_rng(8)
    for chain in (0, wl.chains - 1):
        steps = [0, wl.K - 1, 3, 3, wl.K // 2, 1, wl.K - 2]
        Y = np.stack([rng.standard_normal(wl.d) * (1 + wl.t[i]) for i in steps])
        got = g.batch(steps, Y, chain)
        assert got.shape == (len(steps), wl.d)
        for r, i in enumerate(steps):
            one = g(i, Y[r], chain)
            # same rounding points row by row; only the summation order inside the products may differ
            assert np.allclose(got[r], one, rtol=1e-9, atol=1e-9), (r, np.abs(got[r] - one).max())
        # the rows really are different functions of the step and the chain
        assert not np.allclose(g.batch([5] * len(steps), Y, chain), got)
        if wl.d_cond:
            assert not np.allclose(g.batch(steps, Y, (chain + 1) % wl.chains), got)


def test_stored_trained_network_approximates_the_mixture_posterior_mean():
    """tests/golden/cfg1_trained_mlp.npz (written by tests/golden/make_cfg1_trained_mlp.py) is a network fitted
    to Eq. 4's posterior mean of the cfg-1 mixture: on fresh points of the localization process its drift is
    close to the closed form, far closer than the skip term alone."""
    wl = workloads.make("cfg1_trained")
    base = workloads.make("cfg1_gmm2d")
    net, exact = den.from_workload(wl), den.from_workload(base)
    rng = np.random.default_rng(123)
    err, err_skip, ref = [], [], []
    for _ in range(400):
        i = int(rng.integers(0, wl.K))
        xs = base.means[rng.integers(0, 8)] + base.sigma * rng.standard_normal(2)
        y = base.t[i] * xs + math.sqrt(base.t[i]) * rng.standard_normal(2)
        m = exact(i, y)
        err.append(np.sum((net(i, y) - m) ** 2))
        err_skip.append(np.sum((float(wl.c_skip[i]) * y - m) ** 2))
        ref.append(np.sum(m ** 2))
    rel = math.sqrt(np.sum(err) / np.sum(ref))
    rel_skip = math.sqrt(np.sum(err_skip) / np.sum(ref))
    print(f"trained network: rms error / rms posterior mean = {rel:.3f} (skip term alone {rel_skip:.3f})")
    assert rel < 0.1 and rel < 0.2 * rel_skip
