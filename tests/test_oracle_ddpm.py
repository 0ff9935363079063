"""Pins of the DDPM front end (oracle/ddpm.py) and, without a GPU, the library's host-side
asd_ddpm_schedule against it."""
import numpy as np
import pytest

from oracle import asd as oasd
from oracle import ddpm as oddpm
from oracle import denoisers as oden
from oracle import philox


def _levels(K, lo=1e-3, hi=0.995):
    """alpha-bar of K+1 visited levels, noisy -> clean (a cosine-like ramp)."""
    u = np.linspace(0.0, 1.0, K + 1)
    return lo + (hi - lo) * np.sin(0.5 * np.pi * u) ** 2


@pytest.mark.parametrize("pred", ["x0", "eps", "v"])
def test_sl_mapping_gives_the_posterior_mean(pred):
    """Gaussian data x0 ~ N(mu0, Sigma): feed the exact network output of each prediction type through
    the c_in / c_skip / c_out wrapping and compare with the closed-form SL posterior mean m(t, y)
    (pinned separately by quadrature) at y = sqrt(t (1 + t)) x."""
    rng = np.random.default_rng(0)
    d, K = 3, 12
    ab = _levels(K)
    sch = oddpm.ddpm_schedule(ab, pred, "sl")
    A = rng.standard_normal((d, d))
    Sigma = A @ A.T / d + 0.2 * np.eye(d)
    lam, Q = np.linalg.eigh(Sigma)
    mu0 = rng.standard_normal(d)
    assert np.allclose(sch["t"], ab / (1 - ab)) and np.allclose(sch["sigma2"], np.diff(sch["t"]))
    m = oden.GaussPosteriorMean(sch["t"], mu0, Q, lam)
    m.t = sch["t"]                                     # keep float64 times for this comparison
    for i in range(K):
        x = rng.standard_normal(d) * 1.3
        # E[x0 | x] for x = sqrt(ab) x0 + sqrt(1 - ab) eps, by Gaussian conditioning written out in x
        C = ab[i] * Sigma + (1 - ab[i]) * np.eye(d)
        x0_hat = mu0 + np.sqrt(ab[i]) * Sigma @ np.linalg.solve(C, x - np.sqrt(ab[i]) * mu0)
        eps_hat = (x - np.sqrt(ab[i]) * x0_hat) / np.sqrt(1 - ab[i])
        net = {"x0": x0_hat, "eps": eps_hat, "v": np.sqrt(ab[i]) * eps_hat - np.sqrt(1 - ab[i]) * x0_hat}[pred]
        y = x / sch["x_scale"][i]
        assert np.allclose(sch["c_in"][i] * y, x, rtol=1e-6)
        g = sch["c_skip"][i] * y + sch["c_out"][i] * net
        assert np.allclose(g, m(i, y), rtol=2e-5, atol=2e-5)


@pytest.mark.parametrize("pred,large", [("eps", False), ("x0", True), ("v", False)])
def test_ancestral_mapping_reproduces_the_x_space_sampler(pred, large):
    """The ancestral sampler written directly in x (posterior mean coefficients of x_s and x0_hat, noise
    s) and the chain of Eq. 7 built from the mapped tables give the same path on the same noise."""
    rng = np.random.default_rng(1)
    d, K = 5, 30
    ab = _levels(K)
    sch = oddpm.ddpm_schedule(ab, pred, "ancestral", large)
    W = rng.standard_normal((d, d)) * 0.3

    def net(i, x):                                     # any fixed function of (level, x)
        return np.tanh(W @ x + 0.1 * i)

    def x0_hat(i, x):
        kx, kn = oddpm.prediction_coefficients(ab[i], pred)
        return kx * x + kn * net(i, x)

    x = rng.standard_normal(d)
    xs = philox.xi(7, 3, np.arange(1, K + 1), d)
    # (a) x space, step by step
    xa = x.copy()
    for i in range(K):
        alpha = ab[i] / ab[i + 1]
        beta = 1 - alpha
        mean = (np.sqrt(ab[i + 1]) * beta * x0_hat(i, xa) + np.sqrt(alpha) * (1 - ab[i + 1]) * xa) / (1 - ab[i])
        var = beta if large else beta * (1 - ab[i + 1]) / (1 - ab[i])
        xa = mean + np.sqrt(var) * xs[i]
    # (b) Eq. 7 in y with the mapped schedule; the drift wraps the same network with the float64 scalars
    sched = oasd.Schedule(K=K, eta=np.diff(sch["t"]), sigma=np.sqrt(sch["sigma2"]))
    kx = np.array([oddpm.prediction_coefficients(ab[i], pred)[0] for i in range(K)])
    kn = np.array([oddpm.prediction_coefficients(ab[i], pred)[1] for i in range(K)])

    def g(i, y, chain=0):
        xi_ = sch["x_scale"][i] * y
        return kx[i] * xi_ + kn[i] * net(i, xi_)

    yK = oasd.sequential_ddpm(g, sched, 7, 3, 0, y0=x / sch["x_scale"][0])
    assert np.allclose(sch["x_scale"][K] * yK, xa, rtol=1e-9, atol=1e-9)
    # the float32 tables are those scalars
    assert np.allclose(sch["c_skip"], kx * sch["x_scale"][:K], rtol=1e-6) and np.allclose(sch["c_out"], kn, rtol=1e-6)


@pytest.mark.parametrize("mapping", ["sl", "ancestral"])
@pytest.mark.parametrize("pred", ["x0", "eps", "v"])
def test_library_schedule_matches_the_oracle(pred, mapping):
    from paper_2505_03983_b200 import AsdError, ddpm_schedule
    ab = _levels(50)
    for large in (False, True):
        ours = ddpm_schedule(ab, pred, mapping, large)
        ref = oddpm.ddpm_schedule(ab, pred, mapping, large)
        for k in ("t", "sigma2", "x_scale"):
            assert np.allclose(ours[k], ref[k], rtol=1e-12, atol=0), k
        for k in ("c_in", "c_skip", "c_out"):
            assert np.allclose(ours[k], ref[k], rtol=2e-7, atol=0), k
    with pytest.raises(AsdError):
        ddpm_schedule(ab[::-1].copy(), pred, mapping)
    with pytest.raises(AsdError):
        ddpm_schedule(np.array([0.1, 1.0]), pred, mapping)
