"""Pins for oracle/asd.py against what the paper and the mathematics fix:
Theorem 5 (GRS acceptance probability and output law), Lemma 1 (first slot never
rejected, cursor strictly increasing), Theorem 3 (ASD samples the Euler chain's
law exactly), window 1 == Eq. 7, and a brute-force acceptance probability on d = 2."""
import math

import numpy as np
import pytest
from scipy import stats

import workloads
from oracle import asd, denoisers as den, philox


# ---------------------------------------------------------------- Algorithm 3
def _grs_many(m_hat, m, sigma, n, seed=11):
    d = len(m)
    xs = philox.xi(seed, 0, np.arange(1, n + 1), d)
    us = philox.u(seed, 0, np.arange(1, n + 1))
    out = [asd.grs(u, xi, m_hat, m, sigma) for u, xi in zip(us, xs)]
    x = np.stack([o[0] for o in out])
    b = np.array([o[1] for o in out])
    return x, b, xs


@pytest.mark.parametrize("d,dist,sigma", [(1, 0.7, 1.0), (2, 1.5, 0.6), (5, 0.9, 2.0), (16, 3.0, 1.3)])
def test_grs_acceptance_probability_closed_form(d, dist, sigma):
    """P[b = True] = 1 - TV(N(m^, s^2 I), N(m, s^2 I)) = erfc(|v| / (2 sqrt(2) s))."""
    rng = np.random.default_rng(d)
    m = rng.standard_normal(d)
    dirn = rng.standard_normal(d); dirn /= np.linalg.norm(dirn)
    m_hat = m + dist * dirn
    n = 40_000
    _, b, _ = _grs_many(m_hat, m, sigma, n)
    p = math.erfc(dist / (2 * math.sqrt(2) * sigma))
    assert abs(b.mean() - p) < 4 * math.sqrt(p * (1 - p) / n) + 1e-9


def test_grs_acceptance_quadrature_2d():
    """Integral of min(N(xi), N(xi + v/sigma)) over R^2 on a grid, against the closed
    form and against the accept frequency."""
    v, sigma = np.array([0.8, -0.5]), 0.7
    ax = np.linspace(-9, 9, 1801)
    h = ax[1] - ax[0]
    X0, X1 = np.meshgrid(ax, ax, indexing="ij")
    n0 = np.exp(-(X0 ** 2 + X1 ** 2) / 2) / (2 * math.pi)
    n1 = np.exp(-((X0 + v[0] / sigma) ** 2 + (X1 + v[1] / sigma) ** 2) / 2) / (2 * math.pi)
    quad = np.sum(np.minimum(n0, n1)) * h * h
    closed = math.erfc(np.linalg.norm(v) / (2 * math.sqrt(2) * sigma))
    assert quad == pytest.approx(closed, abs=1e-6)
    m = np.array([0.3, 0.1])
    _, b, _ = _grs_many(m + v, m, sigma, 40_000, seed=5)
    assert abs(b.mean() - quad) < 4 * math.sqrt(quad * (1 - quad) / 40_000)


def test_grs_output_law_and_reflection():
    """x ~ N(m, sigma^2 I) whatever the branch; the rejected branch reflects xi across
    the hyperplane orthogonal to v (an isometry: |x - m| = sigma |xi|)."""
    rng = np.random.default_rng(7)
    d, sigma, n = 4, 0.8, 60_000
    m = rng.standard_normal(d)
    v = np.array([0.9, -0.4, 0.3, 0.2])
    x, b, xs = _grs_many(m + v, m, sigma, n, seed=23)
    assert 0.2 < b.mean() < 0.8                       # both branches exercised
    z = (x - m) / sigma
    assert np.all(np.abs(z.mean(0)) < 4.5 / math.sqrt(n))
    C = np.cov(z.T)
    assert np.max(np.abs(C - np.eye(d))) < 5 * math.sqrt(2 / n)
    e1 = v / np.linalg.norm(v)
    assert stats.kstest(z @ e1, "norm").pvalue > 1e-3
    e2 = np.array([0.4, 0.9, 0.0, 0.0]); e2 -= (e2 @ e1) * e1; e2 /= np.linalg.norm(e2)
    assert stats.kstest(z @ e2, "norm").pvalue > 1e-3
    rej = ~b
    assert np.allclose(np.linalg.norm(z[rej], axis=1), np.linalg.norm(xs[rej], axis=1), rtol=1e-12)
    # component along v flips sign, orthogonal components are untouched
    assert np.allclose(z[rej] @ e1, -(xs[rej] @ e1), atol=1e-12)
    assert np.allclose(z[rej] @ e2, xs[rej] @ e2, atol=1e-12)
    # accepted branch keeps the proposal sample m^ + sigma xi
    assert np.allclose(x[b], (m + v) + sigma * xs[b], atol=1e-12)
    # accepted samples are the ones on the side the proposal and target share
    lr = -(xs @ v) / sigma - (v @ v) / (2 * sigma ** 2)
    assert np.all(b[lr >= 0])


def test_verifier_takes_first_rejection_not_last_accept():
    d = 3
    xis = np.zeros((4, d))
    m = [np.zeros(d)] * 4
    far = np.full(d, 50.0)
    # slot 2 is hopeless (rejected), slots 3, 4 would be accepted on their own
    m_hat = [np.zeros(d), far, np.zeros(d), np.zeros(d)]
    _, n, lr, _ = asd.verifier([0.5] * 4, xis, m_hat, m, [1.0] * 4)
    assert n == 1 and lr[0] == 0.0


# ---------------------------------------------------------------- Algorithm 1
def test_window_one_is_sequential_bit_for_bit():
    for name in ("cfg1_gmm2d", "gauss_small", "mlp_tiny"):
        wl = workloads.make(name)
        g, sch = den.from_workload(wl), asd.make_schedule(wl.t)
        for chain in (0, 3):
            res = asd.asd_sample(g, sch, wl.seed, 100 + chain, chain, 1, d=wl.d)
            y_seq, traj = asd.sequential_ddpm(g, sch, wl.seed, 100 + chain, chain, d=wl.d, return_trajectory=True)
            assert res.rounds == wl.K
            assert np.array_equal(res.y, y_seq)
            assert np.array_equal(res.trajectory, traj)


def test_round_structure_invariants():
    wl = workloads.make("cfg1_gmm2d")
    g, sch = den.from_workload(wl), asd.make_schedule(wl.t)
    for theta in (2, 3, 8, 1000):
        for chain in range(4):
            res = asd.asd_sample(g, sch, wl.seed, chain, chain, theta, d=wl.d)
            K = wl.K
            assert math.ceil(K / theta) <= res.rounds <= math.ceil(K / 2)
            if theta == 2:
                assert res.rounds == math.ceil(K / 2)
            a = 0
            for r in res.records:
                assert r.a_before == a and r.w == min(theta, K - a)
                assert r.ln_ratio[0] == 0.0 and r.n >= 1          # Lemma 1
                assert r.a_after == a + (r.n + 1 if r.n < r.w else r.n)
                a = r.a_after
            assert a == K and res.trajectory.shape == (K + 1, wl.d)
            assert res.model_rows == sum(r.w for r in res.records)


def test_accepted_states_are_the_drafts_and_noise_is_reused():
    """Accepted steps keep y^ = previous + eta v_a + sigma xi_i with the step's own xi_i,
    whichever round reaches it; the rejected step keeps the target mean's distance."""
    wl = workloads.make("gauss_small")
    g, sch = den.from_workload(wl), asd.make_schedule(wl.t)
    res = asd.asd_sample(g, sch, 5, 42, 0, 5, d=wl.d)
    tr = res.trajectory
    for r in res.records:
        v_a = g(r.a_before, tr[r.a_before])
        for k in range(r.n):
            i = r.a_before + k
            xi = philox.xi(5, 42, [i + 1], wl.d)[0]
            assert np.allclose(tr[i + 1], tr[i] + sch.eta[i] * v_a + sch.sigma[i] * xi, atol=1e-12)
        if r.n < r.w:
            i = r.a_before + r.n
            xi = philox.xi(5, 42, [i + 1], wl.d)[0]
            m = tr[i] + sch.eta[i] * g(i, tr[i])
            assert np.linalg.norm(tr[i + 1] - m) == pytest.approx(sch.sigma[i] * np.linalg.norm(xi), rel=1e-10)
            assert r.ln_u[r.n] > r.ln_ratio[r.n]


def test_second_slot_acceptance_brute_force_d2():
    """d = 2, theta = 2, one round from a fixed state: P[both slots accepted] =
    E_{xi_{a+1}} erfc(eta |v_a - g(t_{a+1}, y^_{a+1})| / (2 sqrt 2 sigma_{a+2})), by 2-D
    quadrature over xi_{a+1}, against the frequency over 6000 chains."""
    wl = workloads.make("cfg1_gmm2d")
    g, sch = den.from_workload(wl), asd.make_schedule(wl.t)
    a = 1
    y = np.array([0.2, -0.1])                          # posterior still spread over components
    v_a = g(a, y)
    ax = np.linspace(-7, 7, 281)
    h = ax[1] - ax[0]
    p = 0.0
    for x0 in ax:
        for x1 in ax:
            xi = np.array([x0, x1])
            y1 = y + sch.eta[a] * v_a + sch.sigma[a] * xi
            dist = sch.eta[a + 1] * np.linalg.norm(v_a - g(a + 1, y1))
            p += math.erfc(dist / (2 * math.sqrt(2) * sch.sigma[a + 1])) * math.exp(-(x0 * x0 + x1 * x1) / 2)
    p *= h * h / (2 * math.pi)
    n = 6000
    hits = sum(asd.asd_round(g, sch, 9, c, 0, a, y, 2).n == 2 for c in range(n))
    assert 0.05 < p < 0.95
    assert abs(hits / n - p) < 4 * math.sqrt(p * (1 - p) / n)


# ------------------------------------------------ law of the chain (Theorem 3)
def _euler_gauss_law(t, mu0, Q, lam):
    """Mean and covariance of y_K for the Euler chain on N(mu0, Sigma) from y_0 = 0,
    by the generic recursion mu+ = (I + eta A) mu + eta c, P+ = (I + eta A) P (I + eta A)^T + eta I
    with m(t, y) = A y + c, A = (I + t Sigma)^-1 Sigma, c = (I + t Sigma)^-1 mu0."""
    d = len(mu0)
    Sigma = Q @ np.diag(lam) @ Q.T
    mu, P = np.zeros(d), np.zeros((d, d))
    for i in range(len(t) - 1):
        eta = t[i + 1] - t[i]
        Minv = np.linalg.inv(np.eye(d) + t[i] * Sigma)
        F = np.eye(d) + eta * Minv @ Sigma
        mu = F @ mu + eta * Minv @ mu0
        P = F @ P @ F.T + eta * np.eye(d)
    return mu, P


def test_gauss_chain_closed_form_telescopes():
    """The recursion above has the closed form E y_K = T mu0 and, in Sigma's eigenbasis,
    Var = (1 + T lam)^2 sum_i eta_i / (1 + t_{i+1} lam)^2."""
    wl = workloads.make("gauss_small", K=25)
    Q, lam, mu0 = wl.Q.astype(np.float64), wl.lam.astype(np.float64), wl.mu0.astype(np.float64)
    mu, P = _euler_gauss_law(wl.t, mu0, Q, lam)
    T = wl.t[-1]
    assert np.allclose(mu, T * mu0, rtol=1e-6, atol=1e-6)
    eta = np.diff(wl.t)
    var = (1 + T * lam) ** 2 * np.sum(eta[:, None] / (1 + wl.t[1:, None] * lam[None, :]) ** 2, axis=0)
    assert np.allclose(Q.T @ P @ Q, np.diag(var), rtol=1e-5, atol=1e-5 * var.max())


def test_asd_and_sequential_match_the_analytic_gaussian_law():
    wl = workloads.make("gauss_small", K=24)
    wl.d = 4
    wl.mu0, wl.lam = wl.mu0[:4].copy(), wl.lam[:4].copy() * 3
    wl.Q = np.linalg.qr(wl.Q[:4, :4].astype(np.float64))[0].astype(np.float32)
    g, sch = den.from_workload(wl), asd.make_schedule(wl.t)
    Q, lam, mu0 = wl.Q.astype(np.float64), wl.lam.astype(np.float64), wl.mu0.astype(np.float64)
    mu, P = _euler_gauss_law(np.float32(wl.t).astype(np.float64), mu0, Q, lam)
    n = 2000
    ya = np.stack([asd.asd_sample(g, sch, 1, c, 0, 6, d=4, keep_records=False).y for c in range(n)])
    ys = np.stack([asd.sequential_ddpm(g, sch, 2, c, 0, d=4) for c in range(n)])
    rounds = [asd.asd_sample(g, sch, 1, c, 0, 6, d=4).rounds for c in range(50)]
    assert np.mean(rounds) < 12                        # speculation does happen (K/2 = 12)
    for ysamp in (ya, ys):
        se = np.sqrt(np.diag(P) / n)
        assert np.all(np.abs(ysamp.mean(0) - mu) < 4.5 * se)
        S = np.cov(ysamp.T)
        sd = np.sqrt((np.outer(np.diag(P), np.diag(P)) + P ** 2) / (n - 1))
        assert np.all(np.abs(S - P) < 4.5 * sd)


def test_asd_matches_sequential_in_law_on_the_mixture():
    wl = workloads.make("cfg1_gmm2d", K=40)
    g, sch = den.from_workload(wl), asd.make_schedule(wl.t)
    n = 1000
    ya = np.stack([asd.asd_sample(g, sch, 3, c, 0, 8, d=2, keep_records=False).y for c in range(n)])
    ys = np.stack([asd.sequential_ddpm(g, sch, 4, c, 0, d=2) for c in range(n)])
    T = wl.t[-1]
    for j in range(2):
        assert stats.ks_2samp(ya[:, j], ys[:, j]).pvalue > 1e-3
    # nearest-component occupancy: the two samplers agree (the coarse Euler chain itself is
    # biased away from the equal weights, so the comparison is two-sample)
    c = wl.means.astype(np.float64)
    lab = lambda ysamp: np.bincount(np.argmin(((ysamp[:, None, :] / T - c[None]) ** 2).sum(-1), axis=1),
                                    minlength=len(c))
    table = np.stack([lab(ya), lab(ys)])
    table = table[:, table.sum(0) >= 10]
    assert table.shape[1] >= 2
    assert stats.chi2_contingency(table)[1] > 1e-4


def test_adaptive_window_policy_values_and_law():
    """The per-chain speculation-length rule: hand-computed values, its range, and that Algorithm 1 run
    with it still samples the Euler chain's law (Theorem 3 holds for any theta; the rule looks only at
    the chain's past)."""
    p = asd.AdaptiveWindow(64)
    assert (p.ema8, p.theta()) == (32, 8)               # 2 + 96 // 16
    p.update(8)                                         # whole window of 8 accepted: (32 + 64) >> 1 = 48
    assert (p.ema8, p.theta()) == (48, 11)              # 2 + 144 // 16
    p.update(1)                                         # rejected at once: (48 + 8) >> 1 = 28
    assert (p.ema8, p.theta()) == (28, 7)               # 2 + 84 // 16
    for _ in range(40):
        p.update(1)
    assert (p.ema8, p.theta()) == (8, 3)                # floor: a chain always drafts at least 2 + 1
    for _ in range(40):
        p.update(p.theta())
    assert p.theta() == 64                              # ceiling
    assert asd.AdaptiveWindow(4).theta() == 4 and asd.AdaptiveWindow(2).theta() == 2

    wl = workloads.make("gauss_small", K=24)
    wl.d = 4
    wl.mu0, wl.lam = wl.mu0[:4].copy(), wl.lam[:4].copy() * 3
    wl.Q = np.linalg.qr(wl.Q[:4, :4].astype(np.float64))[0].astype(np.float32)
    g, sch = den.from_workload(wl), asd.make_schedule(wl.t)
    Q, lam, mu0 = wl.Q.astype(np.float64), wl.lam.astype(np.float64), wl.mu0.astype(np.float64)
    mu, P = _euler_gauss_law(np.float32(wl.t).astype(np.float64), mu0, Q, lam)
    n = 2000
    res = [asd.asd_sample(g, sch, 5, c, 0, 16, d=4, adaptive=True) for c in range(n)]
    ya = np.stack([r.y for r in res])
    windows = np.concatenate([[rec.w for rec in r.records] for r in res[:200]])
    assert windows.min() >= 1 and windows.max() <= 16 and len(set(windows)) > 3     # it does adapt
    se = np.sqrt(np.diag(P) / n)
    assert np.all(np.abs(ya.mean(0) - mu) < 4.5 * se)
    S = np.cov(ya.T)
    sd = np.sqrt((np.outer(np.diag(P), np.diag(P)) + P ** 2) / (n - 1))
    assert np.all(np.abs(S - P) < 4.5 * sd)
