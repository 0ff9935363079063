"""TEST INFRASTRUCTURE — CPU oracle, not part of the product path.

The drift g(t_i, y) of the Euler chain (Eq. 7).  In the stochastic-localization
form it is the posterior mean m(t, y) = E[x* | t x* + sqrt(t) xi = y] (Eq. 4).
Three families, each a callable `g(i, y, chain)` with `i` the step index
(time t_i), `y` a float64 vector in R^d and `chain` the position of the chain
in the batch (only the conditioned network looks at it):

GmmPosteriorMean      x* ~ sum_j pi_j N(c_j, s^2 I).  Conditioning on the component:
                      y | j ~ N(t c_j, (t^2 s^2 + t) I), so up to a j-independent
                      constant  l_j = ln pi_j + (<y, c_j> - t |c_j|^2 / 2) / (1 + t s^2);
                      within a component, E[x* | y, j] = (c_j + s^2 y) / (1 + t s^2).
GaussPosteriorMean    x* ~ N(mu0, Sigma), Sigma = Q diag(lam) Q^T:
                      m = (I + t Sigma)^-1 (mu0 + Sigma y), evaluated in Sigma's eigenbasis.
ResMlpDenoiser        the synthetic network of the bf16 workloads.  The paper does not
                      specify a network; the definition (also the library's contract) is
                        x   = [bf16(c_in[i] y) ; bf16(cond) ; bf16(temb(i))]
                        h_0 = bf16(W_in x + b_in)
                        h_l = bf16(h_{l-1} + SiLU(W_l h_{l-1} + b_l)),  l = 1..L
                        g   = c_skip[i] y + c_out[i] (W_out h_L + b_out)
                      with bf16() = round-to-nearest-even to bfloat16, products and
                      sums otherwise exact / float64 here, SiLU(z) = z / (1 + exp(-z)),
                      temb(i): tau = 1000 i / K, half = d_temb / 2,
                      w_f = exp(-ln(10^4) f / half), [sin(tau w_f)]_f ++ [cos(tau w_f)]_f.

Pins (tests/test_oracle_denoisers.py): both closed forms against numerical
integration of the defining conditional expectation (d = 1 and 2), the GMM form
at t = 0 (prior mean) and for one component (Gaussian form), the network against
a plain triple loop, its batched form (several rows, a different step per row)
against the single-point form, and bf16 rounding against torch's cast.
"""
from __future__ import annotations

import numpy as np


def round_bf16(x):
    """Round-to-nearest-even to bfloat16, returned as float64 values."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    b = f.view(np.uint32).astype(np.uint64)
    lsb = (b >> np.uint64(16)) & np.uint64(1)
    b = (b + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return b.astype(np.uint32).view(np.float32).astype(np.float64)


def bf16_bits_to_f64(bits):
    return (np.asarray(bits).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


class GmmPosteriorMean:
    def __init__(self, t, means, weights, sigma):
        self.t = np.asarray(t, dtype=np.float64).astype(np.float32).astype(np.float64)
        self.c = np.asarray(means, dtype=np.float64)            # [n_comp, d]
        self.log_pi = np.log(np.asarray(weights, dtype=np.float64))
        self.s2 = float(np.float32(sigma)) ** 2

    def __call__(self, i, y, chain=0):
        t = self.t[i]
        den = 1.0 + t * self.s2
        logit = self.log_pi + (self.c @ y - 0.5 * t * np.sum(self.c * self.c, axis=1)) / den
        logit = logit - np.max(logit)
        r = np.exp(logit)
        r = r / np.sum(r)
        return (r @ self.c + self.s2 * y) / den


class GaussPosteriorMean:
    def __init__(self, t, mu0, Q, lam):
        self.t = np.asarray(t, dtype=np.float64).astype(np.float32).astype(np.float64)
        self.mu0 = np.asarray(mu0, dtype=np.float64)
        self.Q = np.asarray(Q, dtype=np.float64)
        self.lam = np.asarray(lam, dtype=np.float64)

    def __call__(self, i, y, chain=0):
        t = self.t[i]
        z = self.Q.T @ (self.mu0) + self.lam * (self.Q.T @ y)     # Q^T (mu0 + Sigma y)
        return self.Q @ (z / (1.0 + t * self.lam))


def time_embedding(i, K, d_temb):
    half = d_temb // 2
    tau = 1000.0 * i / K
    f = np.arange(half, dtype=np.float64)
    w = np.exp(-np.log(1.0e4) * f / half)
    return np.concatenate([np.sin(tau * w), np.cos(tau * w)])


def silu(z):
    return z / (1.0 + np.exp(-z))


class ResMlpDenoiser:
    def __init__(self, K, d, d_cond, d_temb, W_in, W_hid, W_out, b_in, b_hid, b_out,
                 c_in, c_skip, c_out, cond):
        self.K, self.d, self.d_cond, self.d_temb = K, d, d_cond, d_temb
        self.W_in = bf16_bits_to_f64(W_in)
        self.W_hid = bf16_bits_to_f64(W_hid)
        self.W_out = bf16_bits_to_f64(W_out)
        self.b_in = np.asarray(b_in, dtype=np.float64)
        self.b_hid = np.asarray(b_hid, dtype=np.float64)
        self.b_out = np.asarray(b_out, dtype=np.float64)
        one = np.ones(K)
        self.c_in = one if c_in is None else np.asarray(c_in, dtype=np.float64)
        self.c_skip = 0 * one if c_skip is None else np.asarray(c_skip, dtype=np.float64)
        self.c_out = one if c_out is None else np.asarray(c_out, dtype=np.float64)
        self.cond = None if cond is None else np.asarray(cond, dtype=np.float64)

    def features(self, i, y, chain):
        parts = [round_bf16(self.c_in[i] * y)]
        if self.d_cond:
            parts.append(round_bf16(self.cond[chain]))
        parts.append(round_bf16(time_embedding(i, self.K, self.d_temb)))
        return np.concatenate(parts)

    def __call__(self, i, y, chain=0):
        x = self.features(i, y, chain)
        h = round_bf16(self.W_in @ x + self.b_in)
        for l in range(self.W_hid.shape[0]):
            h = round_bf16(h + silu(self.W_hid[l] @ h + self.b_hid[l]))
        return self.c_skip[i] * y + self.c_out[i] * (self.W_out @ h + self.b_out)

    def batch(self, steps, Y, chain):
        """The same map applied to several points (rows of Y) of one chain with
        one matrix product per layer; identical arithmetic per row."""
        X = np.stack([self.features(i, y, chain) for i, y in zip(steps, Y)])
        H = round_bf16(X @ self.W_in.T + self.b_in)
        for l in range(self.W_hid.shape[0]):
            H = round_bf16(H + silu(H @ self.W_hid[l].T + self.b_hid[l]))
        steps = np.asarray(steps)
        return self.c_skip[steps, None] * Y + self.c_out[steps, None] * (H @ self.W_out.T + self.b_out)


def from_workload(wl):
    """Build the drift for a workload record (any object with the fields the
    seeded input generator fills in)."""
    if wl.kind == "gmm":
        return GmmPosteriorMean(wl.t, wl.means, wl.weights, wl.sigma)
    if wl.kind == "gauss":
        return GaussPosteriorMean(wl.t, wl.mu0, wl.Q, wl.lam)
    if wl.kind == "mlp":
        return ResMlpDenoiser(wl.K, wl.d, wl.d_cond, wl.d_temb, wl.W_in, wl.W_hid, wl.W_out,
                              wl.b_in, wl.b_hid, wl.b_out, wl.c_in, wl.c_skip, wl.c_out, wl.cond)
    raise ValueError(wl.kind)
