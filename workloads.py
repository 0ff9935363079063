"""Seeded synthetic inputs for the ASD hot path (shared by the CUDA library's
callers and by the CPU oracle's callers).

This module only *draws inputs*: target-distribution parameters, denoiser
weights, conditioning vectors, time grids and the per-step scaling tables the
caller hands to either implementation.  It contains none of the sampler's
arithmetic (no Philox, no posterior means, no accept test); both
implementations receive exactly the arrays produced here.

Workloads (synthetic stand-ins, no dataset or trained weight is used):

  cfg1_gmm2d     d=2, 8-component isotropic Gaussian mixture, K=100, window 8, 16 chains
  cfg2_gauss64   d=64 Gaussian target N(mu, Sigma), K=1000, window 16, 256 chains
  cfg3_policy    action chunk 16x7=112 dims + 64-dim observation, 4-layer residual MLP width 1024
  cfg4_image     d=3x32x32=3072, 6-layer residual MLP width 4096, K=1000, window 32, 32 chains
  sweep_b{B}_w{W}  cfg4 denoiser, B chains x window W, K=1000
  mlp_tiny / mlp_ragged   small residual-MLP cases for parity tests (several tiles + ragged tails)
  cfg1_trained   the cfg-1 problem with a small residual MLP fitted to its posterior mean (stored weights)

All time grids are the uniform stochastic-localization grid t_i = i*T/K with
T = 100 ("linear schedule"), the equal-increment case of the exchangeability
theorem (Theorem 2 of the paper).
"""
from __future__ import annotations

import dataclasses
import re
from typing import Optional

import numpy as np
import torch

T_FINAL = 100.0


@dataclasses.dataclass
class Workload:
    name: str
    kind: str                      # "gmm" | "gauss" | "mlp"
    d: int
    K: int
    window: int
    chains: int
    seed: int
    t: np.ndarray                  # float64 [K+1], strictly increasing
    # gmm
    means: Optional[np.ndarray] = None      # float32 [n_comp, d]
    weights: Optional[np.ndarray] = None    # float32 [n_comp], sums to 1
    sigma: float = 0.0
    # gauss: Sigma = Q diag(lam) Q^T, columns of Q are eigenvectors
    mu0: Optional[np.ndarray] = None        # float32 [d]
    Q: Optional[np.ndarray] = None          # float32 [d, d] row-major
    lam: Optional[np.ndarray] = None        # float32 [d]
    # mlp
    d_cond: int = 0
    d_temb: int = 0
    width: int = 0
    n_layers: int = 0
    W_in: Optional[np.ndarray] = None       # uint16 (bf16 bits) [width, d+d_cond+d_temb]
    W_hid: Optional[np.ndarray] = None      # uint16 [n_layers, width, width]
    W_out: Optional[np.ndarray] = None      # uint16 [d, width]
    b_in: Optional[np.ndarray] = None       # float32 [width]
    b_hid: Optional[np.ndarray] = None      # float32 [n_layers, width]
    b_out: Optional[np.ndarray] = None      # float32 [d]
    c_in: Optional[np.ndarray] = None       # float32 [K]
    c_skip: Optional[np.ndarray] = None     # float32 [K]
    c_out: Optional[np.ndarray] = None      # float32 [K]
    cond: Optional[np.ndarray] = None       # float32 [chains, d_cond]

    @property
    def in_dim(self) -> int:
        return self.d + self.d_cond + self.d_temb


def uniform_grid(K: int, T: float = T_FINAL) -> np.ndarray:
    return np.arange(K + 1, dtype=np.float64) * (T / K)


def _bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bf16 (torch's round-to-nearest-even cast) and
    return the 16-bit patterns."""
    tt = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return tt.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32 (a bit shift)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def _gmm(name, d, n_comp, sigma, K, window, chains, seed, box=4.0) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    means = rng.uniform(-box, box, size=(n_comp, d)).astype(np.float32)
    weights = np.full(n_comp, 1.0 / n_comp, dtype=np.float32)
    return Workload(name=name, kind="gmm", d=d, K=K, window=window, chains=chains, seed=seed,
                    t=uniform_grid(K), means=means, weights=weights, sigma=float(np.float32(sigma)))


def _gauss(name, d, K, window, chains, seed) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    mu0 = rng.standard_normal(d)
    A = rng.standard_normal((d, d))
    Sigma = A @ A.T / d + 0.1 * np.eye(d)
    lam, Q = np.linalg.eigh(Sigma)
    # The target handed to both implementations is *defined* by the float32
    # (mu0, Q, lam) below: Sigma := Q diag(lam) Q^T.
    return Workload(name=name, kind="gauss", d=d, K=K, window=window, chains=chains, seed=seed,
                    t=uniform_grid(K), mu0=mu0.astype(np.float32),
                    Q=np.ascontiguousarray(Q, dtype=np.float32), lam=lam.astype(np.float32))


def _mlp(name, d, d_cond, d_temb, width, n_layers, K, window, chains, seed,
         bias_std: float = 0.0) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    in_dim = d + d_cond + d_temb
    std = 0.02

    def w(shape):
        return _bf16_bits((std * rng.standard_normal(shape, dtype=np.float32)))

    W_in = w((width, in_dim))
    W_hid = w((n_layers, width, width))
    W_out = w((d, width))
    if bias_std > 0:
        b_in = (bias_std * rng.standard_normal(width)).astype(np.float32)
        b_hid = (bias_std * rng.standard_normal((n_layers, width))).astype(np.float32)
        b_out = (bias_std * rng.standard_normal(d)).astype(np.float32)
    else:
        b_in = np.zeros(width, np.float32)
        b_hid = np.zeros((n_layers, width), np.float32)
        b_out = np.zeros(d, np.float32)
    t = uniform_grid(K)
    ti = t[:K]
    # Per-step scaling tables supplied by the caller: unit-variance network input,
    # skip = exact posterior mean of N(0, I) data, small learned correction.
    c_in = np.where(ti > 0, 1.0 / np.sqrt(np.maximum(ti * (1.0 + ti), 1e-300)), 0.0).astype(np.float32)
    c_skip = (1.0 / (1.0 + ti)).astype(np.float32)
    c_out = (0.1 / (1.0 + ti)).astype(np.float32)
    cond = rng.standard_normal((chains, d_cond)).astype(np.float32) if d_cond else np.zeros((chains, 0), np.float32)
    return Workload(name=name, kind="mlp", d=d, K=K, window=window, chains=chains, seed=seed, t=t,
                    d_cond=d_cond, d_temb=d_temb, width=width, n_layers=n_layers,
                    W_in=W_in, W_hid=W_hid, W_out=W_out, b_in=b_in, b_hid=b_hid, b_out=b_out,
                    c_in=c_in, c_skip=c_skip, c_out=c_out, cond=cond)


def make(name: str, *, chains: Optional[int] = None, K: Optional[int] = None,
         window: Optional[int] = None, seed: Optional[int] = None, n_layers: Optional[int] = None) -> Workload:
    """Build a named workload; keyword arguments override chains / K / window / seed and, for the
    network workloads, the number of residual layers (the other shapes stay)."""
    def ov(val, default):
        return default if val is None else val

    s = ov(seed, 0)
    if name == "cfg1_gmm2d":
        return _gmm(name, 2, 8, 0.3, ov(K, 100), ov(window, 8), ov(chains, 16), s)
    if name == "cfg2_gauss64":
        return _gauss(name, 64, ov(K, 1000), ov(window, 16), ov(chains, 256), s)
    if name == "cfg3_policy":
        return _mlp(name, 112, 64, 128, 1024, ov(n_layers, 4), ov(K, 100), ov(window, 16), ov(chains, 64), s)
    if name == "cfg4_image":
        return _mlp(name, 3072, 0, 256, 4096, ov(n_layers, 6), ov(K, 1000), ov(window, 32), ov(chains, 32), s)
    m = re.fullmatch(r"sweep_b(\d+)_w(\d+)", name)
    if m:
        return _mlp(name, 3072, 0, 256, 4096, ov(n_layers, 6), ov(K, 1000), ov(window, int(m.group(2))),
                    ov(chains, int(m.group(1))), s)
    if name == "cfg1_trained":
        # the cfg-1 problem with a small network FITTED to the mixture's closed-form posterior mean in place of the
        # closed form (weights and per-step tables as stored by tests/golden/make_cfg1_trained_mlp.py)
        import os
        z = np.load(os.path.join(os.path.dirname(os.path.abspath(__file__)), "tests", "golden", "cfg1_trained_mlp.npz"))
        Kc = ov(K, 100)
        assert Kc == len(z["c_in"]), "the stored per-step tables are for K = 100"
        return Workload(name=name, kind="mlp", d=2, K=Kc, window=ov(window, 8), chains=ov(chains, 16), seed=s,
                        t=uniform_grid(Kc), d_cond=0, d_temb=int(z["d_temb"]), width=z["W_in"].shape[0],
                        n_layers=z["W_hid"].shape[0], W_in=z["W_in"], W_hid=z["W_hid"], W_out=z["W_out"],
                        b_in=z["b_in"], b_hid=z["b_hid"], b_out=z["b_out"], c_in=z["c_in"], c_skip=z["c_skip"],
                        c_out=z["c_out"], cond=np.zeros((ov(chains, 16), 0), np.float32))
    if name == "mlp_tiny":
        return _mlp(name, 24, 8, 32, 128, 2, ov(K, 40), ov(window, 6), ov(chains, 5), s, bias_std=0.05)
    if name == "mlp_ragged":
        # odd sizes: d not a multiple of 8/16, in_dim padded, width spanning several N tiles
        return _mlp(name, 52, 12, 64, 320, 3, ov(K, 60), ov(window, 12), ov(chains, 37), s, bias_std=0.05)
    if name == "mlp_odd":
        # nothing a multiple of 4: scalar tails in draft / verify / epilogues, width of 72 = 9 x 8
        return _mlp(name, 45, 3, 10, 72, 1, ov(K, 30), ov(window, 9), ov(chains, 7), s, bias_std=0.05)
    if name == "gmm_wide":
        # a wide, odd dimension: many float4 groups per row and a ragged tail in every kernel
        return _gmm(name, 4099, 3, 0.5, ov(K, 12), ov(window, 6), ov(chains, 3), s, box=0.05)
    if name == "gmm_max_d":
        # the largest dimension the library accepts
        return _gmm(name, 65536, 2, 0.5, ov(K, 6), ov(window, 4), ov(chains, 2), s, box=0.02)
    if name == "gmm_odd":
        return _gmm(name, 5, 3, 0.5, ov(K, 50), ov(window, 7), ov(chains, 9), s)
    if name == "gauss_small":
        return _gauss(name, 12, ov(K, 80), ov(window, 5), ov(chains, 11), s)
    if name == "gauss_odd":
        # an odd dimension: a ragged last float4 group and parameter vectors of odd length
        return _gauss(name, 37, ov(K, 60), ov(window, 6), ov(chains, 5), s)
    raise KeyError(name)


SWEEP_CELLS = [(b, w) for b in (1, 8, 64, 512) for w in (4, 16, 64)]
