"""TEST INFRASTRUCTURE — CPU oracle, not part of the product path.

Counter-based randomness of the ASD sampler (Algorithm 1, the two "sample"
lines): the uniforms u_1..u_K and the Gaussians xi_1..xi_K are drawn once per
chain, indexed by the step, and reused by every round that touches that step.
The paper does not say how they are generated; this build fixes the mapping
below (it is part of the library's contract, restated here independently):

  generator  Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11),
             multipliers 0xD2511F53 / 0xCD9E8D57, key increments
             0x9E3779B9 / 0xBB67AE85
  key        (seed low word, seed high word)
  counter    (q, step i in 1..K, chain id, tag)
             tag 0: the four output words give xi_i[4q .. 4q+3]
             tag 1, q = 0: output word 0 gives u_i
  uniform    U(r) = ((r >> 9) + 0.5) * 2**-23   (24 significant bits, in (0,1))
  normal     Box-Muller on word pairs: (r0, r1) -> n0, n1 and (r2, r3) -> n2, n3,
             n_even = sqrt(-2 ln U(r_even)) cos(2 pi U(r_odd)),
             n_odd  = sqrt(-2 ln U(r_even)) sin(2 pi U(r_odd))

Everything after the 32-bit words is evaluated in float64 here.

Pins (tests/test_oracle_philox.py): the published Philox4x32-10 known-answer
vectors, exact values of U at the ends of the word range, Box-Muller against
hand-computed angles, and moment / Kolmogorov-Smirnov checks of 10^6 draws.
"""
from __future__ import annotations

import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = np.uint64(0x9E3779B9)
_W1 = np.uint64(0xBB67AE85)
_MASK = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)

TAG_XI = 0
TAG_U = 1


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten Philox4x32 rounds.  All arguments are broadcastable integer arrays
    holding 32-bit values; returns four uint64 arrays holding 32-bit words."""
    c0, c1, c2, c3, k0, k1 = np.broadcast_arrays(
        *[np.asarray(a, dtype=np.uint64) & _MASK for a in (c0, c1, c2, c3, k0, k1)])
    for r in range(10):
        p0 = _M0 * c0                      # 32x32 -> 64 bit products, exact in uint64
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _S32, p0 & _MASK
        hi1, lo1 = p1 >> _S32, p1 & _MASK
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + _W0) & _MASK
        k1 = (k1 + _W1) & _MASK
    return c0, c1, c2, c3


def uniform_from_word(r):
    """U(r) = ((r >> 9) + 0.5) 2^-23, strictly inside (0, 1)."""
    r = np.asarray(r, dtype=np.uint64)
    return ((r >> np.uint64(9)).astype(np.float64) + 0.5) * (2.0 ** -23)


def box_muller(r_even, r_odd):
    """Two standard normals from two 32-bit words."""
    rad = np.sqrt(-2.0 * np.log(uniform_from_word(r_even)))
    ang = 2.0 * np.pi * uniform_from_word(r_odd)
    return rad * np.cos(ang), rad * np.sin(ang)


def _key(seed: int):
    return seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF


def xi(seed: int, chain: int, steps, d: int) -> np.ndarray:
    """Gaussian vectors xi_i in R^d for the given steps i (1-based, as in
    Algorithm 1); returns float64 [len(steps), d]."""
    steps = np.atleast_1d(np.asarray(steps, dtype=np.int64))
    nq = (d + 3) // 4
    q = np.arange(nq, dtype=np.uint64)[None, :]
    k0, k1 = _key(seed)
    r0, r1, r2, r3 = philox4x32_10(q, steps[:, None].astype(np.uint64), chain, TAG_XI, k0, k1)
    n0, n1 = box_muller(r0, r1)
    n2, n3 = box_muller(r2, r3)
    out = np.stack([n0, n1, n2, n3], axis=-1).reshape(len(steps), 4 * nq)
    return out[:, :d]


def u(seed: int, chain: int, steps) -> np.ndarray:
    """Uniforms u_i for the given steps i (1-based); float64 [len(steps)]."""
    steps = np.atleast_1d(np.asarray(steps, dtype=np.int64))
    k0, k1 = _key(seed)
    r0, _, _, _ = philox4x32_10(0, steps.astype(np.uint64), chain, TAG_U, k0, k1)
    return uniform_from_word(r0)
