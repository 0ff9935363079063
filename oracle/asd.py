"""TEST INFRASTRUCTURE — CPU oracle, not part of the product path.

Plain float64 restatement of the sequential Euler sampler (Eq. 7) and of
Autospeculative Decoding (Algorithms 1-3), one chain at a time, one step at a
time, in the paper's notation.  Only tests, the smoke check and the CPU-baseline
leg of the benchmark may call this; it shares no code with the CUDA library.

Notation (Algorithm 1): cursor a, window end b = min(K, a + theta), drift
v_a = g(t_a, y_a), proposal means m^_{i+1} = y^_i + eta_i v_a, proposal samples
y^_{i+1} = m^_{i+1} + sigma_{i+1} xi_{i+1}, target means
m_{i+1} = y^_i + eta_i g(t_i, y^_i).

Readings of the paper taken here:
 * step size eta_i = t_{i+1} - t_i (Eq. 3; the definition under Eq. 7 has a typo);
 * the Gaussians of Eq. 8 / Eq. 9 have covariance sigma_{i+1}^2 I as in Algorithm 1;
   in the stochastic-localization chain sigma_{i+1}^2 = eta_i (increments given x*
   are N(eta x*, eta I), proof of Theorem 2), which is the default;
 * the target mean of slot i+1 is evaluated at the *proposal sample* y^_i
   (Algorithm 1 writes y_i, which does not exist yet for i > a); for i = a,
   y^_a = y_a, so g(t_a, y_a) = v_a is reused and that slot is never rejected
   (Lemma 1);
 * the Verifier returns the end of the all-accepted prefix (first rejection - 1),
   as Figure 1, the comment "advance until first rejection" and Lemma 1 require;
   the literal max over accepted indices would break Theorem 3;
 * the accept test u <= min(1, ratio) is evaluated as ln u <= min(0, ln ratio),
   ln ratio = -<xi, v>/sigma - |v|^2 / (2 sigma^2) with v = m^ - m (Algorithm 3);
 * the rejected branch divides by |v|^2; it is unreachable for v = 0 (ratio = 1),
   and is guarded anyway;
 * u_i, xi_i are drawn once per step and reused by every round that reaches that
   step (Algorithm 1, first two lines) - see oracle/philox.py for the generator.

Pins (tests/test_oracle_asd.py): acceptance probability 1 - TV (Theorem 5),
output law N(m, sigma^2 I) and the isometry of the reflection, window 1 ==
sequential bit for bit, theta = 2 gives ceil(K/2) rounds, the closed-form law of
the Euler chain on a Gaussian target, brute-force acceptance on d = 2.
"Parity unpinned": the absolute number of rounds per sample (only its bounds
ceil(K/theta) <= R <= ceil(K/2) are fixed by the paper).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Callable, List, Optional

import numpy as np

from . import philox


@dataclasses.dataclass
class Schedule:
    """Per-step tables, rounded to float32 exactly as the library stores them."""
    K: int
    eta: np.ndarray      # eta[i]   = t_{i+1} - t_i,  i = 0..K-1
    sigma: np.ndarray    # sigma[i] = sigma_{i+1}      (std of the step i -> i+1)


def make_schedule(t, sigma2=None) -> Schedule:
    t = np.asarray(t, dtype=np.float64)
    eta = np.diff(t)
    s2 = eta if sigma2 is None else np.asarray(sigma2, dtype=np.float64)
    f32 = lambda a: a.astype(np.float32).astype(np.float64)
    return Schedule(K=len(eta), eta=f32(eta), sigma=f32(np.sqrt(s2)))


# --------------------------------------------------------------------------
# Algorithm 3: Gaussian rejection sampler (reflection coupling)
# --------------------------------------------------------------------------
def grs(u: float, xi: np.ndarray, m_hat: np.ndarray, m: np.ndarray, sigma: float):
    """Returns (x, b, ln_ratio, ln_u)."""
    v = m_hat - m
    vv = float(v @ v)
    ln_ratio = -float(xi @ v) / sigma - vv / (2.0 * sigma * sigma)
    ln_u = math.log(u)
    b = ln_u <= min(0.0, ln_ratio)
    if b or vv == 0.0:
        x = m_hat + sigma * xi
        b = True
    else:
        x = m + sigma * (xi - 2.0 * v * float(v @ xi) / vv)
    return x, b, ln_ratio, ln_u


# --------------------------------------------------------------------------
# Algorithm 2: Verifier
# --------------------------------------------------------------------------
def verifier(us, xis, m_hats, ms, sigmas):
    """All slots go through GRS; returns the GRS outputs, the number n of
    leading accepted slots (j = a + n in the paper's indexing) and diagnostics."""
    zs, bs, ln_ratios, ln_us = [], [], [], []
    for u, xi, m_hat, m, sigma in zip(us, xis, m_hats, ms, sigmas):
        z, b, lr, lu = grs(u, xi, m_hat, m, sigma)
        zs.append(z); bs.append(b); ln_ratios.append(lr); ln_us.append(lu)
    n = 0
    while n < len(bs) and bs[n]:
        n += 1
    return zs, n, np.array(ln_ratios), np.array(ln_us)


@dataclasses.dataclass
class RoundRecord:
    a_before: int
    w: int                     # window actually used, b - a
    n: int                     # accepted prefix length
    a_after: int
    ln_ratio: np.ndarray       # [w]
    ln_u: np.ndarray           # [w]
    y_after: np.ndarray
    new_states: List[np.ndarray]   # y_{a+1} .. y_{a_after}
    points: Optional[List[np.ndarray]] = None   # diagnostics: y^_a .. y^_{b-1}, where the drift was evaluated
    drift: Optional[List[np.ndarray]] = None    # diagnostics: g(t_i, y^_i) at those points (drift[0] = v_a)

    @property
    def margin(self) -> float:
        """Smallest |ln ratio - ln u| over the slots that decide the prefix
        (slots 2 .. min(n+1, w)); slot 1 has ratio exactly 1."""
        last = min(self.n + 1, self.w)
        if last < 2:
            return math.inf
        return float(np.min(np.abs(self.ln_ratio[1:last] - self.ln_u[1:last])))


def _drifts(g: Callable, steps, points, slot):
    if hasattr(g, "batch") and len(steps) > 0:
        return list(g.batch(list(steps), np.stack(points), slot))
    return [g(i, p, slot) for i, p in zip(steps, points)]


# --------------------------------------------------------------------------
# Algorithm 1: one iteration of the while loop
# --------------------------------------------------------------------------
def asd_round(g: Callable, sched: Schedule, seed: int, chain_id: int, slot: int,
              a: int, y: np.ndarray, theta: int) -> RoundRecord:
    K = sched.K
    b = min(K, a + theta)
    w = b - a
    steps = np.arange(a + 1, b + 1)                    # i+1 for i = a..b-1
    xis = philox.xi(seed, chain_id, steps, len(y))     # xi_{a+1} .. xi_b
    us = philox.u(seed, chain_id, steps)               # u_{a+1} .. u_b

    v_a = g(a, y, slot)                                # model call 1
    y_hat = [y]                                        # y^_a = y_a
    m_hat = []
    for k in range(w):                                 # i = a + k
        i = a + k
        m_hat.append(y_hat[k] + sched.eta[i] * v_a)
        y_hat.append(m_hat[k] + sched.sigma[i] * xis[k])

    # model call 2 (parallel): drift at every drafted prefix point; slot i = a reuses v_a
    drift = [v_a] + _drifts(g, range(a + 1, b), y_hat[1:w], slot)
    m = [y_hat[k] + sched.eta[a + k] * drift[k] for k in range(w)]

    zs, n, ln_ratio, ln_u = verifier(us, xis, m_hat, m, sched.sigma[a:b])

    if n < w:                                          # j < b: keep z_{a+1..j+1}
        new_states = zs[: n + 1]
        a_after = a + n + 1
    else:
        new_states = zs[:n]
        a_after = a + n
    return RoundRecord(a, w, n, a_after, ln_ratio, ln_u, new_states[-1], new_states, y_hat[:w], drift)


@dataclasses.dataclass
class AdaptiveWindow:
    """Per-chain choice of the speculation length from the chain's own past (an addition of this
    library: the paper fixes theta; Algorithm 1 is exact for any theta, and a theta that depends only
    on the past is adapted to the filtration used in the proof of Theorem 3).  Integer rule, so that
    it can be reproduced exactly: with p = steps advanced in the round,
        ema8 <- (ema8 + 8 p) >> 1,      theta <- clamp(2 + (3 ema8) // 16, 2, theta_max),
    starting from ema8 = 32 (theta = min(theta_max, 8))."""
    theta_max: int
    ema8: int = 32

    def theta(self) -> int:
        return max(2, min(self.theta_max, 2 + (3 * self.ema8) // 16))

    def update(self, advanced: int) -> None:
        self.ema8 = (self.ema8 + 8 * advanced) >> 1


@dataclasses.dataclass
class ChainResult:
    y: np.ndarray
    rounds: int
    records: List[RoundRecord]
    trajectory: Optional[np.ndarray]
    model_rows: int            # drift evaluations made (pass 1 + pass 2)

    @property
    def min_margin(self) -> float:
        return min((r.margin for r in self.records), default=math.inf)


def asd_sample(g, sched: Schedule, seed: int, chain_id: int, slot: int, theta: int,
               y0=None, d: Optional[int] = None, max_rounds: Optional[int] = None,
               keep_records: bool = True, a0: int = 0, adaptive: bool = False) -> ChainResult:
    """Algorithm 1.  adaptive=True: theta is the upper limit and every round uses AdaptiveWindow's choice."""
    y = np.zeros(d) if y0 is None else np.asarray(y0, dtype=np.float64).copy()
    a, rounds, rows = a0, 0, 0
    records, traj = [], [y.copy()]
    policy = AdaptiveWindow(theta) if adaptive else None
    while a < sched.K and (max_rounds is None or rounds < max_rounds):
        rec = asd_round(g, sched, seed, chain_id, slot, a, y, policy.theta() if adaptive else theta)
        if adaptive:
            policy.update(rec.a_after - rec.a_before)
        rounds += 1
        rows += rec.w                                  # 1 + (w - 1)
        a, y = rec.a_after, rec.y_after
        traj.extend(rec.new_states)
        if keep_records:
            records.append(rec)
    return ChainResult(y, rounds, records, np.stack(traj), rows)


# --------------------------------------------------------------------------
# Eq. 7: the sequential Euler chain with the same xi streams (never uses u)
# --------------------------------------------------------------------------
def sequential_ddpm(g, sched: Schedule, seed: int, chain_id: int, slot: int,
                    y0=None, d: Optional[int] = None, return_trajectory: bool = False):
    y = np.zeros(d) if y0 is None else np.asarray(y0, dtype=np.float64).copy()
    traj = [y.copy()]
    for i in range(sched.K):
        xi = philox.xi(seed, chain_id, [i + 1], len(y))[0]
        y = (y + sched.eta[i] * g(i, y, slot)) + sched.sigma[i] * xi
        if return_trajectory:
            traj.append(y.copy())
    return (y, np.stack(traj)) if return_trajectory else y
