"""TEST INFRASTRUCTURE — CPU oracle, not part of the product path.

DDPM front end: from a DDPM noise schedule (alpha-bar of the K+1 levels visited, in sampling order,
so increasing) and the network's prediction type to the chain of Eq. 7.

Stochastic-localization mapping (Theorem 1; Eq. 4 with x_level = sqrt(ab) x0 + sqrt(1-ab) eps):
dividing by sqrt(ab) and multiplying by t = ab / (1 - ab) gives t x0 + sqrt(t) eps, the SL observation,
so y = (t / sqrt(ab)) x = sqrt(t (1 + t)) x, and the SL increments have variance eta (Theorem 2).

Ancestral mapping (remark after Algorithm 1): the DDPM ancestral step from level s to the less noisy
level r, with alpha = ab_s / ab_r and beta = 1 - alpha, draws from the Gaussian posterior of x_r given
x_s and x0 with x0 replaced by the network's estimate,
    x_r = a x_s + b x0_hat + s xi,   a = sqrt(alpha) (1 - ab_r) / (1 - ab_s),   b = sqrt(ab_r) beta / (1 - ab_s),
    s^2 = beta (1 - ab_r) / (1 - ab_s)   (or beta, the "large" variance).
With A_i = a_0 ... a_{i-1} and y_i = x_i / A_i this is y_{i+1} = y_i + (b_i / A_{i+1}) x0_hat + (s_i / A_{i+1}) xi.

x0_hat = k_x x + k_n net(x): x0-prediction (0, 1); eps-prediction (1 / sqrt(ab), -sqrt((1 - ab) / ab));
v-prediction (sqrt(ab), -sqrt(1 - ab)), from x = sqrt(ab) x0 + sqrt(1-ab) eps and v = sqrt(ab) eps - sqrt(1-ab) x0.

Pins (tests/test_oracle_ddpm.py): the three prediction types against the closed-form posterior mean of a
Gaussian target in SL time; the ancestral mapping against the sampler written directly in x, step by step,
on the same noise.
"""
from __future__ import annotations

import numpy as np


def prediction_coefficients(ab: float, pred: str):
    if pred == "x0":
        return 0.0, 1.0
    if pred == "eps":
        return 1.0 / np.sqrt(ab), -np.sqrt((1.0 - ab) / ab)
    if pred == "v":
        return np.sqrt(ab), -np.sqrt(1.0 - ab)
    raise ValueError(pred)


def ddpm_schedule(alpha_bar, pred="eps", mapping="sl", large_variance=False):
    ab = np.asarray(alpha_bar, dtype=np.float64)
    K = len(ab) - 1
    assert np.all((ab > 0) & (ab < 1)) and np.all(np.diff(ab) > 0)
    if mapping == "sl":
        t = ab / (1.0 - ab)
        sigma2 = np.diff(t)
        x_scale = 1.0 / np.sqrt(t * (1.0 + t))
    elif mapping == "ancestral":
        t, sigma2, x_scale = np.zeros(K + 1), np.zeros(K), np.ones(K + 1)
        for i in range(K):
            alpha = ab[i] / ab[i + 1]
            beta = 1.0 - alpha
            a = np.sqrt(alpha) * (1.0 - ab[i + 1]) / (1.0 - ab[i])
            b = np.sqrt(ab[i + 1]) * beta / (1.0 - ab[i])
            s2 = beta if large_variance else beta * (1.0 - ab[i + 1]) / (1.0 - ab[i])
            x_scale[i + 1] = x_scale[i] * a
            t[i + 1] = t[i] + b / x_scale[i + 1]
            sigma2[i] = s2 / x_scale[i + 1] ** 2
    else:
        raise ValueError(mapping)
    kx, kn = np.array([prediction_coefficients(ab[i], pred) for i in range(K)]).T
    return dict(t=t, sigma2=sigma2, c_in=x_scale[:K].astype(np.float32), c_skip=(kx * x_scale[:K]).astype(np.float32),
                c_out=kn.astype(np.float32), x_scale=x_scale)
