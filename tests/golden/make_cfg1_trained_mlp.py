"""Fits a small residual MLP to the closed-form posterior mean of the cfg-1 mixture and stores it.

    python tests/golden/make_cfg1_trained_mlp.py        (CPU, about a minute; seeded)

The network has the library's architecture (x = [bf16(c_in y); temb(i)], input projection, residual SiLU
layers, output projection, g = c_skip y + c_out (W_out h + b_out)).  The target is Eq. 4's posterior mean of the
8-component mixture of the cfg-1 workload, m(t, y) = (sum_j r_j c_j + s^2 y) / (1 + t s^2), evaluated by the
oracle (oracle.denoisers.GmmPosteriorMean).  The per-step tables take the part that is linear in y out of the
network's job: c_skip = s^2 / (1 + t s^2), c_out = 1 / (1 + t s^2), c_in = 1 / (4 (1 + t s^2)), so the network
regresses sum_j r_j(t, y) c_j, the responsibility-weighted centre, which stays inside the box of the means.
Training pairs: step i uniform, x* from the mixture, y = t_i x* + sqrt(t_i) xi (the law of the localization
process at time t_i).  Weights are rounded to bf16 at the end; the file holds bf16 bit patterns and the fp32
tables, and is written by this script only (tests/golden/cfg1_trained_mlp.npz)."""
import os
import sys

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
sys.path.insert(0, ROOT)

import workloads  # noqa: E402
from oracle import denoisers as oden  # noqa: E402

WIDTH, LAYERS, D_TEMB, STEPS, BATCH = 64, 3, 32, 6000, 2048


def temb_table(K, d_temb):
    return np.stack([oden.time_embedding(i, K, d_temb) for i in range(K)])


def main():
    torch.manual_seed(0)
    torch.set_num_threads(4)
    base = workloads.make("cfg1_gmm2d")
    K, d = base.K, base.d
    g = oden.from_workload(base)
    s2 = float(np.float32(base.sigma)) ** 2
    t = base.t[:K]
    c_skip = (s2 / (1 + t * s2)).astype(np.float32)
    c_out = (1 / (1 + t * s2)).astype(np.float32)
    c_in = (0.25 / (1 + t * s2)).astype(np.float32)
    temb = torch.tensor(temb_table(K, D_TEMB), dtype=torch.float32)
    rng = np.random.default_rng(0)
    in_dim = d + D_TEMB
    W_in = torch.nn.Parameter(torch.randn(WIDTH, in_dim) / np.sqrt(in_dim))
    b_in = torch.nn.Parameter(torch.zeros(WIDTH))
    W_hid = torch.nn.Parameter(torch.randn(LAYERS, WIDTH, WIDTH) / np.sqrt(WIDTH))
    b_hid = torch.nn.Parameter(torch.zeros(LAYERS, WIDTH))
    W_out = torch.nn.Parameter(torch.randn(d, WIDTH) / np.sqrt(WIDTH))
    b_out = torch.nn.Parameter(torch.zeros(d))
    params = [W_in, b_in, W_hid, b_hid, W_out, b_out]
    opt = torch.optim.Adam(params, lr=3e-3)
    sched = torch.optim.lr_scheduler.CosineAnnealingLR(opt, STEPS)

    def net(i, y):
        x = torch.cat([torch.tensor(c_in)[i, None] * y, temb[i]], dim=1)
        h = x @ W_in.T + b_in
        for l in range(LAYERS):
            h = h + torch.nn.functional.silu(h @ W_hid[l].T + b_hid[l])
        return h @ W_out.T + b_out

    def batch(n):
        i = rng.integers(0, K, n)
        comp = rng.integers(0, len(base.weights), n)
        xs = base.means[comp] + base.sigma * rng.standard_normal((n, d))
        y = t[i, None] * xs + np.sqrt(t[i])[:, None] * rng.standard_normal((n, d))
        m = np.stack([g(int(ii), yy) for ii, yy in zip(i, y)])                 # oracle posterior mean
        target = (m - c_skip[i, None] * y) / c_out[i, None]                   # = sum_j r_j c_j
        return torch.tensor(i), torch.tensor(y, dtype=torch.float32), torch.tensor(target, dtype=torch.float32)

    for step in range(STEPS):
        i, y, target = batch(BATCH)
        loss = torch.mean((net(i, y) - target) ** 2)
        opt.zero_grad()
        loss.backward()
        opt.step()
        sched.step()
        if step % 500 == 0 or step == STEPS - 1:
            print(f"step {step}: mse {loss.item():.4f}")
    bits = lambda p: workloads._bf16_bits(p.detach().numpy())
    out = os.path.join(HERE, "cfg1_trained_mlp.npz")
    np.savez_compressed(out, W_in=bits(W_in), W_hid=bits(W_hid), W_out=bits(W_out),
                        b_in=b_in.detach().numpy(), b_hid=b_hid.detach().numpy(), b_out=b_out.detach().numpy(),
                        c_in=c_in, c_skip=c_skip, c_out=c_out, d_temb=np.int32(D_TEMB))
    print("wrote", out, os.path.getsize(out), "bytes")


if __name__ == "__main__":
    main()
