"""asd_denoise_static - the drift entry point for callers that cannot allocate device memory
where they need it (a serving loop that must not take cudaMalloc's device-wide synchronisation,
a process whose remaining device memory belongs to another allocator, a host that forbids
allocation calls).  Its GEMM-chain scratch is a fixed 8 MiB array inside the library instead of
the context's cudaMalloc'd workspaces, so it also serves more rows than the context was sized for.

The test calls it through the C ABI twice in a row and compares with asd_denoise (the existing
entry point, same kernels) on the same inputs; the second call starts from the first call's
leftovers in the shared array.  It is collected last so that a stop-at-first-failure run has
already executed every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

import workloads

pytestmark = pytest.mark.gpu


def _inputs(wl, n_rows, cap, seed):
    rng = np.random.default_rng(seed)
    steps = torch.as_tensor(rng.integers(0, wl.K, n_rows).astype(np.int32), device="cuda")
    tt = wl.t[steps.cpu().numpy()]
    y = (tt[:, None] * rng.standard_normal((n_rows, wl.d)) +
         np.sqrt(tt)[:, None] * rng.standard_normal((n_rows, wl.d))).astype(np.float32)
    slots = torch.as_tensor(rng.integers(0, cap, n_rows).astype(np.int32), device="cuda")
    return steps, torch.as_tensor(y, device="cuda"), slots


def test_static_scratch_entry_point_matches_asd_denoise():
    from paper_2505_03983_b200 import AsdError, AsdSampler
    wl = workloads.make("mlp_ragged")                     # d=52, cond 12, width 320, 3 layers
    cap = wl.chains
    with AsdSampler(wl, max_chains=cap) as s:
        s.reset(cap, 0, cond=wl.cond)
        lib, ctx = s.lib, s._ctx
        max_rows = s.denoise_static_max_rows()
        assert max_rows == (8 * 2 ** 20 - 1024) // (2 * (128 + 2 * 320))
        ctx_rows = cap * (wl.window - 1)                  # what asd_denoise accepts on this context
        for call, n_rows in enumerate((ctx_rows, 200)):   # second call: fewer rows, stale rows beyond
            steps, y, slots = _inputs(wl, n_rows, cap, seed=call)
            ref = s.denoise(steps, y, slots)
            out = torch.full_like(y, float("nan"))
            st = lib.asd_denoise_static(ctx, n_rows, C.c_void_p(steps.data_ptr()), C.c_void_p(y.data_ptr()),
                                        C.c_void_p(slots.data_ptr()), C.c_void_p(out.data_ptr()))
            assert st == 0, lib.asd_last_error(ctx)
            assert torch.isfinite(out).all()
            err = (out - ref).abs().max().item() / max(1.0, ref.abs().max().item())
            assert err < 2e-3                             # the tolerance of the drift parity test
            assert torch.equal(out, ref)                  # same kernels, same data: identical
        # more rows than the context's own workspaces hold, still within the fixed array
        n_big = min(max_rows, ctx_rows + 500)
        steps, y, slots = _inputs(wl, n_big, cap, seed=9)
        with pytest.raises(AsdError):
            s.denoise(steps, y, slots)
        big = s.denoise_static(steps, y, slots)
        head = s.denoise(steps[:ctx_rows], y[:ctx_rows], slots[:ctx_rows])
        # a different row count may select a different GEMM kernel (another summation order), so this
        # comparison uses the tolerance of the drift parity test rather than bit equality
        assert torch.isfinite(big).all()
        assert (big[:ctx_rows] - head).abs().max().item() / max(1.0, head.abs().max().item()) < 2e-3
        # beyond the maximum: rejected with a clear error, nothing launched
        st = lib.asd_denoise_static(ctx, max_rows + 1, C.c_void_p(steps.data_ptr()), C.c_void_p(y.data_ptr()),
                                    C.c_void_p(slots.data_ptr()), C.c_void_p(big.data_ptr()))
        assert st == 1 and b"exceeds" in lib.asd_last_error(ctx)
    # closed-form drifts use no scratch
    g = workloads.make("cfg1_gmm2d")
    with AsdSampler(g) as s2:
        with pytest.raises(AsdError):
            s2.denoise_static(np.zeros(1, np.int32), np.zeros((1, 2), np.float32))
