"""CPU-side checks of the boundary: the shared library loads without a GPU, exports every
symbol declared in include/asd.h, validates arguments on the host, and refuses to compute
without a device (there is no CPU fallback)."""
import ctypes as C
import os
import re

import numpy as np
import pytest
import torch

import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2505_03983_b200 import build, load_library
    build.build()
    return load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "asd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(asd_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    import paper_2505_03983_b200 as pkg
    declared = _declared_functions()
    assert "asd_create" in declared and "asd_round" in declared and "asd_sample" in declared
    assert "asd_sequential_ddpm" in declared
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(pkg.EXPORTED_SYMBOLS) == declared
    assert b"sm_100a" in lib.asd_version()


def test_struct_layout_matches_header():
    from paper_2505_03983_b200 import binding as b
    # pointers 8-byte aligned after the int32 / float fields, as a C compiler lays them out
    assert b._Denoiser.means.offset == 8 and b._Denoiser.sigma.offset == 24 and b._Denoiser.mu0.offset == 32
    assert b._Denoiser.d_cond.offset == 56 and b._Denoiser.W_in.offset == 72
    assert C.sizeof(b._Denoiser) == 144
    assert b._Config.t.offset == 16 and b._Config.den.offset == 40 and C.sizeof(b._Config) == 192
    assert C.sizeof(b._RoundStats) == 32 and C.sizeof(b._RunStats) == 48 and C.sizeof(b._PhaseTime) == 32


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device behaviour")
def test_no_device_means_error_not_fallback(lib):
    from paper_2505_03983_b200 import AsdError, AsdSampler, binding as b
    wl = workloads.make("cfg1_gmm2d")
    with pytest.raises(AsdError):
        AsdSampler(wl)
    # straight through the C ABI: a valid configuration still fails with ASD_ERR_CUDA
    cfg = b._Config()
    t = np.ascontiguousarray(wl.t)
    means, weights = np.ascontiguousarray(wl.means), np.ascontiguousarray(wl.weights)
    cfg.d, cfg.K, cfg.window, cfg.max_chains = 2, wl.K, 8, 4
    cfg.t = t.ctypes.data_as(C.c_void_p)
    cfg.den.kind, cfg.den.n_comp, cfg.den.sigma = 0, 8, 0.3
    cfg.den.means, cfg.den.weights = means.ctypes.data_as(C.c_void_p), weights.ctypes.data_as(C.c_void_p)
    ctx = C.c_void_p()
    assert lib.asd_create(C.byref(cfg), None, C.byref(ctx)) == 4 and not ctx.value
    assert b"no CUDA device" in lib.asd_last_error(None)


def test_host_side_validation(lib):
    from paper_2505_03983_b200 import binding as b
    ctx = C.c_void_p()
    assert lib.asd_create(None, None, C.byref(ctx)) == 1
    cfg = b._Config()
    t = np.array([0.0, 1.0, 2.0])
    cfg.d, cfg.K, cfg.window, cfg.max_chains = 2, 2, 1, 1
    cfg.t = t.ctypes.data_as(C.c_void_p)
    cfg.den.kind = 7
    assert lib.asd_create(C.byref(cfg), None, C.byref(ctx)) == 1
    assert b"unknown denoiser" in lib.asd_last_error(None)
    cfg.window = 0
    assert lib.asd_create(C.byref(cfg), None, C.byref(ctx)) == 1
    cfg.window, cfg.K = 1, 0
    assert lib.asd_create(C.byref(cfg), None, C.byref(ctx)) == 1
    cfg.K = 2
    tbad = np.array([0.0, 2.0, 1.0])
    cfg.t = tbad.ctypes.data_as(C.c_void_p)
    assert lib.asd_create(C.byref(cfg), None, C.byref(ctx)) == 1
    assert b"increasing" in lib.asd_last_error(None)
    # NULL contexts are rejected, never dereferenced
    assert lib.asd_round(None, None) == 1 and lib.asd_reset(None, 1, 0, None, None) == 1
    assert lib.asd_sample(None, None, None, None) == 1 and lib.asd_sequential_ddpm(None, None, None) == 1
    lib.asd_destroy(None)


def test_workloads_are_seeded_and_shaped():
    a, b_ = workloads.make("cfg3_policy"), workloads.make("cfg3_policy")
    assert np.array_equal(a.W_in, b_.W_in) and np.array_equal(a.cond, b_.cond)
    assert a.W_in.shape == (1024, 304) and a.W_hid.shape == (4, 1024, 1024) and a.W_out.shape == (112, 1024)
    w = workloads.bf16_bits_to_f32(a.W_hid)
    assert abs(w.std() - 0.02) < 1e-3 and abs(w.mean()) < 1e-3
    assert a.c_in[0] == 0 and a.c_skip[0] == 1 and np.isclose(a.c_out[0], 0.1)
    g = workloads.make("cfg2_gauss64")
    assert np.allclose(g.Q.T @ g.Q, np.eye(64), atol=1e-5) and g.lam.min() > 0.09
    assert np.allclose(np.diff(g.t), 0.1) and g.t[-1] == 100.0
    c = workloads.make("sweep_b8_w16")
    assert (c.chains, c.window, c.d, c.width, c.n_layers) == (8, 16, 3072, 4096, 6)
