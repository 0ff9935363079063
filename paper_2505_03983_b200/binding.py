"""ctypes binding of the ASD C ABI (include/asd.h).  Same names, argument marshalling only.

There is no CPU fallback: if the shared library has not been built, or no CUDA device is
present, the calls raise."""
from __future__ import annotations

import ctypes as C
import dataclasses
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))

EXPORTED_SYMBOLS = [
    "asd_version", "asd_create", "asd_reset", "asd_round", "asd_sample", "asd_sequential_ddpm",
    "asd_sample_host", "asd_get_state", "asd_set_state", "asd_get_window_state", "asd_set_window_state", "asd_debug_last_round", "asd_denoise",
    "asd_set_profiling", "asd_get_profile", "asd_get_trajectory", "asd_get_prefix_histogram", "asd_ddpm_schedule", "asd_debug_wait_selftest", "asd_denoise_static", "asd_denoise_static_max_rows",
    "asd_last_error", "asd_destroy",
]

STATUS = {0: "ASD_OK", 1: "ASD_ERR_INVALID_ARG", 2: "ASD_ERR_UNSUPPORTED", 3: "ASD_ERR_OOM",
          4: "ASD_ERR_CUDA", 5: "ASD_ERR_STATE", 6: "ASD_ERR_TIMEOUT"}
KIND = {"gmm": 0, "gauss": 1, "mlp": 2}
FLAG_DEBUG_ALL_SLOTS = 1   # ASD_FLAG_DEBUG_ALL_SLOTS
FLAG_ADAPTIVE_WINDOW = 2   # ASD_FLAG_ADAPTIVE_WINDOW
FLAG_LOOKAHEAD = 4         # ASD_FLAG_LOOKAHEAD
FLAG_TRAJECTORY = 8        # ASD_FLAG_TRAJECTORY
FLAG_DEBUG_DUMP = 16       # ASD_FLAG_DEBUG_DUMP


PRED = {"x0": 0, "eps": 1, "v": 2}
MAP = {"sl": 0, "ancestral": 1}


def ddpm_schedule(alpha_bar, pred="eps", mapping="sl", large_variance=False):
    """asd_ddpm_schedule: dict(t, sigma2, c_in, c_skip, c_out, x_scale) for K = len(alpha_bar) - 1 steps."""
    lib = load_library()
    ab = np.ascontiguousarray(alpha_bar, dtype=np.float64)
    K = len(ab) - 1
    t, s2, xs = np.empty(K + 1), np.empty(max(K, 0)), np.empty(K + 1)
    ci, cs, co = (np.empty(max(K, 0), np.float32) for _ in range(3))
    st = lib.asd_ddpm_schedule(K, _np_ptr(ab), PRED[pred], MAP[mapping], int(large_variance), _np_ptr(t), _np_ptr(s2),
                               _np_ptr(ci), _np_ptr(cs), _np_ptr(co), _np_ptr(xs))
    if st != 0:
        raise AsdError(st, "asd_ddpm_schedule: alpha_bar must be strictly increasing inside (0, 1)")
    return dict(t=t, sigma2=s2, c_in=ci, c_skip=cs, c_out=co, x_scale=xs)


class AsdError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"{STATUS.get(status, status)}: {msg}")
        self.status = status


class _Denoiser(C.Structure):
    _fields_ = [
        ("kind", C.c_int32), ("n_comp", C.c_int32), ("means", C.c_void_p), ("weights", C.c_void_p),
        ("sigma", C.c_float), ("mu0", C.c_void_p), ("Q", C.c_void_p), ("lam", C.c_void_p),
        ("d_cond", C.c_int32), ("d_temb", C.c_int32), ("width", C.c_int32), ("n_layers", C.c_int32),
        ("W_in", C.c_void_p), ("W_hid", C.c_void_p), ("W_out", C.c_void_p),
        ("b_in", C.c_void_p), ("b_hid", C.c_void_p), ("b_out", C.c_void_p),
        ("c_in", C.c_void_p), ("c_skip", C.c_void_p), ("c_out", C.c_void_p),
    ]


class _Config(C.Structure):
    _fields_ = [
        ("d", C.c_int32), ("K", C.c_int32), ("window", C.c_int32), ("max_chains", C.c_int32),
        ("t", C.c_void_p), ("sigma2", C.c_void_p), ("seed", C.c_uint64), ("den", _Denoiser),
        ("flags", C.c_uint32),
    ]


class _RoundStats(C.Structure):
    _fields_ = [("n_active_before", C.c_int32), ("n_active_after", C.c_int32),
                ("rows_pass1", C.c_int64), ("rows_pass2", C.c_int64), ("accepted_total", C.c_int64)]


class _RunStats(C.Structure):
    _fields_ = [("rounds_max", C.c_int64), ("rounds_mean", C.c_double), ("rows_total", C.c_int64),
                ("ms_total", C.c_double), ("launches", C.c_int64), ("rows_verified", C.c_int64)]


class _PhaseTime(C.Structure):
    _fields_ = [("name", C.c_char_p), ("launches", C.c_int64), ("ms", C.c_double), ("rows", C.c_int64)]


@dataclasses.dataclass
class RoundStats:
    n_active_before: int
    n_active_after: int
    rows_pass1: int
    rows_pass2: int
    accepted_total: int


@dataclasses.dataclass
class RunStats:
    rounds_max: int
    rounds_mean: float
    rows_total: int
    ms_total: float
    launches: int
    rows_verified: int = 0


def lib_path() -> str:
    return os.path.join(_HERE, "libasd_b200.so")


_LIB = None


def load_library():
    """Load the shared library and declare the prototypes.  Raises if it has not been built."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run `python -m paper_2505_03983_b200.build` "
                          "(or __graft_entry__.build()); there is no fallback path")
    lib = C.CDLL(path)
    vp, i32, u64 = C.c_void_p, C.c_int32, C.c_uint64
    lib.asd_version.restype = C.c_char_p
    lib.asd_version.argtypes = []
    lib.asd_last_error.restype = C.c_char_p
    lib.asd_last_error.argtypes = [vp]
    lib.asd_destroy.restype = None
    lib.asd_destroy.argtypes = [vp]
    protos = {
        "asd_create": [C.POINTER(_Config), vp, C.POINTER(vp)],
        "asd_reset": [vp, i32, u64, vp, vp],
        "asd_round": [vp, C.POINTER(_RoundStats)],
        "asd_sample": [vp, vp, vp, C.POINTER(_RunStats)],
        "asd_sequential_ddpm": [vp, vp, C.POINTER(_RunStats)],
        "asd_sample_host": [vp, i32, u64, vp, vp, i32, vp, vp, C.POINTER(_RunStats)],
        "asd_get_state": [vp, vp, vp, vp],
        "asd_set_state": [vp, vp, vp, vp],
        "asd_debug_wait_selftest": [vp],
        "asd_ddpm_schedule": [i32, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp],
        "asd_get_window_state": [vp, vp, vp],
        "asd_set_window_state": [vp, vp, vp],
        "asd_debug_last_round": [vp, vp, vp, vp],
        "asd_get_trajectory": [vp, vp],
        "asd_get_prefix_histogram": [vp, vp, i32, C.POINTER(i32)],
        "asd_denoise": [vp, i32, vp, vp, vp, vp],
        "asd_denoise_static": [vp, i32, vp, vp, vp, vp],
        "asd_denoise_static_max_rows": [vp, C.POINTER(i32)],
        "asd_set_profiling": [vp, i32],
        "asd_get_profile": [vp, C.POINTER(_PhaseTime), i32, C.POINTER(i32)],
    }
    for name, args in protos.items():
        fn = getattr(lib, name)
        fn.restype = C.c_int
        fn.argtypes = args
    _LIB = lib
    return lib


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dev_ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


class AsdSampler:
    """One library context: asd_create on construction, asd_destroy on close().

    `wl` is any record with the fields of `workloads.Workload` (kind, d, K, window, t and the
    denoiser arrays).  Methods mirror the C entry points; tensors are torch CUDA tensors."""

    def __init__(self, wl, max_chains: Optional[int] = None, window: Optional[int] = None,
                 seed: Optional[int] = None, sigma2: Optional[np.ndarray] = None, stream=None, flags: int = 0):
        import torch
        if not torch.cuda.is_available():
            raise AsdError(4, "no CUDA device: the ASD library has no CPU path")
        self._torch = torch
        self.lib = load_library()
        self.d, self.K = int(wl.d), int(wl.K)
        self.window = int(window if window is not None else wl.window)
        self.max_chains = int(max_chains if max_chains is not None else wl.chains)
        self.d_cond = int(getattr(wl, "d_cond", 0) or 0)
        self.kind = wl.kind
        keep = []  # keep host arrays alive during asd_create

        def f32(a):
            a = np.ascontiguousarray(a, dtype=np.float32); keep.append(a); return _np_ptr(a)

        def u16(a):
            a = np.ascontiguousarray(a, dtype=np.uint16); keep.append(a); return _np_ptr(a)

        def f64(a):
            a = np.ascontiguousarray(a, dtype=np.float64); keep.append(a); return _np_ptr(a)

        den = _Denoiser()
        den.kind = KIND[wl.kind]
        if wl.kind == "gmm":
            den.n_comp = len(wl.weights)
            den.means, den.weights, den.sigma = f32(wl.means), f32(wl.weights), float(wl.sigma)
        elif wl.kind == "gauss":
            den.mu0, den.Q, den.lam = f32(wl.mu0), f32(wl.Q), f32(wl.lam)
        else:
            den.d_cond, den.d_temb, den.width, den.n_layers = wl.d_cond, wl.d_temb, wl.width, wl.n_layers
            den.W_in, den.W_hid, den.W_out = u16(wl.W_in), u16(wl.W_hid), u16(wl.W_out)
            den.b_in, den.b_hid, den.b_out = f32(wl.b_in), f32(wl.b_hid), f32(wl.b_out)
            den.c_in = None if wl.c_in is None else f32(wl.c_in)
            den.c_skip = None if wl.c_skip is None else f32(wl.c_skip)
            den.c_out = None if wl.c_out is None else f32(wl.c_out)
        cfg = _Config()
        cfg.d, cfg.K, cfg.window, cfg.max_chains = self.d, self.K, self.window, self.max_chains
        cfg.t = f64(wl.t)
        cfg.sigma2 = None if sigma2 is None else f64(sigma2)
        cfg.seed = int(seed if seed is not None else wl.seed)
        cfg.den = den
        cfg.flags = int(flags)
        self.seed = cfg.seed
        self.stream = stream
        sptr = C.c_void_p(stream.cuda_stream) if stream is not None else C.c_void_p(
            torch.cuda.current_stream().cuda_stream)
        self._ctx = C.c_void_p()
        st = self.lib.asd_create(C.byref(cfg), sptr, C.byref(self._ctx))
        if st != 0:
            raise AsdError(st, self.lib.asd_last_error(None).decode())
        self.n = 0

    # -- helpers -------------------------------------------------------------------------
    def _check(self, st: int):
        if st != 0:
            raise AsdError(st, self.lib.asd_last_error(self._ctx).decode())

    def _empty(self, shape, dtype):
        return self._torch.empty(shape, dtype=dtype, device="cuda")

    def close(self):
        if getattr(self, "_ctx", None):
            self.lib.asd_destroy(self._ctx)
            self._ctx = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- entry points -------------------------------------------------------------------
    def reset(self, n_chains: int, chain_id_base: int = 0, y0=None, cond=None):
        torch = self._torch
        if y0 is not None:
            y0 = y0.to(device="cuda", dtype=torch.float32).contiguous()
            assert y0.shape == (n_chains, self.d)
        if cond is not None:
            cond = torch.as_tensor(cond).to(device="cuda", dtype=torch.float32).contiguous()
            assert cond.shape == (n_chains, self.d_cond)
        self._check(self.lib.asd_reset(self._ctx, n_chains, chain_id_base, _dev_ptr(y0), _dev_ptr(cond)))
        self.n = n_chains

    def round(self, want_stats: bool = True) -> Optional[RoundStats]:
        if not want_stats:
            self._check(self.lib.asd_round(self._ctx, None))
            return None
        rs = _RoundStats()
        self._check(self.lib.asd_round(self._ctx, C.byref(rs)))
        return RoundStats(rs.n_active_before, rs.n_active_after, rs.rows_pass1, rs.rows_pass2, rs.accepted_total)

    def _run_stats(self, s: _RunStats) -> RunStats:
        return RunStats(s.rounds_max, s.rounds_mean, s.rows_total, s.ms_total, s.launches, s.rows_verified)

    def sample(self):
        torch = self._torch
        y = self._empty((self.n, self.d), torch.float32)
        r = self._empty((self.n,), torch.int32)
        s = _RunStats()
        self._check(self.lib.asd_sample(self._ctx, _dev_ptr(y), _dev_ptr(r), C.byref(s)))
        return y, r, self._run_stats(s)

    def sequential_ddpm(self):
        y = self._empty((self.n, self.d), self._torch.float32)
        s = _RunStats()
        self._check(self.lib.asd_sequential_ddpm(self._ctx, _dev_ptr(y), C.byref(s)))
        return y, self._run_stats(s)

    def sample_host(self, n_chains: int, chain_id_base: int = 0, y0: Optional[np.ndarray] = None,
                    cond: Optional[np.ndarray] = None, sequential: bool = False,
                    y_out: Optional[np.ndarray] = None, rounds_out: Optional[np.ndarray] = None):
        """Host buffers in, host buffers out (numpy or pinned torch CPU tensors viewed as numpy)."""
        if y_out is None:
            y_out = np.empty((n_chains, self.d), np.float32)
        if rounds_out is None:
            rounds_out = np.zeros((n_chains,), np.int32)
        s = _RunStats()
        self._check(self.lib.asd_sample_host(self._ctx, n_chains, chain_id_base, _np_ptr(y0), _np_ptr(cond),
                                             int(sequential), _np_ptr(y_out), _np_ptr(rounds_out), C.byref(s)))
        self.n = n_chains
        return y_out, rounds_out, self._run_stats(s)

    def get_state(self):
        torch = self._torch
        a = self._empty((self.n,), torch.int32)
        y = self._empty((self.n, self.d), torch.float32)
        r = self._empty((self.n,), torch.int32)
        self._check(self.lib.asd_get_state(self._ctx, _dev_ptr(a), _dev_ptr(y), _dev_ptr(r)))
        return a, y, r

    def set_state(self, a=None, y=None, rounds=None):
        torch = self._torch
        a = None if a is None else a.to(device="cuda", dtype=torch.int32).contiguous()
        y = None if y is None else y.to(device="cuda", dtype=torch.float32).contiguous()
        rounds = None if rounds is None else rounds.to(device="cuda", dtype=torch.int32).contiguous()
        self._check(self.lib.asd_set_state(self._ctx, _dev_ptr(a), _dev_ptr(y), _dev_ptr(rounds)))
        torch.cuda.current_stream().synchronize()

    def get_window_state(self):
        """(speculation length of the next round, 8 x running mean of the steps per round), per chain."""
        torch = self._torch
        w, e = self._empty((self.n,), torch.int32), self._empty((self.n,), torch.int32)
        self._check(self.lib.asd_get_window_state(self._ctx, _dev_ptr(w), _dev_ptr(e)))
        torch.cuda.current_stream().synchronize()
        return w, e

    def set_window_state(self, window=None, ema8=None):
        torch = self._torch
        window = None if window is None else window.to(device="cuda", dtype=torch.int32).contiguous()
        ema8 = None if ema8 is None else ema8.to(device="cuda", dtype=torch.int32).contiguous()
        self._check(self.lib.asd_set_window_state(self._ctx, _dev_ptr(window), _dev_ptr(ema8)))
        torch.cuda.current_stream().synchronize()

    def debug_last_round(self):
        torch = self._torch
        lr = self._torch.zeros((self.n, min(self.window, self.K)), dtype=torch.float32, device="cuda")
        lu = self._torch.zeros_like(lr)
        acc = self._empty((self.n,), torch.int32)
        self._check(self.lib.asd_debug_last_round(self._ctx, _dev_ptr(lr), _dev_ptr(lu), _dev_ptr(acc)))
        return lr, lu, acc

    def accepted_last_round(self):
        """Accepted prefix length per chain in the last round (-1: the chain was not active)."""
        acc = self._empty((self.n,), self._torch.int32)
        self._check(self.lib.asd_debug_last_round(self._ctx, None, None, _dev_ptr(acc)))
        return acc

    def get_trajectory(self):
        """(y_0 .. y_K) per chain, [n, K + 1, d]; needs FLAG_TRAJECTORY at construction."""
        traj = self._empty((self.n, self.K + 1, self.d), self._torch.float32)
        self._check(self.lib.asd_get_trajectory(self._ctx, _dev_ptr(traj)))
        return traj

    def prefix_histogram(self) -> np.ndarray:
        """Chain-rounds since the last reset by accepted prefix length (index = length, 0 .. window)."""
        h = np.zeros(min(self.window, self.K) + 1, dtype=np.int64)
        n = C.c_int32(0)
        self._check(self.lib.asd_get_prefix_histogram(self._ctx, _np_ptr(h), len(h), C.byref(n)))
        return h[:n.value]

    def denoise(self, steps, y, slots=None):
        torch = self._torch
        steps = torch.as_tensor(steps).to(device="cuda", dtype=torch.int32).contiguous()
        y = torch.as_tensor(y).to(device="cuda", dtype=torch.float32).contiguous()
        if slots is not None:
            slots = torch.as_tensor(slots).to(device="cuda", dtype=torch.int32).contiguous()
        out = torch.empty_like(y)
        self._check(self.lib.asd_denoise(self._ctx, y.shape[0], _dev_ptr(steps), _dev_ptr(y), _dev_ptr(slots),
                                         _dev_ptr(out)))
        return out

    def set_profiling(self, enable: bool):
        self._check(self.lib.asd_set_profiling(self._ctx, int(enable)))

    def get_profile(self):
        """{phase name: dict(launches, ms, rows)} accumulated since set_profiling(True)."""
        arr = (_PhaseTime * 32)()
        n = C.c_int32(0)
        self._check(self.lib.asd_get_profile(self._ctx, arr, 32, C.byref(n)))
        return {arr[i].name.decode(): dict(launches=arr[i].launches, ms=arr[i].ms, rows=arr[i].rows)
                for i in range(n.value)}

    def denoise_static_max_rows(self) -> int:
        n = C.c_int32(0)
        self._check(self.lib.asd_denoise_static_max_rows(self._ctx, C.byref(n)))
        return n.value

    def denoise_static(self, steps, y, slots=None):
        """asd_denoise_static: same arguments and result as denoise(), but the GEMM chain's scratch
        is the library's fixed 8 MiB array, so the call allocates no device memory (the output
        tensor is allocated here, by torch, before the call; pass `out=` style callers use the C ABI)."""
        torch = self._torch
        steps = torch.as_tensor(steps).to(device="cuda", dtype=torch.int32).contiguous()
        y = torch.as_tensor(y).to(device="cuda", dtype=torch.float32).contiguous()
        if slots is not None:
            slots = torch.as_tensor(slots).to(device="cuda", dtype=torch.int32).contiguous()
        out = torch.empty_like(y)
        self._check(self.lib.asd_denoise_static(self._ctx, y.shape[0], _dev_ptr(steps), _dev_ptr(y),
                                                _dev_ptr(slots), _dev_ptr(out)))
        return out
