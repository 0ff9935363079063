"""GPU parity tests proper: the CUDA library (through the C ABI) against the CPU oracle on the
same seeded inputs.  Tolerances: fp32 states 1e-4 relative L2 (1e-2 for the bf16 network),
accept decisions identical whenever |ln ratio - ln u| > 1e-3, prefix lengths bit-exact under
that margin."""
import math

import numpy as np
import pytest
import torch

import workloads
from oracle import asd as oasd
from oracle import denoisers as oden
from tests._parity import MARGIN, lockstep, oracle_run, rel_l2, tolerances

pytestmark = pytest.mark.gpu


def _sampler(wl, dump=True, **kw):
    """dump=True adds ASD_FLAG_DEBUG_DUMP (ln u / ln ratio per slot, which the lock-step comparison reads);
    the whole-run tests pass dump=False and so run exactly what asd_sample runs by default."""
    from paper_2505_03983_b200 import AsdSampler
    from paper_2505_03983_b200.binding import FLAG_DEBUG_DUMP
    if dump:
        kw["flags"] = kw.get("flags", 0) | FLAG_DEBUG_DUMP
    return AsdSampler(wl, **kw)


def _log(msg):
    print(msg)


# ------------------------------------------------------------------ drift alone
@pytest.mark.parametrize("name,n_rows", [("cfg1_gmm2d", 100), ("gmm_odd", 57), ("gauss_small", 50),
                                         ("cfg2_gauss64", 300), ("mlp_tiny", 23), ("mlp_odd", 19), ("mlp_odd", 300), ("mlp_ragged", 300),
                                         ("mlp_ragged", 1), ("mlp_ragged", 200), ("cfg3_policy", 17),
                                         ("cfg3_policy", 256), ("cfg3_policy", 400), ("cfg3_policy", 512), ("cfg3_policy", 700)])
def test_drift_matches_oracle(name, n_rows):
    wl = workloads.make(name)
    rng = np.random.default_rng(5)
    chains = wl.chains
    cap = max(chains, -(-n_rows // max(wl.window - 1, 1)))
    with _sampler(wl, max_chains=cap) as s:
        cond = None
        if wl.kind == "mlp" and wl.d_cond:
            cond = np.concatenate([wl.cond] * (-(-cap // chains)))[:cap]
            wl.cond = cond
        s.reset(cap, 0, cond=cond)
        steps = rng.integers(0, wl.K, n_rows).astype(np.int32)
        tt = wl.t[steps]
        xstar = rng.standard_normal((n_rows, wl.d))
        y = (tt[:, None] * xstar + np.sqrt(tt)[:, None] * rng.standard_normal((n_rows, wl.d))).astype(np.float32)
        slots = rng.integers(0, cap, n_rows).astype(np.int32)
        out = s.denoise(steps, y, slots).cpu().numpy()
    g = oden.from_workload(wl)
    tol = 2e-3 if wl.kind == "mlp" else 2e-5
    worst = 0.0
    for r in range(n_rows):
        ref = g(int(steps[r]), y[r].astype(np.float64), int(slots[r]))
        err = np.max(np.abs(out[r] - ref)) / max(1.0, np.max(np.abs(ref)))
        worst = max(worst, err)
    _log(f"drift {name} rows={n_rows}: max scaled error {worst:.3e}")
    assert worst < tol


def test_drift_large_row_count_sampled_rows():
    """Row counts at which the CTA-pair GEMM kernel (256 x 256 tiles over two SMs) is selected,
    with a ragged last tile; the oracle is evaluated on a sample of the rows (rows are independent)."""
    wl = workloads.make("cfg3_policy")
    n_rows, cap = 37 * 256 + 77, 700                 # 9549 rows <= 700 chains x 15 slots
    rng = np.random.default_rng(11)
    wl.cond = rng.standard_normal((cap, wl.d_cond)).astype(np.float32)
    with _sampler(wl, max_chains=cap) as s:
        s.reset(cap, 0, cond=wl.cond)
        steps = rng.integers(0, wl.K, n_rows).astype(np.int32)
        tt = wl.t[steps]
        y = (tt[:, None] * rng.standard_normal((n_rows, wl.d)) +
             np.sqrt(tt)[:, None] * rng.standard_normal((n_rows, wl.d))).astype(np.float32)
        slots = rng.integers(0, cap, n_rows).astype(np.int32)
        out = s.denoise(steps, y, slots).cpu().numpy()
    assert np.isfinite(out).all()
    g = oden.from_workload(wl)
    sample = np.unique(np.concatenate([np.arange(0, 300), rng.integers(0, n_rows, 300),
                                       np.arange(n_rows - 200, n_rows), [127, 128, 255, 256, 9471, 9472]]))
    worst = 0.0
    for r in sample:
        ref = g(int(steps[r]), y[r].astype(np.float64), int(slots[r]))
        worst = max(worst, np.max(np.abs(out[r] - ref)) / max(1.0, np.max(np.abs(ref))))
    _log(f"drift cfg3_policy rows={n_rows} (sampled {len(sample)}): max scaled error {worst:.3e}")
    assert worst < 2e-3


@pytest.mark.parametrize("n_layers", [0, 1])
@pytest.mark.parametrize("n_rows,window,chains", [(32256, 64, 512), (32256 - 179, 64, 512), (992, 32, 32), (32, 32, 32)])
def test_drift_cfg4_shapes_without_cascade(n_rows, window, chains, n_layers):
    """The cfg-4 contractions (input 3328 -> 4096 over 52 k-blocks, 4096 -> 4096 over 64 k-blocks, 4096 -> 3072)
    with no or one residual layer, where no rounding cascade can build up, at the row counts of the bench's
    launches: 32256 rows (CTA-pair kernel, 256-wide tiles, several tiles per pair; and a ragged count), 992 rows
    (one tile per pair) and 32 rows (weight-streaming kernel, k split over four CTAs).  Compared on sampled rows
    on the network branch n = g - c_skip y itself, relative to |n| per row, so that the comparison does not
    lean on the skip term: a wrong k-block phase or a misplaced tile changes n by its own size."""
    wl = workloads.make("cfg4_image", n_layers=n_layers, window=window, chains=chains)
    rng = np.random.default_rng(17 + n_layers)
    with _sampler(wl, dump=False) as s:
        s.reset(chains, 0)
        steps = rng.integers(0, wl.K, n_rows).astype(np.int32)
        steps[:3] = [0, 1, wl.K - 1]
        tt = wl.t[steps]
        y = (tt[:, None] * rng.standard_normal((n_rows, wl.d), dtype=np.float32) +
             np.sqrt(tt)[:, None] * rng.standard_normal((n_rows, wl.d), dtype=np.float32)).astype(np.float32)
        out = s.denoise(steps, y).cpu().numpy().astype(np.float64)
    assert np.isfinite(out).all()
    edges = [0, 1, 2, 127, 128, 255, 256, 257, n_rows // 2, n_rows - 257, n_rows - 256, n_rows - 129, n_rows - 128,
             n_rows - 2, n_rows - 1]
    sample = np.unique(np.clip(np.concatenate([edges, rng.integers(0, n_rows, 160)]), 0, n_rows - 1))
    g = oden.from_workload(wl)
    ref = g.batch(list(steps[sample]), y[sample].astype(np.float64), 0)
    skip = wl.c_skip[steps[sample]].astype(np.float64)[:, None] * y[sample]
    branch = ref - skip
    rel = np.linalg.norm(out[sample] - ref, axis=1) / np.linalg.norm(branch, axis=1)
    _log(f"drift cfg4 shapes, {n_layers} residual layer(s), rows={n_rows} (sampled {len(sample)}): "
         f"max |out - ref| / |network branch| {rel.max():.3e}")
    assert rel.max() < 2e-3


def test_drift_cfg4_network_rows():
    """The 6-layer, width-4096 network on a handful of rows.  Its hidden states are rounded to bf16
    after every layer, and two accumulation orders end up rounding most hidden units independently
    (one flipped rounding perturbs every pre-activation of the next layer), so the network branch
    n = g - c_skip y agrees only to bf16 resolution: bound 2^-7 |n| in L2 per row."""
    wl = workloads.make("cfg4_image")
    rng = np.random.default_rng(3)
    n_rows = 40
    with _sampler(wl, max_chains=8) as s:
        s.reset(8, 0)
        steps = rng.integers(0, wl.K, n_rows).astype(np.int32)
        steps[:3] = [0, 1, wl.K - 1]
        tt = wl.t[steps]
        y = (tt[:, None] * rng.standard_normal((n_rows, wl.d)) +
             np.sqrt(tt)[:, None] * rng.standard_normal((n_rows, wl.d))).astype(np.float32)
        out = s.denoise(steps, y).cpu().numpy().astype(np.float64)
    g = oden.from_workload(wl)
    ref = g.batch(list(steps), y.astype(np.float64), 0)
    branch = ref - wl.c_skip[steps].astype(np.float64)[:, None] * y
    rel = np.linalg.norm(out - ref, axis=1) / np.linalg.norm(branch, axis=1)
    _log(f"drift cfg4_image rows={n_rows}: max |out - ref| / |network branch| {rel.max():.3e}")
    assert rel.max() < 2.0 ** -7

@pytest.mark.parametrize("name,check,rounds,cascade", [("cfg2_gauss64", [0, 100, 255], 6, False),
                                                       ("cfg4_image", [0, 13, 31], 3, True)])
def test_lockstep_full_size_configs_sampled_chains(name, check, rounds, cascade):
    """cfg2 (256 chains) and cfg4 (32 chains x window 32, the 6-layer width-4096 network) at their full
    batch sizes; the oracle re-runs a sample of the chains."""
    wl = workloads.make(name)
    with _sampler(wl) as s:
        worst = lockstep(s, wl, wl.chains, rounds, check_chains=check, log=_log, cascade=cascade)
    assert worst["decided"] > 0


def test_lockstep_cfg4_whole_run_sampled_rounds():
    """cfg4 to the end of the run: every 25th round and the round in which the last chain finishes, on
    four chains (the first rounds of all sampled chains are covered above)."""
    wl = workloads.make("cfg4_image")
    with _sampler(wl) as s:
        worst = lockstep(s, wl, wl.chains, 10 ** 6, check_chains=[0, 7, 13, 31], log=_log, cascade=True,
                         check_rounds=lambda r, st: r % 25 == 24 or st.n_active_after == 0)
        a, _, rounds = [t.cpu().numpy() for t in s.get_state()]
    assert np.all(a == wl.K) and worst["rounds"] >= 5 and worst["decided"] > 0
    assert math.ceil(wl.K / wl.window) <= rounds.min() and rounds.max() <= math.ceil(wl.K / 2)


def test_lockstep_bench_workload_sampled_chains():
    """The bench's own launch configuration (cfg-4 network, 512 chains x window 64: 32256 drafted rows
    per round) through a whole run; in seven rounds spread over it (the first two, every 25th, the one in
    which the last chain finishes) the oracle re-runs 16 chains from the GPU's state.  Decisions whose margin
    is inside the reproducibility bound of this network (tests/test_bf16_cascade_cpu.py) are exempt; their
    share is bounded."""
    wl = workloads.make("sweep_b512_w64")
    chains = [0, 1, 37, 64, 100, 127, 128, 200, 255, 256, 300, 383, 384, 450, 510, 511]
    with _sampler(wl) as s:
        worst = lockstep(s, wl, wl.chains, 10 ** 6, chain_base=0, check_chains=chains, log=_log, cascade=True,
                         check_rounds=lambda r, st: r < 2 or r % 25 == 24 or st.n_active_after == 0)
        a, _, rounds = [t.cpu().numpy() for t in s.get_state()]
    assert np.all(a == wl.K) and worst["rounds"] >= 6
    total = worst["decided"] + worst["exempt"]
    _log(f"bench workload: {worst['decided']} decisions compared bit-exactly, {worst['exempt']} exempt of {total}")
    assert total >= 6 * len(chains) // 2 and worst["exempt"] <= 0.4 * total

# ------------------------------------------------------------------ lock-step rounds
@pytest.mark.parametrize("all_slots", [False, True])
@pytest.mark.parametrize("name,chains,rounds", [
    ("cfg1_gmm2d", 16, 60), ("gmm_odd", 9, 30), ("gmm_wide", 3, 6), ("gmm_max_d", 2, 4), ("gauss_small", 11, 40), ("cfg2_gauss64", 24, 12),
    ("mlp_tiny", 5, 25), ("mlp_odd", 7, 12), ("mlp_ragged", 37, 8), ("cfg3_policy", 64, 3)])
def test_lockstep_rounds(name, chains, rounds, all_slots):
    """all_slots=False is the production path (the verify kernel stops at the first rejected slot);
    all_slots=True makes it evaluate the whole window so every ln ratio is compared."""
    from paper_2505_03983_b200.binding import FLAG_DEBUG_ALL_SLOTS
    wl = workloads.make(name, chains=chains)
    with _sampler(wl, flags=FLAG_DEBUG_ALL_SLOTS if all_slots else 0) as s:
        worst = lockstep(s, wl, chains, rounds, chain_base=1000, cond=wl.cond if wl.kind == "mlp" and wl.d_cond else None,
                         log=_log, all_slots=all_slots)
    assert worst["decided"] > 0


@pytest.mark.parametrize("name,chains,rounds,window", [("cfg1_gmm2d", 16, 40, 32), ("cfg2_gauss64", 24, 25, 64),
                                                       ("mlp_ragged", 20, 10, 24), ("cfg3_policy", 32, 4, 64)])
def test_lockstep_adaptive_window(name, chains, rounds, window):
    """ASD_FLAG_ADAPTIVE_WINDOW: every chain drafts with its own speculation length; the oracle is run
    with that length, and the integer rule that updates it is checked against the oracle's."""
    from paper_2505_03983_b200.binding import FLAG_ADAPTIVE_WINDOW
    wl = workloads.make(name, chains=chains, window=window)
    with _sampler(wl, flags=FLAG_ADAPTIVE_WINDOW) as s:
        worst = lockstep(s, wl, chains, rounds, chain_base=500, cond=wl.cond if wl.kind == "mlp" and wl.d_cond else None,
                         log=_log, adaptive=True)
        s.reset(chains, 500, cond=wl.cond if wl.kind == "mlp" and wl.d_cond else None)
        w, e = s.get_window_state()
        assert torch.all(w == min(window, 8)) and torch.all(e == 32)
    assert worst["decided"] > 0


def test_adaptive_window_whole_run_and_invariance():
    """Whole runs with per-chain adaptive windows: chains whose every decision is outside the margin end
    where the oracle's adaptive run ends, a chain's result does not depend on its batch, and the
    sequential sampler is unaffected by the flag."""
    from paper_2505_03983_b200.binding import FLAG_ADAPTIVE_WINDOW
    wl = workloads.make("cfg2_gauss64", chains=16, K=300, window=64)
    with _sampler(wl, flags=FLAG_ADAPTIVE_WINDOW) as s:
        s.reset(16, 40)
        y, rounds, st = s.sample()
        s.reset(3, 45)
        y_part, r_part, _ = s.sample()
        s.reset(16, 40)
        y_seq, _ = s.sequential_ddpm()
    with _sampler(wl) as s0:
        s0.reset(16, 40)
        y_seq0, _ = s0.sequential_ddpm()
        s0.reset(16, 40)
        _, rounds_fixed, _ = s0.sample()
    assert torch.equal(y[5:8], y_part) and torch.equal(rounds[5:8], r_part)
    assert torch.equal(y_seq, y_seq0)
    g, sch = oden.from_workload(wl), oasd.make_schedule(wl.t)
    y, rounds = y.cpu().numpy(), rounds.cpu().numpy()
    compared = 0
    for j in range(16):
        res = oasd.asd_sample(g, sch, wl.seed, 40 + j, j, 64, d=wl.d, adaptive=True)
        if res.min_margin > MARGIN:
            compared += 1
            assert rounds[j] == res.rounds
            assert rel_l2(y[j].astype(np.float64), res.y) < 1e-4
    _log(f"adaptive cfg2 K=300: rounds mean {rounds.mean():.1f} (fixed window 64: {rounds_fixed.float().mean():.1f}), "
         f"drift rows {st.rows_total}, compared {compared}")
    assert compared >= 3


@pytest.mark.parametrize("adaptive", [False, True])
@pytest.mark.parametrize("name,chains,rounds", [("cfg1_gmm2d", 16, 40), ("gmm_odd", 9, 30), ("cfg2_gauss64", 24, 12),
                                                ("mlp_tiny", 5, 25), ("mlp_ragged", 37, 8), ("cfg3_policy", 64, 3)])
def test_lockstep_lookahead(name, chains, rounds, adaptive):
    """ASD_FLAG_LOOKAHEAD: the batched pass also evaluates the drift at the end of each window, and a
    chain that accepted its whole window skips the first model call of its next round.  Every round is
    still the oracle's round from the same state (the saved drift is the drift at that state), and the
    row counts of both passes follow the rule."""
    from paper_2505_03983_b200.binding import FLAG_ADAPTIVE_WINDOW, FLAG_LOOKAHEAD
    wl = workloads.make(name, chains=chains)
    with _sampler(wl, flags=FLAG_LOOKAHEAD | (FLAG_ADAPTIVE_WINDOW if adaptive else 0)) as s:
        worst = lockstep(s, wl, chains, rounds, chain_base=700, cond=wl.cond if wl.kind == "mlp" and wl.d_cond else None,
                         log=_log, adaptive=adaptive, lookahead=True)
    assert worst["decided"] > 0


@pytest.mark.parametrize("name,chains,K", [("cfg1_gmm2d", 33, None), ("cfg2_gauss64", 16, 300), ("gmm_wide", 3, None)])
def test_lookahead_whole_run_equals_default(name, chains, K):
    """The analytic drifts are computed row by row, so moving an evaluation into the previous round's
    batch changes no bit: whole runs with and without look-ahead give the same samples in the same number
    of rounds with fewer sequential model calls, and so does the sequential sampler."""
    from paper_2505_03983_b200.binding import FLAG_LOOKAHEAD
    wl = workloads.make(name, chains=chains) if K is None else workloads.make(name, chains=chains, K=K)
    with _sampler(wl) as s0:
        s0.reset(chains, 11)
        y0, r0, st0 = s0.sample()
        s0.reset(chains, 11)
        q0, _ = s0.sequential_ddpm()
    with _sampler(wl, flags=FLAG_LOOKAHEAD) as s1:
        s1.reset(chains, 11)
        y1, r1, st1 = s1.sample()
        s1.reset(chains, 11)
        q1, sq = s1.sequential_ddpm()
        # a restart after a partial run must not reuse a stale drift
        s1.reset(chains, 11)
        for _ in range(3):
            s1.round(want_stats=False)
        s1.reset(chains, 11)
        y2, r2, _ = s1.sample()
    assert torch.equal(y0, y1) and torch.equal(r0, r1)
    assert torch.equal(y0, y2) and torch.equal(r0, r2)
    assert torch.equal(q0, q1)
    assert sq.rows_total == chains * wl.K          # one drift evaluation per step, as without the flag
    _log(f"look-ahead {name}: drift rows {st0.rows_total} -> {st1.rows_total}, rounds mean {r0.float().mean():.1f}")


@pytest.mark.parametrize("K,window,chains", [(1, 1, 3), (2, 2, 1), (5, 8, 2), (7, 3, 4)])
def test_lookahead_short_chains(K, window, chains):
    """Look-ahead at the ends of its range: a single step (nothing to look ahead to), windows that reach or pass
    the last step (no extra row is drafted there), one chain; with adaptive windows on top."""
    from paper_2505_03983_b200.binding import FLAG_ADAPTIVE_WINDOW, FLAG_LOOKAHEAD
    for name in ("cfg1_gmm2d", "mlp_tiny"):
        wl = workloads.make(name, K=K, window=window, chains=chains)
        cond = wl.cond if wl.kind == "mlp" and wl.d_cond else None
        # (per-chain windows range over 2..window: nothing to adapt for a window of one step)
        for flags in (FLAG_LOOKAHEAD,) + ((FLAG_LOOKAHEAD | FLAG_ADAPTIVE_WINDOW,) if window >= 2 else ()):
            with _sampler(wl, flags=flags) as s:
                lockstep(s, wl, chains, K + 1, chain_base=3, cond=cond, log=None,
                         adaptive=bool(flags & FLAG_ADAPTIVE_WINDOW), lookahead=True)
                a, _, rounds = [t.cpu().numpy() for t in s.get_state()]
                assert np.all(a == K) and np.all(rounds >= 1)
                s.reset(chains, 3, cond=cond)
                y, r, _ = s.sample()
                assert torch.isfinite(y).all() and torch.all(r >= math.ceil(K / max(window, 2)) if K > 1 else r == 1)


def test_lookahead_network_whole_run():
    """Network denoiser: the saved drift comes out of a different GEMM batch, so whole runs agree with the
    oracle's (not bit for bit with the default mode) on chains whose every decision is well outside the
    ln-ratio tolerance of the bf16 network."""
    from paper_2505_03983_b200.binding import FLAG_LOOKAHEAD
    wl = workloads.make("mlp_tiny", chains=24)
    with _sampler(wl, flags=FLAG_LOOKAHEAD) as s:
        s.reset(24, 0, cond=wl.cond)
        y, rounds, st = s.sample()
    with _sampler(wl) as s0:
        s0.reset(24, 0, cond=wl.cond)
        _, _, st0 = s0.sample()
    ref = oracle_run(wl, range(24))
    y, rounds = y.cpu().numpy(), rounds.cpu().numpy()
    tol_y, _ = tolerances(wl.kind)
    compared = 0
    for j, res in enumerate(ref):
        if res.min_margin > 1e-2:
            compared += 1
            assert rounds[j] == res.rounds, (j, rounds[j], res.rounds)
            assert rel_l2(y[j].astype(np.float64), res.y) < tol_y
    _log(f"look-ahead mlp_tiny: compared {compared} of 24, drift rows {st0.rows_total} -> {st.rows_total}")
    assert compared >= 10


@pytest.mark.parametrize("mapping,pred", [("sl", "eps"), ("ancestral", "eps"), ("ancestral", "v")])
def test_ddpm_front_end_chain(mapping, pred):
    """A chain built by asd_ddpm_schedule (non-uniform steps, explicit variances in the ancestral
    mapping, c_skip / c_out of an eps- or v-prediction network) started from noise: lock-step rounds
    and the sequential sampler against the oracle run with the oracle's own copy of the mapping."""
    import torch as th
    from oracle import ddpm as oddpm
    from paper_2505_03983_b200 import ddpm_schedule
    wl = workloads.make("mlp_tiny", K=40, window=8, chains=6)
    u = np.linspace(0.0, 1.0, wl.K + 1)
    ab = 2e-3 + (0.99 - 2e-3) * np.sin(0.5 * np.pi * u) ** 2
    ours, ref = ddpm_schedule(ab, pred, mapping), oddpm.ddpm_schedule(ab, pred, mapping)
    rng = np.random.default_rng(2)
    y0 = (rng.standard_normal((6, wl.d)) / ours["x_scale"][0]).astype(np.float32)
    wl.t, wl.c_in, wl.c_skip, wl.c_out = ours["t"], ours["c_in"], ours["c_skip"], ours["c_out"]
    with _sampler(wl, sigma2=ours["sigma2"]) as s:
        wl.t, wl.c_in, wl.c_skip, wl.c_out = ref["t"], ref["c_in"], ref["c_skip"], ref["c_out"]   # the oracle's copy
        worst = lockstep(s, wl, 6, 12, chain_base=9, cond=wl.cond, log=_log, sigma2=ref["sigma2"],
                         y0=th.as_tensor(y0, device="cuda"))
        s.reset(6, 9, cond=wl.cond, y0=th.as_tensor(y0, device="cuda"))
        y_seq, _ = s.sequential_ddpm()
    assert worst["decided"] > 0
    g, sch = oden.from_workload(wl), oasd.make_schedule(ref["t"], ref["sigma2"])
    for j in range(6):
        yr = oasd.sequential_ddpm(g, sch, wl.seed, 9 + j, j, y0=y0[j].astype(np.float64))
        assert rel_l2(y_seq[j].cpu().numpy().astype(np.float64), yr) < 5e-2


@pytest.mark.parametrize("name,chains,window", [("mlp_ragged", 37, 12), ("mlp_ragged", 2, 12), ("mlp_ragged", 3, 4),
                                                ("mlp_tiny", 5, 6), ("cfg3_policy", 64, 16)])
@pytest.mark.parametrize("graphs", ["1", "0"])
def test_staggered_lanes_equal_plain_rounds(name, chains, window, graphs, monkeypatch):
    """asd_sample as two half-batches half a round apart (one GEMM pass serves the first model call of
    one and the second of the other) must give every chain the state and the round count of the plain
    schedule, bit for bit: per chain nothing changes.  Both with CUDA-graph replay and without.
    The GEMM kernel family is pinned for the comparison: the two schedules present different row counts
    to the GEMM planner, and the skinny kernel (k split over four CTAs) sums in another order than the
    tiled ones."""
    monkeypatch.setenv("ASD_GEMM_MODE", "cta" if chains % 2 else "pair")
    wl = workloads.make(name, chains=chains, window=window)
    cond = wl.cond if wl.d_cond else None
    out = {}
    monkeypatch.setenv("ASD_GRAPHS", graphs)
    for mode in ("0", "1"):
        monkeypatch.setenv("ASD_STAGGER", mode)
        with _sampler(wl, dump=False) as s:
            s.reset(chains, 77, cond=cond)
            y, r, st = s.sample()
            s.reset(chains, 77, cond=cond)           # a second run on the same context
            y2, r2, st2 = s.sample()
        assert torch.equal(y, y2) and torch.equal(r, r2) and st.rows_total == st2.rows_total
        out[mode] = (y, r, st)
    (y0, r0, st0), (y1, r1, st1) = out["0"], out["1"]
    assert torch.equal(r0, r1)
    assert torch.equal(y0, y1)
    assert st0.rows_total == st1.rows_total and st0.rows_verified == st1.rows_verified
    assert st0.rounds_mean == st1.rounds_mean and torch.isfinite(y1).all()


@pytest.mark.parametrize("case", range(12))
def test_lockstep_random_small_shapes(case):
    """Seeded random shapes (dimension, grid length, window, batch, network sizes) of all three drift kinds,
    a few lock-step rounds each, with and without per-chain adaptive windows."""
    from paper_2505_03983_b200.binding import FLAG_ADAPTIVE_WINDOW
    rng = np.random.default_rng(1000 + case)
    kind = ("gmm", "gauss", "mlp")[case % 3]
    K, window, chains = int(rng.integers(3, 70)), int(rng.integers(2, 65)), int(rng.integers(1, 40))
    if kind == "gmm":
        wl = workloads._gmm(f"rand{case}", int(rng.integers(1, 300)), int(rng.integers(1, 6)), 0.4, K, window, chains,
                            case, box=1.0)
    elif kind == "gauss":
        wl = workloads._gauss(f"rand{case}", int(rng.integers(1, 90)), K, window, chains, case)
    else:
        wl = workloads._mlp(f"rand{case}", int(rng.integers(1, 200)), int(rng.integers(0, 20)), 2 * int(rng.integers(0, 20)),
                            8 * int(rng.integers(1, 40)), int(rng.integers(0, 4)), K, window, chains, case, bias_std=0.05)
    cond = wl.cond if wl.kind == "mlp" and wl.d_cond else None
    adaptive = bool(case & 1)
    with _sampler(wl, flags=FLAG_ADAPTIVE_WINDOW if adaptive else 0) as s:
        worst = lockstep(s, wl, chains, 6, chain_base=case * 100, cond=cond, log=_log, adaptive=adaptive)
        s.reset(chains, case * 100, cond=cond)
        y, r, st = s.sample()
    assert torch.isfinite(y).all() and int(r.min()) >= 1 and worst["rounds"] >= 1
    _log(f"random case {case}: {kind} d={wl.d} K={K} window={window} chains={chains} adaptive={adaptive} "
         f"rounds mean {st.rounds_mean:.1f}")


def test_lockstep_window_64_and_window_beyond_K():
    from paper_2505_03983_b200.binding import FLAG_DEBUG_ALL_SLOTS
    wl = workloads.make("gauss_small", K=70, window=64, chains=6)
    with _sampler(wl, flags=FLAG_DEBUG_ALL_SLOTS) as s:
        lockstep(s, wl, 6, 10, log=_log, all_slots=True)
    with _sampler(wl) as s:
        lockstep(s, wl, 6, 10, log=_log)
    wl = workloads.make("cfg1_gmm2d", K=20, window=64, chains=4)     # window > K acts like K
    with _sampler(wl) as s:
        assert s.window == 64
        wl.window = 20
        s.window = 20
        lockstep(s, wl, 4, 10, log=_log)


# ------------------------------------------------------------------ whole runs
@pytest.mark.parametrize("name,chains", [("cfg1_gmm2d", 16), ("gauss_small", 11), ("cfg2_gauss64", 16)])
def test_free_running_matches_oracle(name, chains):
    wl = workloads.make(name, chains=chains)
    with _sampler(wl, dump=False) as s:
        s.reset(chains, 0)
        y, rounds, stats = s.sample()
        y, rounds = y.cpu().numpy(), rounds.cpu().numpy()
    ref = oracle_run(wl, range(chains))
    tol_y, _ = tolerances(wl.kind)
    compared = 0
    for j, res in enumerate(ref):
        if res.min_margin > MARGIN:        # every decision of this chain is outside the margin
            compared += 1
            assert rounds[j] == res.rounds, (j, rounds[j], res.rounds)
            assert rel_l2(y[j].astype(np.float64), res.y) < tol_y
    assert compared >= 3          # a K=1000 chain takes hundreds of decisions; few stay outside the margin throughout
    assert stats.rounds_max == rounds.max() and stats.rounds_mean == pytest.approx(rounds.mean())
    assert math.ceil(wl.K / wl.window) <= rounds.min() and rounds.max() <= math.ceil(wl.K / 2)
    assert stats.launches > 0


@pytest.mark.parametrize("name", ["cfg1_gmm2d", "gauss_small", "mlp_tiny"])
def test_sequential_matches_oracle_and_window_one(name):
    wl = workloads.make(name)
    cond = wl.cond if wl.kind == "mlp" and wl.d_cond else None
    n = wl.chains
    with _sampler(wl) as s:
        s.reset(n, 7, cond=cond)
        y_seq, st = s.sequential_ddpm()
        y_seq = y_seq.cpu().numpy()
        assert st.rows_total == n * wl.K
    with _sampler(wl, window=1) as s1:
        s1.reset(n, 7, cond=cond)
        y_w1, r_w1, _ = s1.sample()
        assert torch.all(r_w1 == wl.K)
        assert np.array_equal(y_w1.cpu().numpy(), y_seq)          # bit for bit
    ref = oracle_run(wl, range(7, 7 + n), slots=list(range(n)), sequential=True)
    tol_y = 5e-2 if wl.kind == "mlp" else 1e-4    # free-running through a random network amplifies rounding;
    for j in range(n):                              # step by step the network path is held to 1e-2 (window-1 lock-step)
        assert rel_l2(y_seq[j].astype(np.float64), ref[j]) < tol_y


def test_batch_and_partition_invariance():
    """A chain's result depends only on its id: alone, inside a batch, or in a shifted partition."""
    wl = workloads.make("cfg2_gauss64", chains=12, K=200)
    with _sampler(wl, dump=False) as s:
        s.reset(12, 100)
        y_all, r_all, _ = s.sample()
        s.reset(5, 104)
        y_part, r_part, _ = s.sample()
        s.reset(1, 107)
        y_one, r_one, _ = s.sample()
    assert torch.equal(y_all[4:9], y_part) and torch.equal(r_all[4:9], r_part)
    assert torch.equal(y_all[7:8], y_one) and torch.equal(r_all[7:8], r_one)


def test_state_save_restore_and_y0():
    wl = workloads.make("gauss_small", chains=8)
    with _sampler(wl) as s:
        s.reset(8, 3)
        y_ref, r_ref, _ = s.sample()
        s.reset(8, 3)
        for _ in range(5):
            s.round(want_stats=False)
        a, y, r = s.get_state()
    with _sampler(wl) as s2:
        s2.reset(8, 3)
        s2.set_state(a, y, r)
        y2, r2, _ = s2.sample()
    assert torch.equal(y2, y_ref) and torch.equal(r2, r_ref)
    # a non-zero starting point is honoured
    with _sampler(wl) as s3:
        y0 = torch.full((8, wl.d), 0.25, device="cuda")
        s3.reset(8, 3, y0=y0)
        s3.round()
        a3, y3, _ = s3.get_state()
    g, sch = oden.from_workload(wl), oasd.make_schedule(wl.t)
    rec = oasd.asd_round(g, sch, wl.seed, 3, 0, 0, np.full(wl.d, 0.25), wl.window)
    assert int(a3[0]) == rec.a_after and rel_l2(y3[0].cpu().numpy().astype(np.float64), rec.y_after) < 1e-4


def test_host_buffer_entry_point():
    wl = workloads.make("cfg1_gmm2d")
    with _sampler(wl) as s:
        s.reset(16, 0)
        y_dev, r_dev, _ = s.sample()
        y_h, r_h, st = s.sample_host(16, 0)
        assert np.array_equal(y_h, y_dev.cpu().numpy()) and np.array_equal(r_h, r_dev.cpu().numpy())
        y_s, _, _ = s.sample_host(16, 0, sequential=True)
        s.reset(16, 0)
        y_sd, _ = s.sequential_ddpm()
        assert np.array_equal(y_s, y_sd.cpu().numpy())


def test_empty_and_degenerate_inputs():
    from paper_2505_03983_b200 import AsdError
    wl = workloads.make("cfg1_gmm2d", K=1, window=1, chains=3)
    with _sampler(wl) as s:
        s.reset(0)
        y, r, st = s.sample()
        assert y.shape == (0, 2) and st.rounds_max == 0
        s.reset(3)
        y, r, _ = s.sample()
        assert torch.all(r == 1)
        with pytest.raises(AsdError):
            s.reset(4)                                   # beyond max_chains
    with pytest.raises(AsdError):
        _sampler(wl, window=0)
    with _sampler(wl, window=10 ** 6, dump=False) as s:      # far beyond K: acts like K
        s.reset(3)
        y2, r2, _ = s.sample()
        assert torch.equal(y2, y) and torch.equal(r2, r)
    with _sampler(wl, dump=False) as s:                      # the ln arrays are kept only on request
        s.reset(3)
        s.round()
        assert torch.all(s.accepted_last_round() == 1)
        with pytest.raises(AsdError):
            s.debug_last_round()
        with pytest.raises(AsdError):
            s.get_trajectory()
    bad = workloads.make("cfg1_gmm2d")
    bad.t = bad.t[::-1].copy()
    with pytest.raises(AsdError):
        _sampler(bad)


def test_degenerate_constant_drift_accepts_everything():
    """A drift that does not depend on the point (zero output weights, no skip) makes proposal and target
    means equal at every slot: ratio exactly 1, |delta|^2 = 0, every window accepted whole, so each chain
    needs exactly ceil(K / window) rounds and ends where the sequential sampler ends, bit for bit."""
    wl = workloads.make("mlp_tiny", K=37, window=6, chains=5)
    wl.W_out[:] = 0
    wl.c_skip[:] = 0
    wl.c_out[:] = 0.5                 # g = 0.5 b_out at every step and point
    with _sampler(wl) as s:
        s.reset(5, 3, cond=wl.cond)
        y, r, st = s.sample()
        s.reset(5, 3, cond=wl.cond)
        st1 = s.round()
        lr, lu, acc = s.debug_last_round()
        s.reset(5, 3, cond=wl.cond)
        y_seq, _ = s.sequential_ddpm()
    assert torch.all(r == math.ceil(37 / 6)) and st.rows_total == 5 * (6 * 6 + 1)
    assert torch.all(acc == 6) and st1.accepted_total == 30 and torch.all(lr == 0)
    assert torch.equal(y, y_seq)
    g, sch = oden.from_workload(wl), oasd.make_schedule(wl.t)
    res = oasd.asd_sample(g, sch, wl.seed, 3, 0, 6, d=wl.d)
    assert res.rounds == 7 and rel_l2(y[0].cpu().numpy().astype(np.float64), res.y) < 1e-5


def test_mixture_law_many_chains():
    """cfg-1 statistical check on the GPU: 65536 ASD chains against 65536 sequential chains (other chain
    ids) on the 8-component mixture - the two samplers have the same law (Theorem 3), compared per
    coordinate (two-sample KS) and by nearest-component occupancy (chi-square)."""
    from scipy import stats
    n = 65536
    wl = workloads.make("cfg1_gmm2d", chains=n)
    with _sampler(wl, dump=False) as s:
        s.reset(n, 0)
        ya, rounds, st = s.sample()
        s.reset(n, n)
        ys, _ = s.sequential_ddpm()
    ya, ys = ya.cpu().numpy().astype(np.float64), ys.cpu().numpy().astype(np.float64)
    _log(f"cfg1 n={n}: rounds mean {st.rounds_mean:.2f} max {st.rounds_max} of K={wl.K}")
    T = wl.t[-1]
    for j in range(2):
        assert stats.ks_2samp(ya[:, j], ys[:, j]).pvalue > 1e-3
    c = wl.means.astype(np.float64)
    lab = lambda y: np.bincount(np.argmin(((y[:, None, :] / T - c[None]) ** 2).sum(-1), axis=1), minlength=len(c))
    table = np.stack([lab(ya), lab(ys)])
    table = table[:, table.sum(0) >= 20]
    assert table.shape[1] >= 4 and stats.chi2_contingency(table)[1] > 1e-3
    # every mode keeps mass: y_K / T lands within 4 component std + the 1/sqrt(T) blur of some mean
    dist = np.sqrt(((ya[:, None, :] / T - c[None]) ** 2).sum(-1)).min(1)
    assert np.mean(dist < 4 * (wl.sigma + 1 / math.sqrt(T))) > 0.99


def test_bounded_wait_runs_out_and_context_survives():
    """Failure path: a wait that nothing completes gives up after its limit, the call reports
    ASD_ERR_TIMEOUT, and the same context then samples as before."""
    wl = workloads.make("mlp_tiny")
    with _sampler(wl) as s:
        s.reset(wl.chains, 0, cond=wl.cond)
        y0, r0, _ = s.sample()
        st = s.lib.asd_debug_wait_selftest(s._ctx)
        assert st == 6 and b"bounded" in s.lib.asd_last_error(s._ctx)        # ASD_ERR_TIMEOUT
        s.reset(wl.chains, 0, cond=wl.cond)
        y1, r1, _ = s.sample()
    assert torch.equal(y0, y1) and torch.equal(r0, r1)


def test_gaussian_target_moments_many_chains():
    """cfg-2 statistical check on the GPU: 16384 ASD chains and 16384 sequential chains against the
    closed-form law of the Euler chain (mean T mu0, eigen-variances (1+T lam)^2 sum eta/(1+t lam)^2)."""
    n = 16384
    wl = workloads.make("cfg2_gauss64", chains=n, K=250)
    Q, lam, mu0 = wl.Q.astype(np.float64), wl.lam.astype(np.float64), wl.mu0.astype(np.float64)
    T = wl.t[-1]
    eta = np.diff(wl.t)
    var = (1 + T * lam) ** 2 * np.sum(eta[:, None] / (1 + wl.t[1:, None] * lam[None, :]) ** 2, axis=0)
    with _sampler(wl, dump=False) as s:
        s.reset(n, 0)
        ya, rounds, st = s.sample()
        s.reset(n, n)
        ys, _ = s.sequential_ddpm()
    _log(f"cfg2 K=250 n={n}: rounds mean {st.rounds_mean:.1f} max {st.rounds_max}")
    for ysamp in (ya.cpu().numpy().astype(np.float64), ys.cpu().numpy().astype(np.float64)):
        z = (ysamp - T * mu0) @ Q                   # eigen-coordinates, independent with variance `var`
        assert np.all(np.abs(z.mean(0)) < 4.5 * np.sqrt(var / n))
        assert np.all(np.abs(z.var(0, ddof=1) - var) < 4.5 * var * math.sqrt(2 / (n - 1)))
        C = np.corrcoef(z.T)
        assert np.max(np.abs(C - np.eye(wl.d))) < 5.5 / math.sqrt(n)


# ------------------------------------------------------------------ sequential path step by step, last rounds
@pytest.mark.parametrize("name,chains", [("mlp_ragged", 37), ("cfg3_policy", 64)])
def test_lockstep_window_one_network(name, chains):
    """The sequential sampler's path (window 1: one model call and one Euler step per round, Eq. 7) on the
    network denoiser, every step of every chain against the oracle from the same state, at the 1e-2 of the
    bf16 configs (measured far below it); free-running comparisons through a random network only bound
    the accumulated effect."""
    wl = workloads.make(name, chains=chains, window=1)
    cond = wl.cond if wl.d_cond else None
    with _sampler(wl) as s:
        worst = lockstep(s, wl, chains, wl.K + 1, chain_base=21, cond=cond, log=_log)
        a, _, rounds = [t.cpu().numpy() for t in s.get_state()]
    assert np.all(a == wl.K) and np.all(rounds == wl.K) and worst["rounds"] == wl.K
    assert worst["y"] < 1e-2


def test_lockstep_cfg3_to_the_last_round():
    """cfg3 from the first round to the one in which the last chain finishes: the short windows at the end of
    the grid and the compaction of finished chains through the GEMM row map."""
    wl = workloads.make("cfg3_policy")
    with _sampler(wl) as s:
        worst = lockstep(s, wl, wl.chains, 10 ** 6, chain_base=5, cond=wl.cond, log=_log)
        a, _, rounds = [t.cpu().numpy() for t in s.get_state()]
    assert np.all(a == wl.K) and worst["rounds"] == rounds.max() and worst["decided"] > 0


# ------------------------------------------------------------------ trajectory, theta = infinity, histogram, streams
@pytest.mark.parametrize("name,chains", [("cfg1_gmm2d", 16), ("gauss_small", 11), ("mlp_tiny", 5)])
def test_trajectory_matches_oracle(name, chains):
    """ASD_FLAG_TRAJECTORY: Algorithm 1's return value (y_0 .. y_K).  Round by round, the rows a chain gained
    are the oracle's new states of that round (accepted proposal samples, then the resampled one); over a
    whole run the rows of well-separated chains are the oracle's trajectory, the last row is y_K bit for bit,
    and the sequential sampler fills the same buffer."""
    from paper_2505_03983_b200.binding import FLAG_TRAJECTORY
    wl = workloads.make(name, chains=chains)
    cond = wl.cond if wl.kind == "mlp" and wl.d_cond else None
    g, sch = oden.from_workload(wl), oasd.make_schedule(wl.t)
    tol_y, _ = tolerances(wl.kind)
    with _sampler(wl, flags=FLAG_TRAJECTORY) as s:
        s.reset(chains, 4, cond=cond)
        checked = 0
        for r in range(8):
            a0, y0, _ = [t.cpu().numpy() for t in s.get_state()]
            s.round()
            acc = s.accepted_last_round().cpu().numpy()
            a1, y1, _ = [t.cpu().numpy() for t in s.get_state()]
            traj = s.get_trajectory().cpu().numpy()
            for j in range(chains):
                assert np.array_equal(traj[j, a1[j]], y1[j]) and np.array_equal(traj[j, a0[j]], y0[j])
                rec = oasd.asd_round(g, sch, wl.seed, 4 + j, j, int(a0[j]), y0[j].astype(np.float64), wl.window)
                if acc[j] != rec.n:
                    continue
                for i, ref in enumerate(rec.new_states):
                    assert rel_l2(traj[j, a0[j] + 1 + i].astype(np.float64), ref) < tol_y
                    checked += 1
        assert checked > chains
        s.reset(chains, 4, cond=cond)
        y, rounds, _ = s.sample()
        traj = s.get_trajectory()
        assert torch.equal(traj[:, wl.K], y) and torch.all(traj[:, 0] == 0) and torch.isfinite(traj).all()
        s.reset(chains, 4, cond=cond)
        y_seq, _ = s.sequential_ddpm()
        traj_seq = s.get_trajectory().cpu().numpy()
        assert np.array_equal(traj_seq[:, wl.K], y_seq.cpu().numpy())
    traj = traj.cpu().numpy().astype(np.float64)
    if wl.kind != "mlp":
        compared = 0
        for j in range(chains):
            res = oasd.asd_sample(g, sch, wl.seed, 4 + j, j, wl.window, d=wl.d)
            if res.min_margin > MARGIN:
                compared += 1
                assert res.trajectory.shape == traj[j].shape
                assert np.max(np.linalg.norm(traj[j] - res.trajectory, axis=1) /
                              np.maximum(np.linalg.norm(res.trajectory, axis=1), 1.0)) < tol_y
            _, tr = oasd.sequential_ddpm(g, sch, wl.seed, 4 + j, j, d=wl.d, return_trajectory=True)
            assert np.max(np.linalg.norm(traj_seq[j] - tr, axis=1) / np.maximum(np.linalg.norm(tr, axis=1), 1.0)) < tol_y
        assert compared >= 2


@pytest.mark.parametrize("name,K,chains,rounds", [("cfg1_gmm2d", 100, 16, 40), ("cfg1_gmm2d", 1000, 6, 12),
                                                  ("gauss_small", 300, 5, 10), ("mlp_tiny", 40, 5, 20),
                                                  ("mlp_ragged", 150, 3, 6)])
def test_lockstep_window_infinity(name, K, chains, rounds):
    """theta = infinity: window = K, every round drafts to the end of the grid (up to 999 slots here), in
    production and all-slots mode; and a whole run."""
    from paper_2505_03983_b200.binding import FLAG_DEBUG_ALL_SLOTS
    wl = workloads.make(name, K=K, window=K, chains=chains)
    cond = wl.cond if wl.kind == "mlp" and wl.d_cond else None
    for flags in (0, FLAG_DEBUG_ALL_SLOTS):
        with _sampler(wl, flags=flags) as s:
            worst = lockstep(s, wl, chains, rounds, chain_base=300, cond=cond, log=_log, all_slots=bool(flags))
            assert worst["decided"] > 0
            s.reset(chains, 300, cond=cond)
            y, r, st = s.sample()
            assert torch.isfinite(y).all() and int(r.min()) >= 1 and int(r.max()) <= math.ceil(K / 2)
    if wl.kind != "mlp":
        ref = oracle_run(wl, range(300, 300 + chains), slots=list(range(chains)))
        y, r = y.cpu().numpy(), r.cpu().numpy()
        compared = 0
        for j, res in enumerate(ref):
            if res.min_margin > MARGIN:
                compared += 1
                assert r[j] == res.rounds and rel_l2(y[j].astype(np.float64), res.y) < 1e-4
        _log(f"theta = infinity {name} K={K}: rounds mean {r.mean():.1f}, compared {compared} whole runs")


def test_prefix_histogram_counts_every_chain_round():
    wl = workloads.make("cfg2_gauss64", chains=24, K=120)
    with _sampler(wl, dump=False) as s:
        s.reset(24, 2)
        counts = np.zeros(wl.window + 1, dtype=np.int64)
        while True:
            st = s.round()
            if st.n_active_before == 0:
                break
            acc = s.accepted_last_round().cpu().numpy()
            counts += np.bincount(acc[acc >= 0], minlength=wl.window + 1)
        hist = s.prefix_histogram()
        _, _, rounds = [t.cpu().numpy() for t in s.get_state()]
        assert np.array_equal(hist, counts) and hist.sum() == rounds.sum() and hist[0] == 0
        s.reset(24, 2)
        _, r, _ = s.sample()
        assert np.array_equal(s.prefix_histogram(), counts)          # same run, same histogram
        s.reset(24, 2)
        assert s.prefix_histogram().sum() == 0
        s.sequential_ddpm()
        h = s.prefix_histogram()
        assert h[1] == 24 * wl.K and h.sum() == h[1]


def test_context_created_on_a_busy_side_stream():
    """asd_create on a non-blocking stream that still has work queued: the tables and weights must be
    ordered with the clearing of their buffers on that stream (not copied through the default stream)."""
    wl = workloads.make("mlp_ragged")
    rng = np.random.default_rng(4)
    n_rows = 64
    steps = rng.integers(0, wl.K, n_rows).astype(np.int32)
    y = rng.standard_normal((n_rows, wl.d)).astype(np.float32) * (1 + wl.t[steps])[:, None].astype(np.float32)
    slots = rng.integers(0, wl.chains, n_rows).astype(np.int32)
    with _sampler(wl, dump=False) as s0:
        s0.reset(wl.chains, 0, cond=wl.cond)
        ref = s0.denoise(steps, y, slots)
        y_ref, r_ref, _ = s0.sample()
    side = torch.cuda.Stream()
    big = torch.empty(1 << 28, dtype=torch.float32, device="cuda")
    with torch.cuda.stream(side):
        for _ in range(100):                     # tens of milliseconds of queued work
            big.mul_(1.0001)
        with _sampler(wl, dump=False, stream=side) as s1:
            s1.reset(wl.chains, 0, cond=torch.as_tensor(wl.cond, device="cuda"))
            out = s1.denoise(steps, y, slots)
            y1, r1, _ = s1.sample()
            side.synchronize()
    torch.cuda.synchronize()
    assert torch.equal(out, ref) and torch.equal(y1, y_ref) and torch.equal(r1, r_ref)

# ------------------------------------------------------------------ chain-resident kernel (closed-form drifts)
@pytest.mark.parametrize("name,chains,kw", [("cfg1_gmm2d", 16, {}), ("cfg2_gauss64", 40, {"K": 300}), ("gmm_odd", 9, {}),
                                            ("gauss_small", 11, {}), ("cfg1_gmm2d", 7, {"K": 200, "window": 200}),
                                            ("gauss_small", 3, {"window": 1}), ("gauss_odd", 5, {})])
@pytest.mark.parametrize("flags", ["plain", "adaptive", "all_slots"])
def test_resident_kernel_equals_per_phase_kernels(name, chains, kw, flags, monkeypatch):
    """asd_sample / asd_sequential_ddpm on the closed-form drifts run Algorithm 1's while loop inside one launch
    (a block per chain).  Same expressions in the same order as the per-phase kernels, so with ASD_RESIDENT=0
    (per-phase kernels, rounds replayed as CUDA graphs) every chain ends in the same bits after the same
    rounds, with the same row statistics, prefix histogram and trajectory."""
    from paper_2505_03983_b200.binding import FLAG_ADAPTIVE_WINDOW, FLAG_DEBUG_ALL_SLOTS, FLAG_TRAJECTORY
    fl = FLAG_TRAJECTORY | {"plain": 0, "adaptive": FLAG_ADAPTIVE_WINDOW, "all_slots": FLAG_DEBUG_ALL_SLOTS}[flags]
    wl = workloads.make(name, chains=chains, **kw)
    out = {}
    for mode in ("0", "1"):
        monkeypatch.setenv("ASD_RESIDENT", mode)
        with _sampler(wl, dump=False, flags=fl) as s:
            s.reset(chains, 90)
            y, r, st = s.sample()
            hist, traj = s.prefix_histogram(), s.get_trajectory()
            wstate = s.get_window_state()
            s.reset(chains, 90)
            y_seq, st_seq = s.sequential_ddpm()
            # stop after a few rounds, resume to the end: the same chain state either way
            s.reset(chains, 90)
            for _ in range(3):
                s.round(want_stats=False)
            y_res, r_res, _ = s.sample()
        out[mode] = (y, r, st, hist, traj, wstate, y_seq, st_seq, y_res, r_res)
    (y0, r0, st0, h0, t0, w0, q0, sq0, yr0, rr0), (y1, r1, st1, h1, t1, w1, q1, sq1, yr1, rr1) = out["0"], out["1"]
    assert st1.launches <= 2 < st0.launches
    assert torch.equal(r0, r1) and torch.equal(y0, y1)
    assert st0.rows_total == st1.rows_total and st0.rows_verified == st1.rows_verified
    assert st0.rounds_max == st1.rounds_max and st0.rounds_mean == st1.rounds_mean
    assert np.array_equal(h0, h1) and torch.equal(t0, t1)
    assert torch.equal(w0[0], w1[0]) and torch.equal(w0[1], w1[1])
    assert torch.equal(q0, q1) and sq0.rows_total == sq1.rows_total == chains * wl.K
    assert torch.equal(yr0, yr1) and torch.equal(rr0, rr1) and torch.equal(yr1, y1)


@pytest.mark.parametrize("name,chains,rounds,kw", [("cfg1_gmm2d", 16, 60, {}), ("gmm_odd", 9, 30, {}), ("gauss_small", 11, 40, {}),
                                                   ("cfg2_gauss64", 24, 12, {}), ("cfg1_gmm2d", 5, 12, {"K": 300, "window": 300}),
                                                   ("gauss_odd", 5, 20, {})])
@pytest.mark.parametrize("adaptive", [False, True])
def test_lockstep_resident_kernel_rounds(name, chains, rounds, kw, adaptive, monkeypatch):
    """The chain-resident kernel limited to one round per launch (ASD_RESIDENT=2 routes asd_round through it),
    round by round against the oracle like the per-phase kernels."""
    from paper_2505_03983_b200.binding import FLAG_ADAPTIVE_WINDOW
    monkeypatch.setenv("ASD_RESIDENT", "2")
    wl = workloads.make(name, chains=chains, **kw)
    with _sampler(wl, flags=FLAG_ADAPTIVE_WINDOW if adaptive else 0) as s:
        worst = lockstep(s, wl, chains, rounds, chain_base=1000, log=_log, adaptive=adaptive)
        st = s.round()
        assert st.rows_pass1 == st.n_active_before
    assert worst["decided"] > 0


def test_trained_network_lockstep_and_rounds():
    """The cfg-1 problem with the small network that was fitted to its posterior mean (stored weights): lock-step
    parity, and over whole runs about as many rounds per sample as with the closed form itself (the acceptance
    behaviour of a true posterior mean, not of a random network).  This network carries the whole drift (c_out of
    order 1, trained weights of order 1), so it is as sensitive as a network can be to the bf16 rounding of its
    two inputs: the library's fp32 drafted point and the oracle's fp64 one differ by 1e-7 relative, which now and
    then rounds c_in y to the neighbouring bf16 value and moves the network branch by up to a few per cent
    (tests/test_bf16_cascade_cpu.py shows the mechanism on the CPU).  ln ratio is therefore compared at the
    bf16-resolution bound of tests/_parity.py and the share of exempt decisions is bounded."""
    wl = workloads.make("cfg1_trained", chains=64)
    with _sampler(wl) as s:
        worst = lockstep(s, wl, 64, 12, chain_base=50, log=_log, cascade=True)
        assert worst["exempt"] <= 0.25 * (worst["exempt"] + worst["decided"])
        s.reset(64, 50)
        y, r, st = s.sample()
    base = workloads.make("cfg1_gmm2d", chains=64)
    with _sampler(base, dump=False) as s0:
        s0.reset(64, 50)
        y0, r0, st0 = s0.sample()
    _log(f"rounds per sample: fitted network {st.rounds_mean:.2f}, closed form {st0.rounds_mean:.2f}")
    assert worst["decided"] > 0 and torch.isfinite(y).all()
    assert abs(st.rounds_mean - st0.rounds_mean) < 0.25 * st0.rounds_mean
    # most chains end in the same mixture component as with the closed form (same noise streams)
    T = base.t[-1]
    c = torch.as_tensor(base.means, device="cuda")
    lab = lambda yy: torch.argmin(((yy[:, None, :] / T - c[None]) ** 2).sum(-1), dim=1)
    assert (lab(y) == lab(y0)).float().mean() > 0.8


@pytest.mark.parametrize("name,chains,rounds", [("mlp_ragged", 37, 8), ("cfg3_policy", 64, 4), ("mlp_odd", 7, 6)])
def test_one_launch_network_kernel(name, chains, rounds, monkeypatch):
    """ASD_MLP_FUSED=1: the whole network in one launch (a cluster of CTAs per 128 rows, the layers chained by
    cluster barriers).  Off by default because it measured slower; kept correct: the drift against the oracle on
    row counts with ragged row blocks, and lock-step rounds."""
    monkeypatch.setenv("ASD_MLP_FUSED", "1")
    wl = workloads.make(name, chains=chains)
    cond = wl.cond if wl.d_cond else None
    rng = np.random.default_rng(2)
    g = oden.from_workload(wl)
    with _sampler(wl) as s:
        s.reset(chains, 0, cond=cond)
        cap = chains * (wl.window - 1)
        for n_rows in (1, min(130, cap), cap):
            steps = rng.integers(0, wl.K, n_rows).astype(np.int32)
            y = (wl.t[steps][:, None] * rng.standard_normal((n_rows, wl.d)) +
                 np.sqrt(wl.t[steps])[:, None] * rng.standard_normal((n_rows, wl.d))).astype(np.float32)
            slots = rng.integers(0, chains, n_rows).astype(np.int32)
            out = s.denoise(steps, y, slots).cpu().numpy()
            for r in np.unique(np.concatenate([[0, n_rows - 1, n_rows // 2], rng.integers(0, n_rows, 20)])):
                ref = g(int(steps[r]), y[r].astype(np.float64), int(slots[r]))
                assert np.max(np.abs(out[r] - ref)) / max(1.0, np.max(np.abs(ref))) < 2e-3
        worst = lockstep(s, wl, chains, rounds, chain_base=60, cond=cond, log=_log)
    assert worst["decided"] > 0


@pytest.mark.parametrize("name", ["cfg1_gmm2d", "mlp_tiny"])
def test_allocation_failure_is_reported_and_leaves_nothing_behind(name, monkeypatch):
    """Failure path of asd_create, injected on the host: the n-th device allocation of the context fails.  The call
    returns ASD_ERR_OOM with a message, frees what it had allocated, and the next context works as usual."""
    from paper_2505_03983_b200 import AsdError
    wl = workloads.make(name)
    cond = wl.cond if wl.kind == "mlp" and wl.d_cond else None
    with _sampler(wl, dump=False) as s:
        s.reset(wl.chains, 0, cond=cond)
        y_ref, r_ref, _ = s.sample()
    free0 = torch.cuda.mem_get_info()[0]
    for n in (0, 1, 4, 9, 17, 24):
        monkeypatch.setenv("ASD_FAIL_ALLOC_AFTER", str(n))
        with pytest.raises(AsdError) as e:
            _sampler(wl, dump=False)
        assert e.value.status == 3 and "allocation" in str(e.value)
    monkeypatch.delenv("ASD_FAIL_ALLOC_AFTER")
    assert torch.cuda.mem_get_info()[0] >= free0 - (8 << 20)          # nothing of the failed contexts is left
    with _sampler(wl, dump=False) as s:
        s.reset(wl.chains, 0, cond=cond)
        y, r, _ = s.sample()
    assert torch.equal(y, y_ref) and torch.equal(r, r_ref)


@pytest.mark.parametrize("name,chains", [("cfg1_gmm2d", 20), ("gauss_small", 11)])
def test_flag_combinations_give_the_same_chains(name, chains):
    """Closed-form drifts are computed point by point, so neither look-ahead reuse, nor keeping the trajectory, nor the
    diagnostics, nor which driver runs the loop (chain-resident kernel or per-phase kernels: look-ahead uses the
    latter) may change a bit of a chain: same samples, rounds, trajectory and prefix histogram for every combination,
    with fixed and with adaptive windows."""
    from paper_2505_03983_b200.binding import (FLAG_ADAPTIVE_WINDOW, FLAG_DEBUG_DUMP, FLAG_LOOKAHEAD, FLAG_TRAJECTORY)
    wl = workloads.make(name, chains=chains)
    for adaptive in (0, FLAG_ADAPTIVE_WINDOW):
        ref = None
        for extra in (0, FLAG_LOOKAHEAD, FLAG_DEBUG_DUMP, FLAG_LOOKAHEAD | FLAG_DEBUG_DUMP):
            with _sampler(wl, dump=False, flags=FLAG_TRAJECTORY | adaptive | extra) as s:
                s.reset(chains, 31)
                y, r, st = s.sample()
                got = (y, r, s.get_trajectory(), torch.as_tensor(s.prefix_histogram()))
            if ref is None:
                ref = got
            else:
                for a, b in zip(ref, got):
                    assert torch.equal(a, b), (adaptive, extra)
