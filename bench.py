#!/usr/bin/env python
"""Benchmark of the ASD hot path on B200.

A "step" is one pass of the whole hot path over one batch: reset the chains and run speculation
rounds (drift at the current points, draft, batched drift at the drafted points, verify,
advance) until every chain has reached step K.  The metric is samples per second.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Under torchrun (N > 1) every rank runs the same number of chains with its own chain ids
(weak scaling, no data-path collective); `value` is all ranks' samples over the max time.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads  # noqa: E402

DEFAULT_WORKLOAD = "sweep_b512_w64"   # cfg-4 denoiser, 512 chains x window 64, K = 1000 (largest cell)
# dram__bytes_read.sum + dram__bytes_write.sum of one pass-2 hidden-layer launch of gemm_pair_kernel<256, EPI_HID>
# at full row count, from one ncu capture of that kernel; set an entry to None when the kernel changes, until the
# counters are taken again
NCU_TRAFFIC_BYTES_PER_LAUNCH = {"sweep_b512_w64": 408_912_896 + 248_380_928}
METRIC = "samples_per_sec"
UNIT = "samples/s"


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        late = False
        if not self.rows:
            # a timed region shorter than nvidia-smi's first report: one query right after it instead
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10).stdout
                self.rows = [[x.strip() for x in line.split(",")] for line in out.splitlines() if line.strip()]
                late = True
            except (OSError, subprocess.SubprocessError):
                pass
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for nm, val in zip(names, r[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        res = dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                   reasons=sorted(reasons), samples=len(sm))
        if late:
            res["note"] = "sampled right after the timed region (it was shorter than the sampling interval)"
        return res


def oracle_sample_rate(wl, budget_s: float, max_rounds: int):
    """Runs the oracle's ASD chain after chain (at most `max_rounds` rounds each) until about
    `budget_s` seconds have passed, and returns (samples per second, with an unfinished chain counted
    by the fraction of its K steps, description)."""
    from oracle import asd as oasd, denoisers as oden
    g = oden.from_workload(wl)
    sch = oasd.make_schedule(wl.t)
    t0 = time.perf_counter()
    done, chains, rounds_total = 0.0, 0, 0
    while chains < wl.chains and (chains == 0 or time.perf_counter() - t0 < 0.5 * budget_s):
        y, a, rounds = np.zeros(wl.d), 0, 0
        slot = chains
        while a < wl.K and rounds < max_rounds and time.perf_counter() - t0 < budget_s:
            rec = oasd.asd_round(g, sch, wl.seed, slot, slot, a, y, wl.window)
            a, y, rounds = rec.a_after, rec.y_after, rounds + 1
        done += a / wl.K
        chains += 1
        rounds_total += rounds
    el = time.perf_counter() - t0
    return done / el, (f"chains 0..{chains - 1}, {rounds_total} rounds = {done:.2f} samples' worth of steps in {el:.1f} s "
                       f"(an unfinished chain counts by its fraction of the K steps)")


def blas_threads():
    try:
        import threadpoolctl
        info = threadpoolctl.threadpool_info()
        return max(int(i.get("num_threads", 1)) for i in info) if info else 1
    except Exception:
        return os.cpu_count() or 1


def oracle_rates(wl, budget_s):
    """The oracle as it stands on all host cores the BLAS uses, and limited to one thread."""
    rate, desc = oracle_sample_rate(wl, budget_s, 10 ** 9)
    out = {"value": rate, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": desc}
    try:
        import threadpoolctl
        with threadpoolctl.threadpool_limits(limits=1):
            r1, d1 = oracle_sample_rate(wl, 0.5 * budget_s, 10 ** 9)
        out["one_core"] = {"value": r1, "unit": UNIT, "cores": 1, "sample": d1}
    except Exception as e:  # pragma: no cover
        out["one_core"] = {"unavailable": repr(e)}
    return out


def compact_config(torch, AsdSampler, wl, peaks, steps=3):
    """One named configuration in brief, on the library's default path (no per-phase events): samples/s, rounds
    per sample, the sequential sampler on the same GPU, and - from a separate pass with the phase events on - the
    share of the time spent in the dominant kernel and its roofline fraction."""
    cond = torch.as_tensor(wl.cond, device="cuda") if wl.kind == "mlp" and wl.d_cond else None
    n = wl.chains
    out = {"chains": n, "K": wl.K, "window": wl.window, "d": wl.d}
    with AsdSampler(wl) as s:
        for _ in range(3):
            s.reset(n, 0, cond=cond); s.sample()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            s.reset(n, 0, cond=cond); _, _, st = s.sample()
        e1.record(); torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        out.update(samples_per_sec=n / (ms / 1e3), ms_per_step=ms, rounds_per_sample=st.rounds_mean,
                   K_over_rounds=wl.K / max(st.rounds_mean, 1e-9), drift_rows_per_sample_over_K=st.rows_total / (n * wl.K),
                   launches_per_step=st.launches)
        s.reset(n, 0, cond=cond); s.sequential_ddpm()
        s.reset(n, 0, cond=cond); _, sq = s.sequential_ddpm()
        out["sequential_gpu_samples_per_sec"] = n / (sq.ms_total / 1e3)
        out["wallclock_speedup_asd"] = sq.ms_total / ms
        s.set_profiling(True)
        s.reset(n, 0, cond=cond); _, _, stp = s.sample()
        prof = s.get_profile()
        s.set_profiling(False)
    total = sum(v["ms"] for v in prof.values()) or 1.0
    if wl.kind == "mlp":
        hid = prof["pass2_gemm_hidden"]
        flops = 2.0 * wl.width * wl.width * hid["rows"] * wl.n_layers
        tf = flops / (hid["ms"] / 1e3) / 1e12 if hid["ms"] > 0 else 0.0
        rows_per_launch = hid["rows"] * wl.n_layers / max(hid["launches"], 1)
        out["dominant_kernel"] = {"phase": "pass2_gemm_hidden", "share_of_phase_time": hid["ms"] / total,
                                  "rows_per_launch": rows_per_launch, "tflops": tf,
                                  "frac_of_sustained_bf16": tf / peaks["bf16_tflops_sustained"],
                                  "weight_stream_gbs": 2.0 * wl.width * wl.width * hid["launches"] / (hid["ms"] / 1e3) / 1e9
                                  if hid["ms"] > 0 else 0.0}
    else:
        name, v = max(prof.items(), key=lambda kv: kv[1]["ms"])
        out["dominant_kernel"] = {"phase": name, "share_of_phase_time": v["ms"] / total,
                                  "note": "per-phase kernels (the timed default path is the chain-resident kernel: "
                                          "one launch per run, latency-bound on a few thousand flops per slot)"}
    return out


def config_of(wl):
    return {"workload": wl.name, "chains_per_gpu": wl.chains, "K": wl.K, "window": wl.window, "d": wl.d,
            "denoiser": wl.kind, "width": wl.width, "layers": wl.n_layers,
            "l2": "working set (weights + activations) larger than L2, no flush needed"
                  if wl.kind == "mlp" and wl.width >= 4096 else "small working set; L2-resident by design"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = workloads.make(args.workload)
    cores = blas_threads()
    for _ in range(args.warmup):
        oracle_sample_rate(wl, 2.0, 1)
    t0 = time.perf_counter()
    rates, desc = [], ""
    for _ in range(args.steps):
        r, desc = oracle_sample_rate(wl, 10.0, 20)
        rates.append(r)
    el = time.perf_counter() - t0
    value = float(np.mean(rates))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * el / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(wl),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "each step: " + desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_ours(args):
    import torch
    from paper_2505_03983_b200 import AsdSampler

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    wl = workloads.make(args.workload)
    n = wl.chains
    base = rank * n                      # each rank owns its own chain ids: partition-invariant results
    cond = wl.cond if wl.kind == "mlp" and wl.d_cond else None
    peaks = read_peaks()
    s = AsdSampler(wl)
    cond_dev = None if cond is None else torch.as_tensor(cond, device="cuda")

    def step():
        s.reset(n, base, cond=cond_dev)
        return s.sample()

    for _ in range(max(args.warmup, 0)):
        step()
    # ---- timed region: device-resident inputs ------------------------------------------------
    # The network workloads are timed with the per-phase events on (the roofline of the dominant kernel is taken
    # over exactly this region).  The closed-form workloads are timed on the library's default path, the
    # chain-resident kernel, which has no phases; their per-phase kernels are timed in the second region below.
    phases_in_main = wl.kind == "mlp"
    s.set_profiling(phases_in_main)
    clocks = ClockSampler(local)
    barrier()
    clocks.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches, rounds_mean, rounds_max, rows, rows_ver = 0, [], [], 0, 0
    ev0.record()
    for _ in range(args.steps):
        y, r, st = step()
        launches += st.launches
        rounds_mean.append(st.rounds_mean); rounds_max.append(st.rounds_max); rows += st.rows_total
        rows_ver += st.rows_verified
    ev1.record()
    barrier()
    clk = clocks.stop()
    ms = ev0.elapsed_time(ev1)
    if phases_in_main:
        prof = s.get_profile()
    s.set_profiling(not phases_in_main)
    # ---- the same steps with the phase events the other way round (off for the network workloads: the events
    # cost a few microseconds per phase, which shows in the launch-bound workloads only; on for the closed-form
    # ones: the per-phase kernels instead of the chain-resident one) --------------------------------
    barrier()
    u0, u1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    u0.record()
    for _ in range(args.steps):
        step()
    u1.record()
    barrier()
    ms_plain = u0.elapsed_time(u1)
    if not phases_in_main:
        prof = s.get_profile()
    s.set_profiling(False)
    # ---- end to end through the host-buffer entry point -------------------------------------------
    y0_h = torch.zeros((n, wl.d), dtype=torch.float32).pin_memory().numpy()
    cond_h = None if cond is None else torch.as_tensor(cond).pin_memory().numpy()
    y_h = torch.empty((n, wl.d), dtype=torch.float32).pin_memory().numpy()
    r_h = torch.zeros((n,), dtype=torch.int32).pin_memory().numpy()
    s.sample_host(n, base, y0_h, cond_h, False, y_h, r_h)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        s.sample_host(n, base, y0_h, cond_h, False, y_h, r_h)
    e1.record()
    barrier()
    ms_e2e = e0.elapsed_time(e1)
    # ---- sequential DDPM (Eq. 7) on the same GPU, one run -------------------------------------------
    s.reset(n, base, cond=cond_dev)
    _, st_seq = s.sequential_ddpm()
    s.close()
    # ---- the verify kernel when it evaluates the whole window (Algorithm 2 as written) ---------------
    from paper_2505_03983_b200.binding import FLAG_ADAPTIVE_WINDOW, FLAG_DEBUG_ALL_SLOTS, FLAG_LOOKAHEAD
    sv = AsdSampler(wl, flags=FLAG_DEBUG_ALL_SLOTS)
    sv.reset(n, base, cond=cond_dev)
    for _ in range(2):
        sv.round(want_stats=False)
    sv.set_profiling(True)
    all_rows, all_chains = 0, 0
    for _ in range(6):
        st_r = sv.round()
        all_rows += st_r.rows_pass2; all_chains += st_r.n_active_before
    ver_all = sv.get_profile()["verify"]
    sv.close()
    def timed_variant(flags):
        """The same steps on a sampler created with `flags`: (ms, mean rounds per sample, drift rows)."""
        sx = AsdSampler(wl, flags=flags)
        for _ in range(2):
            sx.reset(n, base, cond=cond_dev)
            sx.sample()
        barrier()
        x0, x1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        x0.record()
        rnds, nrows = [], 0
        for _ in range(args.steps):
            sx.reset(n, base, cond=cond_dev)
            _, _, st_x = sx.sample()
            rnds.append(st_x.rounds_mean); nrows += st_x.rows_total
        x1.record()
        barrier()
        sx.close()
        return x0.elapsed_time(x1), float(np.mean(rnds)), nrows

    def phase_shares(flags):
        """One step on a sampler created with `flags` with the per-phase events on: {phase: share of the summed phase time}."""
        sx = AsdSampler(wl, flags=flags)
        sx.reset(n, base, cond=cond_dev); sx.sample()
        sx.set_profiling(True)
        sx.reset(n, base, cond=cond_dev); sx.sample()
        pr = sx.get_profile()
        sx.close()
        tot = sum(v["ms"] for v in pr.values()) or 1.0
        return {k: round(v["ms"] / tot, 4) for k, v in pr.items() if v["launches"]}

    ms_adapt, ad_rounds, ad_rows = timed_variant(FLAG_ADAPTIVE_WINDOW)
    ad_shares = phase_shares(FLAG_ADAPTIVE_WINDOW)
    ms_la, la_rounds, la_rows = timed_variant(FLAG_LOOKAHEAD)
    ms_ala, ala_rounds, ala_rows = timed_variant(FLAG_ADAPTIVE_WINDOW | FLAG_LOOKAHEAD)

    t = torch.tensor([ms, ms_e2e, st_seq.ms_total, ms_plain, ms_adapt, ms_la, ms_ala], dtype=torch.float64, device="cuda")
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms, ms_e2e, ms_seq, ms_plain, ms_adapt, ms_la, ms_ala = [float(x) for x in t.cpu()]
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    total = n * world * args.steps
    value = total / (ms / 1e3)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if wl.kind == "mlp" else "f32", "data": "synthetic",
        "config": config_of(wl),
        "rounds_per_sample": float(np.mean(rounds_mean)), "rounds_max": int(max(rounds_max)),
        "K_over_rounds": wl.K / float(np.mean(rounds_mean)),
        "drift_rows_per_sample_over_K": rows / (args.steps * n * wl.K),
        "verified_rows_over_drafted_rows": rows_ver / max(rows - args.steps * n * float(np.mean(rounds_mean)), 1.0),
        "gpu_launches": int(launches),
        "clocks": clk,
        "e2e": {"value": total / (ms_e2e / 1e3), "unit": UNIT,
                "h2d_bytes_per_step": int(y0_h.nbytes + (0 if cond_h is None else cond_h.nbytes)),
                "d2h_bytes_per_step": int(y_h.nbytes + r_h.nbytes)},
        "sequential_gpu": {"value": n * world / (ms_seq / 1e3), "unit": UNIT, "ms": ms_seq,
                           "wallclock_speedup_asd": (ms_seq) / (ms / args.steps)},
        ("without_phase_events" if phases_in_main else "per_phase_kernels_with_events"):
            {"value": total / (ms_plain / 1e3), "unit": UNIT, "ms_per_step": ms_plain / args.steps},
        "adaptive_window": {"value": total / (ms_adapt / 1e3), "unit": UNIT, "ms_per_step": ms_adapt / args.steps,
                            "rounds_per_sample": ad_rounds,
                            "drift_rows_per_sample_over_K": ad_rows / (args.steps * n * wl.K),
                            "phase_time_shares": ad_shares,
                            "note": "same workload, every chain picks its speculation length in 2..window from its "
                                    "own acceptance history (ASD_FLAG_ADAPTIVE_WINDOW); CUDA-graph rounds"},
        "lookahead": {"value": total / (ms_la / 1e3), "unit": UNIT, "ms_per_step": ms_la / args.steps,
                      "rounds_per_sample": la_rounds, "drift_rows_per_sample_over_K": la_rows / (args.steps * n * wl.K),
                      "note": "same workload with ASD_FLAG_LOOKAHEAD: the batched pass also evaluates the end of the "
                              "window, and a chain that accepted its whole window skips its next first model call"},
        "adaptive_window_lookahead": {"value": total / (ms_ala / 1e3), "unit": UNIT, "ms_per_step": ms_ala / args.steps,
                                      "rounds_per_sample": ala_rounds,
                                      "drift_rows_per_sample_over_K": ala_rows / (args.steps * n * wl.K)},
        "phases_ms": {k: round(v["ms"], 3) for k, v in prof.items() if v["launches"]},
    }
    # ---- roofline of the dominant kernel ----------------------------------------------------
    vb_all = 4.0 * wl.d * (all_rows + 3 * all_chains)
    va = vb_all / (ver_all["ms"] / 1e3) / 1e9 if ver_all["ms"] > 0 else 0.0
    line["roofline_verify_whole_window"] = {
        "kernel": "verify_kernel (ASD_FLAG_DEBUG_ALL_SLOTS)", "bound": "hbm", "achieved": va, "peak": peaks["hbm_gbs"],
        "unit": "GB/s", "frac": va / peaks["hbm_gbs"], "launches": ver_all["launches"],
        "avg_launch_ms": ver_all["ms"] / max(ver_all["launches"], 1), "traffic": None,
        "note": "6 rounds with every window slot verified: bytes = 4 d (w + 2) per chain-round (the whole-window "
                "reading of the verify step); instruction issue (Philox + Box-Muller per element) bounds it, not HBM"}
    if wl.kind == "mlp":
        hid = prof["pass2_gemm_hidden"]
        flops = 2.0 * wl.width * wl.width * hid["rows"] * wl.n_layers       # all hidden-layer launches of pass 2
        ach = flops / (hid["ms"] / 1e3) / 1e12 if hid["ms"] > 0 else 0.0
        peak = peaks["bf16_tflops_sustained"]
        rows_per_launch = hid["rows"] * wl.n_layers / max(hid["launches"], 1)
        if rows_per_launch > 256:
            line["roofline"] = {"kernel": "gemm_pair_kernel<BN,EPI_HID> (pass 2 hidden layers)", "bound": "tensor",
                                "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak,
                                "peak_source": peaks["source"] + " (sustained cuBLAS bf16)",
                                "frac_of_burst_peak": ach / peaks["bf16_tflops"],
                                "launches": hid["launches"], "avg_launch_ms": hid["ms"] / max(hid["launches"], 1),
                                "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH.get(wl.name),
                                "algorithmic_bytes_per_full_launch": int(2 * wl.width * (3 * wl.chains * (wl.window - 1) + wl.width))}
        else:
            # few rows: the hidden layers stream their weights (skinny kernel), the bound is HBM
            wbytes = 2.0 * wl.width * wl.width * hid["launches"]
            gbs = wbytes / (hid["ms"] / 1e3) / 1e9 if hid["ms"] > 0 else 0.0
            line["roofline"] = {"kernel": "gemm_skinny_kernel<EPI_HID> (pass 2 hidden layers)", "bound": "hbm",
                                "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                                "peak_source": peaks["source"], "launches": hid["launches"],
                                "avg_launch_ms": hid["ms"] / max(hid["launches"], 1), "traffic": None,
                                "rows_per_launch": rows_per_launch, "tensor_tflops": ach,
                                "note": "algorithmic bytes = the layer's bf16 weights per launch; the launch floor of "
                                        "this system (about 4 us per kernel) is inside the event time"}
        ver = prof["verify"]
        # bytes the verify kernel has to move: every drift row it reads (it stops after the first
        # rejection, so this is less than the 4 d (w - 1) per chain-round of reading the whole window),
        # plus y^/v reads and the y write (3 * 4 d per chain-round)
        vbytes = 4.0 * wl.d * (rows_ver + 3 * ver["rows"])
        vach = vbytes / (ver["ms"] / 1e3) / 1e9 if ver["ms"] > 0 else 0.0
        # the same step when the whole window is read: drafted rows + 3 rows per chain-round
        wbytes = 4.0 * wl.d * ((rows - ver["rows"]) + 3 * ver["rows"])
        line["roofline_verify"] = {"kernel": "verify_kernel", "bound": "hbm", "achieved": vach, "peak": peaks["hbm_gbs"],
                                   "unit": "GB/s", "frac": vach / peaks["hbm_gbs"], "peak_source": peaks["source"],
                                   "launches": ver["launches"], "avg_launch_ms": ver["ms"] / max(ver["launches"], 1),
                                   "traffic": None,
                                   "whole_window_bytes_over_time": {
                                       "achieved": wbytes / (ver["ms"] / 1e3) / 1e9 if ver["ms"] > 0 else 0.0,
                                       "unit": "GB/s",
                                       "frac": (wbytes / (ver["ms"] / 1e3) / 1e9 / peaks["hbm_gbs"]) if ver["ms"] > 0 else 0.0,
                                       "note": "4 d (w + 2) bytes per chain-round, the step as Algorithm 2 states it, over "
                                               "the same kernel time: what stopping at the first rejection is worth "
                                               "against a kernel that reads the whole window (not a bandwidth claim)"},
                                   "note": "bytes = drift rows actually read (the kernel stops at the first rejection) + "
                                           "3 rows per chain-round; bound by instruction issue (Philox + Box-Muller per "
                                           "element) and by the longest accepted prefix, not by HBM"}
    else:
        ver = prof["verify"]  # per-phase kernels, second region: the same chains, the same rounds as the first
        vbytes = 4.0 * wl.d * (rows_ver + 3 * ver["rows"])
        vach = vbytes / (ver["ms"] / 1e3) / 1e9 if ver["ms"] > 0 else 0.0
        line["roofline"] = {"kernel": "verify_kernel", "bound": "hbm", "achieved": vach, "peak": peaks["hbm_gbs"],
                            "unit": "GB/s", "frac": vach / peaks["hbm_gbs"], "peak_source": peaks["source"],
                            "launches": ver["launches"], "avg_launch_ms": ver["ms"] / max(ver["launches"], 1),
                            "traffic": None,
                            "note": "the per-phase verify kernel, timed in the second region; at this size it is bound "
                                    "by launch latency, and the default path (value) does not launch it at all"}
    # ---- CPU oracle on a bounded sample (rank 0, N = 1 only) -----------------------------------
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = oracle_rates(wl, 20.0)
    # ---- every named configuration in brief (N = 1 only; each costs well under a second of GPU time) ----
    if world == 1 and not args.no_configs:
        import dataclasses
        cfgs = {}
        for name in ("cfg1_gmm2d", "cfg2_gauss64", "cfg3_policy", "cfg4_image"):
            if name == wl.name:
                continue
            if name == "cfg4_image" and wl.kind == "mlp" and wl.width == 4096 and wl.n_layers == 6 and wl.K == 1000:
                w4 = dataclasses.replace(wl, name=name, window=32, chains=32)   # the same seeded weights
            else:
                w4 = workloads.make(name)
            cfgs[name] = compact_config(torch, AsdSampler, w4, peaks)
        # the cfg-1 problem with a small network fitted to its closed-form posterior mean (stored weights): rounds per
        # sample on a true posterior mean represented by the bf16 network, next to the closed form's (cfg1_gmm2d)
        wt = workloads.make("cfg1_trained", chains=256)
        cfgs["cfg1_trained_mlp_256_chains"] = compact_config(torch, AsdSampler, wt, peaks)
        cfgs["cfg1_gmm2d_256_chains"] = compact_config(torch, AsdSampler, workloads.make("cfg1_gmm2d", chains=256), peaks)
        # theta = infinity (window = K: every round drafts to the end of the grid), the paper's upper limit of the
        # algorithmic speed-up
        cfgs["cfg1_gmm2d_theta_inf"] = compact_config(torch, AsdSampler, workloads.make("cfg1_gmm2d", window=100), peaks)
        cfgs["cfg2_gauss64_theta_inf"] = compact_config(torch, AsdSampler, workloads.make("cfg2_gauss64", window=1000, chains=64), peaks)
        line["configs"] = cfgs
        # the batch x window sweep on the cfg-4 denoiser in brief (the full lines: --sweep)
        if wl.kind == "mlp" and wl.width == 4096 and wl.n_layers == 6 and wl.K == 1000:
            sweep = {}
            for b, w in workloads.SWEEP_CELLS:
                cell = dataclasses.replace(wl, name=f"sweep_b{b}_w{w}", window=w, chains=b)
                c = compact_config(torch, AsdSampler, cell, peaks, steps=1 if b * w >= 4096 else 2)
                sweep[cell.name] = {k: c[k] for k in ("samples_per_sec", "rounds_per_sample", "drift_rows_per_sample_over_K",
                                                      "sequential_gpu_samples_per_sec", "wallclock_speedup_asd")}
                sweep[cell.name]["dominant_kernel"] = {k: round(v, 4) if isinstance(v, float) else v
                                                       for k, v in c["dominant_kernel"].items()}
            line["sweep"] = sweep
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the brief block on the other named configurations")
    ap.add_argument("--sweep", action="store_true",
                    help="run the 12 cells of the batch x window sweep on the cfg-4 denoiser, one JSON line per cell")
    ap.add_argument("--profile-rounds", type=int, default=0,
                    help="profiling aid: reset, run this many speculation rounds, print nothing timed and exit "
                         "(a short, bounded launch sequence for ncu captures)")
    ap.add_argument("--all-slots", action="store_true",
                    help="with --profile-rounds: create the sampler with ASD_FLAG_DEBUG_ALL_SLOTS (every window slot verified)")
    args = ap.parse_args()
    if args.profile_rounds > 0:
        import torch
        from paper_2505_03983_b200 import AsdSampler
        from paper_2505_03983_b200.binding import FLAG_DEBUG_ALL_SLOTS
        wl = workloads.make(args.workload)
        with AsdSampler(wl, flags=FLAG_DEBUG_ALL_SLOTS if args.all_slots else 0) as s:
            cond = torch.as_tensor(wl.cond, device="cuda") if wl.kind == "mlp" and wl.d_cond else None
            s.reset(wl.chains, 0, cond=cond)
            for _ in range(args.profile_rounds):
                st = s.round()
            print(json.dumps({"profile_rounds": args.profile_rounds, "workload": wl.name,
                              "last_round": {"active": st.n_active_before, "rows_pass2": st.rows_pass2,
                                             "accepted": st.accepted_total}}))
    elif args.sweep:
        for b, w in workloads.SWEEP_CELLS:
            args.workload, args.no_cpu_baseline, args.no_configs = f"sweep_b{b}_w{w}", True, True
            run_ours(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
