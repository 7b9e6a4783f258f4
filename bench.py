#!/usr/bin/env python
"""Benchmark of the speculative patch decoder: committed patches/s on workload C1.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload C1]

One "step" is one whole speculative forecast (instance norm, prefill of both models, the
round loop draft -> verify -> accept -> rollback until T patches are committed, de-normalise)
over one batch of synthetic series.  `value` = committed patches per second with the inputs
resident in HBM; `e2e` = the same through the host-buffer entry point (pinned host input and
output, copies inside the timed region).  With N > 1 (torchrun) every rank decodes its own
batch on its own GPU (the path shards by series with no exchange step: weak scaling, no
collective); times are CUDA-event times, max over ranks.

`--impl reference` times the CPU oracle (fp64, as it stands) on a bounded sample of the same
workload on the host cores, rank 0 only.
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

METRIC = "committed_patches_per_s"
UNIT = "patches/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C1")
    ap.add_argument("--tau", type=float, default=None)
    ap.add_argument("--K", type=int, default=None)
    ap.add_argument("--cpu-series", type=int, default=None, help="series per oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--others", default="C2,C4", help="comma list of further workloads to profile briefly ('' = none)")
    return ap.parse_args()


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
            except ValueError:
                continue
            for name, v in zip(names, r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------ CPU oracle leg
def oracle_sample(wl, K, tau, n_series, repeats):
    """Time the oracle's speculative forecast on the first `n_series` series; returns patches/s."""
    import torch
    from oracle import tsfm_oracle as orc
    from tests import parity
    from tsfm_inputs import build_models, make_series
    tw, dw = build_models(wl)
    tm, dm = parity.oracle_models(wl, tw, dw)
    s = make_series(wl, n_series)
    times = []
    for r in range(repeats):
        t0 = time.perf_counter()
        orc.forecast_speculative(tm, dm, s, wl.ctx_len, wl.horizon, K, tau, wl.forecast_seed + r)
        times.append(time.perf_counter() - t0)
    total = float(np.sum(times))
    return n_series * wl.n_patches * repeats / total, total, torch.get_num_threads()


def run_reference(args, wl, K, tau):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_series = args.cpu_series or min(wl.batch, 8)
    # warm-up steps and timed steps, each one bounded sample
    for _ in range(args.warmup):
        oracle_sample(wl, K, tau, n_series, 1)
    t0 = time.perf_counter()
    val, total, cores = oracle_sample(wl, K, tau, n_series, args.steps)
    ms = (time.perf_counter() - t0) * 1e3 / args.steps
    sample = f"{n_series} of {wl.batch} series of {wl.name} per step, full forecast (T={wl.n_patches})"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "B": wl.batch, "ctx_len": wl.ctx_len, "P": wl.patch_len,
                   "H": wl.horizon, "K": K, "tau": tau},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------ other workloads (informational)
def profile_workload(name, hbm_peak, tf_peak):
    """One warm speculative and target-only forecast of another workload plus one profiled forecast:
    where the tensor-bound verification GEMMs (C2) and the KV-bound attention (C4) stand against the
    measured peaks.  Not part of the headline metric."""
    import torch
    import paper_2511_18191_b200 as tsfm
    from tsfm_inputs import build_models, make_series, workload
    wl = workload(name)
    tw, dw = build_models(wl)
    dec = tsfm.SpecDecoder.for_workload(wl, tw, dw, max_K=wl.K)
    s = make_series(wl)
    ctx = torch.from_numpy(np.ascontiguousarray(s[:, :wl.ctx_len])).cuda()
    for _ in range(2):
        _, st = dec.forecast(ctx, wl.horizon, wl.K, wl.tau, wl.forecast_seed)
        _, st_t = dec.target_only(ctx, wl.horizon)
    d, dt = st.as_dict(), st_t.as_dict()
    tsfm.tsfm_spec_set_profiling(dec.h, True)
    dec.forecast(ctx, wl.horizon, wl.K, wl.tau, wl.forecast_seed, stats=False)
    prof = tsfm.tsfm_spec_kernel_profile(dec.h)
    tsfm.tsfm_spec_set_profiling(dec.h, False)
    dec.close()
    tot = sum(v["ms_total"] for v in prof.values())
    kernels = {}
    for k, v in sorted(prof.items(), key=lambda kv: -kv[1]["ms_total"])[:3]:
        gbs, tfs = v["bytes"] / v["ms_total"] / 1e6, v["flops"] / v["ms_total"] / 1e9
        kernels[k] = {"share": round(v["ms_total"] / tot, 3), "avg_launch_us": round(v["ms_total"] * 1e3 / v["launches"], 2),
                      "GB/s": round(gbs, 1), "frac_hbm": round(gbs / hbm_peak, 4),
                      "TFLOP/s": round(tfs, 1), "frac_tensor": round(tfs / tf_peak, 4)}
    return {"ms_per_forecast": d["ms_total"], "ms_target_only": dt["ms_total"],
            "phases_ms": {k: d[k] for k in ("ms_prefill", "ms_draft", "ms_verify", "ms_accept")},
            "rounds": d["rounds"], "accepted_over_tested": d["proposals_accepted"] / max(d["proposals_tested"], 1),
            "B": wl.batch, "patches_per_s": wl.batch * wl.n_patches / (d["ms_total"] * 1e-3),
            "kernels_event_timed": kernels}


# ------------------------------------------------------------------ multi-rank host logic
def rank_workload(wl, rank: int):
    """Every rank decodes its own batch: same shapes and weights, different series."""
    return wl.with_(series_seed=wl.series_seed + 7919 * rank)


def max_over_ranks(ms: float, world: int, device="cuda") -> float:
    """The job's time is the slowest rank's: one scalar all-reduce(MAX) after the timed region."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, series_per_rank: int, patches: int, steps: int, ms: float) -> float:
    """Committed patches per second of the whole job (all ranks), given the max-over-ranks time."""
    return world * series_per_rank * patches * steps / (ms * 1e-3)


def throughput_law(stats, to_stats, K, T):
    """Predicted speedup S(K) = E[L] / (c K + v) of the paper's Eq. 8 from this run's own measurements:
    acceptance rate alpha = accepted / tested, c = draft step time / target step time, v = verification
    pass time / target step time (phase clocks of the decoder), E[L] of Eq. 7."""
    rounds = max(stats["rounds"], 1)
    step = to_stats["ms_verify"] / T
    if step <= 0:
        return None
    alpha = stats["proposals_accepted"] / max(stats["proposals_tested"], 1)
    c = stats["ms_draft"] / (rounds * K) / step
    v = stats["ms_verify"] / rounds / step
    e_l = float(K + 1) if alpha >= 1.0 else (1.0 - alpha ** (K + 1)) / (1.0 - alpha)
    import paper_2511_18191_b200 as tsfm
    k_star, s_star = tsfm.tsfm_advise_block_size(alpha, c, v, 32)
    return {"alpha": alpha, "c": c, "v": v, "E_L": e_l, "predicted_speedup": e_l / (c * K + v),
            "advised_K": k_star, "predicted_speedup_at_advised_K": s_star}


# ------------------------------------------------------------------ our arm
def run_ours(args, wl, K, tau):
    import torch
    import torch.distributed as dist
    import paper_2511_18191_b200 as tsfm
    from tsfm_inputs import build_models, make_series

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decoder has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    peak_src = "measured" if "hbm_gbs" in peaks else "fallback"

    tw, dw = build_models(wl)
    dec = tsfm.SpecDecoder.for_workload(wl, tw, dw, max_K=K, device=f"cuda:{local}")
    # every rank decodes its own batch of B series (different series per rank)
    s = make_series(rank_workload(wl, rank))
    ctx_host = torch.from_numpy(np.ascontiguousarray(s[:, :wl.ctx_len])).pin_memory()
    ctx = ctx_host.cuda()
    B, H, T = wl.batch, wl.horizon, wl.n_patches
    out = torch.empty((B, H), device="cuda")
    out_host = torch.empty((B, H)).pin_memory()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")     # > 126 MB of L2
    stream = torch.cuda.current_stream()

    def timed(fn, steps, seeds0):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        for i in range(steps):
            flush.fill_(i & 0xFF)
            ev[i][0].record(stream)
            fn(seeds0 + i)
            ev[i][1].record(stream)
        barrier()
        return max_over_ranks(sum(a.elapsed_time(b) for a, b in ev), world)

    spec = lambda seed: tsfm.tsfm_spec_forecast(dec.h, ctx, B, wl.ctx_len, H, K, tau, seed, out, None)
    tonly = lambda seed: tsfm.tsfm_target_only_forecast(dec.h, ctx, B, wl.ctx_len, H, out, None)
    donly = lambda seed: tsfm.tsfm_draft_only_forecast(dec.h, ctx, B, wl.ctx_len, H, out, None)
    spec_host = lambda seed: tsfm.tsfm_spec_forecast_host(dec.h, ctx_host, B, wl.ctx_len, H, K, tau, seed, out_host, None)

    seed0 = wl.forecast_seed
    for i in range(args.warmup):
        spec(seed0 + i)
        tonly(0)
        donly(0)
        spec_host(seed0 + i)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = tsfm.tsfm_launch_count()
    ms_spec = timed(spec, args.steps, seed0)
    launches = tsfm.tsfm_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    ms_tonly = timed(tonly, args.steps, 0)
    ms_donly = timed(donly, args.steps, 0)
    # accuracy of the three arms against the synthetic ground-truth tail (normalised series: plain MSE)
    truth = torch.from_numpy(np.ascontiguousarray(s[:, wl.ctx_len:wl.ctx_len + H])).cuda()
    mse = {}
    for name, fn in (("target_only", tonly), ("draft_only", donly), ("speculative", spec)):
        fn(seed0)
        mse[name] = float(((out - truth) ** 2).mean().item())
    ms_e2e = timed(spec_host, args.steps, seed0)

    # one forecast for the acceptance counters, then one profiled forecast for per-kernel times
    _, st = dec.forecast(ctx, H, K, tau, seed0)
    stats = st.as_dict()
    _, st_t = dec.target_only(ctx, H)
    to_stats = st_t.as_dict()
    tsfm.tsfm_spec_set_profiling(dec.h, True)
    flush.fill_(1)
    n_prof = 3
    for i in range(n_prof):
        spec(seed0 + i)
    prof = tsfm.tsfm_spec_kernel_profile(dec.h)
    tsfm.tsfm_spec_set_profiling(dec.h, False)

    units = world * B * T * args.steps
    value = whole_job_value(world, B, T, args.steps, ms_spec)
    result = None
    if rank == 0:
        total_ms = sum(v["ms_total"] for v in prof.values())
        top = max(prof.items(), key=lambda kv: kv[1]["ms_total"])
        name, p = top
        achieved = p["bytes"] / (p["ms_total"] * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": name, "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                    "frac": achieved / hbm_peak, "peak_source": peak_src, "traffic": None,
                    "launches_per_step": p["launches"] / n_prof,
                    "avg_launch_us": p["ms_total"] * 1e3 / p["launches"],
                    "share_of_kernel_time": p["ms_total"] / total_ms,
                    "achieved_tflops": p["flops"] / (p["ms_total"] * 1e-3) / 1e12,
                    "kernel_shares": {k: round(v["ms_total"] / total_ms, 4) for k, v in prof.items()}}
        # The per-kernel events above bracket launches made one by one from the host, so each
        # duration carries the launch gap around it.  The timed region itself replays a graph with
        # programmatic dependent launches; this kernel's time inside it is estimated as its share
        # of the profiled kernel time x the graph's step time (an estimate, reported beside the
        # directly measured figure, not instead of it).
        in_graph_us = roofline["share_of_kernel_time"] * (ms_spec / args.steps) * 1e3 / roofline["launches_per_step"]
        bytes_per_launch = p["bytes"] / p["launches"]
        roofline["in_graph_estimate"] = {"avg_launch_us": in_graph_us,
                                         "achieved": bytes_per_launch / (in_graph_us * 1e-6) / 1e9,
                                         "frac": bytes_per_launch / (in_graph_us * 1e-6) / 1e9 / hbm_peak}
        tested, acc = stats["proposals_tested"], stats["proposals_accepted"]
        result = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_spec / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": wl.name, "B": B, "ctx_len": wl.ctx_len, "P": wl.patch_len, "H": H, "K": K,
                       "tau": tau, "series_per_gpu": B, "l2": "flushed between steps (256 MB write)",
                       "sharding": "by series, no collective"},
            "e2e": {"value": units / (ms_e2e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": B * wl.ctx_len * 4, "d2h_bytes_per_step": B * H * 4},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": roofline,
            "target_only": {"value": units / (ms_tonly * 1e-3), "unit": UNIT, "ms_per_step": ms_tonly / args.steps},
            "draft_only": {"value": units / (ms_donly * 1e-3), "unit": UNIT, "ms_per_step": ms_donly / args.steps},
            "speedup_vs_target_only": ms_tonly / ms_spec,
            "mse_vs_truth": mse,
            "throughput_law": throughput_law(stats, to_stats, K, T),
            "acceptance": {"accepted_over_tested": acc / max(tested, 1), "rounds": stats["rounds"],
                           "mean_yield": (sum(l * c for l, c in enumerate(stats["L_hist"])) /
                                          max(sum(stats["L_hist"]), 1))},
        }
        if not args.no_cpu_baseline and world == 1:
            n_series = args.cpu_series or min(B, 32)
            val, total, cores = oracle_sample(wl, K, tau, n_series, 3)
            result["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                                      "sample": f"{n_series} of {B} series of {wl.name}, full forecast, 3 repeats, "
                                                f"{total:.1f} s"}
    dec.close()
    if result is not None and world == 1 and args.others:
        tf_peak = float(peaks.get("bf16_tflops_sustained", 1400.0))
        result["other_workloads"] = {"peaks": {"hbm_gbs": hbm_peak, "bf16_tflops_sustained": tf_peak, "source": peak_src}}
        for name in [n for n in args.others.split(",") if n]:
            try:
                result["other_workloads"][name] = profile_workload(name, hbm_peak, tf_peak)
            except Exception as e:          # informational: never lose the headline line
                result["other_workloads"][name] = {"error": repr(e)}
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if result is not None:
        print(json.dumps(result))


def main():
    args = parse_args()
    from tsfm_inputs import workload
    wl = workload(args.workload)
    K = args.K or wl.K
    tau = args.tau or wl.tau
    if args.impl == "reference":
        run_reference(args, wl, K, tau)
    else:
        run_ours(args, wl, K, tau)


if __name__ == "__main__":
    main()
