"""Parity protocol between the CUDA decoder and the CPU oracle (shared by the GPU tests,
the smoke check and nothing else).

Decisions (accept / reject, first-rejection index, committed length) must agree exactly,
except decisions whose margin |l_i - log u_i| is below `margin` (1e-3 in fp32, 5e-2 in bf16):
those are counted, and the oracle is re-run forced onto the GPU's decisions before values
are compared.  Values are compared PER SERIES: max-abs 1e-4 (fp32) or relative RMS 3e-2
(bf16) for every single series; the figure over all compared series together is reported
as information only.  Near-margin flips are bounded (at most 2 % of the compared decisions,
and at least one allowed), and the decoder's own count of near-margin decisions is checked
against the oracle's.
"""
from __future__ import annotations

import math
import multiprocessing as mp
import os

import numpy as np

from oracle import tsfm_oracle as orc

MARGIN = {"f32": 1e-3, "bf16": 5e-2}
VALUE_TOL = {"f32": ("max_abs", 1e-4), "bf16": ("rel_rms", 3e-2)}
# how far the two sides' statistics l_i may sit apart when both call a decision "near the margin":
# decisions whose distance to the margin is below this band may be classified differently
NEAR_BAND = {"f32": 1e-4, "bf16": 2e-2}
MAX_FLIP_FRACTION = 0.02


def oracle_models(wl, tw, dw):
    t = orc.make_model(tw, wl.target.n_layers, wl.target.d_model, wl.target.n_heads, wl.target.d_ff, wl.patch_len)
    d = orc.make_model(dw, wl.draft.n_layers, wl.draft.d_model, wl.draft.n_heads, wl.draft.d_ff, wl.patch_len)
    return t, d


def value_error(kind: str, got: np.ndarray, want: np.ndarray) -> float:
    got = np.asarray(got, dtype=np.float64)
    if kind == "max_abs":
        return float(np.abs(got - want).max())
    return float(np.sqrt(np.mean((got - want) ** 2)) / np.sqrt(np.mean(want ** 2)))


def per_series_errors(kind: str, got: np.ndarray, want: np.ndarray) -> np.ndarray:
    """The value error of every row (series) on its own."""
    return np.array([value_error(kind, got[i:i + 1], want[i:i + 1]) for i in range(len(want))])


def gpu_decisions(n_accept: np.ndarray, K: int, b: int):
    """Per-round forced-decision lists of series b from the GPU trace ([R, B] n_accept, -1 = finished)."""
    rounds = []
    for r in range(n_accept.shape[0]):
        n = int(n_accept[r, b])
        if n < 0:
            break
        rounds.append([True] * n + ([False] if n < K else []))
    return rounds


# ---------------------------------------------------------------- oracle runs, one series each
# Series are independent, so the oracle's per-series runs are spread over worker processes (fork:
# the fp64 weights are shared copy-on-write; the workers run numpy only and never touch CUDA).
_JOB = {}


def _one_series(b):
    j = _JOB
    try:
        from threadpoolctl import threadpool_limits
        limiter = threadpool_limits(limits=1)
    except Exception:                                   # pragma: no cover
        limiter = None
    s = j["series"][b:b + 1]
    if j["mode"] == "spec":
        out, tr = orc.forecast_speculative(j["target"], j["draft"], s, j["ctx"], j["H"], j["K"], j["tau"], j["seed"],
                                           forced=[j["forced"][b]], series_index0=b, variant=j["variant"])
        recs = [(list(r.ell), list(r.log_u), list(r.decisions)) for r in tr.rounds[0]]
        res = (out[0], recs)
    else:
        res = (orc.forecast_target_only(j["target"], s, j["ctx"], j["H"])[0], None)
    del limiter
    return res


def _run_jobs(ids, job):
    global _JOB
    _JOB = job
    ids = list(ids)
    n_proc = min(len(ids), max(1, (os.cpu_count() or 1)))
    heavy = job["target"].n_layers * job["target"].d_model >= 8 * 512
    if n_proc < 2 or not heavy or len(ids) < 4:
        return [_one_series(b) for b in ids]
    with mp.get_context("fork").Pool(n_proc) as pool:
        return pool.map(_one_series, ids, chunksize=1)


def oracle_target_only(target, series, ctx_len, H, ids):
    """Eq. 1 by the oracle for the series in `ids` (rows in that order)."""
    res = _run_jobs(ids, dict(mode="target", target=target, draft=None, series=series, ctx=ctx_len, H=H))
    return np.stack([r[0] for r in res])


def compare_forecast(wl, target, draft, series, H, K, tau, seed, gpu_out, gpu_nacc, series_ids, dtype=None,
                     variant=None, gpu_ell=None, gpu_logu=None):
    """Compare GPU results for the series in `series_ids` with the oracle.

    Returns a dict with the worst per-series value error, the pooled one, the number of decisions
    compared, the number of near-margin flips and both sides' near-margin counts (the GPU's only
    when its trace of l_i and log u_i is passed); raises AssertionError on any violation.
    """
    dtype = dtype or wl.dtype
    margin = MARGIN[dtype]
    kind, tol = VALUE_TOL[dtype]
    ids = list(series_ids)
    T = -(-H // wl.patch_len)
    forced = {}
    for b in ids:
        forced[b] = gpu_decisions(gpu_nacc, K, b)
        # the GPU's rounds must cover the horizon exactly
        L = [sum(f) + 1 for f in forced[b]]
        assert sum(L[:-1]) < T <= sum(L), f"series {b}: GPU rounds {L} do not cover T={T}"
    res = _run_jobs(ids, dict(mode="spec", target=target, draft=draft, series=series, ctx=wl.ctx_len, H=H, K=K,
                              tau=tau, seed=seed, forced=forced, variant=variant))
    flips = n_dec = near_oracle = near_gpu = in_band = 0
    ell_gap = 0.0
    for b, (_, recs) in zip(ids, res):
        for r, (ells, lus, decs) in enumerate(recs):
            for i, (ell, lu, dec) in enumerate(zip(ells, lus, decs)):
                natural = lu <= min(ell, 0.0)
                n_dec += 1
                gap = abs(ell - lu)
                near_oracle += gap < margin
                in_band += abs(gap - margin) < NEAR_BAND[dtype]
                if gpu_ell is not None:
                    g_gap = abs(float(gpu_ell[r, b, i]) - float(gpu_logu[r, b, i]))
                    near_gpu += g_gap < margin
                    ell_gap = max(ell_gap, abs(float(gpu_ell[r, b, i]) - ell))
                if natural != dec:
                    flips += 1
                    assert gap < margin, (
                        f"series {b} round {r} pos {i}: GPU decided {dec}, oracle {natural}, "
                        f"margin {gap:.4g} >= {margin}")
    assert flips <= max(1, math.ceil(MAX_FLIP_FRACTION * n_dec)), f"{flips} near-margin flips in {n_dec} decisions"
    if gpu_ell is not None:
        # both sides count the same decisions as near the margin, up to those that sit on its edge
        assert abs(near_gpu - near_oracle) <= flips + in_band, (near_gpu, near_oracle, flips, in_band)
    want = np.stack([r[0] for r in res])
    got = np.asarray(gpu_out)[ids]
    each = per_series_errors(kind, got, want)
    worst = int(np.argmax(each))
    assert each[worst] <= tol, f"series {ids[worst]}: {kind} error {each[worst]:.4g} > {tol} (all: {np.round(each, 5)})"
    return {"error": float(each[worst]), "worst_series": ids[worst], "pooled_error": value_error(kind, got, want),
            "kind": kind, "series": len(ids), "decisions": n_dec, "near_margin_flips": flips,
            "near_margin_oracle": near_oracle, "near_margin_gpu": near_gpu if gpu_ell is not None else None,
            "max_ell_gap": ell_gap}


def gpu_near_margin_total(n_accept, ell, log_u, K, margin):
    """Tested decisions of a whole GPU trace ([R, B], [R, B, K] x 2) with |l - log u| < margin: what
    the decoder's own counter must show."""
    n = np.asarray(n_accept)
    tested = np.minimum(n + 1, K)                              # -1 (finished) -> 0
    pos = np.arange(K)[None, None, :]
    mask = pos < tested[:, :, None]
    return int((mask & (np.abs(np.asarray(ell) - np.asarray(log_u)) < margin)).sum())
