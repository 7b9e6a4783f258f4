"""Parity protocol between the CUDA decoder and the CPU oracle (shared by the GPU tests,
the smoke check and nothing else).

Decisions (accept / reject, first-rejection index, committed length) must agree exactly,
except decisions whose margin |l_i - log u_i| is below `margin` (1e-3 in fp32, 5e-2 in bf16):
those are counted, and the oracle is re-run forced onto the GPU's decisions before values
are compared.  Values: max-abs 1e-4 (fp32) or relative RMS 3e-2 (bf16).
"""
from __future__ import annotations

import numpy as np

from oracle import tsfm_oracle as orc

MARGIN = {"f32": 1e-3, "bf16": 5e-2}
VALUE_TOL = {"f32": ("max_abs", 1e-4), "bf16": ("rel_rms", 3e-2)}


def oracle_models(wl, tw, dw):
    t = orc.make_model(tw, wl.target.n_layers, wl.target.d_model, wl.target.n_heads, wl.target.d_ff, wl.patch_len)
    d = orc.make_model(dw, wl.draft.n_layers, wl.draft.d_model, wl.draft.n_heads, wl.draft.d_ff, wl.patch_len)
    return t, d


def value_error(kind: str, got: np.ndarray, want: np.ndarray) -> float:
    got = np.asarray(got, dtype=np.float64)
    if kind == "max_abs":
        return float(np.abs(got - want).max())
    return float(np.sqrt(np.mean((got - want) ** 2)) / np.sqrt(np.mean(want ** 2)))


def gpu_decisions(n_accept: np.ndarray, K: int, b: int):
    """Per-round forced-decision lists of series b from the GPU trace ([R, B] n_accept, -1 = finished)."""
    rounds = []
    for r in range(n_accept.shape[0]):
        n = int(n_accept[r, b])
        if n < 0:
            break
        rounds.append([True] * n + ([False] if n < K else []))
    return rounds


def compare_forecast(wl, target, draft, series, H, K, tau, seed, gpu_out, gpu_nacc, series_ids, dtype=None,
                     variant=None):
    """Compare GPU results for the series in `series_ids` with the oracle.

    Returns a dict with the value error, the number of decisions compared, the number of
    near-margin flips; raises AssertionError on any violation.
    """
    dtype = dtype or wl.dtype
    margin = MARGIN[dtype]
    kind, tol = VALUE_TOL[dtype]
    ctx = wl.ctx_len
    flips = 0
    n_dec = 0
    outs = []
    for b in series_ids:
        s = series[b:b + 1]
        forced = [gpu_decisions(gpu_nacc, K, b)]
        T = -(-H // wl.patch_len)
        # the GPU's rounds must cover the horizon exactly
        L = [sum(f) + 1 for f in forced[0]]
        assert sum(L[:-1]) < T <= sum(L), f"series {b}: GPU rounds {L} do not cover T={T}"
        out, tr = orc.forecast_speculative(target, draft, s, ctx, H, K, tau, seed, forced=forced, series_index0=b,
                                           variant=variant)
        for r, rec in enumerate(tr.rounds[0]):
            for i, (ell, lu, dec) in enumerate(zip(rec.ell, rec.log_u, rec.decisions)):
                natural = lu <= min(ell, 0.0)
                n_dec += 1
                if natural != dec:
                    flips += 1
                    assert abs(ell - lu) < margin, (
                        f"series {b} round {r} pos {i}: GPU decided {dec}, oracle {natural}, "
                        f"margin {abs(ell - lu):.4g} >= {margin}")
        outs.append(out[0])
    want = np.stack(outs)
    got = np.asarray(gpu_out)[list(series_ids)]
    err = value_error(kind, got, want)
    assert err <= tol, f"{kind} error {err:.4g} > {tol}"
    return {"error": err, "kind": kind, "decisions": n_dec, "near_margin_flips": flips}
