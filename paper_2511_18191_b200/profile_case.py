"""Small, self-terminating cases of the decoder's kernels, meant to be run under a profiler.

    python -m paper_2511_18191_b200.profile_case gemm --M 160 --N 1536 --K 512 --reps 3
    python -m paper_2511_18191_b200.profile_case forecast --workload C1 --reps 2
    python -m paper_2511_18191_b200.profile_case forecast --workload C4 --target-layers 2 --mode target_only

`gemm` runs the bf16 tensor-core contraction alone on random operands (optionally over a ring of
weight matrices larger than the L2 cache, so that DRAM counters describe a cold weight stream).
`forecast` runs whole forecasts of a workload, optionally with fewer target layers, a smaller
batch or a shorter horizon so that a capture holds little device memory and ends quickly.
"""
from __future__ import annotations

import argparse
import sys

import numpy as np


def run_gemm(a):
    import torch
    from . import binding as tsfm
    g = torch.Generator(device="cpu").manual_seed(1)
    A = torch.randn((a.M, a.K), generator=g).to(torch.bfloat16).cuda()
    n_w = max(1, a.ring)
    Ws = [(torch.randn((a.N, a.K), generator=g) / a.K ** 0.5).to(torch.bfloat16).cuda() for _ in range(n_w)]
    C = torch.empty((a.M, a.N), device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    backend = tsfm.TSFM_GEMM_WS if a.backend == "ws" else tsfm.TSFM_GEMM_AUTO
    for i in range(a.reps):
        tsfm.tsfm_gemm_bf16(s, A, Ws[i % n_w], C, a.M, a.N, a.K, backend)
    torch.cuda.synchronize()
    print(f"gemm M={a.M} N={a.N} K={a.K}: {a.reps} launches over {n_w} weight matrices, "
          f"checksum {float(C.double().sum()):.6g}")


def run_forecast(a):
    import torch
    from . import binding as tsfm
    from tsfm_inputs import build_models, make_series, workload
    wl = workload(a.workload)
    over = {}
    if a.target_layers:
        over["target"] = type(wl.target)(a.target_layers, wl.target.d_model, wl.target.n_heads, wl.target.d_ff)
        if wl.draft_mode != "separate":
            over["draft"] = type(wl.draft)(min(wl.draft.n_layers, a.target_layers), wl.draft.d_model,
                                           wl.draft.n_heads, wl.draft.d_ff)
    if a.batch:
        over["batch"] = a.batch
    if a.horizon:
        over["horizon"] = a.horizon
    if over:
        wl = wl.with_(**over)
    K = a.K or wl.K
    tw, dw = build_models(wl)
    # kernels inside a graph with a conditional node cannot be profiled one by one: --exec stream
    # launches the same kernels directly
    mode = tsfm.TSFM_EXEC_STREAM if a.exec == "stream" else tsfm.TSFM_EXEC_GRAPH
    dec = tsfm.SpecDecoder.for_workload(wl, tw, dw, max_K=K, exec_mode=mode)
    s = make_series(wl)
    ctx = torch.from_numpy(np.ascontiguousarray(s[:, :wl.ctx_len])).cuda()
    out = torch.empty((wl.batch, wl.horizon), device="cuda")
    for i in range(a.reps):
        if a.mode == "target_only":
            tsfm.tsfm_target_only_forecast(dec.h, ctx, wl.batch, wl.ctx_len, wl.horizon, out, None)
        else:
            tsfm.tsfm_spec_forecast(dec.h, ctx, wl.batch, wl.ctx_len, wl.horizon, K, a.tau or wl.tau,
                                    wl.forecast_seed + i, out, None)
    torch.cuda.synchronize()
    print(f"{a.mode} forecast {wl.name}: B={wl.batch} layers={wl.target.n_layers} H={wl.horizon} K={K}, "
          f"{a.reps} calls, {tsfm.tsfm_launch_count()} kernel launches, checksum {float(out.double().sum()):.6g}")
    dec.close()


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    sub = ap.add_subparsers(dest="cmd", required=True)
    g = sub.add_parser("gemm")
    g.add_argument("--M", type=int, required=True)
    g.add_argument("--N", type=int, required=True)
    g.add_argument("--K", type=int, required=True)
    g.add_argument("--reps", type=int, default=3)
    g.add_argument("--ring", type=int, default=1, help="number of distinct weight matrices cycled through")
    g.add_argument("--backend", default="auto", choices=["auto", "ws"],
                   help="auto: tensor-memory kernel; ws: the small-batch kernel with a resident weight tile")
    f = sub.add_parser("forecast")
    f.add_argument("--workload", default="C1")
    f.add_argument("--mode", default="spec", choices=["spec", "target_only"])
    f.add_argument("--target-layers", type=int, default=0)
    f.add_argument("--batch", type=int, default=0)
    f.add_argument("--horizon", type=int, default=0)
    f.add_argument("--K", type=int, default=0)
    f.add_argument("--tau", type=float, default=0.0)
    f.add_argument("--reps", type=int, default=2)
    f.add_argument("--exec", default="graph", choices=["graph", "stream"])
    a = ap.parse_args(argv)
    (run_gemm if a.cmd == "gemm" else run_forecast)(a)


if __name__ == "__main__":
    main(sys.argv[1:])
