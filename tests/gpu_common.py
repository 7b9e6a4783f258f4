"""Helpers of the GPU tests: build a decoder + inputs for a workload."""
from __future__ import annotations

import functools
import os

import numpy as np
import torch

import paper_2511_18191_b200 as tsfm
from tsfm_inputs import build_models, make_series


@functools.lru_cache(maxsize=2)
def _models(wl_key):
    """Weights depend on the model shapes and seeds only: consecutive tests on one workload (a sweep
    over K, tau or the execution mode) reuse them."""
    return build_models(wl_key)


def make_decoder(wl, backend=tsfm.TSFM_GEMM_AUTO, max_K=None, batch=None, exec_mode=tsfm.TSFM_EXEC_GRAPH):
    # TSFM_TEST_CHECK_BOUNDS=1 runs every test of the suite in the decoder's bounds-checking mode
    if os.environ.get("TSFM_TEST_CHECK_BOUNDS") == "1":
        exec_mode |= tsfm.TSFM_EXEC_CHECK_BOUNDS
    tw, dw = _models(wl.with_(batch=1, horizon=wl.patch_len, K=1, tau=1.0, ctx_len=2 * wl.patch_len, series_recipe="c1",
                              series_seed=0, forecast_seed=0, K_sweep=(), tau_sweep=(), eps_sweep=()))
    dec = tsfm.SpecDecoder.for_workload(wl, tw, dw, max_K=max_K, batch=batch, gemm_backend=backend,
                                        exec_mode=exec_mode)
    return dec, tw, dw


def series_on_device(wl, batch=None):
    s = make_series(wl, batch)
    ctx = torch.from_numpy(np.ascontiguousarray(s[:, :wl.ctx_len])).cuda()
    return s, ctx
