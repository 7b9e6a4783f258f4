"""Helpers of the GPU tests: build a decoder + inputs for a workload."""
from __future__ import annotations

import numpy as np
import torch

import paper_2511_18191_b200 as tsfm
from tsfm_inputs import build_models, make_series


def make_decoder(wl, backend=tsfm.TSFM_GEMM_AUTO, max_K=None, batch=None, exec_mode=tsfm.TSFM_EXEC_GRAPH):
    tw, dw = build_models(wl)
    dec = tsfm.SpecDecoder.for_workload(wl, tw, dw, max_K=max_K, batch=batch, gemm_backend=backend,
                                        exec_mode=exec_mode)
    return dec, tw, dw


def series_on_device(wl, batch=None):
    s = make_series(wl, batch)
    ctx = torch.from_numpy(np.ascontiguousarray(s[:, :wl.ctx_len])).cuda()
    return s, ctx
