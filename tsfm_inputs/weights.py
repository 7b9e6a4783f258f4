"""Seeded random weights for the patch transformers.

Tensor inventory of one model (no biases, every linear stored
``[out_features, in_features]``):

    W_emb [d, P]
    per layer l: g1 [d], Wq Wk Wv Wo [d, d], g2 [d], W1 [d_ff, d], W2 [d, d_ff]
    g_f [d], W_head [P, d]

Linears are Xavier-normal, std = sqrt(2 / (fan_in + fan_out)); gains are 1.
Values are float32 arrays; for ``dtype == "bf16"`` every linear is rounded to
the nearest bf16 value (ties to even) here, so that every consumer sees exactly
the same numbers.
"""
from __future__ import annotations

from typing import Dict, List

import numpy as np

from .configs import Arch, Workload

Weights = Dict[str, np.ndarray]


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def tensor_names(n_layers: int) -> List[str]:
    names = ["W_emb"]
    for l in range(n_layers):
        names += [f"layers.{l}.{t}" for t in ("g1", "Wq", "Wk", "Wv", "Wo", "g2", "W1", "W2")]
    names += ["g_f", "W_head"]
    return names


def _shape(name: str, arch: Arch, patch_len: int, patch_in: int = 0):
    d, f, p = arch.d_model, arch.d_ff, patch_len
    t = name.split(".")[-1]
    return {"W_emb": (d, patch_in or p), "g1": (d,), "g2": (d,), "g_f": (d,),
            "Wq": (d, d), "Wk": (d, d), "Wv": (d, d), "Wo": (d, d),
            "W1": (f, d), "W2": (d, f), "W_head": (p, d)}[t]


def make_model(arch: Arch, patch_len: int, seed: int, dtype: str, stream: int = 0, patch_in: int = 0) -> Weights:
    """Xavier-normal weights; ``stream`` separates target (0) and draft (1) draws.  ``patch_in``
    (0 = patch_len) is the length of an input token: the embedding is [d, patch_in]."""
    rng = np.random.default_rng([int(seed), int(stream), 0x7511])
    w: Weights = {}
    for name in tensor_names(arch.n_layers):
        shape = _shape(name, arch, patch_len, patch_in)
        if len(shape) == 1:
            w[name] = np.ones(shape, dtype=np.float32)
            continue
        fan_out, fan_in = shape
        std = np.float32(np.sqrt(2.0 / (fan_in + fan_out)))
        t = rng.standard_normal(shape, dtype=np.float32) * std
        w[name] = round_to_bf16(t) if dtype == "bf16" else t
    return w


def layer_skip_draft(target: Weights, n_layers: int) -> Weights:
    """Draft = the target's first ``n_layers`` layers + its final norm and head (aliases)."""
    w: Weights = {"W_emb": target["W_emb"], "g_f": target["g_f"], "W_head": target["W_head"]}
    for name in tensor_names(n_layers):
        if name.startswith("layers."):
            w[name] = target[name]
    return {n: w[n] for n in tensor_names(n_layers)}


def perturbed_draft(target: Weights, n_layers: int, eps: float, seed: int, dtype: str) -> Weights:
    """Draft = target + eps * std(tensor) * N(0, 1) per linear; gains untouched.

    eps == 0 returns tensors with bit-identical values.
    """
    rng = np.random.default_rng([int(seed), 0x9e37])
    w: Weights = {}
    for name in tensor_names(n_layers):
        t = target[name]
        if t.ndim == 1:
            w[name] = t.copy()
            continue
        noise = rng.standard_normal(t.shape, dtype=np.float32)
        if eps == 0.0:
            w[name] = t.copy()
            continue
        p = t + np.float32(eps) * np.float32(t.std()) * noise
        w[name] = round_to_bf16(p) if dtype == "bf16" else p.astype(np.float32)
    return w


def build_models(wl: Workload):
    """(target weights, draft weights) for a workload."""
    tgt = make_model(wl.target, wl.patch_len, wl.weight_seed, wl.dtype, stream=0, patch_in=wl.patch_in)
    if wl.draft_mode == "layer_skip" and wl.late_layer_scale != 1.0:
        # a draft that tracks its target: the layers the draft lacks contribute less to the residual stream
        for l in range(wl.draft.n_layers, wl.target.n_layers):
            for t in ("Wo", "W2"):
                w = tgt[f"layers.{l}.{t}"] * np.float32(wl.late_layer_scale)
                tgt[f"layers.{l}.{t}"] = round_to_bf16(w) if wl.dtype == "bf16" else w.astype(np.float32)
    if wl.draft_mode == "layer_skip":
        drf = layer_skip_draft(tgt, wl.draft.n_layers)
    elif wl.draft_mode == "perturbed":
        drf = perturbed_draft(tgt, wl.draft.n_layers, wl.draft_eps, wl.perturb_seed, wl.dtype)
    else:
        drf = make_model(wl.draft, wl.patch_len, wl.weight_seed, wl.dtype, stream=1, patch_in=wl.patch_in)
    return tgt, drf
