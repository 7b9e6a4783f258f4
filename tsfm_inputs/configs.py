"""The five synthetic workloads (C0..C4): shapes, decoding knobs and seeds.

The shapes follow the paper's workload classes (contexts of a few thousand
steps, patches of 32-96 steps, horizons 336-2048, batch 1-1024 with channels
folded into the batch, block size K 1-8; per-family tables of the paper's
appendix B); the concrete numbers are this build's benchmark definitions.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Tuple


@dataclass(frozen=True)
class Arch:
    """Decoder-only patch transformer shape."""
    n_layers: int
    d_model: int
    n_heads: int
    d_ff: int

    @property
    def d_head(self) -> int:
        return self.d_model // self.n_heads

    def n_params(self, patch_len: int) -> int:
        d, f, p = self.d_model, self.d_ff, patch_len
        per_layer = 4 * d * d + 2 * d * f + 2 * d
        return d * p + self.n_layers * per_layer + d + p * d


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int            # B series
    ctx_len: int          # context steps
    patch_len: int        # P
    horizon: int          # H steps
    K: int                # default block size
    tau: float            # default acceptance temperature (the paper's sigma)
    dtype: str            # "f32" | "bf16"
    target: Arch
    draft: Arch
    draft_mode: str       # "separate" | "layer_skip" | "perturbed"
    series_recipe: str    # key into series.make_series
    K_sweep: Tuple[int, ...] = ()
    tau_sweep: Tuple[float, ...] = ()
    eps_sweep: Tuple[float, ...] = ()
    draft_eps: float = 0.0          # perturbation size for "perturbed" drafts
    patch_in: int = 0               # steps per input token; 0 = patch_len (patch tokens)
    late_layer_scale: float = 1.0   # layer-skip drafts: factor on Wo and W2 of the target layers the draft lacks
    weight_seed: int = 0
    perturb_seed: int = 1
    series_seed: int = 1000
    forecast_seed: int = 2021

    @property
    def token_len(self) -> int:
        """P_in: steps per input token."""
        return self.patch_in or self.patch_len

    @property
    def n_ctx_tokens(self) -> int:
        return self.ctx_len // self.token_len

    @property
    def n_patches(self) -> int:
        return -(-self.horizon // self.patch_len)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS = {
    "C0": Workload("C0", 1, 672, 96, 384, 2, 1.0, "f32",
                   Arch(2, 128, 4, 512), Arch(1, 64, 2, 256), "separate", "c0",
                   series_seed=1000),
    "C1": Workload("C1", 32, 2880, 96, 720, 4, 1.0, "bf16",
                   Arch(8, 512, 8, 2048), Arch(2, 512, 8, 2048), "layer_skip", "c1",
                   tau_sweep=(0.5, 1.0, 2.0), series_seed=1001),
    "C2": Workload("C2", 256, 2880, 96, 720, 4, 1.0, "bf16",
                   Arch(24, 1024, 16, 4096), Arch(2, 256, 4, 1024), "separate", "c2",
                   series_seed=1002),
    "C3": Workload("C3", 1024, 672, 96, 1440, 4, 1.0, "bf16",
                   Arch(12, 768, 12, 3072), Arch(12, 768, 12, 3072), "perturbed", "c1",
                   K_sweep=(1, 2, 4, 8), eps_sweep=(0.0, 1e-3, 1e-2, 1e-1),
                   draft_eps=1e-2, series_seed=1003),
    "C4": Workload("C4", 64, 8192, 32, 2048, 8, 1.0, "bf16",
                   Arch(24, 1280, 20, 5120), Arch(4, 384, 6, 1536), "separate", "c4",
                   series_seed=1004),
    # The point-token family of the paper's appendix B (its Time-MoE table: input patch 1, a horizon
    # head of 64 steps, K = 3, bf16, a draft of about a quarter of the target's size): tokens are
    # single points, a committed patch is 64 of them.  Context, horizon and model sizes are scaled
    # down from the table's 3072 / 1536 / 453 M so that the oracle decodes a series in seconds.
    "C5": Workload("C5", 16, 768, 64, 384, 3, 1.0, "bf16",
                   Arch(6, 512, 8, 2048), Arch(2, 256, 4, 1024), "separate", "c1",
                   patch_in=1, series_seed=1005),
}


def workload(name: str, **overrides) -> Workload:
    w = WORKLOADS[name]
    return w.with_(**overrides) if overrides else w
