"""ctypes binding of libtsfm_spec.so: argument marshalling only.

Every function mirrors the C entry point of the same name in include/tsfm.h.  torch is used
for device memory and streams; no step of the decoding path runs in Python.  There is no
fallback: if the shared library is missing or cannot be loaded, importing this module fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np

from . import build as _build

TSFM_OK = 0
TSFM_ERR_ARG, TSFM_ERR_SHAPE, TSFM_ERR_ARCH, TSFM_ERR_CUDA, TSFM_ERR_TIMEOUT, TSFM_ERR_INTERNAL = -1, -2, -3, -4, -5, -6
TSFM_F32, TSFM_BF16 = 0, 1
TSFM_DRAFT_SEPARATE, TSFM_DRAFT_LAYER_SKIP = 0, 1
TSFM_GEMM_AUTO, TSFM_GEMM_SIMT, TSFM_GEMM_WS = 0, 1, 2
TSFM_EXEC_GRAPH, TSFM_EXEC_STREAM, TSFM_EXEC_NO_PDL, TSFM_EXEC_NO_COMPACT, TSFM_EXEC_CHECK_BOUNDS = 0, 1, 2, 4, 8
TSFM_MAX_K = 32

EXPORTS = [
    "tsfm_weights_bytes", "tsfm_weights_offset", "tsfm_weights_bytes_io", "tsfm_weights_offset_io", "tsfm_spec_create", "tsfm_spec_forecast", "tsfm_spec_forecast_variant",
    "tsfm_target_only_forecast", "tsfm_draft_only_forecast", "tsfm_spec_forecast_host", "tsfm_target_only_forecast_host",
    "tsfm_spec_last_trace", "tsfm_accept_round", "tsfm_model_forward", "tsfm_gemm_bf16", "tsfm_gemm_bf16_static",
    "tsfm_spec_debug_guard", "tsfm_spec_set_profiling", "tsfm_spec_kernel_profile", "tsfm_advise_block_size", "tsfm_spec_destroy", "tsfm_launch_count", "tsfm_strerror", "tsfm_last_cuda_error",
]


class tsfm_arch(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32), ("d_ff", C.c_int32)]


class tsfm_cfg(C.Structure):
    _fields_ = [("target", tsfm_arch), ("draft", tsfm_arch),
                ("patch_len", C.c_int32), ("dtype", C.c_int32), ("draft_mode", C.c_int32),
                ("max_batch", C.c_int32), ("max_ctx_tokens", C.c_int32),
                ("max_horizon_patches", C.c_int32), ("max_K", C.c_int32), ("gemm_backend", C.c_int32),
                ("rms_eps", C.c_float), ("norm_eps", C.c_float), ("rope_base", C.c_float),
                ("exec_mode", C.c_int32), ("patch_in", C.c_int32), ("stream", C.c_void_p)]


class tsfm_weights(C.Structure):
    _fields_ = [("blob", C.c_void_p), ("bytes", C.c_size_t)]


class tsfm_stats(C.Structure):
    _fields_ = [("rounds", C.c_int64), ("proposals_drafted", C.c_int64), ("proposals_tested", C.c_int64),
                ("proposals_accepted", C.c_int64), ("patches_committed", C.c_int64),
                ("near_margin_decisions", C.c_int64),
                ("tested_by_pos", C.c_int64 * TSFM_MAX_K), ("accepted_by_pos", C.c_int64 * TSFM_MAX_K),
                ("L_hist", C.c_int64 * (TSFM_MAX_K + 2)),
                ("ms_total", C.c_float), ("ms_prefill", C.c_float), ("ms_draft", C.c_float),
                ("ms_verify", C.c_float), ("ms_accept", C.c_float),
                ("device_status", C.c_int32), ("reserved0", C.c_int32)]

    def as_dict(self):
        d = {k: getattr(self, k) for k, _ in self._fields_ if k not in ("tested_by_pos", "accepted_by_pos", "L_hist", "reserved0")}
        d["tested_by_pos"] = list(self.tested_by_pos)
        d["accepted_by_pos"] = list(self.accepted_by_pos)
        d["L_hist"] = list(self.L_hist)
        return d


class tsfm_variant(C.Structure):
    _fields_ = [("sigma_q", C.c_float), ("fallback_noise", C.c_float), ("sample_proposals", C.c_int32),
                ("no_tempering", C.c_int32)]


class tsfm_kernel_stat(C.Structure):
    _fields_ = [("name", C.c_char * 24), ("launches", C.c_int64), ("ms_total", C.c_double),
                ("bytes", C.c_double), ("flops", C.c_double)]


def _load() -> C.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python paper_2511_18191_b200/build.py` "
                          "(nvcc, sm_100a); there is no fallback implementation")
    lib = C.CDLL(path)
    i32, f32, u64, vp, sz = C.c_int32, C.c_float, C.c_uint64, C.c_void_p, C.c_size_t
    lib.tsfm_weights_bytes.restype = sz
    lib.tsfm_weights_bytes.argtypes = [C.POINTER(tsfm_arch), i32, i32]
    lib.tsfm_weights_offset.restype = sz
    lib.tsfm_weights_offset.argtypes = [C.POINTER(tsfm_arch), i32, i32, i32, C.c_char_p]
    lib.tsfm_weights_bytes_io.restype = sz
    lib.tsfm_weights_bytes_io.argtypes = [C.POINTER(tsfm_arch), i32, i32, i32]
    lib.tsfm_weights_offset_io.restype = sz
    lib.tsfm_weights_offset_io.argtypes = [C.POINTER(tsfm_arch), i32, i32, i32, i32, C.c_char_p]
    lib.tsfm_spec_create.restype = C.c_int
    lib.tsfm_spec_create.argtypes = [C.POINTER(tsfm_weights), C.POINTER(tsfm_weights), C.POINTER(tsfm_cfg), C.POINTER(vp)]
    for name in ("tsfm_spec_forecast", "tsfm_spec_forecast_host"):
        fn = getattr(lib, name)
        fn.restype = C.c_int
        fn.argtypes = [vp, vp, i32, i32, i32, i32, f32, u64, vp, C.POINTER(tsfm_stats)]
    lib.tsfm_spec_forecast_variant.restype = C.c_int
    lib.tsfm_spec_forecast_variant.argtypes = [vp, vp, i32, i32, i32, i32, f32, u64, C.POINTER(tsfm_variant), vp,
                                               C.POINTER(tsfm_stats)]
    for name in ("tsfm_target_only_forecast", "tsfm_draft_only_forecast", "tsfm_target_only_forecast_host"):
        fn = getattr(lib, name)
        fn.restype = C.c_int
        fn.argtypes = [vp, vp, i32, i32, i32, vp, C.POINTER(tsfm_stats)]
    lib.tsfm_spec_last_trace.restype = C.c_int
    lib.tsfm_spec_last_trace.argtypes = [vp, i32, C.POINTER(i32), vp, vp, vp]
    lib.tsfm_accept_round.restype = C.c_int
    lib.tsfm_accept_round.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, f32, f32, u64, i32, i32, vp, vp, vp, vp, vp, vp]
    lib.tsfm_model_forward.restype = C.c_int
    lib.tsfm_model_forward.argtypes = [vp, i32, vp, i32, i32, vp]
    lib.tsfm_gemm_bf16.restype = C.c_int
    lib.tsfm_gemm_bf16.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32]
    lib.tsfm_gemm_bf16_static.restype = C.c_int
    lib.tsfm_gemm_bf16_static.argtypes = [vp, vp, vp, vp, i32, i32, i32]
    lib.tsfm_spec_debug_guard.restype = C.c_int
    lib.tsfm_spec_debug_guard.argtypes = [vp, i32, i32, C.POINTER(i32)]
    lib.tsfm_spec_set_profiling.restype = C.c_int
    lib.tsfm_spec_set_profiling.argtypes = [vp, i32]
    lib.tsfm_spec_kernel_profile.restype = C.c_int
    lib.tsfm_spec_kernel_profile.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(tsfm_kernel_stat)]
    lib.tsfm_advise_block_size.restype = C.c_int32
    lib.tsfm_advise_block_size.argtypes = [C.c_double, C.c_double, C.c_double, i32, C.POINTER(C.c_double)]
    lib.tsfm_spec_destroy.restype = C.c_int
    lib.tsfm_spec_destroy.argtypes = [vp]
    lib.tsfm_launch_count.restype = C.c_int64
    lib.tsfm_launch_count.argtypes = []
    lib.tsfm_strerror.restype = C.c_char_p
    lib.tsfm_strerror.argtypes = [C.c_int]
    lib.tsfm_last_cuda_error.restype = C.c_char_p
    lib.tsfm_last_cuda_error.argtypes = []
    return lib


lib = _load()


class TsfmError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib.tsfm_strerror(code).decode()
        if code in (TSFM_ERR_CUDA, TSFM_ERR_INTERNAL):
            msg += " (" + lib.tsfm_last_cuda_error().decode() + ")"
        super().__init__(f"{where}: {msg} [{code}]")


def _check(code: int, where: str) -> None:
    if code != TSFM_OK:
        raise TsfmError(code, where)


def _ptr(t) -> Optional[int]:
    """Address of a torch tensor / numpy array (None -> NULL)."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _arch(a) -> tsfm_arch:
    return tsfm_arch(a.n_layers, a.d_model, a.n_heads, a.d_ff)


def _dtype_code(dtype: str) -> int:
    return {"f32": TSFM_F32, "bf16": TSFM_BF16}[dtype]


# ---------------------------------------------------------------- weight blobs
def tsfm_weights_bytes(arch, patch_len: int, dtype: str) -> int:
    a = _arch(arch)
    return int(lib.tsfm_weights_bytes(C.byref(a), patch_len, _dtype_code(dtype)))


def tsfm_weights_offset(arch, patch_len: int, dtype: str, layer: int, name: str) -> int:
    a = _arch(arch)
    return int(lib.tsfm_weights_offset(C.byref(a), patch_len, _dtype_code(dtype), layer, name.encode()))


def tsfm_weights_bytes_io(arch, patch_in: int, patch_len: int, dtype: str) -> int:
    a = _arch(arch)
    return int(lib.tsfm_weights_bytes_io(C.byref(a), patch_in, patch_len, _dtype_code(dtype)))


def tsfm_weights_offset_io(arch, patch_in: int, patch_len: int, dtype: str, layer: int, name: str) -> int:
    a = _arch(arch)
    return int(lib.tsfm_weights_offset_io(C.byref(a), patch_in, patch_len, _dtype_code(dtype), layer, name.encode()))


def pack_weights(weights: Dict[str, np.ndarray], arch, patch_len: int, dtype: str, patch_in: int = 0) -> np.ndarray:
    """Serialise a name -> float32 array dict into the blob layout of include/tsfm.h (host bytes)."""
    total = tsfm_weights_bytes_io(arch, patch_in, patch_len, dtype)
    if total == 0:
        raise ValueError("unsupported model shape")
    blob = np.zeros(total, dtype=np.uint8)
    hdr = blob[:36].view(np.int32)
    hdr[:] = [0x4D465354, 1, _dtype_code(dtype), arch.n_layers, arch.d_model, arch.n_heads, arch.d_ff, patch_len,
              patch_in]
    for name, w in weights.items():
        parts = name.split(".")
        layer, short = (int(parts[1]), parts[2]) if parts[0] == "layers" else (-1, name)
        off = tsfm_weights_offset_io(arch, patch_in, patch_len, dtype, layer, short)
        if off == 0:
            raise ValueError(f"no slot for tensor {name}")
        w32 = np.ascontiguousarray(w, dtype=np.float32)
        if w32.ndim == 1 or dtype == "f32":
            raw = w32.view(np.uint8).reshape(-1)
        else:                                   # values are already bf16-representable: keep the top half
            u = w32.view(np.uint32)
            if np.any(u & 0xFFFF):
                raise ValueError(f"tensor {name} is not bf16-representable")
            raw = (u >> 16).astype(np.uint16).view(np.uint8).reshape(-1)
        blob[off:off + raw.size] = raw
    return blob


# ---------------------------------------------------------------- decoder handle
def tsfm_spec_create(target_blob, draft_blob, cfg: tsfm_cfg) -> int:
    """target_blob / draft_blob: torch.uint8 CUDA tensors (kept alive by the caller). Returns the handle."""
    tw = tsfm_weights(_ptr(target_blob), target_blob.numel())
    dw = tsfm_weights(_ptr(draft_blob), draft_blob.numel()) if draft_blob is not None else None
    h = C.c_void_p()
    _check(lib.tsfm_spec_create(C.byref(tw), C.byref(dw) if dw is not None else None, C.byref(cfg), C.byref(h)),
           "tsfm_spec_create")
    return h.value


def tsfm_spec_destroy(h: int) -> None:
    _check(lib.tsfm_spec_destroy(h), "tsfm_spec_destroy")


def tsfm_spec_forecast(h, series, B, ctx_len, H, K, tau, seed, out, stats: Optional[tsfm_stats] = None) -> None:
    _check(lib.tsfm_spec_forecast(h, _ptr(series), B, ctx_len, H, K, tau, seed, _ptr(out),
                                  C.byref(stats) if stats is not None else None), "tsfm_spec_forecast")


def tsfm_spec_forecast_variant(h, series, B, ctx_len, H, K, tau, seed, variant: Optional[tsfm_variant], out,
                               stats: Optional[tsfm_stats] = None) -> None:
    _check(lib.tsfm_spec_forecast_variant(h, _ptr(series), B, ctx_len, H, K, tau, seed,
                                          C.byref(variant) if variant is not None else None, _ptr(out),
                                          C.byref(stats) if stats is not None else None), "tsfm_spec_forecast_variant")


def tsfm_target_only_forecast(h, series, B, ctx_len, H, out, stats: Optional[tsfm_stats] = None) -> None:
    _check(lib.tsfm_target_only_forecast(h, _ptr(series), B, ctx_len, H, _ptr(out),
                                         C.byref(stats) if stats is not None else None), "tsfm_target_only_forecast")


def tsfm_draft_only_forecast(h, series, B, ctx_len, H, out, stats: Optional[tsfm_stats] = None) -> None:
    _check(lib.tsfm_draft_only_forecast(h, _ptr(series), B, ctx_len, H, _ptr(out),
                                        C.byref(stats) if stats is not None else None), "tsfm_draft_only_forecast")


def tsfm_spec_forecast_host(h, series, B, ctx_len, H, K, tau, seed, out, stats: Optional[tsfm_stats] = None) -> None:
    _check(lib.tsfm_spec_forecast_host(h, _ptr(series), B, ctx_len, H, K, tau, seed, _ptr(out),
                                       C.byref(stats) if stats is not None else None), "tsfm_spec_forecast_host")


def tsfm_target_only_forecast_host(h, series, B, ctx_len, H, out, stats: Optional[tsfm_stats] = None) -> None:
    _check(lib.tsfm_target_only_forecast_host(h, _ptr(series), B, ctx_len, H, _ptr(out),
                                              C.byref(stats) if stats is not None else None),
           "tsfm_target_only_forecast_host")


def tsfm_spec_last_trace(h, B: int, K: int, cap_rounds: int):
    """Returns (n_accept [R, B] int32, ell [R, B, K] f32, log_u [R, B, K] f32) as numpy arrays."""
    n_acc = np.empty((cap_rounds, B), dtype=np.int32)
    ell = np.empty((cap_rounds, B, K), dtype=np.float32)
    log_u = np.empty((cap_rounds, B, K), dtype=np.float32)
    r = C.c_int32(0)
    _check(lib.tsfm_spec_last_trace(h, cap_rounds, C.byref(r), _ptr(n_acc), _ptr(ell), _ptr(log_u)),
           "tsfm_spec_last_trace")
    R = r.value
    return n_acc[:R], ell[:R], log_u[:R]


def tsfm_accept_round(stream, x, mu_q, mu_p, B, K, P, T, sigma_p, sigma_q, seed, round_idx, series0,
                      forced_u, done, commit, n_accept, ell, log_u) -> None:
    _check(lib.tsfm_accept_round(stream, _ptr(x), _ptr(mu_q), _ptr(mu_p), B, K, P, T, sigma_p, sigma_q, seed,
                                 round_idx, series0, _ptr(forced_u), _ptr(done), _ptr(commit), _ptr(n_accept),
                                 _ptr(ell), _ptr(log_u)), "tsfm_accept_round")


def tsfm_model_forward(h, which: int, tokens, B: int, n: int, out) -> None:
    _check(lib.tsfm_model_forward(h, which, _ptr(tokens), B, n, _ptr(out)), "tsfm_model_forward")


def tsfm_gemm_bf16(stream, A, W, Cout, M: int, N: int, Kd: int, backend: int) -> None:
    _check(lib.tsfm_gemm_bf16(stream, _ptr(A), _ptr(W), _ptr(Cout), M, N, Kd, backend), "tsfm_gemm_bf16")


TSFM_STATIC_GEMM_MAX_ELEMS = 1 << 20


def tsfm_gemm_bf16_static(stream, A, W, Cout, M: int, N: int, Kd: int) -> None:
    """The contraction of tsfm_gemm_bf16 without any device allocation (scratch is a fixed array inside
    the library; M * N <= TSFM_STATIC_GEMM_MAX_ELEMS; calls on one device must not overlap)."""
    code = lib.tsfm_gemm_bf16_static(stream, _ptr(A), _ptr(W), _ptr(Cout), M, N, Kd)
    if code == TSFM_ERR_SHAPE:
        raise TsfmError(code, "tsfm_gemm_bf16_static: " + lib.tsfm_last_cuda_error().decode())
    _check(code, "tsfm_gemm_bf16_static")


def tsfm_spec_debug_guard(h, region: int = -1, damage: bool = False) -> int:
    """Bounds-checking mode: number of guard regions; region >= 0 damages / restores one byte of it."""
    n = C.c_int32(0)
    _check(lib.tsfm_spec_debug_guard(h, region, int(bool(damage)), C.byref(n)), "tsfm_spec_debug_guard")
    return n.value


def tsfm_spec_set_profiling(h, enable: bool) -> None:
    _check(lib.tsfm_spec_set_profiling(h, int(bool(enable))), "tsfm_spec_set_profiling")


def tsfm_spec_kernel_profile(h):
    """Per-kernel {name: dict(launches, ms_total, bytes, flops)} of the launches since profiling was enabled."""
    arr = (tsfm_kernel_stat * 32)()
    n = C.c_int32(0)
    _check(lib.tsfm_spec_kernel_profile(h, 32, C.byref(n), arr), "tsfm_spec_kernel_profile")
    return {arr[i].name.decode(): dict(launches=arr[i].launches, ms_total=arr[i].ms_total, bytes=arr[i].bytes,
                                       flops=arr[i].flops) for i in range(n.value)}


def tsfm_advise_block_size(alpha: float, c: float, v: float, max_K: int):
    """(K, predicted speedup) by the marginal-gain rule; K == 0 on invalid arguments."""
    s = C.c_double(0.0)
    k = int(lib.tsfm_advise_block_size(alpha, c, v, max_K, C.byref(s)))
    return k, s.value


def tsfm_launch_count() -> int:
    return int(lib.tsfm_launch_count())


# ---------------------------------------------------------------- convenience wrapper
class SpecDecoder:
    """Owns device copies of the weight blobs and a decoder handle for one workload shape."""

    def __init__(self, target_w, draft_w, target_arch, draft_arch, patch_len: int, dtype: str,
                 draft_mode: str, max_batch: int, max_ctx_tokens: int, max_horizon_patches: int, max_K: int,
                 gemm_backend: int = TSFM_GEMM_AUTO, exec_mode: int = TSFM_EXEC_GRAPH, device: str = "cuda:0",
                 patch_in: int = 0):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.patch_len, self.dtype = patch_len, dtype
        self.target_blob = torch.from_numpy(pack_weights(target_w, target_arch, patch_len, dtype, patch_in)).to(self.device)
        self.draft_blob = None
        if draft_mode != "layer_skip":
            self.draft_blob = torch.from_numpy(pack_weights(draft_w, draft_arch, patch_len, dtype, patch_in)).to(self.device)
        cfg = tsfm_cfg()
        cfg.target, cfg.draft = _arch(target_arch), _arch(draft_arch)
        cfg.patch_len, cfg.dtype = patch_len, _dtype_code(dtype)
        cfg.patch_in = patch_in
        cfg.draft_mode = TSFM_DRAFT_LAYER_SKIP if draft_mode == "layer_skip" else TSFM_DRAFT_SEPARATE
        cfg.max_batch, cfg.max_ctx_tokens = max_batch, max_ctx_tokens
        cfg.max_horizon_patches, cfg.max_K = max_horizon_patches, max_K
        cfg.gemm_backend = gemm_backend
        cfg.exec_mode = exec_mode
        cfg.rms_eps, cfg.norm_eps, cfg.rope_base = 1e-6, 1e-5, 1e4
        cfg.stream = torch.cuda.current_stream(self.device).cuda_stream
        self.cfg = cfg
        self.max_T, self.max_K = max_horizon_patches, max_K
        self.h = tsfm_spec_create(self.target_blob, self.draft_blob, cfg)

    @classmethod
    def for_workload(cls, wl, target_w, draft_w, max_K: Optional[int] = None, batch: Optional[int] = None, **kw):
        ks = max(wl.K_sweep) if wl.K_sweep else wl.K
        return cls(target_w, draft_w, wl.target, wl.draft, wl.patch_len, wl.dtype,
                   "layer_skip" if wl.draft_mode == "layer_skip" else "separate",
                   batch or wl.batch, wl.n_ctx_tokens, wl.n_patches, max_K or ks, patch_in=wl.patch_in, **kw)

    def close(self):
        if getattr(self, "h", None):
            tsfm_spec_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def forecast(self, series, H: int, K: int, tau: float, seed: int, out=None, stats: bool = True,
                 variant: Optional[tsfm_variant] = None):
        """series: CUDA float32 [B, ctx_len]. Returns (out [B, H] CUDA, tsfm_stats | None)."""
        B, ctx_len = series.shape
        if out is None:
            out = self.torch.empty((B, H), dtype=self.torch.float32, device=series.device)
        st = tsfm_stats() if stats else None
        if variant is None:
            tsfm_spec_forecast(self.h, series, B, ctx_len, H, K, tau, seed, out, st)
        else:
            tsfm_spec_forecast_variant(self.h, series, B, ctx_len, H, K, tau, seed, variant, out, st)
        return out, st

    def target_only(self, series, H: int, out=None, stats: bool = True):
        B, ctx_len = series.shape
        if out is None:
            out = self.torch.empty((B, H), dtype=self.torch.float32, device=series.device)
        st = tsfm_stats() if stats else None
        tsfm_target_only_forecast(self.h, series, B, ctx_len, H, out, st)
        return out, st

    def draft_only(self, series, H: int, out=None, stats: bool = True):
        B, ctx_len = series.shape
        if out is None:
            out = self.torch.empty((B, H), dtype=self.torch.float32, device=series.device)
        st = tsfm_stats() if stats else None
        tsfm_draft_only_forecast(self.h, series, B, ctx_len, H, out, st)
        return out, st

    def last_trace(self, B: int, K: int):
        return tsfm_spec_last_trace(self.h, B, K, self.max_T)

    def model_forward(self, which: int, tokens):
        B, n, _ = tokens.shape                                # [B, n, P_in]
        out = self.torch.empty((B, n, self.patch_len), dtype=tokens.dtype, device=tokens.device)
        tsfm_model_forward(self.h, which, tokens, B, n, out)
        return out
