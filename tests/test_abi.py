"""The C-ABI library: it loads, exports every symbol the header declares, and its host-only
entry points and argument checks behave as documented (no GPU needed)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    src = open(os.path.join(ROOT, "include", "tsfm.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(tsfm_[a-z0-9_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    import paper_2511_18191_b200 as tsfm
    names = declared_functions()
    assert "tsfm_spec_create" in names and "tsfm_spec_forecast" in names and "tsfm_target_only_forecast" in names
    for n in names:
        assert hasattr(tsfm.lib, n), n
    assert sorted(tsfm.EXPORTS) == names
    for n in names:                                   # the Python binding carries the same names
        assert hasattr(tsfm, n) or n in ("tsfm_strerror", "tsfm_last_cuda_error"), n


def test_blob_layout_and_packing():
    import paper_2511_18191_b200 as tsfm
    from tsfm_inputs import Arch, make_model
    arch, P = Arch(2, 128, 4, 512), 96
    for dtype, e in (("f32", 4), ("bf16", 2)):
        total = tsfm.tsfm_weights_bytes(arch, P, dtype)
        offs = [tsfm.tsfm_weights_offset(arch, P, dtype, -1, "W_emb")]
        for l in range(2):
            offs += [tsfm.tsfm_weights_offset(arch, P, dtype, l, n) for n in ("g1", "Wq", "Wk", "Wv", "Wo", "g2", "W1", "W2")]
        offs += [tsfm.tsfm_weights_offset(arch, P, dtype, -1, "g_f"), tsfm.tsfm_weights_offset(arch, P, dtype, -1, "W_head")]
        assert offs[0] == 256 and all(o % 256 == 0 for o in offs) and offs == sorted(offs) and offs[-1] < total
        wq, wk = offs[2], offs[3]
        assert wk - wq == 128 * 128 * e                # Wq, Wk, Wv adjacent: one [3d, d] matrix
        w = make_model(arch, P, 0, dtype)
        blob = tsfm.pack_weights(w, arch, P, dtype)
        assert blob.size == total and list(blob[:32].view(np.int32)) == [0x4D465354, 1, e == 2, 2, 128, 4, 512, 96]
        if dtype == "f32":
            got = blob[wq:wq + 128 * 128 * 4].view(np.float32).reshape(128, 128)
        else:
            got = (blob[wq:wq + 128 * 128 * 2].view(np.uint16).astype(np.uint32) << 16).view(np.float32).reshape(128, 128)
        np.testing.assert_array_equal(got, w["layers.0.Wq"])
    assert tsfm.tsfm_weights_bytes(Arch(2, 100, 4, 512), P, "f32") == 0
    assert tsfm.tsfm_weights_offset(arch, P, "f32", 5, "Wq") == 0
    assert tsfm.tsfm_weights_offset(arch, P, "f32", 0, "nope") == 0


def test_argument_validation_needs_no_device_and_never_falls_back():
    import torch
    import paper_2511_18191_b200 as tsfm
    lib = tsfm.lib
    assert lib.tsfm_spec_create(None, None, None, None) == tsfm.TSFM_ERR_ARG
    assert lib.tsfm_spec_forecast(None, None, 1, 96, 96, 1, 1.0, 0, None, None) == tsfm.TSFM_ERR_ARG
    assert lib.tsfm_target_only_forecast(None, None, 1, 96, 96, None, None) == tsfm.TSFM_ERR_ARG
    assert lib.tsfm_spec_destroy(None) == tsfm.TSFM_ERR_ARG
    assert lib.tsfm_accept_round(None, None, None, None, 1, 1, 1, 1, 1.0, 1.0, 0, 0, 0, None, None, None, None, None, None) == tsfm.TSFM_ERR_ARG
    assert lib.tsfm_gemm_bf16(None, None, None, None, 1, 1, 64, 0) == tsfm.TSFM_ERR_ARG
    assert lib.tsfm_strerror(tsfm.TSFM_ERR_TIMEOUT).decode().startswith("bounded")
    assert tsfm.tsfm_launch_count() >= 0
    if not torch.cuda.is_available():
        # a valid create on a machine without a device fails loudly: there is no CPU path
        cfg = tsfm.tsfm_cfg()
        cfg.target = cfg.draft = tsfm.tsfm_arch(1, 64, 2, 64)
        cfg.patch_len, cfg.dtype, cfg.max_batch, cfg.max_ctx_tokens = 16, 0, 1, 2
        cfg.max_horizon_patches, cfg.max_K = 1, 1
        cfg.rms_eps, cfg.norm_eps, cfg.rope_base = 1e-6, 1e-5, 1e4
        buf = (C.c_char * 1024)()
        w = tsfm.tsfm_weights(C.addressof(buf), 1 << 30)
        h = C.c_void_p()
        rc = lib.tsfm_spec_create(C.byref(w), C.byref(w), C.byref(cfg), C.byref(h))
        assert rc in (tsfm.TSFM_ERR_CUDA, tsfm.TSFM_ERR_ARCH) and not h.value


def test_block_size_advice_agrees_with_the_oracle_rule():
    import paper_2511_18191_b200 as tsfm
    from oracle import tsfm_oracle as orc
    for alpha in (0.0, 0.2, 0.6, 0.9, 0.99, 1.0):
        for c in (0.04, 0.25, 1.0):
            for v in (1.0, 1.44, 2.5):
                k, s = tsfm.tsfm_advise_block_size(alpha, c, v, 32)
                best = orc.best_block_size(alpha, c, v, 32)
                assert s == pytest.approx(orc.predicted_speedup(alpha, k, c, v), rel=1e-12)
                assert s == pytest.approx(orc.predicted_speedup(alpha, best, c, v), rel=1e-9)
    assert tsfm.tsfm_advise_block_size(1.5, 0.1, 1.0, 8)[0] == 0
    assert tsfm.tsfm_advise_block_size(0.5, 0.0, 1.0, 8)[0] == 0
    assert tsfm.tsfm_advise_block_size(0.5, 0.1, 1.0, 0)[0] == 0


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2511_18191_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read(), f
