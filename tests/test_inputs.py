"""The seeded generators: determinism, shapes, bf16 rounding, recipe structure."""
import numpy as np
import torch

from tsfm_inputs import WORKLOADS, build_models, make_series, round_to_bf16, workload, tensor_names


def test_workload_shapes_match_the_benchmark_definitions():
    want = {"C0": (7, 4, 0.42, 0.062), "C1": (30, 8, 25.3, 6.4), "C2": (30, 8, 302.0, 1.6),
            "C3": (7, 15, 85.1, 85.1), "C4": (256, 64, 472.0, 7.1)}
    for name, (n, t, pt, pd) in want.items():
        w = WORKLOADS[name]
        assert (w.n_ctx_tokens, w.n_patches) == (n, t)
        assert abs(w.target.n_params(w.patch_len) / 1e6 - pt) / pt < 0.01
        assert abs(w.draft.n_params(w.patch_len) / 1e6 - pd) / pd < 0.02


def test_round_to_bf16_matches_torch():
    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32) * 3
    x[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]       # ties
    want = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    np.testing.assert_array_equal(round_to_bf16(x), want)


def test_weights_are_deterministic_xavier_and_rounded():
    wl = workload("C0")
    a, d = build_models(wl)
    b, _ = build_models(wl)
    assert list(a) == tensor_names(2) and list(d) == tensor_names(1)
    assert all(np.array_equal(a[k], b[k]) for k in a)
    assert abs(a["layers.0.W1"].std() / np.sqrt(2 / (128 + 512)) - 1) < 0.02
    assert a["layers.0.W1"].shape == (512, 128) and a["W_head"].shape == (96, 128)
    assert np.all(a["g_f"] == 1)
    small = workload("C1", target=WORKLOADS["C0"].target, draft=WORKLOADS["C0"].target.__class__(1, 128, 4, 512))
    t, dr = build_models(small)
    assert np.array_equal(round_to_bf16(t["layers.1.Wq"]), t["layers.1.Wq"])
    assert dr["layers.0.Wq"] is t["layers.0.Wq"]


def test_series_recipes():
    for name in WORKLOADS:
        wl = WORKLOADS[name]
        s = make_series(wl, batch=4)
        assert s.shape == (4, wl.ctx_len + wl.horizon) and s.dtype == np.float32
        np.testing.assert_allclose(s.mean(axis=1), 0, atol=1e-4)
        np.testing.assert_allclose(s.std(axis=1), 1, atol=1e-3)
        np.testing.assert_array_equal(s, make_series(wl, batch=4))
    # C0: the daily cycle dominates after detrending
    s = make_series(WORKLOADS["C0"])[0].astype(np.float64)
    t = np.arange(s.size)
    s = s - np.polyval(np.polyfit(t, s, 1), t)
    spec = np.abs(np.fft.rfft(s))
    assert abs(s.size / np.argmax(spec[1:] + 0) - 24) < 1.5 or abs(s.size / (np.argmax(spec[1:]) + 1) - 24) < 1.5
