"""Pins for the oracle's transformer forward.

The paper prints no activations, so the network is pinned to library routines (torch's
rms_norm / gelu / scaled_dot_product_attention / linear in fp64, an implementation independent
of the oracle's numpy code) and to mathematical invariants chosen so that a dropped term, a
wrong sign, a wrong index or a transposed operand fails at least one of them.
"""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import tsfm_oracle as orc
from tsfm_inputs import Arch, make_model as make_weights, layer_skip_draft, perturbed_draft


def model(arch=Arch(3, 48, 4, 96), P=10, seed=1, gains=True):
    w = make_weights(arch, P, seed, "f32")
    if gains:                                  # non-trivial gains so that they are exercised
        rng = np.random.default_rng(5)
        for k in w:
            if w[k].ndim == 1:
                w[k] = (1.0 + 0.3 * rng.standard_normal(w[k].shape)).astype(np.float32)
    return orc.make_model(w, arch.n_layers, arch.d_model, arch.n_heads, arch.d_ff, P)


def torch_forward(m: orc.Model, z: np.ndarray) -> np.ndarray:
    """The same network from torch library routines (fp64), RoPE via complex multiplication."""
    w = {k: torch.from_numpy(v) for k, v in m.w.items()}
    n, H, dh = z.shape[0], m.n_heads, m.d_head
    x = F.linear(torch.from_numpy(z).double(), w["W_emb"])
    half = dh // 2
    freqs = torch.outer(torch.arange(n, dtype=torch.float64),
                        1e4 ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh))
    rot = torch.polar(torch.ones_like(freqs), freqs)            # e^{i pos theta_j}

    def rope(t):                                                # t: [n, H, dh], pairs (j, j + dh/2)
        c = torch.complex(t[..., :half], t[..., half:]) * rot[:, None, :]
        return torch.cat([c.real, c.imag], dim=-1)

    for l in range(m.n_layers):
        p = f"layers.{l}."
        a = F.rms_norm(x, (m.d_model,), w[p + "g1"], eps=1e-6)
        q = rope(F.linear(a, w[p + "Wq"]).view(n, H, dh)).transpose(0, 1)
        k = rope(F.linear(a, w[p + "Wk"]).view(n, H, dh)).transpose(0, 1)
        v = F.linear(a, w[p + "Wv"]).view(n, H, dh).transpose(0, 1)
        ctx = F.scaled_dot_product_attention(q, k, v, is_causal=True)
        x = x + F.linear(ctx.transpose(0, 1).reshape(n, -1), w[p + "Wo"])
        h = F.rms_norm(x, (m.d_model,), w[p + "g2"], eps=1e-6)
        x = x + F.linear(F.gelu(F.linear(h, w[p + "W1"])), w[p + "W2"])
    return F.linear(F.rms_norm(x, (m.d_model,), w["g_f"], eps=1e-6), w["W_head"]).numpy()


def test_forward_matches_torch_library_routines():
    for arch, P in [(Arch(3, 48, 4, 96), 10), (Arch(1, 64, 2, 256), 96), (Arch(2, 32, 1, 64), 4)]:
        m = model(arch, P)
        z = np.random.default_rng(0).standard_normal((9, P))
        np.testing.assert_allclose(orc.forward(m, z), torch_forward(m, z), rtol=1e-10, atol=1e-11)


def test_gelu_is_x_times_normal_cdf():
    from scipy.stats import norm
    x = np.linspace(-6, 6, 101)
    np.testing.assert_allclose(orc.gelu(x), x * norm.cdf(x), rtol=1e-12, atol=1e-15)
    assert orc.gelu(np.array([1.0]))[0] == pytest.approx(0.8413447460685429, rel=1e-14)


def test_rmsnorm_output_has_unit_rms_and_applies_gain():
    x = np.random.default_rng(0).standard_normal((5, 64)) * 7.0
    y = orc.rmsnorm(x, np.ones(64))
    np.testing.assert_allclose(np.sqrt((y * y).mean(axis=-1)), 1.0, rtol=1e-6)
    g = np.arange(1, 65, dtype=np.float64)
    np.testing.assert_allclose(orc.rmsnorm(x, g), y * g, rtol=1e-14)
    np.testing.assert_allclose(orc.rmsnorm(3.0 * x, g), orc.rmsnorm(x, g), rtol=1e-6)


def test_rope_properties():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((6, 3, 8))
    np.testing.assert_array_equal(orc.rope(x[:1], np.array([0])), x[:1])       # position 0 = identity
    r = orc.rope(x, np.arange(6))
    np.testing.assert_allclose((r * r).sum(-1), (x * x).sum(-1), rtol=1e-13)  # a rotation
    # scores depend on the position difference only
    q, k = rng.standard_normal((2, 1, 1, 8))
    s = lambda m, n: float((orc.rope(q, np.array([m])) * orc.rope(k, np.array([n]))).sum())
    assert s(5, 2) == pytest.approx(s(13, 10), rel=1e-12)
    assert s(5, 2) != pytest.approx(s(2, 5), rel=1e-3)
    # first pair (j = 0, j + d_h/2) rotates by exactly `pos` radians
    e = np.zeros((1, 1, 8)); e[0, 0, 0] = 1.0
    out = orc.rope(e, np.array([2]))[0, 0]
    assert out[0] == pytest.approx(math.cos(2.0)) and out[4] == pytest.approx(math.sin(2.0))
    # slowest pair: theta = base^(-2 (d_h/2 - 1) / d_h)
    e = np.zeros((1, 1, 8)); e[0, 0, 3] = 1.0
    out = orc.rope(e, np.array([7]))[0, 0]
    assert out[7] == pytest.approx(math.sin(7.0 * 1e4 ** (-6.0 / 8.0)))


def test_single_token_attention_returns_the_value_path():
    """With one token the softmax is 1, so attention adds W_o W_v a regardless of q and k."""
    m = model(Arch(1, 32, 4, 64), 6)
    z = np.random.default_rng(2).standard_normal((1, 6))
    w = m.w
    x = z @ w["W_emb"].T
    a = orc.rmsnorm(x, w["layers.0.g1"])
    x = x + (a @ w["layers.0.Wv"].T) @ w["layers.0.Wo"].T
    h = orc.rmsnorm(x, w["layers.0.g2"])
    x = x + orc.gelu(h @ w["layers.0.W1"].T) @ w["layers.0.W2"].T
    want = orc.rmsnorm(x, w["g_f"]) @ w["W_head"].T
    np.testing.assert_allclose(orc.forward(m, z), want, rtol=1e-12)


def test_forward_is_causal_and_position_dependent():
    m = model()
    rng = np.random.default_rng(3)
    z = rng.standard_normal((8, 10))
    full = orc.forward(m, z)
    for n in (1, 4, 7):
        np.testing.assert_allclose(orc.forward(m, z[:n]), full[:n], rtol=0, atol=1e-12)
    z2 = z.copy(); z2[5] += 1.0
    out2 = orc.forward(m, z2)
    np.testing.assert_array_equal(out2[:5], full[:5])
    assert np.abs(out2[5:] - full[5:]).max() > 1e-3
    # earlier tokens matter (attention is not diagonal), and order matters (RoPE)
    z3 = z.copy(); z3[0] += 1.0
    assert np.abs(orc.forward(m, z3)[7] - full[7]).max() > 1e-4
    z4 = z.copy(); z4[[0, 1]] = z4[[1, 0]]
    assert np.abs(orc.forward(m, z4)[7] - full[7]).max() > 1e-5


def test_kv_cached_forward_matches_full_recompute_and_rolls_back():
    m = model()
    z = np.random.default_rng(4).standard_normal((11, 10))
    full = orc.forward(m, z)
    c = orc.KVCache.empty(m)
    a = orc.forward(m, z[:6], c)
    b = orc.forward(m, z[6:9], c)
    assert c.length == 9
    np.testing.assert_allclose(np.concatenate([a, b]), full[:9], rtol=0, atol=1e-12)
    c.truncate(7)                                   # ragged rollback, then different continuation
    alt = np.concatenate([z[:7], z[9:11]])
    np.testing.assert_allclose(orc.forward(m, z[9:11], c), orc.forward(m, alt)[7:], rtol=0, atol=1e-12)


def test_heads_are_split_contiguously():
    """Zeroing W_o's columns of head h must equal removing that head's value contribution."""
    m = model(Arch(1, 32, 4, 64), 6, gains=False)
    z = np.random.default_rng(6).standard_normal((5, 6))
    base = orc.forward(m, z)
    w2 = dict(m.w)
    wo = w2["layers.0.Wo"].copy(); wo[:, 8:16] = 0.0   # head 1 = features 8..15
    wv = w2["layers.0.Wv"].copy(); wv[8:16, :] = 0.0
    ma = orc.Model(1, 32, 4, 64, 6, {**w2, "layers.0.Wo": wo})
    mb = orc.Model(1, 32, 4, 64, 6, {**w2, "layers.0.Wv": wv})
    np.testing.assert_allclose(orc.forward(ma, z), orc.forward(mb, z), rtol=0, atol=1e-12)
    assert np.abs(orc.forward(ma, z) - base).max() > 1e-4


def test_layer_skip_and_perturbed_drafts():
    arch = Arch(4, 32, 4, 64)
    tw = make_weights(arch, 8, 0, "bf16")
    dw = layer_skip_draft(tw, 2)
    assert dw["layers.1.W1"] is tw["layers.1.W1"] and "layers.2.Wq" not in dw
    assert dw["W_head"] is tw["W_head"] and dw["g_f"] is tw["g_f"]
    p0 = perturbed_draft(tw, 4, 0.0, 1, "bf16")
    assert all(np.array_equal(p0[k], tw[k]) for k in tw)
    p1 = perturbed_draft(tw, 4, 0.1, 1, "bf16")
    rel = np.std(p1["layers.0.Wq"] - tw["layers.0.Wq"]) / np.std(tw["layers.0.Wq"])
    assert 0.08 < rel < 0.12
    assert np.array_equal(p1["g_f"], tw["g_f"])
