"""CPU oracle for Gaussian speculative decoding of continuous patches (fp64).

TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, obviously-correct
restatement of what the decoding path computes, written from the paper.  It is
imported by the tests, by the smoke check and by the benchmark's CPU-baseline
leg, and by nothing else; the CUDA library shares no code with it.

What follows the paper, and where:

* patch-autoregressive decoding, T = ceil(H / P) sequential target forwards
  (Preliminaries, Eq. 1)                                   -> forecast_target_only
* Gaussian surrogate heads with a supplied shared scale sigma (Section 3.1,
  Eq. 4) and the 1/d-scaled log likelihood ratio (Section 3.2, Eq. 5)
                                                           -> log_ratio
* mean-propagating proposals x_i = mu_q^(i), target-mean fallback r = 0, bonus
  patch on full acceptance (Section 3.3, Eq. 6)            -> speculative_round
* left-to-right acceptance, stop at the first rejection (Section 3.2;
  Algorithm 1)                                             -> speculative_round
* one causal verification pass over [h, x_1..x_K] read at the K+1 prefix
  boundaries, instance statistics frozen on the context (Section 3.4; boundary
  index N-1+i, appendix B "Per-Family Boundary Indexing")  -> speculative_round
* capped-geometric block length and dependence band (Eq. 7; appendix
  propositions on block length and dependence)             -> capped_geometric_*
* input tokens shorter than the predicted patch (the point-token family of
  appendix B: input patch length P_in, a horizon head of P steps): a patch is
  P / P_in tokens and the boundary of prefix i sits at token
  N - 1 + i (P / P_in) (appendix B "Per-Family Boundary Indexing")
                                                           -> speculative_round, boundary_indices

The paper fixes the decoding rule but not the network: it says only
"decoder-only Transformer / point head".  The transformer below (pre-norm,
RMSNorm, rotate-half RoPE on the patch index, exact-erf GELU MLP, linear patch
embedding and linear mean head, no biases) is this build's reading.  Forward
numerics are therefore NOT pinned by any value the paper prints; they are
pinned to library routines and mathematical invariants instead (see
tests/test_oracle_forward.py).  The decoding rule is pinned to the paper's
Figure 1 example, its sigma -> 0 and draft == target statements, Proposition 1
and the capped-geometric law (tests/test_oracle_rule.py).

Uniform draws: Philox4x32-10 (Salmon et al., SC'11), key = (seed low, seed
high), counter = (series, round, position, 0), first output word w,
u = ((w >> 9) + 0.5) * 2^-23, so u is never 0 or 1 and is exact in fp32.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np
from scipy.special import erf as _erf

RMS_EPS = 1e-6
NORM_EPS = 1e-5
ROPE_BASE = 1e4

# ----------------------------------------------------------------------------
# Philox4x32-10 (counter-based uniforms)
# ----------------------------------------------------------------------------
_PHILOX_M0 = 0xD2511F53
_PHILOX_M1 = 0xCD9E8D57
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85
_MASK32 = 0xFFFFFFFF


def philox4x32_10(counter: Sequence[int], key: Sequence[int]) -> List[int]:
    """Ten rounds of Philox-4x32 on a 128-bit counter with a 64-bit key."""
    c0, c1, c2, c3 = (int(c) & _MASK32 for c in counter)
    k0, k1 = (int(k) & _MASK32 for k in key)
    for _ in range(10):
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> 32, p0 & _MASK32
        hi1, lo1 = p1 >> 32, p1 & _MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & _MASK32, lo1, (hi0 ^ c3 ^ k1) & _MASK32, lo0
        k0 = (k0 + _PHILOX_W0) & _MASK32
        k1 = (k1 + _PHILOX_W1) & _MASK32
    return [c0, c1, c2, c3]


def uniform_from_word(w: int) -> float:
    """23-bit uniform in (0, 1): (2m + 1) / 2^24 with m = w >> 9."""
    return ((int(w) >> 9) + 0.5) * 2.0 ** -23


def acceptance_uniform(seed: int, series: int, rnd: int, pos: int) -> float:
    """u for proposal ``pos`` (0-based) of round ``rnd`` of series ``series``."""
    key = (seed & _MASK32, (seed >> 32) & _MASK32)
    return uniform_from_word(philox4x32_10((series, rnd, pos, 0), key)[0])


NOISE_PROPOSAL = 0x10000000      # counter word 3 of the proposal-noise stream
NOISE_FALLBACK = 0x20000000      # ... of the fallback / bonus noise stream


def standard_normals(seed: int, series: int, rnd: int, pos: int, stream: int, n: int) -> np.ndarray:
    """n standard normal draws for the sampled variants of Section 3.3 (proposal noise, fallback
    noise).  Box-Muller on Philox words: element pair (2j, 2j+1) takes the counter
    (series, round, position, stream | j), u1, u2 from output words 0 and 1 on the same 23-bit grid
    as the acceptance uniforms, z = sqrt(-2 ln u1) * (cos, sin)(2 pi u2)."""
    key = (seed & _MASK32, (seed >> 32) & _MASK32)
    out = np.empty(n)
    for j in range((n + 1) // 2):
        w = philox4x32_10((series, rnd, pos, stream | j), key)
        u1, u2 = uniform_from_word(w[0]), uniform_from_word(w[1])
        rad = math.sqrt(-2.0 * math.log(u1))
        out[2 * j] = rad * math.cos(2.0 * math.pi * u2)
        if 2 * j + 1 < n:
            out[2 * j + 1] = rad * math.sin(2.0 * math.pi * u2)
    return out


@dataclass
class Variant:
    """Knobs of the general rule (Sections 3.2-3.3, Algorithm 1); the deployed scheme is the default.

    sigma_q:           draft surrogate scale (None = sigma_p: the determinant term vanishes)
    sample_proposals:  x_i = mu_q^(i) + sigma_q * eps instead of the mean
    fallback_noise:    r in t = mu_p + r * eps for the correction and the bonus patch
    tempering:         False drops the 1/d factor of Eq. 5 (component ablation)
    """
    sigma_q: Optional[float] = None
    sample_proposals: bool = False
    fallback_noise: float = 0.0
    tempering: bool = True


# ----------------------------------------------------------------------------
# The network (this build's reading; see the header)
# ----------------------------------------------------------------------------
@dataclass
class Model:
    n_layers: int
    d_model: int
    n_heads: int
    d_ff: int
    patch_len: int                # P: steps predicted per forward (length of a committed patch)
    w: Dict[str, np.ndarray]

    @property
    def d_head(self) -> int:
        return self.d_model // self.n_heads

    @property
    def patch_in(self) -> int:
        """P_in: steps per input token (= P for the patch-token families, 1 for point tokens)."""
        return self.w["W_emb"].shape[1]

    @property
    def tokens_per_patch(self) -> int:
        return self.patch_len // self.patch_in


def make_model(weights: Dict[str, np.ndarray], n_layers: int, d_model: int, n_heads: int,
               d_ff: int, patch_len: int) -> Model:
    w = {k: np.asarray(v, dtype=np.float64) for k, v in weights.items()}
    assert w["W_emb"].shape[0] == d_model and patch_len % w["W_emb"].shape[1] == 0
    assert w["W_head"].shape == (patch_len, d_model)
    return Model(n_layers, d_model, n_heads, d_ff, patch_len, w)


def rmsnorm(x: np.ndarray, g: np.ndarray) -> np.ndarray:
    return g * x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + RMS_EPS)


def gelu(x: np.ndarray) -> np.ndarray:
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


def rope(x: np.ndarray, pos: np.ndarray) -> np.ndarray:
    """Rotate-half RoPE.  x: [n, heads, d_h]; pos: [n] absolute token indices."""
    d_h = x.shape[-1]
    half = d_h // 2
    theta = ROPE_BASE ** (-2.0 * np.arange(half, dtype=np.float64) / d_h)
    ang = pos.astype(np.float64)[:, None] * theta[None, :]          # [n, half]
    cos, sin = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


def softmax_rows(s: np.ndarray) -> np.ndarray:
    e = np.exp(s - s.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


@dataclass
class KVCache:
    """Per-series keys/values of every layer, grown by ``forward``; ``length`` is ragged."""
    k: List[np.ndarray]
    v: List[np.ndarray]
    length: int = 0

    @staticmethod
    def empty(model: Model) -> "KVCache":
        z = lambda: np.zeros((0, model.n_heads, model.d_head))
        return KVCache([z() for _ in range(model.n_layers)], [z() for _ in range(model.n_layers)], 0)

    def truncate(self, length: int) -> None:
        assert 0 <= length <= self.length
        self.k = [a[:length] for a in self.k]
        self.v = [a[:length] for a in self.v]
        self.length = length


def forward(model: Model, z: np.ndarray, cache: Optional[KVCache] = None) -> np.ndarray:
    """Next-patch means at every input position.

    z: [n, P_in] input tokens.  Row t of the result is the model's mean for the
    P steps that follow tokens 0..t (of the cache plus ``z``).  With a cache the
    new tokens sit at positions cache.length .. cache.length + n - 1 and their
    keys/values are appended; without one this is the full recomputation.
    """
    w, H, dh = model.w, model.n_heads, model.d_head
    n = z.shape[0]
    start = 0 if cache is None else cache.length
    pos = np.arange(start, start + n)
    x = z.astype(np.float64) @ w["W_emb"].T                          # [n, d]
    for l in range(model.n_layers):
        p = f"layers.{l}."
        a = rmsnorm(x, w[p + "g1"])
        q = rope((a @ w[p + "Wq"].T).reshape(n, H, dh), pos)
        k = rope((a @ w[p + "Wk"].T).reshape(n, H, dh), pos)
        v = (a @ w[p + "Wv"].T).reshape(n, H, dh)
        if cache is not None:
            k = np.concatenate([cache.k[l], k], axis=0)
            v = np.concatenate([cache.v[l], v], axis=0)
            cache.k[l], cache.v[l] = k, v
        ctx = np.empty((n, H, dh))
        for h in range(H):
            s = q[:, h, :] @ k[:, h, :].T / math.sqrt(dh)            # [n, start + n]
            key_pos = np.arange(start + n)
            s = np.where(key_pos[None, :] <= pos[:, None], s, -np.inf)
            ctx[:, h, :] = softmax_rows(s) @ v[:, h, :]
        x = x + ctx.reshape(n, H * dh) @ w[p + "Wo"].T
        m = rmsnorm(x, w[p + "g2"])
        x = x + gelu(m @ w[p + "W1"].T) @ w[p + "W2"].T
    if cache is not None:
        cache.length = start + n
    return rmsnorm(x, w["g_f"]) @ w["W_head"].T


# ----------------------------------------------------------------------------
# Instance normalisation, frozen on the context (Section 3.4)
# ----------------------------------------------------------------------------
def instance_stats(context: np.ndarray):
    c = np.asarray(context, dtype=np.float64)
    m = c.mean()
    sd = math.sqrt(np.mean((c - m) ** 2) + NORM_EPS)
    return m, sd


# ----------------------------------------------------------------------------
# Acceptance rule (Section 3.2, Eq. 5) and one round (Algorithm 1)
# ----------------------------------------------------------------------------
def energy(u: np.ndarray) -> float:
    """Per-dimension energy ||u||_d^2 = ||u||^2 / d."""
    u = np.asarray(u, dtype=np.float64)
    return float(np.dot(u, u)) / u.size


def log_ratio(x, mu_p, mu_q, sigma_p: float, sigma_q: float) -> float:
    """l_i = -||x-mu_p||_d^2 / 2 sigma_p^2 + ||x-mu_q||_d^2 / 2 sigma_q^2 + 0.5 log(sigma_q^2/sigma_p^2)."""
    x = np.asarray(x, dtype=np.float64)
    return (-energy(x - mu_p) / (2.0 * sigma_p ** 2)
            + energy(x - mu_q) / (2.0 * sigma_q ** 2)
            + 0.5 * math.log(sigma_q ** 2 / sigma_p ** 2))


def accept(ell: float, u: float) -> bool:
    """u <= min(1, e^l), taken in the log domain: log u <= min(l, 0)."""
    return math.log(u) <= min(ell, 0.0)


@dataclass
class RoundRecord:
    """What one round of one series did (the parity harness compares these)."""
    n_accept: int                 # leading accepted proposals
    L: int                        # untruncated yield n_accept + 1
    committed: int                # patches kept after truncation to the horizon
    ell: List[float]              # l_i for every tested position
    log_u: List[float]            # log u_i for every tested position
    decisions: List[bool]         # accept/reject for every tested position
    mu_q: np.ndarray              # [K, P] proposals
    mu_p: np.ndarray              # [K+1, P] boundary predictions


def speculative_round(hist: np.ndarray, target: Model, draft: Model, K: int, sigma: float,
                      uniforms: Sequence[float],
                      forced: Optional[Sequence[bool]] = None,
                      caches=None, variant: Optional[Variant] = None,
                      proposal_eps: Optional[np.ndarray] = None,
                      fallback_eps: Optional[np.ndarray] = None) -> RoundRecord:
    """Algorithm 1 for one series; mean proposals and r = 0 unless ``variant`` says otherwise.

    With a variant the standard-normal draws are inputs: ``proposal_eps`` [K, P] for the sampled
    proposals, ``fallback_eps`` [K+1, P] (row i for a correction at position i, row K for the bonus).

    hist: [n, P] context + committed patches (normalised space).  ``uniforms``
    supplies u_1..u_K.  ``forced`` (optional) overrides the decisions, used to
    replay another implementation's accept/reject sequence.  ``caches`` is an
    optional (target KVCache, draft KVCache) pair holding a prefix of ``hist``
    (their lengths count tokens); without it both models recompute from scratch.

    The models read the sequence as tokens of P_in steps (P / P_in of them per
    patch); the target's prediction after prefix i is read at token index
    N - 1 + i (P / P_in), N the token count of ``hist``.
    """
    n = hist.shape[0]
    tc, dc = caches if caches is not None else (None, None)

    def run(model, cache, patches):
        tokens = patches.reshape(-1, model.patch_in)
        if cache is None:
            return forward(model, tokens)
        out = forward(model, tokens[cache.length:], cache)
        return np.concatenate([np.zeros((tokens.shape[0] - out.shape[0], out.shape[1])), out], axis=0)

    var = variant or Variant()
    sigma_q = sigma if var.sigma_q is None else var.sigma_q
    props: List[np.ndarray] = []
    means: List[np.ndarray] = []
    for i in range(K):                                    # draft rollout
        toks = np.concatenate([hist] + [p[None, :] for p in props], axis=0)
        mu = run(draft, dc, toks)[-1]
        means.append(mu)
        props.append(mu + sigma_q * proposal_eps[i] if var.sample_proposals else mu)
    x = np.stack(props, axis=0)                           # x_i = mu_q^(i) (+ sigma_q eps)
    mu_q = np.stack(means, axis=0)
    o = run(target, tc, np.concatenate([hist, x], axis=0))
    at = boundary_indices(n * target.tokens_per_patch, K, target.tokens_per_patch)
    mu_p = o[at]                                          # boundaries N-1+i(P/P_in), i = 0..K
    if var.fallback_noise != 0.0:
        mu_p = mu_p + var.fallback_noise * np.asarray(fallback_eps, dtype=np.float64)
    ell, log_u, dec = [], [], []
    n_acc = 0
    for i in range(K):
        mp_i = o[at[i]]                                   # the statistic uses the noise-free target mean
        l_i = log_ratio(x[i], mp_i, mu_q[i], sigma, sigma_q)
        if not var.tempering:
            l_i *= x.shape[1]                             # l_i is (1/d) log p/q: undo the 1/d
        ok = accept(l_i, uniforms[i]) if forced is None else bool(forced[i])
        ell.append(l_i)
        log_u.append(math.log(uniforms[i]))
        dec.append(ok)
        if not ok:
            break
        n_acc += 1
    return RoundRecord(n_acc, n_acc + 1, n_acc + 1, ell, log_u, dec, x, mu_p)


def boundary_indices(n_tokens: int, K: int, tokens_per_patch: int = 1) -> np.ndarray:
    """Token indices at which the target's predictions mu_p^(1..K+1) are read in the pass over
    [h, x_1..x_K]: N - 1 + i (P / P_in), i = 0..K, with N the token count of h."""
    return n_tokens - 1 + tokens_per_patch * np.arange(K + 1)


def committed_patches(rec: RoundRecord) -> np.ndarray:
    """x_1..x_n followed by mu_p^(n+1) (correction if n < K, bonus if n = K)."""
    return np.concatenate([rec.mu_q[:rec.n_accept], rec.mu_p[rec.n_accept][None, :]], axis=0)


# ----------------------------------------------------------------------------
# Whole forecasts
# ----------------------------------------------------------------------------
def _patches(ctx_norm: np.ndarray, P: int) -> np.ndarray:
    assert ctx_norm.size % P == 0
    return ctx_norm.reshape(-1, P)


def forecast_target_only(target: Model, series: np.ndarray, ctx_len: int, H: int,
                         use_cache: bool = True) -> np.ndarray:
    """Eq. 1: T = ceil(H/P) sequential target forwards per series. series: [B, >= ctx_len]."""
    P = target.patch_len
    T = -(-H // P)
    out = np.empty((series.shape[0], H))
    for b in range(series.shape[0]):
        m, sd = instance_stats(series[b, :ctx_len])
        hist = _patches((series[b, :ctx_len].astype(np.float64) - m) / sd, P)
        cache = KVCache.empty(target) if use_cache else None
        for _ in range(T):
            tokens = hist.reshape(-1, target.patch_in)
            if cache is None:
                mu = forward(target, tokens)[-1]
            else:
                mu = forward(target, tokens[cache.length:], cache)[-1]
            hist = np.concatenate([hist, mu[None, :]], axis=0)
        out[b] = (hist[-T:].reshape(-1) * sd + m)[:H]
    return out


@dataclass
class ForecastTrace:
    rounds: List[List[RoundRecord]] = field(default_factory=list)   # [series][round]

    def yields(self) -> np.ndarray:
        return np.array([r.L for s in self.rounds for r in s])

    def counts_by_position(self, K: int):
        tested = np.zeros(K, dtype=np.int64)
        accepted = np.zeros(K, dtype=np.int64)
        for s in self.rounds:
            for r in s:
                for i, d in enumerate(r.decisions):
                    tested[i] += 1
                    accepted[i] += int(d)
        return tested, accepted


def forecast_speculative(target: Model, draft: Model, series: np.ndarray, ctx_len: int, H: int,
                         K: int, tau: float, seed: int,
                         forced: Optional[List[List[Sequence[bool]]]] = None,
                         use_cache: bool = True, series_index0: int = 0,
                         variant: Optional[Variant] = None):
    """Algorithm 1 looped until T = ceil(H/P) patches are committed, per series.

    Every round drafts K and verifies K+1; the committed list of the last round
    is truncated to the patches still missing.  ``series_index0`` offsets the
    series id used in the uniform counter (to decode a sub-batch of a larger
    batch).  Returns (out [B, H], ForecastTrace).
    """
    P = target.patch_len
    T = -(-H // P)
    out = np.empty((series.shape[0], H))
    trace = ForecastTrace()
    for b in range(series.shape[0]):
        m, sd = instance_stats(series[b, :ctx_len])
        hist = _patches((series[b, :ctx_len].astype(np.float64) - m) / sd, P)
        caches = (KVCache.empty(target), KVCache.empty(draft)) if use_cache else None
        done, rnd, recs = 0, 0, []
        while done < T:
            us = [acceptance_uniform(seed, series_index0 + b, rnd, i) for i in range(K)]
            f = None if forced is None else forced[b][rnd]
            pe = fe = None
            if variant is not None and variant.sample_proposals:
                pe = np.stack([standard_normals(seed, series_index0 + b, rnd, i, NOISE_PROPOSAL, P) for i in range(K)])
            if variant is not None and variant.fallback_noise != 0.0:
                fe = np.stack([standard_normals(seed, series_index0 + b, rnd, i, NOISE_FALLBACK, P) for i in range(K + 1)])
            rec = speculative_round(hist, target, draft, K, tau, us, forced=f, caches=caches, variant=variant,
                                    proposal_eps=pe, fallback_eps=fe)
            new = committed_patches(rec)[: T - done]
            rec.committed = new.shape[0]
            hist = np.concatenate([hist, new], axis=0)
            done += new.shape[0]
            rnd += 1
            recs.append(rec)
            if caches is not None:                       # roll both caches back
                keep = hist.shape[0] - 1                 # everything but the newest patch
                for c, mdl in zip(caches, (target, draft)):
                    c.truncate(min(c.length, keep * mdl.tokens_per_patch))
        trace.rounds.append(recs)
        out[b] = (hist[-T:].reshape(-1) * sd + m)[:H]
    return out, trace


# ----------------------------------------------------------------------------
# Throughput law (Eq. 7, Eq. 8 and the dependence proposition)
# ----------------------------------------------------------------------------
def capped_geometric_pmf(alpha: float, K: int) -> np.ndarray:
    """P(L = l), l = 1..K+1."""
    p = [(1.0 - alpha) * alpha ** (l - 1) for l in range(1, K + 1)] + [alpha ** K]
    return np.array(p)


def capped_geometric_mean(alpha: float, K: int) -> float:
    """E[L] = sum_{j=0}^{K} alpha^j = (1 - alpha^(K+1)) / (1 - alpha)."""
    return float(sum(alpha ** j for j in range(K + 1)))


def predicted_speedup(alpha: float, K: int, c: float, v: float) -> float:
    """S(K) = E[L] / (c K + v)."""
    return capped_geometric_mean(alpha, K) / (c * K + v)


def marginal_gain_holds(alpha: float, K: int, c: float, v: float) -> bool:
    """Marginal-gain condition (appendix proposition on block-size selection):
    S(K+1) >= S(K)  iff  alpha^(K+1) (c K + v) >= c E[L_K]."""
    return alpha ** (K + 1) * (c * K + v) >= c * capped_geometric_mean(alpha, K)


def best_block_size(alpha: float, c: float, v: float, max_K: int) -> int:
    """argmax over K = 1..max_K of S(K) = E[L_K] / (c K + v), by brute force (smallest K on ties)."""
    best, best_s = 1, -1.0
    for K in range(1, max_K + 1):
        s_k = predicted_speedup(alpha, K, c, v)
        if s_k > best_s * (1.0 + 1e-15):
            best, best_s = K, s_k
    return best
