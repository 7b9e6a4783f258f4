"""Pins for the oracle's decoding rule: what the paper and the mathematics fix.

Every test here runs on CPU.  None of them re-types the oracle's own formula as its
expected value: expectations come from the paper's worked example (Figure 1), its limit
statements (sigma -> 0, draft == target), Proposition 1's closed form, the capped-geometric
law, published Philox known answers, and brute force.
"""
import math
import os

import numpy as np
import pytest

from oracle import tsfm_oracle as orc
from tsfm_inputs import Arch, make_model as make_weights, perturbed_draft

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def tiny_models(P=8, seed=3, same=False):
    ta, da = Arch(2, 32, 4, 64), Arch(1, 16, 2, 32)
    tw = make_weights(ta, P, seed, "f32", stream=0)
    target = orc.make_model(tw, ta.n_layers, ta.d_model, ta.n_heads, ta.d_ff, P)
    if same:
        return target, target
    dw = make_weights(da, P, seed, "f32", stream=1)
    return target, orc.make_model(dw, da.n_layers, da.d_model, da.n_heads, da.d_ff, P)


def toy_series(B, n, seed=0):
    rng = np.random.default_rng(seed)
    t = np.arange(n)[None, :]
    return np.sin(2 * np.pi * t / 12.0 + rng.uniform(0, 6, (B, 1))) + 0.1 * rng.standard_normal((B, n))


# ---------------------------------------------------------------- Philox ----
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l[0] != "#"]
    assert len(rows) == 2
    for r in rows:
        v = [int(x, 16) for x in r]
        assert orc.philox4x32_10(v[0:4], v[4:6]) == v[6:10]


def test_philox_is_a_bijection_of_the_counter_and_uniforms_are_open_interval():
    seen = {tuple(orc.philox4x32_10((i, 0, 0, 0), (1, 2))) for i in range(2000)}
    assert len(seen) == 2000
    assert orc.uniform_from_word(0) == 2.0 ** -24
    assert orc.uniform_from_word(0xFFFFFFFF) == 1.0 - 2.0 ** -24
    assert np.float32(orc.uniform_from_word(0x12345678)) == orc.uniform_from_word(0x12345678)
    us = np.array([orc.acceptance_uniform(2021, b, r, k)
                   for b in range(20) for r in range(20) for k in range(10)])
    assert abs(us.mean() - 0.5) < 0.02 and abs(us.var() - 1 / 12) < 0.01
    assert orc.acceptance_uniform(2021, 1, 0, 0) != orc.acceptance_uniform(2021, 0, 1, 0)
    assert orc.acceptance_uniform(2021, 0, 0, 1) != orc.acceptance_uniform(2021, 0, 1, 0)
    assert orc.acceptance_uniform(2021, 3, 4, 5) != orc.acceptance_uniform(2022, 3, 4, 5)
    assert orc.acceptance_uniform(2021 + (7 << 32), 3, 4, 5) != orc.acceptance_uniform(2021, 3, 4, 5)


# ---------------------------------------------------- Eq. 5: the statistic ----
def test_log_ratio_is_the_tempered_gaussian_log_density_ratio():
    """Eq. 5 is (1/d) log[p(x)/q(x)] for isotropic Gaussians: check against scipy's densities."""
    from scipy.stats import multivariate_normal as mvn
    rng = np.random.default_rng(0)
    for d, sp, sq in [(4, 0.7, 0.7), (6, 0.5, 1.3), (3, 2.0, 0.4)]:
        x, mp, mq = rng.standard_normal((3, d))
        want = (mvn.logpdf(x, mp, sp ** 2 * np.eye(d)) - mvn.logpdf(x, mq, sq ** 2 * np.eye(d))) / d
        assert orc.log_ratio(x, mp, mq, sp, sq) == pytest.approx(want, rel=1e-12, abs=1e-12)


def test_mean_proposal_collapses_to_the_distance_gate():
    """Eq. 6: x = mu_q, sigma_p = sigma_q = sigma  =>  alpha = exp(-Delta^2 / 2 sigma^2)."""
    mq = np.array([1.0, 2.0, 3.0, 4.0])
    mp = mq + np.array([0.5, -0.5, 0.5, -0.5])        # Delta^2 = 0.25
    for sigma in (0.25, 1.0, 3.0):
        assert math.exp(orc.log_ratio(mq, mp, mq, sigma, sigma)) == pytest.approx(
            math.exp(-0.25 / (2 * sigma ** 2)), rel=1e-13)
    assert orc.log_ratio(mq, mq, mq, 1.0, 1.0) == 0.0
    assert orc.accept(0.0, 1.0 - 2.0 ** -24)          # Delta = 0: always accepted
    # without the 1/d tempering the same gap at P = 96 would give exp(-96 * 0.125) ~ 6e-6
    assert math.exp(96 * orc.log_ratio(mq, mp, mq, 1.0, 1.0)) < 1e-5


def test_accept_is_u_le_alpha():
    rng = np.random.default_rng(1)
    for _ in range(2000):
        ell = rng.normal(0, 2)
        u = rng.uniform(1e-9, 1)
        if abs(u - min(1.0, math.exp(ell))) < 1e-12:
            continue
        assert orc.accept(ell, u) == (u <= min(1.0, math.exp(ell)))
    assert orc.accept(800.0, 0.999)                   # overflow-safe


def test_a_non_finite_statistic_is_a_rejection():
    """A NaN (or -inf) statistic never passes the test u <= min(1, e^l): the comparison is false, the
    proposal is rejected and the target's own prediction takes its place."""
    for ell in (float("nan"), float("-inf")):
        for u in (2.0 ** -24, 0.5, 1.0 - 2.0 ** -24):
            assert not orc.accept(ell, u)
    # an infinite or NaN proposal makes the statistic non-finite whatever the draft mean is
    mu = np.zeros(8)
    for bad in (np.inf, -np.inf, np.nan):
        x = mu.copy()
        x[3] = bad
        for mu_q in (x, mu):                              # mean proposal (x = mu_q) and a finite draft mean
            l = orc.log_ratio(x, mu, mu_q, 1.0, 1.0)
            assert not l > -np.inf or math.isnan(l)
            assert not orc.accept(l, 2.0 ** -24)


# ------------------------------------------- Algorithm 1 / Figure 1 example ----
def _scripted_round(decisions, K=4):
    """Drive one round with uniforms chosen to realise a given accept/reject script."""
    target, draft = tiny_models()
    hist = toy_series(1, 40, seed=5)[0].reshape(-1, 8)
    probe = orc.speculative_round(hist, target, draft, K, 1.0, [2.0 ** -24] * K)
    assert probe.n_accept == K                        # u ~ 0 accepts everything, so all l_i known
    us = []
    for i in range(K):
        a = math.exp(min(probe.ell[i], 0.0))
        want = decisions[i] if i < len(decisions) else True
        us.append(a * 0.5 if want else a + 0.5 * (1 - a))
    return hist, target, draft, orc.speculative_round(hist, target, draft, K, 1.0, us), probe


def test_figure1_example():
    g = dict(l.split(None, 1) for l in open(os.path.join(GOLDEN, "figure1_round.txt")) if l[0] != "#")
    K = int(g["K"])
    script = [w == "accept" for w in g["decisions"].split()]
    hist, target, draft, rec, probe = _scripted_round(script, K)
    assert rec.n_accept == int(g["n_accept"]) and rec.L == int(g["yield"])
    assert len(rec.decisions) == int(g["tested"])     # x_4 never tested
    got = orc.committed_patches(rec)
    assert got.shape[0] == 3
    np.testing.assert_array_equal(got[0], rec.mu_q[0])
    np.testing.assert_array_equal(got[1], rec.mu_q[1])
    np.testing.assert_array_equal(got[2], rec.mu_p[2])  # the target's own mu_p^(3), not x_3
    assert not np.array_equal(got[2], rec.mu_q[2])
    # mu_p^(3) is what the target alone predicts after [h, x_1, x_2]
    alone = orc.forward(target, np.concatenate([hist, rec.mu_q[:2]], axis=0))[-1]
    np.testing.assert_allclose(got[2], alone, rtol=0, atol=1e-12)


def test_every_outcome_of_a_round_by_brute_force():
    """All K+1 outcomes: n leading accepts commit x_1..x_n then mu_p^(n+1); full acceptance adds the bonus."""
    K = 3
    for n in range(K + 1):
        script = [True] * n + [False]
        hist, target, draft, rec, probe = _scripted_round(script, K)
        assert rec.n_accept == n and rec.L == n + 1
        assert len(rec.decisions) == min(n + 1, K)
        got = orc.committed_patches(rec)
        assert got.shape[0] == n + 1
        np.testing.assert_array_equal(got[:n], probe.mu_q[:n])
        np.testing.assert_array_equal(got[n], probe.mu_p[n])
    # a later "accept" after a rejection is never looked at
    _, _, _, rec, _ = _scripted_round([False, True, True], K)
    assert rec.n_accept == 0 and len(rec.decisions) == 1


def test_proposals_are_the_draft_rollout_and_boundaries_are_prefix_forwards():
    """mu_q^(i) = draft on h + x_{1:i-1}; mu_p^(i) = target on h + x_{1:i-1} (single-pass property)."""
    target, draft = tiny_models()
    hist = toy_series(1, 48, seed=7)[0].reshape(-1, 8)
    K = 3
    rec = orc.speculative_round(hist, target, draft, K, 1.0, [0.5] * K)
    toks = hist
    for i in range(K):
        np.testing.assert_allclose(rec.mu_q[i], orc.forward(draft, toks)[-1], atol=1e-12)
        np.testing.assert_allclose(rec.mu_p[i], orc.forward(target, toks)[-1], atol=1e-12)
        toks = np.concatenate([toks, rec.mu_q[i][None]], axis=0)
    np.testing.assert_allclose(rec.mu_p[K], orc.forward(target, toks)[-1], atol=1e-12)


# --------------------------------------------- limit statements of the paper ----
@pytest.mark.parametrize("use_cache", [False, True])
def test_draft_equals_target_accepts_everything_and_reproduces_target_only(use_cache):
    target, _ = tiny_models(same=True)
    s = toy_series(3, 40 + 60, seed=2)
    K, H = 3, 60
    ref = orc.forecast_target_only(target, s, 40, H, use_cache=use_cache)
    out, tr = orc.forecast_speculative(target, target, s, 40, H, K, 0.3, 2021, use_cache=use_cache)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-10)
    T = -(-H // 8)
    for recs in tr.rounds:
        assert all(r.n_accept == K and r.L == K + 1 for r in recs)
        assert len(recs) == -(-T // (K + 1))
        assert sum(r.committed for r in recs) == T


def test_sigma_to_zero_recovers_target_only_with_zero_acceptance():
    target, draft = tiny_models()
    s = toy_series(2, 40 + 48, seed=4)
    ref = orc.forecast_target_only(target, s, 40, 48)
    out, tr = orc.forecast_speculative(target, draft, s, 40, 48, 3, 1e-6, 2021)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-10)
    assert all(r.n_accept == 0 and r.L == 1 for recs in tr.rounds for r in recs)
    assert all(len(recs) == 6 for recs in tr.rounds)


# ------------------------------- point tokens: P_in < P, strided boundaries ----
def point_token_models(P=8, P_in=2, seed=5, same=False):
    ta, da = Arch(2, 32, 4, 64), Arch(1, 16, 2, 32)
    tw = make_weights(ta, P, seed, "f32", stream=0, patch_in=P_in)
    target = orc.make_model(tw, ta.n_layers, ta.d_model, ta.n_heads, ta.d_ff, P)
    if same:
        return target, target
    dw = make_weights(da, P, seed, "f32", stream=1, patch_in=P_in)
    return target, orc.make_model(dw, da.n_layers, da.d_model, da.n_heads, da.d_ff, P)


def test_boundary_indices_follow_the_per_family_rule():
    """Prefix i is read at token N - 1 + i (P / P_in): with patch tokens that is N - 1 + i; with
    point tokens and a 64-step head, 64 tokens further per prefix."""
    assert list(orc.boundary_indices(30, 4)) == [29, 30, 31, 32, 33]
    assert list(orc.boundary_indices(3072, 3, 64)) == [3071, 3135, 3199, 3263]
    t, _ = point_token_models(P=8, P_in=2)
    assert t.patch_in == 2 and t.tokens_per_patch == 4


@pytest.mark.parametrize("P_in", [1, 2, 4, 8])
def test_strided_boundaries_are_prefix_forwards(P_in):
    """The single-pass property with input tokens shorter than a patch: the prediction read at
    token N - 1 + i (P / P_in) of the one causal pass over [h, x_1..x_K] is what a forward over
    h + x_{1:i} alone gives at its last token -- for the draft rollout as for the verification."""
    P, K = 8, 3
    target, draft = point_token_models(P, P_in)
    hist = toy_series(1, 48, seed=7)[0].reshape(-1, P)
    rec = orc.speculative_round(hist, target, draft, K, 1.0, [0.5] * K)
    seq = hist
    for i in range(K):
        np.testing.assert_allclose(rec.mu_q[i], orc.forward(draft, seq.reshape(-1, P_in))[-1], atol=1e-12)
        np.testing.assert_allclose(rec.mu_p[i], orc.forward(target, seq.reshape(-1, P_in))[-1], atol=1e-12)
        seq = np.concatenate([seq, rec.mu_q[i][None]], axis=0)
    np.testing.assert_allclose(rec.mu_p[K], orc.forward(target, seq.reshape(-1, P_in))[-1], atol=1e-12)
    # a wrong stride would read a prediction made from an incomplete patch: those differ
    o = orc.forward(target, np.concatenate([hist, rec.mu_q], axis=0).reshape(-1, P_in))
    if P_in < P:
        assert not np.allclose(o[hist.shape[0] * (P // P_in) - 1 + 1], rec.mu_p[1])


def test_point_token_forecasts_keep_the_rule_level_invariants():
    """draft == target accepts everything and reproduces target-only decoding; the KV-cached and the
    full-recompute forecasts agree; every round commits between 1 and K + 1 patches, T in total."""
    P, P_in, K, H = 8, 2, 3, 44
    target, draft = point_token_models(P, P_in)
    s = toy_series(3, 40 + H, seed=2)
    same, _ = point_token_models(P, P_in, same=True)
    out, tr = orc.forecast_speculative(same, same, s, 40, H, K, 1.0, 3)
    np.testing.assert_allclose(out, orc.forecast_target_only(same, s, 40, H), atol=1e-10)
    assert all(r.n_accept == K for recs in tr.rounds for r in recs)
    a, tra = orc.forecast_speculative(target, draft, s, 40, H, K, 2.0, 9, use_cache=True)
    b, trb = orc.forecast_speculative(target, draft, s, 40, H, K, 2.0, 9, use_cache=False)
    np.testing.assert_allclose(a, b, atol=1e-10)
    T = -(-H // P)
    for recs in tra.rounds:
        assert all(1 <= r.L <= K + 1 for r in recs) and sum(r.committed for r in recs) == T
    np.testing.assert_allclose(orc.forecast_target_only(target, s, 40, H, use_cache=True),
                               orc.forecast_target_only(target, s, 40, H, use_cache=False), atol=1e-10)


@pytest.mark.parametrize("K,tau,H", [(1, 1.0, 40), (2, 2.0, 44), (4, 1.5, 64), (8, 3.0, 50)])
def test_round_yield_and_total(K, tau, H):
    target, draft = tiny_models()
    s = toy_series(4, 40 + H, seed=K)
    out, tr = orc.forecast_speculative(target, draft, s, 40, H, K, tau, 7)
    T = -(-H // 8)
    assert out.shape == (4, H) and np.isfinite(out).all()
    for recs in tr.rounds:
        assert all(1 <= r.L <= K + 1 and r.L == r.n_accept + 1 for r in recs)
        assert all(1 <= r.committed <= r.L for r in recs)
        assert all(r.committed == r.L for r in recs[:-1])      # only the last round truncates
        assert sum(r.committed for r in recs) == T
        assert len(recs) <= T


def test_cached_and_full_recompute_forecasts_agree():
    target, draft = tiny_models()
    s = toy_series(2, 40 + 56, seed=9)
    a, ta = orc.forecast_speculative(target, draft, s, 40, 56, 3, 2.0, 11, use_cache=False)
    b, tb = orc.forecast_speculative(target, draft, s, 40, 56, 3, 2.0, 11, use_cache=True)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-10)
    assert [[r.n_accept for r in x] for x in ta.rounds] == [[r.n_accept for r in x] for x in tb.rounds]
    assert sum(r.n_accept for x in ta.rounds for r in x) > 0     # the test exercises acceptance
    assert sum(1 for x in ta.rounds for r in x if r.n_accept < 3) > 0


def test_forced_decisions_are_replayed():
    target, draft = tiny_models()
    s = toy_series(1, 40 + 40, seed=1)
    forced = [[[True, False, True], [False], [True, True, True]]]
    out, tr = orc.forecast_speculative(target, draft, s, 40, 40, 3, 1.0, 5, forced=forced)
    assert [r.n_accept for r in tr.rounds[0]] == [1, 0, 3]
    assert [r.committed for r in tr.rounds[0]] == [2, 1, 2]


def test_instance_statistics_are_frozen_on_the_context():
    """Changing the tail (future) of a series cannot change the forecast; scaling the context rescales it."""
    target, draft = tiny_models()
    s = toy_series(1, 40 + 24, seed=3)
    s2 = s.copy()
    s2[:, 40:] += 100.0
    a, _ = orc.forecast_speculative(target, draft, s, 40, 24, 2, 1.0, 5)
    b, _ = orc.forecast_speculative(target, draft, s2, 40, 24, 2, 1.0, 5)
    np.testing.assert_array_equal(a, b)
    # eps under the square root is 1e-5, so affine equivariance holds to ~1e-5 relative
    c, _ = orc.forecast_speculative(target, draft, 3.0 * s + 7.0, 40, 24, 2, 1.0, 5)
    np.testing.assert_allclose(c, 3.0 * a + 7.0, rtol=0, atol=2e-4)
    m, sd = orc.instance_stats(np.array([1.0, 2.0, 3.0, 6.0]))
    assert m == 3.0 and sd == pytest.approx(math.sqrt(3.5 + 1e-5), rel=1e-15)


# --------------------------------------------------- Proposition 1 (fidelity) ----
def test_proposition1_by_enumerating_every_uniform():
    """E||Y - mu_p||_d^2 = Delta^2 exp(-Delta^2 / 2 sigma^2) <= 2 sigma^2 / e, maximum at Delta^2 = 2 sigma^2."""
    m = np.arange(2 ** 23, dtype=np.float64)
    log_u = np.log((m + 0.5) * 2.0 ** -23)            # every value u can take
    rng = np.random.default_rng(0)
    d = 12
    for sigma in (0.3, 1.0):
        worst = 0.0
        for gap2 in (0.0, 0.1 * sigma ** 2, 2 * sigma ** 2, 5 * sigma ** 2, 40 * sigma ** 2):
            mu_p = rng.standard_normal(d)
            dirn = rng.standard_normal(d)
            mu_q = mu_p + dirn / np.linalg.norm(dirn) * math.sqrt(gap2 * d)
            ell = orc.log_ratio(mu_q, mu_p, mu_q, sigma, sigma)
            frac = np.count_nonzero(log_u <= min(ell, 0.0)) / log_u.size
            assert all(orc.accept(ell, math.exp(lu)) == (lu <= min(ell, 0.0)) for lu in log_u[::400000])
            got = frac * orc.energy(mu_q - mu_p)       # Y = mu_q w.p. frac, else mu_p
            want = gap2 * math.exp(-gap2 / (2 * sigma ** 2))
            assert got == pytest.approx(want, abs=gap2 * 2.0 ** -22 + 1e-12)
            assert got <= 2 * sigma ** 2 / math.e + 1e-6
            worst = max(worst, got)
            # tail: P(||Y - mu_p||^2 > t) <= exp(-t / 2 sigma^2)
            for t in (0.5 * gap2, 2.0 * gap2):
                p_tail = frac if gap2 > t else 0.0
                assert p_tail <= math.exp(-t / (2 * sigma ** 2)) + 2.0 ** -22
        assert worst == pytest.approx(2 * sigma ** 2 / math.e, rel=1e-5)   # attained at Delta^2 = 2 sigma^2


# --------------------------------------------------- capped-geometric law ----
def test_capped_geometric_law_closed_forms():
    for a in (0.0, 0.2, 0.8, 0.97):
        for K in (1, 3, 8):
            pmf = orc.capped_geometric_pmf(a, K)
            assert pmf.sum() == pytest.approx(1.0, abs=1e-14)
            mean = float((np.arange(1, K + 2) * pmf).sum())
            assert orc.capped_geometric_mean(a, K) == pytest.approx(mean, rel=1e-13)
            if a < 1:
                assert mean == pytest.approx((1 - a ** (K + 1)) / (1 - a), rel=1e-13)
    assert orc.capped_geometric_mean(1.0, 4) == 5.0
    assert orc.predicted_speedup(0.8, 4, 0.04, 1.0) == pytest.approx((1 - 0.8 ** 5) / 0.2 / 1.16)


def test_measured_yield_follows_the_capped_geometric_law():
    """Rounds with i.i.d. acceptance at rate a: the round machinery must reproduce P(L = l)."""
    target, _ = tiny_models(same=True)
    tw = {k: v.astype(np.float32) for k, v in target.w.items()}
    dw = perturbed_draft(tw, 2, 0.35, 1, "f32")
    draft = orc.make_model(dw, 2, 32, 4, 64, 8)
    K, H = 4, 8 * 24
    s = toy_series(24, 40 + H, seed=12)
    out, tr = orc.forecast_speculative(target, draft, s, 40, H, K, 0.6, 99)
    tested, accepted = tr.counts_by_position(K)
    assert tested[0] > 100 and 0.15 < accepted.sum() / tested.sum() < 0.95
    rate = accepted / np.maximum(tested, 1)
    L = tr.yields()
    # exact identity on the run's own data: mean(L) = sum_l prod_{i<l} a_i
    tail = sum(np.prod(rate[:l]) for l in range(K + 1))
    assert L.mean() == pytest.approx(tail, rel=1e-12)
    # dependence band (appendix proposition): f(min a_i) <= mean(L) <= f(max a_i)
    lo = orc.capped_geometric_mean(rate[tested > 0].min(), K)
    hi = orc.capped_geometric_mean(rate[tested > 0].max(), K)
    assert lo - 1e-12 <= L.mean() <= hi + 1e-12
    # pooled rate: the law's E[L] within sampling error of the measured mean
    pooled = accepted.sum() / tested.sum()
    assert abs(orc.capped_geometric_mean(pooled, K) - L.mean()) < 0.35


def test_simulated_rounds_match_the_pmf():
    """Drive rounds with synthetic energies so acceptance is exactly i.i.d. with known alpha."""
    K, alpha, n = 3, 0.7, 40000
    ell = math.log(alpha)
    counts = np.zeros(K + 2)
    for r in range(n):
        L = 1
        for i in range(K):
            if not orc.accept(ell, orc.acceptance_uniform(5, 0, r, i)):
                break
            L += 1
        counts[L] += 1
    np.testing.assert_allclose(counts[1:] / n, orc.capped_geometric_pmf(alpha, K), atol=0.01)


# ----------------------------------------------------------------------------
# Sampled variants (Sec. 3.3 "Fallback Correction and Sampled Variants"; Algorithm 1 with r > 0)
# ----------------------------------------------------------------------------
def test_standard_normals_are_standard_and_streams_differ():
    z = np.concatenate([orc.standard_normals(7, s, 0, 0, orc.NOISE_PROPOSAL, 96) for s in range(400)])
    assert abs(z.mean()) < 0.02 and abs(z.var() - 1.0) < 0.03
    assert abs(np.mean(z ** 4) - 3.0) < 0.15                        # Gaussian kurtosis
    assert abs(np.mean(np.abs(z) > 1.959964) - 0.05) < 0.005        # two-sided 5 % tail
    a = orc.standard_normals(7, 1, 2, 3, orc.NOISE_PROPOSAL, 8)
    b = orc.standard_normals(7, 1, 2, 3, orc.NOISE_FALLBACK, 8)
    assert not np.allclose(a, b)
    np.testing.assert_array_equal(a[:5], orc.standard_normals(7, 1, 2, 3, orc.NOISE_PROPOSAL, 5))   # prefix-stable


def test_standard_normals_invert_to_the_philox_words_they_were_made_from():
    """Box-Muller is invertible: an (even, odd) element pair gives back its two uniforms,
    z0^2 + z1^2 = -2 ln u1 and atan2(z1, z0) = 2 pi u2.  That fixes which Philox word feeds the
    radius and which the angle, the cosine branch on even and the sine branch on odd elements, and
    the counter layout (series, round, position, stream | pair index)."""
    seed, series, rnd, pos = 0x1234567800000009, 5, 2, 3
    key = (seed & 0xFFFFFFFF, seed >> 32)
    for stream in (orc.NOISE_PROPOSAL, orc.NOISE_FALLBACK):
        z = orc.standard_normals(seed, series, rnd, pos, stream, 10)
        for j in range(5):
            w = orc.philox4x32_10((series, rnd, pos, stream | j), key)
            u1, u2 = orc.uniform_from_word(w[0]), orc.uniform_from_word(w[1])
            assert z[2 * j] ** 2 + z[2 * j + 1] ** 2 == pytest.approx(-2.0 * math.log(u1), rel=1e-12)
            ang = math.atan2(z[2 * j + 1], z[2 * j]) % (2.0 * math.pi)
            assert ang == pytest.approx(2.0 * math.pi * u2, abs=1e-9)


def test_sampled_proposals_accept_at_the_equal_covariance_rate_in_one_dimension():
    """Equal-covariance acceptance (appendix proposition): with x ~ q = N(mu_q, s^2) and the
    untempered ratio, the mean acceptance is 2 Phi(-Delta / 2), Delta = |mu_p - mu_q| / s.  In one
    dimension the 1/d tempering is the identity, so the rule as implemented must reproduce it."""
    from scipy.stats import norm
    rng = np.random.default_rng(5)
    s, mu_q = 0.7, np.array([0.3])
    for delta in (0.5, 1.0, 2.0):
        mu_p = mu_q + delta * s
        x = mu_q + s * rng.standard_normal((200000, 1))
        ell = np.array([orc.log_ratio(xi, mu_p, mu_q, s, s) for xi in x[:20000]])
        alpha = np.minimum(1.0, np.exp(ell)).mean()
        assert alpha == pytest.approx(2 * norm.cdf(-delta / 2), abs=0.01)


def test_round_with_sampled_proposals_fallback_noise_and_unequal_scales():
    """Algorithm 1 in its general form, step by step against its definition: x_i = mu_q^(i) + sigma_q eps_i
    where mu_q^(i) is the draft's mean given the SAMPLED x_1..x_{i-1}; the statistic is Eq. 5 with both
    energies and the determinant term; a rejection commits mu_p^(i) + r eps, full acceptance the bonus
    mu_p^(K+1) + r eps."""
    tgt, drf = tiny_models(P=8)
    P, K, sp, sq, r = 8, 3, 0.9, 0.5, 0.25
    hist = toy_series(1, 5 * P, seed=2)[0].reshape(5, P)
    rng = np.random.default_rng(9)
    pe, fe = rng.standard_normal((K, P)), rng.standard_normal((K + 1, P))
    var = orc.Variant(sigma_q=sq, sample_proposals=True, fallback_noise=r)
    for script in ([True, True, True], [True, False], [False]):
        rec = orc.speculative_round(hist, tgt, drf, K, sp, [0.5] * K, forced=script, variant=var,
                                    proposal_eps=pe, fallback_eps=fe)
        # proposals: rebuilt by per-prefix draft forwards on the sampled tokens
        toks = hist.copy()
        for i in range(K):
            mu = orc.forward(drf, toks)[-1]
            np.testing.assert_allclose(rec.mu_q[i], mu + sq * pe[i], rtol=0, atol=1e-12)
            toks = np.concatenate([toks, rec.mu_q[i][None, :]], axis=0)
        # statistic of the first tested position, written out from Eq. 5
        mu_q1 = orc.forward(drf, hist)[-1]
        mu_p1 = orc.forward(tgt, hist)[-1]
        x1 = rec.mu_q[0]
        want = (-np.sum((x1 - mu_p1) ** 2) / P / (2 * sp ** 2) + np.sum((x1 - mu_q1) ** 2) / P / (2 * sq ** 2)
                + 0.5 * math.log(sq ** 2 / sp ** 2))
        assert rec.ell[0] == pytest.approx(want, rel=1e-12)
        n = rec.n_accept
        assert n == sum(script[:script.index(False)] if False in script else script)
        commit = orc.committed_patches(rec)
        np.testing.assert_array_equal(commit[:n], rec.mu_q[:n])
        clean = orc.forward(tgt, np.concatenate([hist, rec.mu_q[:n]], axis=0))[-1]
        np.testing.assert_allclose(commit[n], clean + r * fe[n], rtol=0, atol=1e-12)


def test_dropping_the_tempering_multiplies_the_statistic_by_d_and_kills_acceptance():
    """Component ablation (Table 2, row "w/o 1/d tempering"): the untempered log ratio is d times
    the tempered one, and at patch dimensions acceptance collapses."""
    tgt, drf = tiny_models(P=8)
    P, K = 8, 2
    hist = toy_series(1, 4 * P, seed=4)[0].reshape(4, P)
    a = orc.speculative_round(hist, tgt, drf, K, 1.0, [0.999] * K, forced=[True, True])
    b = orc.speculative_round(hist, tgt, drf, K, 1.0, [0.999] * K, forced=[True, True],
                              variant=orc.Variant(tempering=False))
    np.testing.assert_allclose(np.array(b.ell), P * np.array(a.ell), rtol=1e-12)
    s = toy_series(6, 4 * P + 6 * P, seed=5)
    _, tr_t = orc.forecast_speculative(tgt, drf, s, 4 * P, 6 * P, K, 1.0, 3)
    _, tr_u = orc.forecast_speculative(tgt, drf, s, 4 * P, 6 * P, K, 1.0, 3, variant=orc.Variant(tempering=False))
    acc = lambda tr: sum(sum(r.decisions) for sr in tr.rounds for r in sr)
    assert acc(tr_u) <= acc(tr_t)


def test_variant_defaults_reproduce_the_deployed_scheme_and_noise_is_seeded():
    tgt, drf = tiny_models(P=8)
    P = 8
    s = toy_series(3, 4 * P + 5 * P, seed=6)
    base, _ = orc.forecast_speculative(tgt, drf, s, 4 * P, 5 * P, 2, 1.0, 11)
    same, _ = orc.forecast_speculative(tgt, drf, s, 4 * P, 5 * P, 2, 1.0, 11, variant=orc.Variant())
    np.testing.assert_array_equal(base, same)
    v = orc.Variant(sample_proposals=True, fallback_noise=0.3)
    n1, _ = orc.forecast_speculative(tgt, drf, s, 4 * P, 5 * P, 2, 1.0, 11, variant=v)
    n2, _ = orc.forecast_speculative(tgt, drf, s, 4 * P, 5 * P, 2, 1.0, 11, variant=v)
    n3, _ = orc.forecast_speculative(tgt, drf, s, 4 * P, 5 * P, 2, 1.0, 12, variant=v)
    np.testing.assert_array_equal(n1, n2)
    assert not np.allclose(n1, base) and not np.allclose(n1, n3)
    # a series decoded alone (same series id) sees the same noise as inside the batch
    solo, _ = orc.forecast_speculative(tgt, drf, s[1:2], 4 * P, 5 * P, 2, 1.0, 11, variant=v, series_index0=1)
    np.testing.assert_array_equal(solo[0], n1[1])


def test_marginal_gain_condition_is_equivalent_to_a_speedup_gain_and_finds_the_best_block():
    """Prop. (marginal-gain condition for K): S(K+1) >= S(K) iff alpha^(K+1)(cK+v) >= c E[L_K];
    stepping K up while it holds lands on the brute-force argmax of Eq. 8."""
    for alpha in (0.05, 0.3, 0.6, 0.8, 0.95, 0.999):
        for c in (0.02, 0.1, 0.25, 0.5, 1.0):
            for v in (1.0, 1.4, 2.5):
                K = 1
                while K < 32 and orc.marginal_gain_holds(alpha, K, c, v):
                    K += 1
                for k in range(1, 12):
                    lhs = orc.predicted_speedup(alpha, k + 1, c, v) >= orc.predicted_speedup(alpha, k, c, v) * (1 - 1e-12)
                    assert lhs == orc.marginal_gain_holds(alpha, k, c, v) or \
                        abs(orc.predicted_speedup(alpha, k + 1, c, v) - orc.predicted_speedup(alpha, k, c, v)) < 1e-12
                best = orc.best_block_size(alpha, c, v, 32)
                assert orc.predicted_speedup(alpha, K, c, v) == pytest.approx(orc.predicted_speedup(alpha, best, c, v), rel=1e-12)
