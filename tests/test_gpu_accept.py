"""The fused accept kernel (Eq. 5, first rejection, correction / bonus, Philox) against the oracle."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import tsfm_oracle as orc

pytestmark = pytest.mark.gpu


def run_accept(x, mu_q, mu_p, T, sp, sq, seed, rnd, series0, forced_u, done):
    import paper_2511_18191_b200 as tsfm
    B, K, P = x.shape
    dev = "cuda"
    t = lambda a, dt=torch.float32: None if a is None else torch.tensor(np.asarray(a), dtype=dt, device=dev).contiguous()
    xd, qd, pd, fd = t(x), t(mu_q), t(mu_p), t(forced_u)
    dd = t(done, torch.int32)
    commit = torch.full((B, K + 1, P), float("nan"), device=dev)
    nacc = torch.full((B,), -7, dtype=torch.int32, device=dev)
    ell = torch.zeros((B, K), device=dev)
    logu = torch.zeros((B, K), device=dev)
    tsfm.tsfm_accept_round(torch.cuda.current_stream().cuda_stream, xd, qd, pd, B, K, P, T, sp, sq, seed, rnd,
                           series0, fd, dd, commit, nacc, ell, logu)
    torch.cuda.synchronize()
    return commit.cpu().numpy(), nacc.cpu().numpy(), ell.cpu().numpy(), logu.cpu().numpy(), dd.cpu().numpy()


@pytest.mark.parametrize("B,K,P", [(1, 2, 96), (32, 4, 96), (256, 4, 96), (1024, 8, 96), (64, 8, 32), (5, 1, 16), (7, 32, 48)])
def test_accept_matches_oracle(B, K, P):
    rng = np.random.default_rng(B * 100 + K)
    mu_p = rng.standard_normal((B, K + 1, P)).astype(np.float32)
    gap = rng.uniform(0.0, 2.0, (B, K, 1)).astype(np.float32)
    x = (mu_p[:, :K] + gap * rng.standard_normal((B, K, P))).astype(np.float32)
    x[0, :] = mu_p[0, :K]                                    # Delta = 0: always accepted
    done = np.zeros(B, dtype=np.int32)
    T, seed, rnd, s0, tau = 1000, 2021 + (5 << 32), 3, 11, 0.9
    commit, nacc, ell, logu, done2 = run_accept(x, x, mu_p, T, tau, tau, seed, rnd, s0, None, done)
    flips = 0
    for b in range(B):
        n = 0
        alive = True
        for i in range(K):
            l = orc.log_ratio(x[b, i], mu_p[b, i], x[b, i], tau, tau)
            u = orc.acceptance_uniform(seed, s0 + b, rnd, i)
            assert logu[b, i] == pytest.approx(math.log(u), abs=2e-6)
            assert ell[b, i] == pytest.approx(l, rel=2e-5, abs=1e-6)
            if alive:
                ok = orc.accept(l, u)
                if ok:
                    n += 1
                else:
                    alive = False
        if n != nacc[b]:
            # only a decision inside the fp32 margin may differ
            i = min(n, nacc[b])
            l = orc.log_ratio(x[b, i], mu_p[b, i], x[b, i], tau, tau)
            assert abs(l - math.log(orc.acceptance_uniform(seed, s0 + b, rnd, i))) < 1e-3
            flips += 1
            continue
        want = np.concatenate([x[b, :n], mu_p[b, n:n + 1]], axis=0)
        np.testing.assert_array_equal(commit[b, :n + 1], want)
        assert done2[b] == n + 1
    assert nacc[0] == K
    assert flips <= max(1, B // 200)


def test_figure1_example_with_scripted_uniforms():
    g = dict(l.split(None, 1) for l in open(os.path.join(os.path.dirname(__file__), "golden", "figure1_round.txt")) if l[0] != "#")
    K, P = int(g["K"]), 96
    rng = np.random.default_rng(0)
    mu_p = rng.standard_normal((1, K + 1, P)).astype(np.float32)
    x = (mu_p[:, :K] + 0.8 * rng.standard_normal((1, K, P))).astype(np.float32)
    alphas = [math.exp(min(orc.log_ratio(x[0, i], mu_p[0, i], x[0, i], 1.0, 1.0), 0.0)) for i in range(K)]
    script = [w == "accept" for w in g["decisions"].split()] + [True]
    u = np.array([[a * 0.5 if ok else a + 0.5 * (1 - a) for a, ok in zip(alphas, script)]], dtype=np.float32)
    commit, nacc, ell, logu, done = run_accept(x, x, mu_p, 100, 1.0, 1.0, 0, 0, 0, u, np.zeros(1, np.int32))
    assert nacc[0] == int(g["n_accept"]) and done[0] == int(g["yield"])
    np.testing.assert_array_equal(commit[0, 0], x[0, 0])
    np.testing.assert_array_equal(commit[0, 1], x[0, 1])
    np.testing.assert_array_equal(commit[0, 2], mu_p[0, 2])      # the target's mu_p^(3), not x_3
    assert np.isnan(commit[0, 3:]).all()                         # nothing else committed, no bonus


def test_every_outcome_truncation_and_finished_series():
    K, P = 3, 32
    B = K + 3
    rng = np.random.default_rng(1)
    mu_p = rng.standard_normal((B, K + 1, P)).astype(np.float32)
    x = (mu_p[:, :K] + 0.5 * rng.standard_normal((B, K, P))).astype(np.float32)
    u = np.full((B, K), 1e-6, dtype=np.float32)               # accept ...
    for b in range(K):
        u[b, b] = 1.0 - 1e-6                                    # ... except a scripted first rejection
    T = 10
    done = np.array([0, 0, 0, 0, T - 2, T], dtype=np.int32)    # series 4 truncates, series 5 finished
    commit, nacc, ell, logu, done2 = run_accept(x, x, mu_p, T, 1.0, 1.0, 0, 0, 0, u, done)
    assert list(nacc) == [0, 1, 2, 3, 3, -1]
    assert list(done2) == [1, 2, 3, 4, T, T]
    for b in range(4):
        n = nacc[b]
        np.testing.assert_array_equal(commit[b, :n], x[b, :n])
        np.testing.assert_array_equal(commit[b, n], mu_p[b, n])
    assert np.isnan(commit[5]).all()


def test_general_statistic_with_unequal_scales():
    """Eq. 5 in full: sampled proposals (x != mu_q) and sigma_q != sigma_p exercise all three terms."""
    B, K, P = 16, 4, 96
    rng = np.random.default_rng(2)
    mu_p = rng.standard_normal((B, K + 1, P)).astype(np.float32)
    mu_q = (mu_p[:, :K] + 0.3 * rng.standard_normal((B, K, P))).astype(np.float32)
    x = (mu_q + 0.7 * rng.standard_normal((B, K, P))).astype(np.float32)
    sp, sq = 1.1, 0.6
    commit, nacc, ell, logu, done = run_accept(x, mu_q, mu_p, 100, sp, sq, 9, 0, 0, None, np.zeros(B, np.int32))
    for b in range(B):
        for i in range(K):
            assert ell[b, i] == pytest.approx(orc.log_ratio(x[b, i], mu_p[b, i], mu_q[b, i], sp, sq), rel=3e-5, abs=2e-6)


def test_non_finite_proposals_are_rejected_and_the_target_corrects():
    """A NaN or infinite proposal makes Eq. 5's statistic NaN (with mean proposals the draft term is
    inf - inf).  A NaN never passes the test: the position is a rejection, and the committed patch
    there is the target's own prediction -- on the GPU as in the oracle."""
    B, K, P = 5, 3, 32
    rng = np.random.default_rng(3)
    mu_p = rng.standard_normal((B, K + 1, P)).astype(np.float32)
    x = (mu_p[:, :K] + 0.1 * rng.standard_normal((B, K, P))).astype(np.float32)
    x[0, 1, 5] = np.nan
    x[1, 0, :] = np.inf
    x[2, 2, 3] = -np.inf
    mu_q = x.copy()
    mu_q[3] = mu_p[3, :K]                                     # series 3: finite draft mean, infinite proposal
    x[3, 1, 0] = np.inf
    u = np.full((B, K), 2.0 ** -24, dtype=np.float32)         # accepts every finite statistic
    commit, nacc, ell, logu, done = run_accept(x, mu_q, mu_p, 100, 1.0, 1.0, 0, 0, 0, u, np.zeros(B, np.int32))
    want_n = [1, 0, 2, 1, 3]
    for b in range(B):
        n = 0
        for i in range(K):                                    # the oracle's decisions on the same inputs
            if not orc.accept(orc.log_ratio(x[b, i], mu_p[b, i], mu_q[b, i], 1.0, 1.0), float(u[b, i])):
                break
            n += 1
        assert n == want_n[b] == nacc[b], (b, n, nacc[b])
        assert done[b] == n + 1
        np.testing.assert_array_equal(commit[b, n], mu_p[b, n])     # the target's mean replaces the rejected patch
        np.testing.assert_array_equal(commit[b, :n], x[b, :n])
