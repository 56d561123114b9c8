"""Pins for the acceptance statistic, the reflection coupling and the first-rejection scan."""
import itertools

import numpy as np
from scipy import stats

from oracle import spec


def test_log_ratio_is_the_difference_of_gaussian_log_densities():
    """log alpha = log N(x~; mu, sigma^2 I) - log N(x~; mu^, sigma^2 I) at x~ = mu^ + sigma xi."""
    rng = np.random.default_rng(1)
    for D in (1, 3, 32, 160):
        mu_hat, mu, xi = rng.normal(size=D), rng.normal(size=D), rng.normal(size=D)
        sigma = 0.37
        x = mu_hat + sigma * xi
        ref = stats.norm.logpdf(x, mu, sigma).sum() - stats.norm.logpdf(x, mu_hat, sigma).sum()
        assert abs(spec.log_accept_ratio(mu_hat, mu, sigma, xi) - ref) < 1e-10 * max(1.0, abs(ref))
    # sigma_scale s: the same identity with both densities widened to s*sigma at the same x~
    s = 1.7
    x = mu_hat + sigma * xi
    ref = stats.norm.logpdf(x, mu, s * sigma).sum() - stats.norm.logpdf(x, mu_hat, s * sigma).sum()
    got = spec.log_accept_ratio(mu_hat, mu, sigma, xi / s, s)   # x~ - mu^ = (s sigma)(xi/s)
    assert abs(got - ref) < 1e-9 * abs(ref)


def test_decision_rules():
    a0 = spec.Accept(mode=0)
    assert spec.accepted(-0.5, a0, np.log(0.5)) and not spec.accepted(-0.8, a0, np.log(0.5))
    assert spec.accepted(3.0, a0, np.log(0.999999))                       # alpha > 1 always passes
    a1 = spec.Accept(mode=1, lam=0.6)
    assert spec.accepted(np.log(0.61), a1, None) and not spec.accepted(np.log(0.59), a1, None)
    assert spec.accepted(5.0, spec.Accept(mode=1, lam=1.0), None)          # p = min(1, alpha) = 1
    assert not spec.accepted(-1e-9, spec.Accept(mode=1, lam=1.0), None)


def test_reflection_is_a_householder_map():
    rng = np.random.default_rng(2)
    D = 12
    m_r, m_s, xt = rng.normal(size=D), rng.normal(size=D), rng.normal(size=D)
    x = spec.reflect(xt, m_r, m_s)
    e = (m_r - m_s) / np.linalg.norm(m_r - m_s)
    assert abs(np.linalg.norm(x - m_s) - np.linalg.norm(xt - m_r)) < 1e-12          # isometry
    assert abs(np.dot(x - m_s, e) + np.dot(xt - m_r, e)) < 1e-12                    # flips along e
    P = np.eye(D) - np.outer(e, e)
    assert np.allclose(P @ (x - m_s), P @ (xt - m_r), atol=1e-12)                   # keeps the rest
    back = spec.reflect(x, m_s, m_r)                                                # involution
    assert np.allclose(back, xt, atol=1e-12)
    # shape is preserved and 1-D reduces to x = m_s - (x~ - m_r)
    assert spec.reflect(xt.reshape(3, 4), m_r.reshape(3, 4), m_s.reshape(3, 4)).shape == (3, 4)
    assert np.allclose(spec.reflect(np.array([0.9]), np.array([0.5]), np.array([0.2])), [0.2 - 0.4])


def test_accept_or_reflect_samples_the_target_gaussian():
    """10^5 draws: the coupled output is N(m_s, sigma^2 I) and the acceptance frequency is the
    overlap of two equal-variance Gaussians, 2 Phi(-|Delta| / (2 sigma))."""
    rng = np.random.default_rng(3)
    D, sigma, N = 6, 0.8, 100_000
    m_r = rng.normal(size=D)
    for dist in (0.378 * sigma, 1.0 * sigma, 2.5 * sigma):
        dirn = rng.normal(size=D); dirn /= np.linalg.norm(dirn)
        m_s = m_r - dist * dirn
        out = np.empty((N, D)); n_acc = 0
        acc = spec.Accept(mode=0)
        for i in range(N):
            xi = rng.normal(size=D)
            la = spec.log_accept_ratio(m_r, m_s, sigma, xi)
            if spec.accepted(la, acc, np.log(rng.random())):
                out[i] = m_r + sigma * xi; n_acc += 1
            else:
                out[i] = spec.reflect(m_r + sigma * xi, m_r, m_s)
        expect = 2 * stats.norm.cdf(-dist / (2 * sigma))
        assert abs(n_acc / N - expect) < 4 * np.sqrt(expect * (1 - expect) / N)
        z = (out - m_s) / sigma
        orth = np.linalg.svd(np.vstack([dirn, np.eye(D)]).T)[0][:, 1]
        orth -= dirn * np.dot(orth, dirn); orth /= np.linalg.norm(orth)
        assert stats.kstest(z @ dirn, "norm").pvalue > 0.01
        assert stats.kstest(z @ orth, "norm").pvalue > 0.01
        assert stats.kstest(z[:, 0], "norm").pvalue > 0.01


def test_first_rejection_brute_force():
    for K in range(0, 5):
        for pat in itertools.product([True, False], repeat=K):
            j = spec.first_rejection(list(pat))
            rejected = [i + 1 for i, a in enumerate(pat) if not a]
            assert j == (min(rejected) if rejected else None)
            if j is not None:
                assert all(pat[: j - 1]) and not pat[j - 1]
