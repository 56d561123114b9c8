"""Pins for the oracle's DDPM scheduler tables and posterior."""
import numpy as np

from oracle import ddpm


def test_tables_against_running_products():
    S = ddpm.Schedule(100, 1e-4, 0.02)
    ab, prev = 1.0, 1.0
    for t in range(100):
        beta = 1e-4 + (0.02 - 1e-4) * t / 99
        prev, ab = ab, ab * (1.0 - beta)
        assert abs(S.abar[t] - ab) < 1e-14 and abs(S.abar_prev[t] - prev) < 1e-14
    assert S.sigma[0] == 0.0 and np.all(S.sigma[1:] > 0)


def test_posterior_is_the_bayes_product_of_forward_gaussians():
    """q(x_{t-1} | x_t, x0) ∝ N(x_t; sqrt(alpha_t) x_{t-1}, beta_t) N(x_{t-1}; sqrt(abar_{t-1}) x0, 1-abar_{t-1}):
    precision and mean by completing the square, not by the closed form the oracle uses."""
    S = ddpm.Schedule()
    rng = np.random.default_rng(0)
    for t in (1, 2, 17, 50, 99):
        x_t, x0 = rng.normal(size=5), rng.normal(size=5)
        prec = S.alpha[t] / S.beta[t] + 1.0 / (1.0 - S.abar[t - 1])
        mean = (np.sqrt(S.alpha[t]) * x_t / S.beta[t] + np.sqrt(S.abar[t - 1]) * x0 / (1.0 - S.abar[t - 1])) / prec
        eps = (x_t - np.sqrt(S.abar[t]) * x0) / np.sqrt(1.0 - S.abar[t])      # the eps that yields x0_hat = x0
        assert np.allclose(S.posterior_mean(x_t, eps, t), mean, rtol=0, atol=1e-12)
        assert abs(S.sigma[t] ** 2 - 1.0 / prec) < 1e-15
    # t = 0: the "posterior" is the point mass at x0_hat
    x_t, eps = rng.normal(size=5), rng.normal(size=5)
    assert np.allclose(S.posterior_mean(x_t, eps, 0), S.x0_hat(x_t, eps, 0), atol=1e-12)


def test_clip_and_step():
    S = ddpm.Schedule()
    x_t, eps, xi = np.array([3.0, -3.0]), np.array([-2.0, 2.0]), np.array([1.0, -1.0])
    assert np.all(np.abs(S.x0_hat(x_t, eps, 60, clip=1.0)) == 1.0)
    x_prev, mu = S.step(x_t, eps, 60, xi)
    assert np.allclose(x_prev - mu, S.sigma[60] * xi)


def test_late_stage_sensitivity_grows():
    """d = c_t (eps_hat - eps) with c_t = beta_t / (sqrt(alpha_t (1-abar_t)) sigma_t): the same network
    disagreement costs far more acceptance late in denoising (the collapse the paper describes
    for the standard variance, Sec. 3.2)."""
    S = ddpm.Schedule()
    t = np.arange(1, 100)
    c = S.beta[t] / (np.sqrt(S.alpha[t] * (1 - S.abar[t])) * S.sigma[t])
    # c_t is the eps-coefficient of the posterior mean divided by sigma_t
    e = np.array([1.0]); x = np.array([0.3])
    for tt in (1, 50):
        num = (S.posterior_mean(x, 0 * e, tt) - S.posterior_mean(x, e, tt)) / S.sigma[tt]
        assert abs(num[0] - c[tt - 1]) < 1e-12
    assert abs(c[49] - 0.2145) < 1e-3 and abs(c[0] - 1.735) < 1e-2
    assert np.all(np.diff(c[:40]) < 0)          # monotone growth towards t -> 1


def test_sinusoidal_embedding():
    e = ddpm.sinusoidal_embedding(7, 8)
    f = [1.0, 0.1, 0.01, 0.001]
    assert np.allclose(e, [np.sin(7 * x) for x in f] + [np.cos(7 * x) for x in f], atol=1e-12)
    assert np.allclose(ddpm.sinusoidal_embedding(0, 6), [0, 0, 0, 1, 1, 1])
