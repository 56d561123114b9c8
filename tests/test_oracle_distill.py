"""Pins of the distillation-objective oracle (Sec. 3.2): identities that a dropped coefficient or a wrong sigma breaks."""
import math

import numpy as np

from oracle import ddpm, distill, nets, philox
from paper_2512_15773_b200 import inputs

S = ddpm.Schedule(100, 1e-4, 0.02)


def test_equal_networks_give_zero_loss_and_certain_acceptance():
    wl = dict(inputs.WORKLOADS["toy_mlp"])
    base = nets.make_denoiser(inputs.make_net(1, wl, "base"), S)
    rng = np.random.default_rng(0)
    x0s = rng.normal(size=(12, wl["H"], wl["A"]))
    obs = inputs.make_obs(0, 12, wl["To"], wl["Do"])
    assert distill.distill_loss(S, base, base, x0s, obs, 3) == (0.0, 0.0, 0.0, 1.0)


def test_constant_offset_between_the_networks_has_a_closed_form():
    """If the drafter's output is the base's plus a constant delta in every element, the normalised mean offset is
    d = -c_t delta with c_t = beta_t / (sqrt(alpha_t (1 - abar_t)) sigma_t): 0.2145 at t = 50 and 1.735 at t = 1 for the
    linear 1e-4..0.02 schedule -- the growth towards t -> 0 the paper describes for the late denoising stage."""
    base = lambda x, t, o: 0.3 * x
    delta = 0.05
    drafter = lambda x, t, o: 0.3 * x + delta
    x0 = np.random.default_rng(1).normal(size=(16, 2)); eps = np.random.default_rng(2).normal(size=(16, 2))
    for t, c_print in ((50, 0.2145), (1, 1.735)):
        pred, q = distill.sample_terms(S, base, drafter, x0, t, eps, None)
        c_t = S.beta[t] / (math.sqrt(S.alpha[t] * (1.0 - S.abar[t])) * S.sigma[t])
        assert abs(c_t - c_print) < 6e-4 * max(1.0, c_print)
        assert abs(pred - 32 * delta ** 2) < 1e-12 and abs(q - 32 * (c_t * delta) ** 2) < 1e-10
    assert distill.sample_terms(S, base, drafter, x0, 0, eps, None)[1] is None        # sigma_0 = 0: no normalised term


def test_loss_is_the_weighted_sum_and_the_acceptance_is_the_gaussian_overlap():
    base = nets.make_denoiser(inputs.make_gauss_params(0.7, 0.5), S)
    drafter = nets.make_denoiser(inputs.make_gauss_params(0.95, 0.4), S)
    x0s = np.random.default_rng(3).normal(0.7, 0.5, size=(200, 1, 1))
    Lp, Ln, L, acc = distill.distill_loss(S, base, drafter, x0s, None, 11, lambda1=2.0, lambda2=0.5)
    assert Lp > 0 and Ln > 0 and abs(L - (2.0 * Lp + 0.5 * Ln)) < 1e-12 and 0.0 < acc < 1.0
    # per sample: overlap of N(mu, sigma^2) and N(mu^, sigma^2) = 2 Phi(-|d|/2); 1-D check against a direct integral
    t = min(99, int(philox.uniform(11, 0, 0) * 100))
    eps = philox.x_init(11, 0, 1).reshape(1, 1)
    _, q = distill.sample_terms(S, base, drafter, x0s[0], t, eps, None)
    if q is not None:
        d = math.sqrt(q)
        z = np.linspace(-12, 12 + d, 400001)
        pdf = lambda m: np.exp(-0.5 * (z - m) ** 2) / math.sqrt(2 * math.pi)
        overlap = np.trapezoid(np.minimum(pdf(0.0), pdf(d)), z)
        assert abs(overlap - math.erfc(d / (2 * math.sqrt(2)))) < 1e-6


# ----------------------------------------------------------------------------- the distillation step (Gaussian drafter)
def _gauss_pair(m, s):
    return nets.make_denoiser(inputs.make_gauss_params(m, s), S)


def test_gauss_gradient_matches_finite_differences_of_the_pinned_loss():
    base = _gauss_pair(0.7, 0.5)
    x0s = np.random.default_rng(5).normal(0.7, 0.5, size=(96, 4, 2))
    m, s, l1, l2, seed = 0.95, 0.4, 1.5, 0.25, 17
    Lp, Ln, L, gm, gs = distill.gauss_distill_grad(S, base, m, s, x0s, None, seed, l1, l2)
    ref = distill.distill_loss(S, base, _gauss_pair(m, s), x0s, None, seed, l1, l2)
    assert abs(Lp - ref[0]) < 1e-12 * max(1, ref[0]) and abs(Ln - ref[1]) < 1e-10 * max(1, ref[1]) and abs(L - ref[2]) < 1e-10 * max(1, ref[2])
    h = 1e-6
    f = lambda mm, ss: distill.distill_loss(S, base, _gauss_pair(mm, ss), x0s, None, seed, l1, l2)[2]
    fd_m = (f(m + h, s) - f(m - h, s)) / (2 * h)
    fd_s = (f(m, s + h) - f(m, s - h)) / (2 * h)
    assert abs(gm - fd_m) < 1e-6 * max(1.0, abs(fd_m)) and abs(gs - fd_s) < 1e-6 * max(1.0, abs(fd_s))
    assert abs(gm) > 1e-3 and abs(gs) > 1e-3
    # each term alone (a dropped weight or a wrong c_t would survive a test of the sum only at one (lambda1, lambda2))
    for a, b in ((1.0, 0.0), (0.0, 1.0)):
        g = distill.gauss_distill_grad(S, base, m, s, x0s, None, seed, a, b)
        fa = lambda mm, ss: distill.distill_loss(S, base, _gauss_pair(mm, ss), x0s, None, seed, a, b)[2]
        assert abs(g[3] - (fa(m + h, s) - fa(m - h, s)) / (2 * h)) < 1e-6 * max(1.0, abs(g[3]))
        assert abs(g[4] - (fa(m, s + h) - fa(m, s - h)) / (2 * h)) < 1e-6 * max(1.0, abs(g[4]))


def test_gauss_distillation_descends_to_the_base_parameters():
    """The base's own parameters are a fixed point (zero loss, zero gradient); small steps decrease L monotonically
    and carry (m0, s0) to the base's."""
    base = _gauss_pair(0.7, 0.5)
    x0s = np.random.default_rng(6).normal(0.7, 0.5, size=(128, 1, 1))
    out = distill.gauss_distill_grad(S, base, 0.7, 0.5, x0s, None, 3)
    assert out[2] < 1e-24 and abs(out[3]) < 1e-12 and abs(out[4]) < 1e-12
    m, s, last = 0.95, 0.4, None
    for it in range(400):
        Lp, Ln, L, gm, gs, m, s = distill.gauss_distill_step(S, base, m, s, x0s, None, 3, 1.0, 1.0, lr=0.02)
        assert last is None or L <= last * (1 + 1e-12)
        last = L
    assert abs(m - 0.7) < 5e-3 and abs(s - 0.5) < 5e-3 and last < 1e-3
