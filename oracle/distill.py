"""Distillation objective of the drafter against the frozen base model (Sec. 3.2, "Draft model"), numpy fp64.
Test infrastructure: only tests/, the smoke check and bench.py's CPU baseline may import this package.

For a clean action chunk x0, a timestep t and Gaussian noise eps, the noisy latent is the forward-process sample
    x_t = sqrt(abar_t) x0 + sqrt(1 - abar_t) eps,
and with m = M(x_t, t), m^ = M^(x_t, t) the two networks' outputs and mu, mu^ the DDPM posterior means they give,
    L_pred = E | m^ - m |^2,      L_norm = E | (mu^ - mu) / sigma_t |^2,      L = lambda1 L_pred + lambda2 L_norm.
Norms are over the whole chunk latent, expectations are sample means over (t, x0, eps).

What the paper does not fix, and is read here: t is uniform on {0..T-1}; sigma_0 = 0, so samples that draw t = 0
enter L_pred only and L_norm averages over the samples with t >= 1; the draws come from the counter-based
generator -- t_n = floor(T u) with u the uniform of (seed, sample n, timestep code 0), eps the INIT-stream normals
of (seed, n).  The last output is not in the paper: the mean over t >= 1 of 2 Phi(-|d| / 2), d = (mu^ - mu)/sigma_t,
the probability that the likelihood-ratio test of Sec. 3.1 accepts a draft with that mean offset (closed form for
two Gaussians of equal covariance) -- what L_norm is a proxy for.
"""
import math

import numpy as np

from . import philox


def sample_terms(sched, base, drafter, x0, t, eps, obs, clip=0.0):
    """(|m^ - m|^2, |d|^2 or None at t = 0) for one sample."""
    x_t = np.sqrt(sched.abar[t]) * x0 + np.sqrt(1.0 - sched.abar[t]) * eps
    m, mh = base(x_t, t, obs), drafter(x_t, t, obs)
    pred = float(np.sum((mh - m) ** 2))
    if t == 0:
        return pred, None
    d = (sched.posterior_mean(x_t, mh, t, clip) - sched.posterior_mean(x_t, m, t, clip)) / sched.sigma[t]
    return pred, float(np.sum(d * d))


def distill_loss(sched, base, drafter, x0s, obs, seed, lambda1=1.0, lambda2=1.0, clip=0.0):
    """Returns (L_pred, L_norm, L, mean acceptance probability) over the samples x0s [N, H, A]."""
    preds, norms, accs = [], [], []
    for n, x0 in enumerate(x0s):
        t = min(sched.T - 1, int(philox.uniform(seed, n, 0) * sched.T))
        eps = philox.x_init(seed, n, x0.size).reshape(x0.shape)
        p, q = sample_terms(sched, base, drafter, np.asarray(x0, dtype=np.float64), t, eps, None if obs is None else obs[n], clip)
        preds.append(p)
        if q is not None:
            norms.append(q)
            accs.append(math.erfc(math.sqrt(q) / (2.0 * math.sqrt(2.0))))
    L_pred = float(np.mean(preds))
    L_norm = float(np.mean(norms)) if norms else 0.0
    return L_pred, L_norm, lambda1 * L_pred + lambda2 * L_norm, (float(np.mean(accs)) if accs else 1.0)


def gauss_distill_grad(sched, base, m0, s0, x0s, obs, seed, lambda1=1.0, lambda2=1.0):
    """Gradient of L = lambda1 L_pred + lambda2 L_norm with respect to the parameters theta = (m0, s0) of the
    closed-form Gaussian drafter  m^(x, t) = sqrt(1 - abar)(x - sqrt(abar) m0) / (abar s0^2 + 1 - abar), the base
    model frozen (Sec. 3.2, "Draft Model Training": only theta is updated).  Same draws as distill_loss.

    With v = abar s0^2 + 1 - abar:
        d m^ / d m0 = -sqrt(1 - abar) sqrt(abar) / v,
        d m^ / d s0 = -sqrt(1 - abar) (x - sqrt(abar) m0) 2 abar s0 / v^2,
    and, the posterior mean being affine in the network output (no clipping),
        (mu^ - mu) / sigma_t = -c_t (m^ - m),   c_t = c_x0(t) sqrt(1 - abar_t) / (sqrt(abar_t) sigma_t),
    so  dL/dtheta = sum_n (lambda1 / N + [t_n >= 1] lambda2 c_{t_n}^2 / N_1) 2 <m^_n - m_n, d m^_n / d theta>,
    N_1 the number of samples with t_n >= 1.  Returns (L_pred, L_norm, L, dL/dm0, dL/ds0)."""
    N = len(x0s)
    rows = []
    for n, x0 in enumerate(x0s):
        t = min(sched.T - 1, int(philox.uniform(seed, n, 0) * sched.T))
        eps = philox.x_init(seed, n, x0.size).reshape(x0.shape)
        ab = sched.abar[t]
        x_t = np.sqrt(ab) * np.asarray(x0, dtype=np.float64) + np.sqrt(1.0 - ab) * eps
        m = base(x_t, t, None if obs is None else obs[n])
        v = ab * s0 * s0 + 1.0 - ab
        mh = np.sqrt(1.0 - ab) * (x_t - np.sqrt(ab) * m0) / v
        dm = -np.sqrt(1.0 - ab) * np.sqrt(ab) / v * np.ones_like(x_t)
        ds = -np.sqrt(1.0 - ab) * (x_t - np.sqrt(ab) * m0) * 2.0 * ab * s0 / (v * v)
        r = mh - m
        c2 = 0.0
        if t >= 1:
            c_t = sched.c_x0[t] * np.sqrt(1.0 - ab) / (np.sqrt(ab) * sched.sigma[t])
            c2 = c_t * c_t
        rows.append((float(np.sum(r * r)), c2, t >= 1, 2.0 * float(np.sum(r * dm)), 2.0 * float(np.sum(r * ds))))
    N1 = sum(1 for r in rows if r[2])
    L_pred = sum(r[0] for r in rows) / N
    L_norm = sum(r[0] * r[1] for r in rows) / N1 if N1 else 0.0
    gm = sum((lambda1 / N + (lambda2 * r[1] / N1 if r[2] else 0.0)) * r[3] for r in rows)
    gs = sum((lambda1 / N + (lambda2 * r[1] / N1 if r[2] else 0.0)) * r[4] for r in rows)
    return L_pred, L_norm, lambda1 * L_pred + lambda2 * L_norm, gm, gs


def gauss_distill_step(sched, base, m0, s0, x0s, obs, seed, lambda1=1.0, lambda2=1.0, lr=0.1):
    """One plain gradient step theta <- theta - lr dL/dtheta.  Returns (L_pred, L_norm, L, dL/dm0, dL/ds0, m0', s0');
    the losses are those before the step."""
    Lp, Ln, L, gm, gs = gauss_distill_grad(sched, base, m0, s0, x0s, obs, seed, lambda1, lambda2)
    return Lp, Ln, L, gm, gs, m0 - lr * gm, s0 - lr * gs
