"""DDPM scheduler S: the tables and the one-step posterior the paper calls "the DDPM scheduler".

The paper never writes S out (Sec. 3.2, "Draft Generation Procedure": x_{t-1} = S(m_t, t, x_t);
"Verification of Speculative Drafts": S yields a conditional mean mu_i and a standard deviation
sigma_i per candidate).  The textbook form (Ho et al. 2020, Eqs. 6-7, with the posterior-variance
choice) is used:

    beta_t linear from beta0 to beta1 over t = 0..T-1,  alpha_t = 1 - beta_t,
    abar_t = prod_{s<=t} alpha_s,  abar_{-1} := 1,
    x0_hat = (x_t - sqrt(1 - abar_t) eps) / sqrt(abar_t)          (clipped to +-clip iff clip > 0)
    mu     = sqrt(abar_{t-1}) beta_t / (1 - abar_t) * x0_hat
             + sqrt(alpha_t) (1 - abar_{t-1}) / (1 - abar_t) * x_t
    sigma_t^2 = beta_t (1 - abar_{t-1}) / (1 - abar_t),  so sigma_0 = 0
    x_{t-1} = mu + sigma_t xi.

Time convention: a network called with timestep t receives the latent "at t"; the transition
"at t" produces the latent at t-1; the latent at -1 is the clean action chunk.
"""
import numpy as np


class Schedule:
    def __init__(self, T=100, beta0=1e-4, beta1=0.02):
        self.T = T
        self.beta = np.linspace(beta0, beta1, T, dtype=np.float64)
        self.alpha = 1.0 - self.beta
        self.abar = np.cumprod(self.alpha)
        self.abar_prev = np.concatenate([[1.0], self.abar[:-1]])
        self.sigma = np.sqrt(self.beta * (1.0 - self.abar_prev) / (1.0 - self.abar))
        # coefficients of x0_hat and x_t in the posterior mean
        self.c_x0 = np.sqrt(self.abar_prev) * self.beta / (1.0 - self.abar)
        self.c_xt = np.sqrt(self.alpha) * (1.0 - self.abar_prev) / (1.0 - self.abar)

    def x0_hat(self, x_t, eps, t, clip=0.0):
        x0 = (x_t - np.sqrt(1.0 - self.abar[t]) * eps) / np.sqrt(self.abar[t])
        if clip > 0.0:
            x0 = np.clip(x0, -clip, clip)
        return x0

    def posterior_mean(self, x_t, eps, t, clip=0.0):
        """mu(x_t, eps, t): mean of the Gaussian reverse transition taken at timestep t."""
        return self.c_x0[t] * self.x0_hat(x_t, eps, t, clip) + self.c_xt[t] * x_t

    def step(self, x_t, eps, t, xi, clip=0.0):
        """x_{t-1} = mu + sigma_t xi; returns (x_{t-1}, mu)."""
        mu = self.posterior_mean(x_t, eps, t, clip)
        return mu + self.sigma[t] * xi, mu


def sinusoidal_embedding(tau, dim):
    """[sin(tau f_i) | cos(tau f_i)], f_i = 10000^(-i / (dim/2)), i = 0..dim/2-1."""
    half = dim // 2
    f = 10000.0 ** (-np.arange(half, dtype=np.float64) / half)
    return np.concatenate([np.sin(tau * f), np.cos(tau * f)])
