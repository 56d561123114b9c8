"""Acceptance / fidelity trade-off of the lossy speculative knobs on the 1-D Gaussian toy.

    python -m paper_2512_15773_b200.sweep [--envs 100000] [--K 6]

The paper makes the acceptance threshold lambda and the sigma scale tunable (Sec. 3.2, "Verification
of Speculative Drafts"; Sec. 3.3 action space) to keep acceptance high; both leave the exact
likelihood-ratio test, so the sampled law moves away from vanilla DDPM's.  On data ~ N(m0, s0^2)
with the closed-form optimal denoiser as base model and a perturbed one as drafter, every reverse
transition is affine-Gaussian and the law of vanilla DDPM's output is known in closed form, so the
damage can be measured: the Kolmogorov-Smirnov distance between `envs` GPU samples and that law,
beside the acceptance rate and the base forwards per chunk.  One JSON line per setting.
"""
import argparse
import json

import numpy as np

M0, S0 = 0.7, 0.5                      # data law; the drafter believes in (M0 + 0.25, 0.8 S0)


def vanilla_output_law(T=100, beta0=1e-4, beta1=0.02, m0=M0, s0=S0):
    """Mean and standard deviation of x_{-1} when every step uses the optimal denoiser of N(m0, s0^2)
    data: with eps* affine in x the transition is x' = a_t x + b_t + sigma_t xi, so the Gaussian law is
    propagated by mean <- a mean + b, var <- a^2 var + sigma^2 from x_T ~ N(0, 1)."""
    beta = np.linspace(beta0, beta1, T)
    alpha = 1.0 - beta
    abar = np.cumprod(alpha)
    abar_prev = np.concatenate([[1.0], abar[:-1]])
    mean, var = 0.0, 1.0
    for t in range(T - 1, -1, -1):
        c0 = np.sqrt(abar_prev[t]) * beta[t] / (1.0 - abar[t])
        ct = np.sqrt(alpha[t]) * (1.0 - abar_prev[t]) / (1.0 - abar[t])
        sig2 = beta[t] * (1.0 - abar_prev[t]) / (1.0 - abar[t])
        den = abar[t] * s0 * s0 + 1.0 - abar[t]
        # eps* = g (x - sqrt(abar) m0), x0_hat = (x - sqrt(1-abar) eps*) / sqrt(abar)
        g = np.sqrt(1.0 - abar[t]) / den
        k = (1.0 - np.sqrt(1.0 - abar[t]) * g) / np.sqrt(abar[t])          # x0_hat = k x + l
        l = np.sqrt(1.0 - abar[t]) * g * m0
        a, b = c0 * k + ct, c0 * l
        mean, var = a * mean + b, a * a * var + sig2
    return mean, np.sqrt(var)


def ks_distance(x, mean, std):
    """sup |F_n - F| against N(mean, std^2)."""
    from math import erf, sqrt
    z = np.sort((x - mean) / std)
    F = 0.5 * (1.0 + np.vectorize(erf)(z / sqrt(2.0)))
    n = len(z)
    return float(max(np.max(np.arange(1, n + 1) / n - F), np.max(F - np.arange(0, n) / n)))


def settings():
    yield dict(mode=0, lam=1.0, s=1.0, label="lossless (U <= alpha, s = 1)")
    for s in (1.5, 2.0, 3.0):
        yield dict(mode=0, lam=1.0, s=s, label=f"U <= alpha, sigma scale {s}")
    for lam in (0.9, 0.6, 0.3, 0.1):
        yield dict(mode=1, lam=lam, s=1.0, label=f"threshold p >= {lam}")
    yield dict(mode=1, lam=0.6, s=2.0, label="threshold p >= 0.6, sigma scale 2")


def main():
    import torch
    from . import binding, inputs
    ap = argparse.ArgumentParser()
    ap.add_argument("--envs", type=int, default=100_000)
    ap.add_argument("--K", type=int, default=6)
    ap.add_argument("--seed", type=int, default=1234)
    args = ap.parse_args()
    B = args.envs
    cfg = binding.make_config(1, 1, 0, 0, dict(arch="gauss"), dict(arch="gauss"), max_B=B, max_K=args.K, precision=0)
    smp = binding.Sampler(cfg)
    smp.load_weights(binding.BASE, inputs.make_gauss_params(M0, S0))
    smp.load_weights(binding.DRAFT, inputs.make_gauss_params(M0 + 0.25, 0.8 * S0))
    mean, std = vanilla_output_law()
    out = torch.zeros(B, 1, 1, device="cuda")
    for st in settings():
        smp.reset_stats()
        smp.sample_chunk(None, B, args.K, binding.AcceptT(st["mode"], st["lam"], st["s"], 1), args.seed, out)
        x = out.cpu().numpy().reshape(-1).astype(np.float64)
        s = smp.stats()
        print(json.dumps(dict(setting=st["label"], mode=st["mode"], lam=st["lam"], sigma_scale=st["s"], K=args.K, envs=B,
                              acceptance=s["drafts_accepted"] / max(s["drafts_tested"], 1),
                              base_forwards_per_chunk=s["env_rounds"] / B, ks_distance=ks_distance(x, mean, std),
                              ks_noise_floor=1.36 / np.sqrt(B), sample_mean=float(x.mean()), sample_std=float(x.std()),
                              law_mean=mean, law_std=std)))
    smp.close()


if __name__ == "__main__":
    main()
