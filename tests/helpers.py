"""Shared set-up for the GPU parity tests: one workload -> (CUDA sampler, oracle denoisers, obs)."""
import numpy as np

from oracle import ddpm, nets, spec
from paper_2512_15773_b200 import binding, inputs


def small_xfmr_workload(precision, d=128, heads=4, layers=2, dd=128, dlayers=1, H=16, A=2, To=2, Do=20, gamma=0.05):
    return dict(H=H, A=A, To=To, Do=Do, T=100, precision=precision,
                base=dict(arch="xfmr", layers=layers, d=d, heads=heads),
                draft=dict(arch="xfmr", layers=dlayers, d=dd, heads=heads), gamma=gamma)


def setup(wl, max_B, max_K, seed=1, use_graph=1, draft_is_base=False, precision=None, clip=0.0, drafter=0, verifier=0):
    prec = wl["precision"] if precision is None else precision
    cfg = binding.make_config(wl["H"], wl["A"], wl["To"], wl["Do"], wl["base"],
                              wl["base"] if draft_is_base else wl["draft"], T=wl["T"], max_B=max_B, max_K=max_K,
                              precision=prec, use_graph=use_graph, clip=clip, drafter=drafter, verifier=verifier)
    S = ddpm.Schedule(wl["T"], 1e-4, 0.02)
    frozen = wl["draft"]["arch"] == "frozen" and not draft_is_base
    if wl["base"]["arch"] == "gauss":
        pb, pd = wl["base_params"], wl.get("draft_params")
    else:
        pb = inputs.make_net(seed, wl, "base", bf16=(prec == 1))
        pd = pb if (draft_is_base or frozen) else inputs.make_net(seed + 1, wl, "draft", bf16=(prec == 1))
    smp = binding.Sampler(cfg)
    smp.load_weights(binding.BASE, pb)
    base = nets.make_denoiser(pb, S)
    if frozen:      # drafter-free: nothing to load, the oracle's drafter wraps its base
        return smp, S, base, spec.FrozenTargetDraft(base)
    smp.load_weights(binding.DRAFT, pd)
    return smp, S, base, nets.make_denoiser(pd, S)


def accept_t(mode=0, lam=1.0, sigma_scale=1.0, bonus=1):
    return binding.AcceptT(mode, lam, sigma_scale, bonus)


def oracle_accept(a):
    return spec.Accept(mode=a.mode, lam=a.lam, sigma_scale=a.sigma_scale, bonus=bool(a.bonus))


def max_rel(got, ref):
    """max |got - ref| / max |ref|: the 'max relative error' the tolerances are stated in."""
    return float(np.max(np.abs(got - ref)) / max(np.max(np.abs(ref)), 1e-30))


# ------------------------------------------------------------------------------------------------
# Round-level comparison of the CUDA path with the oracle, one environment at a time.
#
# The accept statistic depends on the two networks only through their difference at the SAME input:
# mu^_k - mu_k = -(c_x0 sqrt(1-abar)/sqrt(abar)) (eps^ - eps), so  d = -(c_tau / s) (eps^ - eps)  with
# c_tau = c_x0 sqrt(1-abar_tau) / (sqrt(abar_tau) sigma_tau).  If both network outputs are within the
# stated max-relative tolerance tol of the oracle's (|delta eps|_inf <= tol max|eps|), then
#     |delta d|_2 <= eta := (c_tau / s) sqrt(D) tol (max|eps^| + max|eps|)
# and, from  l = -1/2 |d|^2 - <d, xi>,
#     |l_gpu - l_oracle| <= eta (|d| + |xi|) + eta^2 / 2.
# A decision may differ from the oracle's only where |l_oracle - log thr| < 1e-3 + that bound.
# ------------------------------------------------------------------------------------------------
BAND = 1e-3


def logalpha_bound(S, tau, sigma_scale, eps_hat, eps, mu_hat, mu, xi, tol_eps):
    D = eps.size
    c_tau = S.c_x0[tau] * np.sqrt(1.0 - S.abar[tau]) / (np.sqrt(S.abar[tau]) * S.sigma[tau]) / sigma_scale
    eta = c_tau * np.sqrt(D) * tol_eps * (np.max(np.abs(eps_hat)) + np.max(np.abs(eps)))
    d = (mu_hat - mu).reshape(-1) / (sigma_scale * S.sigma[tau])
    return float(eta * (np.linalg.norm(d) + np.linalg.norm(xi)) + 0.5 * eta * eta)


def gpu_own_jstar(la_gpu, log_thr, K_eff, mode):
    """First k whose dumped statistic fails the test the kernel applies, and whether any of those
    comparisons sits within float rounding of the threshold (then the host cannot re-decide it)."""
    j, fragile = K_eff + 1, False
    for k in range(1, K_eff + 1):
        v = min(0.0, float(la_gpu[k - 1])) if mode == 1 else float(la_gpu[k - 1])
        fragile |= abs(v - log_thr[k - 1]) <= 4e-6 * max(1.0, abs(log_thr[k - 1]))
        if v < log_thr[k - 1]:
            j = k
            break
    return j, fragile


def check_round_env(S, noise, acc, b, t0, K, d, g, tol_eps, tol_x):
    """Compare one environment's round.  d: the oracle's dump; g: dict(xt [K+1, D], mh [K, D], eps [K+1, D],
    la [K], j, t_new, x_new [D], t_oracle, x_oracle) from tsdp_round.  Asserts everything that does not depend
    on a decision; returns True if the decisions were checked too (j*, t, committed latent), False if a
    deciding statistic lay inside the tolerated band and the two sides took different decisions."""
    Ke = d["K_eff"]
    s = acc.sigma_scale
    log_thr, bounds = [], []
    for k in range(1, Ke + 1):
        tau = t0 - k + 1
        assert np.max(np.abs(g["xt"][k] - d["x_tilde"][k].reshape(-1))) < tol_x, (b, k)
        assert np.max(np.abs(g["mh"][k - 1] - d["mu_hat"][k].reshape(-1))) < tol_x, (b, k)
        log_thr.append(float(np.log(noise.u(b, tau))) if acc.mode == 0 else float(np.log(acc.lam)))
        bounds.append(logalpha_bound(S, tau, s, d["eps_hat"][k], d["eps"][k - 1], d["mu_hat"][k], d["mu"][k],
                                     d["xi"][k].reshape(-1), tol_eps))
    for k in range(d["n_base"]):
        assert max_rel(g["eps"][k], d["eps"][k].reshape(-1)) < tol_eps, (b, k)
    # the statistic itself, within what the denoiser tolerance allows
    for k in range(1, Ke + 1):
        lo = d["log_alpha"][k - 1]
        assert abs(g["la"][k - 1] - lo) <= bounds[k - 1] + 1e-4 * max(1.0, abs(lo)), (b, k, g["la"][k - 1], lo, bounds[k - 1])
    # the kernel's decision follows from its own statistic, exactly
    j_own, fragile = gpu_own_jstar(g["la"], log_thr, Ke, acc.mode)
    if not fragile:
        assert g["j"] == j_own, (b, g["j"], j_own)
    # the oracle's decisions up to and including its first rejection are the ones that matter
    jo = d["jstar"]
    near = False
    for k in range(1, min(jo, Ke) + 1):
        v = min(0.0, d["log_alpha"][k - 1]) if acc.mode == 1 else d["log_alpha"][k - 1]
        near |= abs(v - log_thr[k - 1]) < BAND + bounds[k - 1]
    if g["j"] != jo:
        assert near, (b, g["j"], jo, d["log_alpha"], log_thr, bounds)
        return False
    assert g["t_new"] == g["t_oracle"], (b, g["t_new"], g["t_oracle"])
    assert np.max(np.abs(g["x_new"].reshape(-1) - g["x_oracle"].reshape(-1))) < 3 * tol_x, b
    return True
