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
