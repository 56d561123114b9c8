"""Parity at the sizes and in the launch configuration the benchmark times, on sampled outputs.

The full serving batch (256 environments x 11 candidates x 16 tokens = 45 056 token rows through the
persistent 148-CTA GEMM, the tensor-core attentions and the fused acceptance kernel) is run once; a few
environments are then recomputed one by one by the oracle."""
import numpy as np
import pytest
import torch

from oracle import ddpm, nets, spec
from paper_2512_15773_b200 import binding, inputs
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def test_serving_round_at_bench_size_sampled_environments():
    wl = dict(inputs.WORKLOADS["serving_xfmr"])
    B, K, seed = wl["B"], wl["K"], 7
    smp, S, base, draft = hp.setup(wl, max_B=B, max_K=K, drafter=0)
    D = wl["H"] * wl["A"]; shape = (wl["H"], wl["A"])
    obs = inputs.make_obs(100, B, wl["To"], wl["Do"])
    noise = spec.PhiloxNoise(seed)
    rng = np.random.default_rng(0)
    t0s = rng.integers(0, 100, size=B).astype(np.int32)
    t0s[:4] = [99, 50, 3, 0]
    x0 = rng.normal(size=(B, D)).astype(np.float32)
    dx = torch.tensor(x0, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    h_t = t0s.copy()
    d_xt = torch.zeros(B, K + 1, D, device="cuda"); d_mh = torch.zeros(B, K, D, device="cuda")
    d_eps = torch.zeros(B, K + 1, D, device="cuda"); d_la = torch.zeros(B, K, device="cuda")
    h_j = np.zeros(B, dtype=np.int32)
    acc = hp.accept_t(sigma_scale=1.5)
    smp.round(dobs, B, K, acc, seed, dx, h_t, d_xt, d_mh, d_eps, d_la, h_j)
    xt, mh, eps, la = d_xt.cpu().numpy(), d_mh.cpu().numpy(), d_eps.cpu().numpy(), d_la.cpu().numpy()
    x_new = dx.cpu().numpy()
    checked = 0
    envs = (0, 1, 2, 3, 100, 255)
    for b in envs:
        xo, to, d = spec.spec_round(S, base, draft, noise, b, obs[b], x0[b].astype(np.float64).reshape(shape), int(t0s[b]), K,
                                    hp.oracle_accept(acc))
        g = dict(xt=xt[b], mh=mh[b], eps=eps[b], la=la[b], j=int(h_j[b]), t_new=int(h_t[b]), x_new=x_new[b],
                 t_oracle=to, x_oracle=xo)
        checked += hp.check_round_env(S, noise, hp.oracle_accept(acc), b, int(t0s[b]), K, d, g, 2e-2, 3e-3)
    assert checked >= len(envs) - 1, checked
    smp.close()


def test_vla_shaped_dit_forward_at_full_width_sampled_candidates():
    """Full width and sequence of the VLA-scale expert (d = 1024, 16 heads, 50 tokens, 256 context tokens,
    GEMMs up to 4096 x 4096), two blocks deep so that the oracle stays affordable."""
    wl = dict(inputs.WORKLOADS["vla_dit"])
    wl["base"] = dict(wl["base"], layers=2); wl["draft"] = dict(wl["draft"], layers=1)
    wl["gamma"] = 1.0
    N = 40                                   # 2000 token rows: 16 row tiles, ragged
    smp, S, base, draft = hp.setup(wl, max_B=N, max_K=1)
    rng = np.random.default_rng(1)
    x = rng.normal(size=(N, wl["H"], wl["A"])).astype(np.float32)
    tau = rng.integers(0, 100, size=N).astype(np.int32)
    obs = inputs.make_obs(5, N, wl["To"], wl["Do"])
    dx = torch.tensor(x, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    for which, net in ((binding.BASE, base), (binding.DRAFT, draft)):
        out = torch.zeros_like(dx)
        smp.denoise(which, dx, tau, dobs, N, out)
        got = out.cpu().numpy()
        for n in (0, 17, 39):
            ref = net(x[n].astype(np.float64), int(tau[n]), obs[n])
            assert hp.max_rel(got[n], ref) < 2e-2, (which, n)
    smp.close()


def test_mid_size_batch_both_head_widths():
    """1200 candidates x 16 token rows: the GEMMs run with their TMA-store tiles (128 x 256 for the base, 128 x 128
    for the drafter), several waves of the attention kernels; head widths 64 and 32."""
    wl = dict(inputs.WORKLOADS["pusht_xfmr"], precision=1, gamma=1.0)
    N = 1200
    smp, S, base, draft = hp.setup(wl, max_B=N, max_K=1)
    rng = np.random.default_rng(2)
    x = rng.normal(size=(N, wl["H"], wl["A"])).astype(np.float32)
    tau = rng.integers(0, 100, size=N).astype(np.int32)
    obs = inputs.make_obs(6, N, wl["To"], wl["Do"])
    dx = torch.tensor(x, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    for which, net in ((binding.BASE, base), (binding.DRAFT, draft)):
        out = torch.zeros_like(dx)
        smp.denoise(which, dx, tau, dobs, N, out)
        got = out.cpu().numpy()
        assert np.isfinite(got).all()
        for n in (0, 1, 7, 599, 1199):
            ref = net(x[n].astype(np.float64), int(tau[n]), obs[n])
            assert hp.max_rel(got[n], ref) < 2e-2, (which, n)
    smp.close()


def test_robomimic_unet_at_full_width_sampled_candidates():
    """The conv UNet at the width the benchmark times (channels 256 / 512 / 1024, kernel-5 convolutions with
    K = 5 C_in up to 7680 through the tensor-core GEMM's convolution addressing) and at its batch-32 row counts:
    288 candidates = 5760 / 3456 / 2304 padded rows per level, several waves of row tiles with ragged tails.
    A few candidates are recomputed by the oracle."""
    wl = dict(inputs.WORKLOADS["robomimic_unet"], gamma=1.0)
    N = 32 * 9
    smp, S, base, draft = hp.setup(wl, max_B=N, max_K=1)
    rng = np.random.default_rng(3)
    x = rng.normal(size=(N, wl["H"], wl["A"])).astype(np.float32)
    tau = rng.integers(0, 100, size=N).astype(np.int32)
    tau[:2] = [99, 0]
    obs = inputs.make_obs(8, N, wl["To"], wl["Do"])
    dx = torch.tensor(x, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    out = torch.zeros_like(dx)
    smp.denoise(binding.BASE, dx, tau, dobs, N, out)
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    for n in (0, 1, 143, 287):
        ref = base(x[n].astype(np.float64), int(tau[n]), obs[n])
        assert hp.max_rel(got[n], ref) < 2e-2, n
    smp.close()


def test_robomimic_unet_at_full_width_batch_one_split_reduction():
    """The same UNet at the row counts of a batch-1 round (9 candidates = 180 / 108 / 72 padded rows per level): every
    level is one or two row tiles, so the convolution GEMMs split their K = 1280 .. 7680 reductions into parts that
    run on otherwise idle SMs and the GroupNorm kernel adds the partial sums.  Every candidate against the oracle."""
    wl = dict(inputs.WORKLOADS["robomimic_unet"], gamma=1.0)
    N = 9
    smp, S, base, draft = hp.setup(wl, max_B=N, max_K=1)
    rng = np.random.default_rng(13)
    x = rng.normal(size=(N, wl["H"], wl["A"])).astype(np.float32)
    tau = rng.integers(0, 100, size=N).astype(np.int32)
    tau[:2] = [99, 0]
    obs = inputs.make_obs(9, N, wl["To"], wl["Do"])
    dx = torch.tensor(x, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    out = torch.zeros_like(dx)
    smp.denoise(binding.BASE, dx, tau, dobs, N, out)
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    for n in (0, 1, 4, 8):
        ref = base(x[n].astype(np.float64), int(tau[n]), obs[n])
        assert hp.max_rel(got[n], ref) < 2e-2, n
    smp.close()


def _round_sampled(wl, B, K, seed, t0s, envs, acc=None):
    """One round at full width from random states; the listed environments are recomputed by the oracle."""
    acc = acc or hp.accept_t()
    smp, S, base, draft = hp.setup(wl, max_B=B, max_K=K)
    D = wl["H"] * wl["A"]; shape = (wl["H"], wl["A"])
    obs = inputs.make_obs(50, B, wl["To"], wl["Do"])
    noise = spec.PhiloxNoise(seed)
    rng = np.random.default_rng(seed)
    x0 = rng.normal(size=(B, D)).astype(np.float32)
    dx = torch.tensor(x0, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    h_t = np.array(t0s, dtype=np.int32)
    d_xt = torch.zeros(B, K + 1, D, device="cuda"); d_mh = torch.zeros(B, K, D, device="cuda")
    d_eps = torch.zeros(B, K + 1, D, device="cuda"); d_la = torch.zeros(B, K, device="cuda")
    h_j = np.zeros(B, dtype=np.int32)
    smp.round(dobs, B, K, acc, seed, dx, h_t, d_xt, d_mh, d_eps, d_la, h_j)
    xt, mh, eps, la = d_xt.cpu().numpy(), d_mh.cpu().numpy(), d_eps.cpu().numpy(), d_la.cpu().numpy()
    x_new = dx.cpu().numpy()
    checked = 0
    for b in envs:
        xo, to, d = spec.spec_round(S, base, draft, noise, b, obs[b], x0[b].astype(np.float64).reshape(shape), int(t0s[b]), K,
                                    hp.oracle_accept(acc))
        g = dict(xt=xt[b], mh=mh[b], eps=eps[b], la=la[b], j=int(h_j[b]), t_new=int(h_t[b]), x_new=x_new[b],
                 t_oracle=to, x_oracle=xo)
        checked += hp.check_round_env(S, noise, hp.oracle_accept(acc), b, int(t0s[b]), K, d, g, 2e-2, 3e-3)
    assert smp.check_guards() > 0
    smp.close()
    return checked


def test_vla_shaped_round_at_full_width_sampled_environments():
    """A whole speculative round of the VLA-scale pairing at full width (d = 1024 / 512, 50 tokens, 256 context tokens,
    K = 16; two base blocks and one drafter block so that the oracle stays affordable): compacted candidate list with a
    finished environment and short windows in it, the two-CTA GEMM on the K >= 1024 shapes, context cross-attention
    grouped by slot through the plan's slot offsets."""
    wl = dict(inputs.WORKLOADS["vla_dit"])
    wl["base"] = dict(wl["base"], layers=2); wl["draft"] = dict(wl["draft"], layers=1)
    B, K = 12, 16
    t0s = [99, 50, 7, 0, -1, 30, 3, 99, 12, 64, 1, 80]
    checked = _round_sampled(wl, B, K, 17, t0s, envs=(0, 2, 3))
    assert checked >= 2


def test_robomimic_shaped_round_at_full_width_sampled_environments():
    """The conv UNet at its real channel widths verified against the 4-block transformer drafter's drafts, one round,
    ragged windows and a finished environment; two environments through the oracle."""
    wl = dict(inputs.WORKLOADS["robomimic_unet"])
    B, K = 10, 8
    t0s = [99, 40, 3, -1, 0, 70, 5, 99, 20, 1]
    checked = _round_sampled(wl, B, K, 23, t0s, envs=(1, 2))
    assert checked >= 1
