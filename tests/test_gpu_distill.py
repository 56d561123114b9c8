"""GPU parity of the distillation-objective evaluation (tsdp_distill_loss) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import distill
from paper_2512_15773_b200 import binding, inputs
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _case(wl, N, seed, precision=None, draft_is_base=False):
    smp, S, base, draft = hp.setup(wl, max_B=N, max_K=2, precision=precision, draft_is_base=draft_is_base)
    rng = np.random.default_rng(seed)
    x0 = rng.normal(0.0, 0.7, size=(N, wl["H"], wl["A"])).astype(np.float32)
    obs = inputs.make_obs(9, N, wl["To"], wl["Do"])
    got = smp.distill_loss(torch.tensor(x0, device="cuda"), torch.tensor(obs, dtype=torch.float32, device="cuda"), N, seed,
                           lambda1=1.5, lambda2=0.25)
    ref = distill.distill_loss(S, base, draft, x0.astype(np.float64), obs, seed, lambda1=1.5, lambda2=0.25)
    smp.close()
    return got, ref


def test_distill_loss_fp32_mlp_matches_oracle():
    got, ref = _case(dict(inputs.WORKLOADS["toy_mlp"]), 64, 5)
    for g, r in zip(got, ref):
        assert abs(g - r) < 1e-4 * max(abs(r), 1e-6), (got, ref)
    assert abs(got[2] - (1.5 * got[0] + 0.25 * got[1])) < 1e-9 * max(1.0, got[2])


def test_distill_loss_bf16_transformer_matches_oracle():
    # sums of squared differences of two bf16 forwards: the relative error of a difference is larger than that of an output
    got, ref = _case(dict(inputs.WORKLOADS["pusht_xfmr"], gamma=1.0), 40, 6, precision=1)
    assert abs(got[0] - ref[0]) < 5e-2 * ref[0] and abs(got[1] - ref[1]) < 5e-2 * ref[1], (got, ref)
    assert abs(got[3] - ref[3]) < 2e-2


def test_distill_loss_of_equal_networks_is_zero():
    got, ref = _case(dict(inputs.WORKLOADS["toy_mlp"]), 16, 7, draft_is_base=True)
    assert got == (0.0, 0.0, 0.0, 1.0) and ref == (0.0, 0.0, 0.0, 1.0)


def test_distill_loss_rejects_a_frozen_drafter_and_bad_sizes():
    wl = dict(inputs.WORKLOADS["toy_mlp"], draft=dict(arch="frozen"))
    smp, *_ = hp.setup(wl, max_B=4, max_K=2)
    x0 = torch.zeros(4, wl["H"], wl["A"], device="cuda")
    obs = torch.zeros(4, wl["To"], wl["Do"], device="cuda")
    with pytest.raises(binding.TsdpError):
        smp.distill_loss(x0, obs, 4, 1)
    smp.close()
    smp, *_ = hp.setup(dict(inputs.WORKLOADS["toy_mlp"]), max_B=4, max_K=2)
    with pytest.raises(binding.TsdpError):
        smp.distill_loss(x0, obs, 5, 1)
    smp.close()


def _gauss_wl(m_b, s_b, m_d, s_d, H=4, A=2):
    return dict(H=H, A=A, To=0, Do=0, T=100, precision=0, base=dict(arch="gauss"), draft=dict(arch="gauss"),
                base_params=inputs.make_gauss_params(m_b, s_b), draft_params=inputs.make_gauss_params(m_d, s_d))


def test_distill_step_matches_oracle_step_by_step():
    """tsdp_distill_step on the closed-form Gaussian drafter: losses, gradient and the updated parameters against the
    oracle, chained over several steps (each step starts from the parameters the GPU's previous step left)."""
    from oracle import ddpm, nets
    wl = _gauss_wl(0.7, 0.5, 0.95, 0.4)
    N = 96
    smp, S, base, _ = hp.setup(wl, max_B=N, max_K=2)
    x0 = np.random.default_rng(5).normal(0.7, 0.5, size=(N, wl["H"], wl["A"])).astype(np.float32)
    d_x0 = torch.tensor(x0, device="cuda")
    m, s = np.float32(0.95), np.float32(0.4)
    for it in range(6):
        got = smp.distill_step(d_x0, None, N, 100 + it, lambda1=1.5, lambda2=0.25, lr=0.05)
        ref = distill.gauss_distill_step(S, base, float(m), float(s), x0.astype(np.float64), None, 100 + it, 1.5, 0.25, lr=0.05)
        for g, r in zip(got[:5], ref[:5]):
            assert abs(g - r) < 2e-4 * max(abs(r), 1e-3), (it, got, ref)
        assert abs(got[5] - ref[5]) < 1e-5 and abs(got[6] - ref[6]) < 1e-5, (it, got, ref)
        m, s = np.float32(got[5]), np.float32(got[6])
    # the loss entry point sees the updated drafter
    L = smp.distill_loss(d_x0, None, N, 7)
    ref = distill.distill_loss(S, base, nets.make_denoiser(inputs.make_gauss_params(float(m), float(s)), S), x0.astype(np.float64), None, 7)
    assert abs(L[2] - ref[2]) < 1e-4 * max(ref[2], 1e-6)
    smp.close()


def test_distillation_raises_acceptance_on_the_gaussian_toy():
    """Train the drafter from (0.95, 0.4) towards the base's (0.7, 0.5) and sample before / after: the loss falls
    monotonically on a fixed batch, the parameters approach the base's, and the sampler's acceptance rises and its
    base forwards per chunk fall."""
    wl = _gauss_wl(0.7, 0.5, 0.95, 0.4, H=1, A=1)
    B, N, K = 4096, 512, 6
    smp, *_ = hp.setup(wl, max_B=B, max_K=K)
    out = torch.zeros(B, 1, 1, device="cuda")

    def sample():
        smp.reset_stats()
        smp.sample_chunk(None, B, K, hp.accept_t(), 42, out)
        st = smp.stats()
        return st["drafts_accepted"] / st["drafts_tested"], st["env_rounds"] / B

    acc0, fw0 = sample()
    x0 = torch.tensor(np.random.default_rng(8).normal(0.7, 0.5, size=(N, 1, 1)).astype(np.float32), device="cuda")
    last = None
    for it in range(300):
        r = smp.distill_step(x0, None, N, 3, lr=0.02)
        assert last is None or r[2] <= last * (1 + 1e-5)
        last = r[2]
    assert abs(r[5] - 0.7) < 2e-2 and abs(r[6] - 0.5) < 2e-2 and last < 5e-3
    acc1, fw1 = sample()
    assert acc1 > acc0 + 0.01 and acc1 > 0.99 and fw1 < fw0
    with pytest.raises(binding.TsdpError):      # only the Gaussian drafter has a backward pass
        s2, *_ = hp.setup(dict(inputs.WORKLOADS["toy_mlp"]), max_B=4, max_K=2)
        try:
            s2.distill_step(torch.zeros(4, 16, 2, device="cuda"), torch.zeros(4, 1, 20, device="cuda"), 4, 1)
        finally:
            s2.close()
    smp.close()
