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
