"""Host helpers of the trade-off sweep, and (GPU) the lossy acceptance modes against the oracle."""
import numpy as np
import pytest
from scipy import stats

from paper_2512_15773_b200 import inputs, sweep


def test_vanilla_output_law_matches_the_oracle_side_recursion():
    from tests.test_oracle_chain import _analytic_marginal
    m, s = sweep.vanilla_output_law()
    mo, so = _analytic_marginal()
    assert abs(m - mo) < 1e-12 and abs(s - so) < 1e-12


def test_ks_distance_is_the_textbook_statistic():
    x = np.random.default_rng(1).normal(0.3, 2.0, size=5000)
    assert abs(sweep.ks_distance(x, 0.3, 2.0) - stats.kstest((x - 0.3) / 2.0, "norm").statistic) < 1e-12
    assert sweep.ks_distance(x, 1.3, 2.0) > 0.15


@pytest.mark.gpu
@pytest.mark.parametrize("mode,lam,s", [(1, 0.6, 1.0), (0, 1.0, 2.0), (1, 0.3, 2.0)])
def test_lossy_modes_on_gpu_match_oracle_chain_by_chain(mode, lam, s):
    import torch
    from oracle import ddpm, nets, spec
    from tests import helpers as hp
    B, K = 400, 6
    wl = dict(H=1, A=1, To=0, Do=0, T=100, precision=0, base=dict(arch="gauss"), draft=dict(arch="gauss"),
              base_params=inputs.make_gauss_params(sweep.M0, sweep.S0),
              draft_params=inputs.make_gauss_params(sweep.M0 + 0.25, 0.8 * sweep.S0))
    smp, S, base, draft = hp.setup(wl, max_B=B, max_K=K)
    acc = hp.accept_t(mode=mode, lam=lam, sigma_scale=s)
    out = torch.zeros(B, 1, 1, device="cuda")
    smp.reset_stats()
    smp.sample_chunk(None, B, K, acc, 77, out)
    x = out.cpu().numpy().reshape(-1)
    st = smp.stats()
    noise = spec.TableNoise(77, range(B), 100, 1)
    n_match, accepted, tested = 0, 0, 0
    for b in range(B):
        xo, so = spec.sample_chunk(S, base, draft, noise, b, None, (1, 1), K, hp.oracle_accept(acc))
        accepted += so["accepted"]; tested += so["accepted"] + so["rejections"]
        n_match += abs(x[b] - xo[0, 0]) < 1e-3
    assert n_match >= B - 2                                      # a near-tie may flip a decision in fp32
    assert abs(st["drafts_accepted"] - accepted) <= 0.01 * accepted
    smp.close()
