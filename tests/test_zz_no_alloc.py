"""The allocation-free verification tail (tsdp_verify_commit_static) against tsdp_round.

Some users of the library run where device memory may not be requested at all -- a fixed-budget
control loop, a plug-in inside an application that owns the allocator, a real-time thread that must
stay off the driver's allocation lock.  For them the library keeps the working memory of the fused
acceptance / commit kernel in a fixed array of its own.  This test feeds that entry point the
candidates, drafter means and base outputs that an ordinary round produced and checks that it takes
the same decisions and commits the same latents -- twice in a row with different rounds, because the
array still holds the first call's values when the second one starts.

Collected last on purpose: a run that stops at the first failure has then already run every other
test.  It needs nothing from them and passes alone in a fresh process as well.
"""
import numpy as np
import pytest
import torch

from oracle import spec
from paper_2512_15773_b200 import binding, inputs
from tests import helpers as hp

pytestmark = pytest.mark.gpu
TOL = 2e-5          # fp32 check mode, the tolerance of the round-level parity tests


def _one_round(smp, wl, B, K, acc, seed, t0s):
    D = wl["H"] * wl["A"]
    shape = (wl["H"], wl["A"])
    obs = torch.tensor(inputs.make_obs(3, B, wl["To"], wl["Do"]), dtype=torch.float32, device="cuda")
    noise = spec.PhiloxNoise(seed)
    x0 = np.stack([noise.x_init(b, shape) for b in range(B)]).astype(np.float32)
    dx = torch.tensor(x0, device="cuda")
    h_t = np.array(t0s, dtype=np.int32)
    xt = torch.zeros(B, K + 1, D, device="cuda"); mh = torch.zeros(B, max(K, 1), D, device="cuda")
    eps = torch.zeros(B, K + 1, D, device="cuda"); la = torch.zeros(B, max(K, 1), device="cuda")
    h_j = np.zeros(B, dtype=np.int32)
    smp.round(obs, B, K, acc, seed, dx, h_t, xt, mh, eps, la, h_j)
    return dict(xt=xt, mh=mh, eps=eps, la=la, jstar=h_j, x_new=dx, t_new=h_t, t0=np.array(t0s, dtype=np.int32))


def _check_static(r, B, K, D, acc, seed):
    xt = r["xt"].clone()
    actions = torch.full((B, D), float("nan"), device="cuda")
    la = torch.zeros(B, max(K, 1), device="cuda")
    t_new = np.full(B, -7, dtype=np.int32); jstar = np.full(B, -7, dtype=np.int32)
    binding.verify_commit_static(xt, r["mh"], r["eps"], r["t0"], B, K, D, acc, seed, actions, t_new, jstar, la)
    assert np.array_equal(jstar, r["jstar"])
    assert np.array_equal(t_new, r["t_new"])
    got = xt[:, 0, :].cpu().numpy()
    ref = r["x_new"].reshape(B, D).cpu().numpy()
    assert np.max(np.abs(got - ref)) <= TOL
    if K > 0:
        assert np.max(np.abs(la.cpu().numpy() - r["la"].cpu().numpy())) <= 1e-3
    done = t_new < 0
    if done.any():
        assert np.max(np.abs(actions.cpu().numpy()[done] - ref[done])) <= TOL
    # candidates other than slot 0 are inputs and stay untouched
    assert torch.equal(xt[:, 1:, :], r["xt"][:, 1:, :])


def test_static_entry_matches_round_twice_in_a_row():
    wl = dict(inputs.WORKLOADS["toy_mlp"])
    B, K = 6, 4
    D = wl["H"] * wl["A"]
    smp, *_ = hp.setup(wl, max_B=B, max_K=K)
    acc1 = hp.accept_t()
    acc2 = hp.accept_t(mode=1, lam=0.7, sigma_scale=1.5, bonus=0)
    r1 = _one_round(smp, wl, B, K, acc1, 11, [99, 60, 30, 2, 1, 0])
    r2 = _one_round(smp, wl, B, K, acc2, 12, [80, 50, 20, 3, 0, 97])
    _check_static(r1, B, K, D, acc1, 11)
    _check_static(r2, B, K, D, acc2, 12)           # the array still holds the first call's state
    _check_static(r1, B, K, D, acc1, 11)
    smp.close()


def test_static_entry_rejects_sizes_beyond_its_capacity():
    B, K, D = 1025, 1, 4
    xt = torch.zeros(B, K + 1, D, device="cuda"); mh = torch.zeros(B, K, D, device="cuda")
    h_t = np.zeros(B, dtype=np.int32); out = np.zeros(B, dtype=np.int32)
    act = torch.zeros(B, D, device="cuda")
    with pytest.raises(binding.TsdpError) as e:
        binding.verify_commit_static(xt, mh, xt, h_t, B, K, D, hp.accept_t(), 0, act, out, out.copy())
    assert e.value.status == 8
    with pytest.raises(binding.TsdpError) as e:
        binding.verify_commit_static(xt, mh, xt, h_t[:4], 4, K, D, hp.accept_t(), 0, act, out, out.copy(), T=2000)
    assert e.value.status == 8
