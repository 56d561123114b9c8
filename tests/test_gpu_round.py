"""GPU parity, round and chunk level, against the fp64 oracle on the same seeds."""
import numpy as np
import pytest
import torch
from scipy import stats

from oracle import spec
from paper_2512_15773_b200 import binding, inputs
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _round_parity(wl, B, K, acc, seed, tol_eps, tol_x, t0s, precision=None, drafter=0, verifier=0, min_checked=None):
    """One round from given (x, t) on both sides.  Intermediates are compared for every environment; the decision
    (j*, new t, committed latent) for every environment too, except where the two sides decided differently AND
    the oracle's deciding statistic lies within 1e-3 + the bound the denoiser tolerance implies (helpers.py).
    At least `min_checked` environments (default: all but one) must have been compared in full."""
    smp, S, base, draft = hp.setup(wl, max_B=B, max_K=max(K, 1), precision=precision, drafter=drafter, verifier=verifier)
    shape = (wl["H"], wl["A"]); D = wl["H"] * wl["A"]
    obs = inputs.make_obs(3, B, wl["To"], wl["Do"])
    noise = spec.PhiloxNoise(seed)
    x0 = np.stack([noise.x_init(b, shape) for b in range(B)]).astype(np.float32)
    dx = torch.tensor(x0, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    h_t = np.array(t0s, dtype=np.int32)
    d_xt = torch.zeros(B, K + 1, D, device="cuda"); d_mh = torch.zeros(B, max(K, 1), D, device="cuda")
    d_eps = torch.zeros(B, K + 1, D, device="cuda"); d_la = torch.zeros(B, max(K, 1), device="cuda")
    h_j = np.zeros(B, dtype=np.int32)
    smp.round(dobs, B, K, acc, seed, dx, h_t, d_xt, d_mh, d_eps, d_la, h_j)
    xt, mh, eps, la = (v.cpu().numpy() for v in (d_xt, d_mh, d_eps, d_la))
    x_new = dx.cpu().numpy()
    checked = 0
    for b in range(B):
        xo, to, d = spec.spec_round(S, base, draft, noise, b, obs[b], x0[b].astype(np.float64), int(t0s[b]), K,
                                    hp.oracle_accept(acc))
        g = dict(xt=xt[b], mh=mh[b], eps=eps[b], la=la[b], j=int(h_j[b]), t_new=int(h_t[b]), x_new=x_new[b],
                 t_oracle=to, x_oracle=xo)
        checked += hp.check_round_env(S, noise, hp.oracle_accept(acc), b, int(t0s[b]), K, d, g, tol_eps, tol_x)
    smp.close()
    assert checked >= (B - 1 if min_checked is None else min_checked), (checked, B)
    return checked


def test_round_toy_mlp_fp32():
    wl = dict(inputs.WORKLOADS["toy_mlp"])
    for K, bonus in ((4, 1), (3, 0), (0, 1)):
        _round_parity(wl, 6, K, hp.accept_t(bonus=bonus), 11, 1e-4, 2e-5, [99, 60, 30, 2, 1, 0])
    _round_parity(wl, 4, 4, hp.accept_t(mode=1, lam=0.7, sigma_scale=1.5), 12, 1e-4, 2e-5, [80, 50, 20, 3])


@pytest.mark.parametrize("precision,tol_eps,tol_x", [(0, 1e-4, 2e-5), (1, 2e-2, 3e-3)])
def test_round_transformer(precision, tol_eps, tol_x):
    wl = dict(inputs.WORKLOADS["pusht_xfmr"], precision=precision)
    _round_parity(wl, 5, 8, hp.accept_t(), 21, tol_eps, tol_x, [99, 70, 40, 5, 0])


@pytest.mark.parametrize("drafter", [1, 2])
def test_round_transformer_bf16_both_drafters(drafter):
    """Layer-by-layer drafter and the persistent cluster drafter against the oracle, same round."""
    wl = dict(inputs.WORKLOADS["pusht_xfmr"], precision=1)
    _round_parity(wl, 5, 8, hp.accept_t(), 21, 2e-2, 3e-3, [99, 70, 40, 5, 0], drafter=drafter)
    # more environments than clusters fit at once, ragged K_eff, A = 7
    wl7 = hp.small_xfmr_workload(1, d=256, heads=4, layers=2, dd=128, dlayers=2, H=16, A=7, To=3, Do=9, gamma=0.05)
    _round_parity(wl7, 23, 6, hp.accept_t(sigma_scale=1.5), 5, 2e-2, 3e-3, [99 - 4 * i for i in range(22)] + [2],
                  drafter=drafter)


def test_cluster_kernels_with_cluster_barriers_give_the_same_bits(monkeypatch):
    """The two ways a cluster hands a stage over (st.async stores counted on mbarriers; plain distributed-shared-memory
    stores and a cluster barrier) move the same values: a round must come out bit for bit the same."""
    wl = dict(inputs.WORKLOADS["pusht_xfmr"], precision=1)
    B, K, D = 3, 8, wl["H"] * wl["A"]
    outs = []
    for legacy in (False, True):
        if legacy:
            monkeypatch.setenv("TSDP_NO_ASYNC_BCAST", "1")
        smp, *_ = hp.setup(wl, max_B=B, max_K=K, drafter=2, verifier=2)
        obs = torch.tensor(inputs.make_obs(3, B, wl["To"], wl["Do"]), dtype=torch.float32, device="cuda")
        x = torch.tensor(np.random.default_rng(0).normal(size=(B, D)).astype(np.float32), device="cuda")
        h_t = np.array([90, 50, 3], dtype=np.int32)
        xt = torch.zeros(B, K + 1, D, device="cuda"); mh = torch.zeros(B, K, D, device="cuda"); ep = torch.zeros(B, K + 1, D, device="cuda")
        smp.round(obs, B, K, hp.accept_t(), 4, x, h_t, xt, mh, ep, None, None)
        outs.append((xt.clone(), mh.clone(), ep.clone(), x.clone()))
        smp.close()
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_cluster_kernels_without_the_cross_attention_fold(monkeypatch):
    """The cluster kernel's own query / output projections and attention over the memory tokens (what it runs when
    (1 + obs_tokens) * heads exceeds its 16 folded rows), selected here through the environment variable."""
    monkeypatch.setenv("TSDP_NO_FOLD", "1")
    wl = dict(inputs.WORKLOADS["pusht_xfmr"], precision=1)
    _round_parity(wl, 2, 8, hp.accept_t(), 21, 2e-2, 3e-3, [99, 40], drafter=2, verifier=2)


@pytest.mark.parametrize("case", ["resident", "streamed"])
def test_cluster_drafter_matches_layered_drafter(case):
    """resident: the PushT drafter, whose weight slices live in shared memory; streamed: a 4-block d = 256
    drafter (Robomimic-shaped), too large for that, whose slices are read through the L2."""
    if case == "resident":
        wl = dict(inputs.WORKLOADS["pusht_xfmr"], precision=1)
    else:
        wl = dict(H=16, A=10, To=2, Do=24, T=100, precision=1, gamma=0.05,
                  base=dict(arch="xfmr", layers=1, d=128, heads=4), draft=dict(arch="xfmr", layers=4, d=256, heads=4))
    B, K, D = 3, 8, wl["H"] * wl["A"]
    outs = []
    for drafter in (1, 2):
        smp, *_ = hp.setup(wl, max_B=B, max_K=K, drafter=drafter)
        obs = torch.tensor(inputs.make_obs(3, B, wl["To"], wl["Do"]), dtype=torch.float32, device="cuda")
        x = torch.tensor(np.random.default_rng(0).normal(size=(B, D)).astype(np.float32), device="cuda")
        h_t = np.array([90, 50, 3], dtype=np.int32)
        xt = torch.zeros(B, K + 1, D, device="cuda"); mh = torch.zeros(B, K, D, device="cuda")
        smp.round(obs, B, K, hp.accept_t(), 4, x, h_t, xt, mh, None, None, None)
        outs.append((xt.cpu().numpy(), mh.cpu().numpy()))
        smp.close()
    for b, t0 in enumerate((90, 50, 3)):          # draft slots beyond K_eff = min(K, t) are not part of the round
        Ke = min(K, t0)
        assert np.max(np.abs(outs[0][0][b, :Ke + 1] - outs[1][0][b, :Ke + 1])) < 3e-3
        assert np.max(np.abs(outs[0][1][b, :Ke] - outs[1][1][b, :Ke])) < 3e-3


def _chunk_parity(wl, B, K, acc, seed, tol_final, precision=None, schedule=None, drafter=0, verifier=0):
    smp, S, base, draft = hp.setup(wl, max_B=B, max_K=max(K, 1) if schedule is None else 10, precision=precision,
                                   drafter=drafter, verifier=verifier)
    shape = (wl["H"], wl["A"])
    obs = inputs.make_obs(4, B, wl["To"], wl["Do"])
    dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    out = torch.zeros(B, *shape, device="cuda")
    osched = None
    if schedule is not None:
        Ks, Ss = schedule
        smp.set_schedule(Ks, [hp.accept_t(sigma_scale=s) for s in Ss])
        osched = lambda r, t: (Ks[min(r, len(Ks) - 1)], spec.Accept(sigma_scale=Ss[min(r, len(Ks) - 1)]))
    smp.reset_stats()
    smp.sample_chunk(dobs, B, K, acc, seed, out)
    got = out.cpu().numpy()
    st = smp.stats()
    tot = dict(accepted=0, draft_evals=0, rounds=0, rej=0, bonus=0)
    n_match = 0
    for b in range(B):
        xo, so = spec.sample_chunk(S, base, draft, spec.PhiloxNoise(seed), b, obs[b], shape, K, hp.oracle_accept(acc),
                                   schedule=osched)
        tot["accepted"] += so["accepted"]; tot["draft_evals"] += so["draft_evals"]; tot["rounds"] += so["rounds"]
        tot["rej"] += so["rejections"]; tot["bonus"] += so["bonus"]
        if np.max(np.abs(got[b] - xo)) < tol_final:
            n_match += 1
    assert st["steps_advanced"] == 100 * B and st["chunks"] == B
    assert st["drafts_accepted"] + st["rejections"] + st["bonus_steps"] == 100 * B
    # NFE rule of the paper (Sec. 4): a base forward counts 1, a drafter call draft_layers / base_layers
    ratio = wl["draft"]["layers"] / wl["base"]["layers"]
    assert abs(st["nfe"] - (st["env_rounds"] + st["draft_evals"] * ratio)) < 1e-3
    smp.close()
    return n_match, tot, st


def test_request_counters_and_process_reward_match_oracle():
    """Per-request counters (drafts proposed / accepted, rounds, steps) against the oracle's chunk statistics, and
    the intermediate reward of Sec. 3.3 computed on the device against the oracle's formula."""
    from oracle import sched as osched
    wl = dict(inputs.WORKLOADS["toy_mlp"])
    B, K, seed = 8, 4, 5
    smp, S, base, draft = hp.setup(wl, max_B=B, max_K=K)
    shape = (wl["H"], wl["A"])
    obs = inputs.make_obs(4, B, wl["To"], wl["Do"])
    dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    out = torch.zeros(B, *shape, device="cuda")
    acc = hp.accept_t()
    smp.sample_chunk(dobs, B, K, acc, seed, out)
    cnt = smp.request_counts(B)
    rew = smp.process_reward(100.0, 400, 8, B)
    got = out.cpu().numpy()
    assert (cnt[:, 3] == 100).all() and (cnt[:, 1] <= cnt[:, 0]).all()
    n_same = 0
    for b in range(B):
        xo, so = spec.sample_chunk(S, base, draft, spec.PhiloxNoise(seed), b, obs[b], shape, K, hp.oracle_accept(acc))
        # the reward follows from the device's own counters whatever the trajectory did
        ref = osched.process_reward(int(cnt[b, 1]), int(cnt[b, 0]), int(cnt[b, 3]), 100.0, 400, 8)
        assert abs(rew[b] - ref) < 1e-6 * max(1.0, ref)
        if np.max(np.abs(got[b] - xo)) < 3e-2:       # same trajectory (no near-tie flip): same counters
            n_same += 1
            assert cnt[b, 0] == so["draft_evals"] and cnt[b, 1] == so["accepted"] and cnt[b, 2] == so["rounds"]
    assert n_same >= B - 1
    # continuous batching: the counters follow the request, not the slot
    N = 20
    obs2 = inputs.make_obs(6, N, wl["To"], wl["Do"])
    out2 = torch.zeros(N, *shape, device="cuda")
    smp.serve(torch.tensor(obs2, dtype=torch.float32, device="cuda"), N, B, K, acc, seed, out2)
    cnt2 = smp.request_counts(N)
    assert (cnt2[:, 3] == 100).all() and (cnt2[:, 2] >= 100 // (K + 1)).all()
    st = smp.stats()
    smp.close()


def _frozen(wl):
    return dict(wl, draft=dict(arch="frozen"))


def test_frozen_target_drafts_round_parity():
    """Drafter-free rounds (every draft reuses the base output at the round's start) against the oracle: fp32 MLP,
    bf16 transformer with the layer-by-layer kernels, and with the cluster kernel supplying both base passes."""
    _round_parity(_frozen(inputs.WORKLOADS["toy_mlp"]), 6, 4, hp.accept_t(), 11, 1e-4, 2e-5, [99, 60, 30, 2, 1, 0])
    wl = _frozen(dict(inputs.WORKLOADS["pusht_xfmr"], gamma=1.0))
    _round_parity(wl, 3, 6, hp.accept_t(), 7, 2e-2, 3e-3, [99, 40, 3], precision=1, verifier=1)
    _round_parity(wl, 2, 4, hp.accept_t(), 8, 2e-2, 3e-3, [80, 20], precision=1, verifier=2)


def test_frozen_target_drafts_chunk_and_accounting():
    wl = _frozen(inputs.WORKLOADS["toy_mlp"])
    B, K, seed = 8, 5, 21
    smp, S, base, draft = hp.setup(wl, max_B=B, max_K=K)
    shape = (wl["H"], wl["A"])
    obs = inputs.make_obs(4, B, wl["To"], wl["Do"])
    dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    out = torch.zeros(B, *shape, device="cuda")
    acc = hp.accept_t()
    # K = 1: the only draft is the base model's own step -> vanilla DDPM, sample by sample
    van = torch.zeros_like(out)
    smp.sample_chunk(dobs, B, 0, acc, seed, van)
    smp.reset_stats()
    smp.sample_chunk(dobs, B, 1, acc, seed, out)
    st = smp.stats()
    assert torch.equal(out, van) and st["rejections"] == 0 and st["drafts_accepted"] == st["draft_evals"]
    # K = 5 against the oracle, and the NFE rule: one batched verification per round plus one base pass per drafting round
    smp.reset_stats()
    smp.sample_chunk(dobs, B, K, acc, seed, out)
    st = smp.stats()
    got = out.cpu().numpy()
    n_match, rounds, drounds = 0, 0, 0
    for b in range(B):
        xo, so = spec.sample_chunk(S, base, draft, spec.PhiloxNoise(seed), b, obs[b], shape, K, hp.oracle_accept(acc))
        ok = np.max(np.abs(got[b] - xo)) < 3e-2
        n_match += ok
        rounds += so["rounds"]; drounds += so["draft_rounds"]
    assert n_match >= B - 1
    if n_match == B:
        assert st["env_rounds"] == rounds and st["draft_rounds"] == drounds
    assert abs(st["nfe"] - (st["env_rounds"] + st["draft_rounds"])) < 1e-9 and st["steps_advanced"] == 100 * B
    # the frozen drafter takes no weights
    with pytest.raises(binding.TsdpError):
        smp.load_weights(binding.DRAFT, inputs.make_net(3, inputs.WORKLOADS["toy_mlp"], "draft"))
    smp.close()


def test_chunk_toy_mlp_fp32_matches_oracle_exactly_in_structure():
    wl = dict(inputs.WORKLOADS["toy_mlp"])
    B = 8
    n_match, tot, st = _chunk_parity(wl, B, 4, hp.accept_t(), 5, 3e-2)
    # fp32 check mode: a near-tie flip is possible in principle but rare; allow one environment
    assert n_match >= B - 1
    if n_match == B:
        assert st["drafts_accepted"] == tot["accepted"] and st["draft_evals"] == tot["draft_evals"]
        assert st["env_rounds"] == tot["rounds"] and st["rejections"] == tot["rej"]


def _chunk_walk(wl, B, K, acc, seed, tol_eps, tol_x, tol_final, precision=None, drafter=0, verifier=0, max_flagged=1):
    """A whole chunk, every round of every environment compared.

    The product call (tsdp_sample_chunk) runs first.  Then the chunk is walked round by round through tsdp_round:
    each round starts, on BOTH sides, from the state the CUDA path committed in the round before, so a decision
    that legitimately flipped inside the tolerated band (helpers.check_round_env) does not end the comparison --
    the rounds after it are still checked at the round tolerances.  An environment is `flagged` once such a flip
    happened.  For every environment that was never flagged, the product call's chunk, the walk's chunk and the
    oracle's own independent chunk must agree within tol_final, and the statistics must agree exactly when no
    environment was flagged."""
    smp, S, base, draft = hp.setup(wl, max_B=B, max_K=max(K, 1), precision=precision, drafter=drafter, verifier=verifier)
    shape = (wl["H"], wl["A"]); D = wl["H"] * wl["A"]; T = wl["T"]
    obs = inputs.make_obs(4, B, wl["To"], wl["Do"])
    dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    noise = spec.PhiloxNoise(seed)
    oacc = hp.oracle_accept(acc)
    out = torch.zeros(B, *shape, device="cuda")
    smp.reset_stats()
    smp.sample_chunk(dobs, B, K, acc, seed, out)
    got = out.cpu().numpy()
    st = smp.stats()
    assert st["steps_advanced"] == T * B and st["chunks"] == B
    assert st["drafts_accepted"] + st["rejections"] + st["bonus_steps"] == T * B
    ratio = wl["draft"]["layers"] / wl["base"]["layers"]
    assert abs(st["nfe"] - (st["env_rounds"] + st["draft_evals"] * ratio)) < 1e-3
    # the walk
    x = np.stack([noise.x_init(b, shape) for b in range(B)]).astype(np.float32).reshape(B, D)
    t = np.full(B, T - 1, dtype=np.int32)
    flagged = np.zeros(B, dtype=bool)
    rounds_checked = rounds_total = 0
    d_xt = torch.zeros(B, K + 1, D, device="cuda"); d_mh = torch.zeros(B, max(K, 1), D, device="cuda")
    d_eps = torch.zeros(B, K + 1, D, device="cuda"); d_la = torch.zeros(B, max(K, 1), device="cuda")
    while (t >= 0).any():
        x_in, t_in = x.copy(), t.copy()
        dx = torch.tensor(x_in, device="cuda"); h_t = t_in.copy(); h_j = np.zeros(B, dtype=np.int32)
        smp.round(dobs, B, K, acc, seed, dx, h_t, d_xt, d_mh, d_eps, d_la, h_j)
        xt, mh, eps, la = (v.cpu().numpy() for v in (d_xt, d_mh, d_eps, d_la))
        x = dx.cpu().numpy(); t = h_t
        for b in range(B):
            if t_in[b] < 0:
                assert h_j[b] == -1 and t[b] == -1 and np.array_equal(x[b], x_in[b])      # finished: untouched
                continue
            xo, to, d = spec.spec_round(S, base, draft, noise, b, obs[b], x_in[b].astype(np.float64).reshape(shape),
                                        int(t_in[b]), K, oacc)
            g = dict(xt=xt[b], mh=mh[b], eps=eps[b], la=la[b], j=int(h_j[b]), t_new=int(t[b]), x_new=x[b],
                     t_oracle=to, x_oracle=xo)
            ok = hp.check_round_env(S, noise, oacc, b, int(t_in[b]), K, d, g, tol_eps, tol_x)
            flagged[b] |= not ok
            rounds_checked += ok; rounds_total += 1
    # the oracle's own chunks, from its own x_T and its own states
    tot = dict(accepted=0, draft_evals=0, rounds=0, rej=0, prop=np.zeros(T, int), test=np.zeros(T, int), acc=np.zeros(T, int))
    for b in range(B):
        xo, so = spec.sample_chunk(S, base, draft, noise, b, obs[b], shape, K, oacc)
        for k_, v_ in (("accepted", "accepted"), ("draft_evals", "draft_evals"), ("rounds", "rounds"), ("rej", "rejections"),
                       ("prop", "prop_hist"), ("test", "test_hist"), ("acc", "acc_hist")):
            tot[k_] = tot[k_] + so[v_]
        if not flagged[b]:
            assert np.max(np.abs(got[b] - xo)) < tol_final, b
            assert np.max(np.abs(x[b].reshape(shape) - xo)) < tol_final, b
            assert np.max(np.abs(x[b].reshape(shape) - got[b])) < tol_final, b
    assert flagged.sum() <= max_flagged, (flagged, rounds_checked, rounds_total)
    if not flagged.any():      # same decisions everywhere: every counter and the per-timestep histograms agree exactly
        assert st["drafts_accepted"] == tot["accepted"] and st["draft_evals"] == tot["draft_evals"]
        assert st["env_rounds"] == tot["rounds"] and st["rejections"] == tot["rej"]
        assert np.array_equal(st["hist_drafted"], tot["prop"]) and np.array_equal(st["hist_tested"], tot["test"])
        assert np.array_equal(st["hist_accepted"], tot["acc"])
    smp.close()
    return int(flagged.sum()), rounds_checked, rounds_total


@pytest.mark.parametrize("precision,drafter,verifier", [(0, 0, 0), (1, 1, 1), (1, 2, 1), (1, 2, 2)])
def test_chunk_pusht_transformer(precision, drafter, verifier):
    wl = dict(inputs.WORKLOADS["pusht_xfmr"], precision=precision)
    tol_eps, tol_x = (1e-4, 2e-5) if precision == 0 else (2e-2, 3e-3)
    _chunk_walk(wl, 3, 8, hp.accept_t(), 9, tol_eps, tol_x, 3e-2, precision=precision, drafter=drafter, verifier=verifier,
                max_flagged=0 if precision == 0 else 1)


def test_chunk_statistics_and_histograms_match_the_oracle_fp32():
    """Per-timestep histograms of drafts proposed / tested / accepted (the axis of the paper's acceptance-versus-
    timestep figure, Sec. 3.2) and every counter, against the oracle's, on chunks whose decisions all agree."""
    wl = dict(inputs.WORKLOADS["toy_mlp"])
    flagged, checked, total = _chunk_walk(wl, 8, 4, hp.accept_t(), 5, 1e-4, 2e-5, 3e-2, max_flagged=0)
    assert checked == total and total >= 8 * 20


@pytest.mark.parametrize("precision,tol_eps,tol_x", [(0, 1e-4, 2e-5), (1, 2e-2, 3e-3)])
def test_round_dit(precision, tol_eps, tol_x):
    """One speculative round with the adaptive-LayerNorm transformer as base and drafter."""
    wl = dict(H=10, A=4, To=16, Do=8, T=100, precision=precision, gamma=0.05,
              base=dict(arch="dit", layers=2, d=128, heads=4), draft=dict(arch="dit", layers=1, d=128, heads=2))
    _round_parity(wl, 4, 5, hp.accept_t(), 33, tol_eps, tol_x, [99, 60, 3, 0])


def test_chunk_dit_fp32():
    wl = dict(H=10, A=4, To=16, Do=8, T=100, precision=0, gamma=0.05,
              base=dict(arch="dit", layers=2, d=128, heads=4), draft=dict(arch="dit", layers=1, d=128, heads=2))
    B = 3
    n_match, tot, st = _chunk_parity(wl, B, 6, hp.accept_t(), 41, 3e-2)
    assert n_match >= B - 1


@pytest.mark.parametrize("precision,tol_eps,tol_x", [(0, 1e-4, 2e-5), (1, 2e-2, 3e-3)])
def test_round_unet_base_transformer_drafter(precision, tol_eps, tol_x):
    """Robomimic-shaped pairing: conv UNet base verified against a transformer drafter's drafts."""
    wl = dict(H=16, A=10, To=2, Do=24, T=100, precision=precision, gamma=0.05,
              base=dict(arch="unet", layers=2, d=128, heads=8, temb=32), draft=dict(arch="xfmr", layers=1, d=128, heads=4))
    _round_parity(wl, 4, 5, hp.accept_t(), 51, tol_eps, tol_x, [99, 60, 3, 0])


def test_chunk_with_round_schedule_fp32():
    wl = hp.small_xfmr_workload(0, d=128, heads=4, layers=1, dd=128, dlayers=1, H=16, A=7, To=2, Do=64, gamma=0.03)
    Ks, Ss = inputs.markov_schedule(0, 40)
    n_match, tot, st = _chunk_parity(wl, 4, 10, hp.accept_t(), 13, 3e-2, schedule=(Ks, Ss))
    assert n_match >= 3


def test_drafter_equal_to_base_accepts_everything_and_equals_vanilla():
    for wl in (dict(inputs.WORKLOADS["toy_mlp"]), hp.small_xfmr_workload(1)):
        B = 4
        # bit-identity needs the same kernels on both sides: the layer-by-layer drafter and verifier
        smp, S, base, _ = hp.setup(wl, max_B=B, max_K=6, draft_is_base=True, drafter=1, verifier=1)
        obs = torch.tensor(inputs.make_obs(4, B, wl["To"], wl["Do"]), dtype=torch.float32, device="cuda")
        ref = torch.zeros(B, wl["H"], wl["A"], device="cuda")
        smp.sample_chunk(obs, B, 0, hp.accept_t(), 77, ref)                  # K = 0: vanilla DDPM
        st0 = smp.stats()
        assert st0["env_rounds"] == 100 * B and st0["draft_evals"] == 0
        for K, bonus in ((6, 1), (1, 0), (3, 1)):
            smp.reset_stats()
            out = torch.zeros_like(ref)
            smp.sample_chunk(obs, B, K, hp.accept_t(bonus=bonus), 77, out)
            st = smp.stats()
            assert st["rejections"] == 0 and st["drafts_accepted"] == st["draft_evals"]
            assert torch.equal(out, ref)
            if K == 1 and bonus == 0:
                assert st["env_rounds"] == 100 * B                           # T base forwards per chunk
        smp.close()


def test_cluster_kernel_as_drafter_and_verifier_reproduces_vanilla_bit_for_bit():
    """Batch 1 with the cluster kernel on both sides: the same arithmetic drafts and verifies, so with
    drafter == base every draft is accepted and the chunk equals vanilla DDPM (K = 0) exactly."""
    wl = hp.small_xfmr_workload(1)
    smp, *_ = hp.setup(wl, max_B=1, max_K=6, draft_is_base=True, drafter=2, verifier=2)
    obs = torch.tensor(inputs.make_obs(4, 1, wl["To"], wl["Do"]), dtype=torch.float32, device="cuda")
    ref = torch.zeros(1, wl["H"], wl["A"], device="cuda")
    smp.sample_chunk(obs, 1, 0, hp.accept_t(), 77, ref)
    for K in (6, 3):
        smp.reset_stats()
        out = torch.zeros_like(ref)
        smp.sample_chunk(obs, 1, K, hp.accept_t(), 77, out)
        st = smp.stats()
        assert st["rejections"] == 0 and st["drafts_accepted"] == st["draft_evals"]
        assert torch.equal(out, ref)
    smp.close()


@pytest.mark.parametrize("B,K", [(1, 8), (2, 4)])
def test_round_transformer_cluster_verifier(B, K):
    """Verification forward through the cluster kernel (one cluster per candidate) against the oracle."""
    wl = dict(inputs.WORKLOADS["pusht_xfmr"], precision=1)
    smp, S, base, draft = hp.setup(wl, max_B=B, max_K=K, drafter=2, verifier=2)
    smp.close()
    _round_parity_cfg = dict(drafter=2, verifier=2)
    _round_parity(wl, B, K, hp.accept_t(), 21, 2e-2, 3e-3, [99, 40][:B], **_round_parity_cfg)


def test_cluster_drafter_equal_to_base_is_accepted_almost_always():
    """Same weights through two different kernels (cluster drafter vs tensor-core base): the means
    differ by rounding only, so nearly every draft passes the likelihood-ratio test."""
    wl = hp.small_xfmr_workload(1)
    B = 4
    smp, *_ = hp.setup(wl, max_B=B, max_K=6, draft_is_base=True, drafter=2)
    obs = torch.tensor(inputs.make_obs(4, B, wl["To"], wl["Do"]), dtype=torch.float32, device="cuda")
    out = torch.zeros(B, wl["H"], wl["A"], device="cuda")
    smp.sample_chunk(obs, B, 6, hp.accept_t(), 77, out)
    st = smp.stats()
    assert st["steps_advanced"] == 100 * B and torch.isfinite(out).all()
    assert st["drafts_accepted"] >= 0.95 * st["drafts_tested"]
    smp.close()


def test_gaussian_toy_on_gpu_matches_analytic_marginal():
    """10^5 one-dimensional chains on the GPU, vanilla and speculative, against the analytic marginal."""
    from tests.test_oracle_chain import _analytic_marginal, M0, S0
    B = 100_000
    wl = dict(H=1, A=1, To=0, Do=0, T=100, precision=0, base=dict(arch="gauss"), draft=dict(arch="gauss"),
              base_params=inputs.make_gauss_params(M0, S0), draft_params=inputs.make_gauss_params(M0 + 0.25, 0.8 * S0))
    smp, *_ = hp.setup(wl, max_B=B, max_K=6)
    mean, std = _analytic_marginal()
    for K in (0, 6):
        smp.reset_stats()
        out = torch.zeros(B, 1, 1, device="cuda")
        smp.sample_chunk(None, B, K, hp.accept_t(), 1234, out)
        x = out.cpu().numpy().reshape(-1).astype(np.float64)
        assert stats.kstest((x - mean) / std, "norm").pvalue > 0.01
        st = smp.stats()
        if K:
            assert 0.2 < st["drafts_accepted"] / st["drafts_tested"] < 0.98
    # same seed, same chains as the oracle's KS pin: spot-check a few environments sample by sample
    from oracle import ddpm, nets
    S = ddpm.Schedule()
    base = nets.make_denoiser(wl["base_params"], S); draft = nets.make_denoiser(wl["draft_params"], S)
    for b in (0, 1, 99_999):
        xo, _ = spec.sample_chunk(S, base, draft, spec.PhiloxNoise(1234), b, None, (1, 1), 6, spec.Accept())
        assert abs(x[b] - xo[0, 0]) < 1e-3
    smp.close()


def test_gaussian_toy_with_frozen_target_drafts_keeps_the_marginal_on_gpu():
    """Drafter-free rounds are lossless too: 10^5 chains on the GPU against the analytic marginal, and a few of them
    sample by sample against the oracle; rejections do occur (the frozen output drifts from the base's)."""
    from tests.test_oracle_chain import _analytic_marginal, M0, S0
    from oracle import ddpm, nets
    B = 100_000
    wl = dict(H=1, A=1, To=0, Do=0, T=100, precision=0, base=dict(arch="gauss"), draft=dict(arch="frozen"),
              base_params=inputs.make_gauss_params(M0, S0))
    smp, *_ = hp.setup(wl, max_B=B, max_K=6)
    mean, std = _analytic_marginal()
    out = torch.zeros(B, 1, 1, device="cuda")
    smp.reset_stats()
    smp.sample_chunk(None, B, 6, hp.accept_t(), 1234, out)
    x = out.cpu().numpy().reshape(-1).astype(np.float64)
    assert stats.kstest((x - mean) / std, "norm").pvalue > 0.01
    st = smp.stats()
    assert st["rejections"] > 0 and st["drafts_accepted"] < st["drafts_tested"] and st["steps_advanced"] == 100 * B
    S = ddpm.Schedule()
    base = nets.make_denoiser(wl["base_params"], S)
    for b in (0, 7, 99_999):
        xo, _ = spec.sample_chunk(S, base, spec.FrozenTargetDraft(base), spec.PhiloxNoise(1234), b, None, (1, 1), 6, spec.Accept())
        assert abs(x[b] - xo[0, 0]) < 1e-3
    smp.close()


def test_argument_errors_on_device():
    wl = dict(inputs.WORKLOADS["toy_mlp"])
    cfg = binding.make_config(wl["H"], wl["A"], wl["To"], wl["Do"], wl["base"], wl["draft"], max_B=2, max_K=4, precision=0)
    smp = binding.Sampler(cfg)
    out = torch.zeros(2, 16, 2, device="cuda"); obs = torch.zeros(2, 1, 20, device="cuda")
    with pytest.raises(binding.TsdpError) as e:
        smp.sample_chunk(obs, 2, 4, hp.accept_t(), 0, out)
    assert e.value.status == 2                                                # weights not loaded
    blob = binding.pack_weights(inputs.make_net(1, wl, "base"))
    with pytest.raises(binding.TsdpError) as e:
        smp.load_weights(binding.BASE, blob[:-1])
    assert e.value.status == 3
    bad = blob.copy(); bad[5] = np.nan
    with pytest.raises(binding.TsdpError) as e:
        smp.load_weights(binding.BASE, bad)
    assert e.value.status == 6
    smp.load_weights(binding.BASE, blob)
    smp.load_weights(binding.DRAFT, inputs.make_net(2, wl, "draft"))
    for B, K in ((3, 4), (2, 5), (0, 1)):
        with pytest.raises(binding.TsdpError) as e:
            smp.sample_chunk(obs, B, K, hp.accept_t(), 0, out)
        assert e.value.status == 1
    with pytest.raises(binding.TsdpError):
        smp.sample_chunk(obs, 2, 4, hp.accept_t(mode=1, lam=1.5), 0, out)
    smp.sample_chunk(obs, 2, 4, hp.accept_t(), 0, out)
    assert torch.isfinite(out).all()
    smp.close()


def test_call_latency_ring_percentiles():
    """tsdp_stats reports the median and 99th percentile of the device time of the last chunk calls; checked against
    CUDA events recorded around the same calls on the same stream."""
    wl = dict(inputs.WORKLOADS["toy_mlp"])
    smp, *_ = hp.setup(wl, max_B=2, max_K=4)
    obs = torch.tensor(inputs.make_obs(4, 2, wl["To"], wl["Do"]), dtype=torch.float32, device="cuda")
    out = torch.zeros(2, wl["H"], wl["A"], device="cuda")
    smp.sample_chunk(obs, 2, 4, hp.accept_t(), 1, out)
    smp.reset_stats()
    assert smp.stats()["call_ms_samples"] == 0
    n, ms = 7, []
    for i in range(n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        smp.sample_chunk(obs, 2, 4 if i else 0, hp.accept_t(), 10 + i, out)      # the first call is vanilla: the slowest
        e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1))
    st = smp.stats()
    assert st["call_ms_samples"] == n
    assert 0 < st["call_ms_p50"] <= st["call_ms_p99"] <= max(ms) * 1.05
    assert abs(st["call_ms_p50"] - float(np.median(ms))) < 0.25 * float(np.median(ms)) + 0.05
    assert st["call_ms_p99"] > 1.5 * st["call_ms_p50"]                           # the K = 0 call stands out
    # the ring keeps the last TSDP_LATENCY_RING calls only
    for i in range(260):
        smp.sample_chunk(obs, 2, 4, hp.accept_t(), 100 + i, out)
    assert smp.stats()["call_ms_samples"] == 256
    smp.close()
