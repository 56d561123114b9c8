"""Continuous batching (tsdp_serve): N requests through fewer slots give, request by request, the
chunks of one big batch -- the refill inside the acceptance kernel changes scheduling, not results."""
import numpy as np
import pytest
import torch
from scipy import stats

from oracle import spec
from paper_2512_15773_b200 import binding, inputs
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _serve_vs_batch(wl, N, slots, K, acc, seed, drafter=0, precision=None):
    smp, S, base, draft = hp.setup(wl, max_B=N, max_K=max(K, 1), precision=precision, drafter=drafter)
    obs = inputs.make_obs(8, N, wl["To"], wl["Do"])
    dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    ref = torch.zeros(N, wl["H"], wl["A"], device="cuda")
    smp.reset_stats()
    smp.sample_chunk(dobs, N, K, acc, seed, ref)
    st_ref = smp.stats()
    out = torch.full_like(ref, float("nan"))
    smp.reset_stats()
    smp.serve(dobs, N, slots, K, acc, seed, out)
    st = smp.stats()
    assert st["chunks"] == N and st["steps_advanced"] == 100 * N
    assert torch.equal(out, ref)
    # per-request work is identical; only the number of batched rounds differs
    for k in ("env_rounds", "draft_evals", "drafts_accepted", "rejections", "bonus_steps"):
        assert st[k] == st_ref[k], k
    smp.close()
    return obs, ref.cpu().numpy(), (S, base, draft), st, st_ref


def test_serve_toy_mlp_fp32_equals_batch_and_oracle():
    wl = dict(inputs.WORKLOADS["toy_mlp"])
    N, slots, K, seed = 20, 6, 4, 17
    obs, got, (S, base, draft), st, st_ref = _serve_vs_batch(wl, N, slots, K, hp.accept_t(), seed)
    # a late request against the oracle: request i uses the noise streams of environment i
    n_match = 0
    for i in (0, 7, 13, 19):
        xo, _ = spec.sample_chunk(S, base, draft, spec.PhiloxNoise(seed), i, obs[i], (wl["H"], wl["A"]), K, spec.Accept())
        n_match += np.max(np.abs(got[i] - xo)) < 3e-2
    assert n_match >= 3
    assert st["rounds"] > st_ref["rounds"]                      # fewer slots, more batched rounds


@pytest.mark.parametrize("drafter", [1, 2])
def test_serve_transformer_bf16_equals_batch(drafter):
    wl = dict(inputs.WORKLOADS["pusht_xfmr"], precision=1)
    _serve_vs_batch(wl, 11, 4, 8, hp.accept_t(), 23, drafter=drafter)


def test_serve_grows_its_buffers_beyond_max_b_and_keeps_the_law():
    """5000 one-dimensional requests through 512 slots of a context built for 512."""
    from paper_2512_15773_b200 import sweep
    N, slots = 5000, 512
    wl = dict(H=1, A=1, To=0, Do=0, T=100, precision=0, base=dict(arch="gauss"), draft=dict(arch="gauss"),
              base_params=inputs.make_gauss_params(sweep.M0, sweep.S0),
              draft_params=inputs.make_gauss_params(sweep.M0 + 0.25, 0.8 * sweep.S0))
    smp, *_ = hp.setup(wl, max_B=slots, max_K=6)
    out = torch.zeros(N, 1, 1, device="cuda")
    smp.reset_stats()
    smp.serve(None, N, slots, 6, hp.accept_t(), 99, out)
    st = smp.stats()
    assert st["chunks"] == N and st["steps_advanced"] == 100 * N
    x = out.cpu().numpy().reshape(-1).astype(np.float64)
    mean, std = sweep.vanilla_output_law()
    assert stats.kstest((x - mean) / std, "norm").pvalue > 0.01
    with pytest.raises(binding.TsdpError):
        smp.serve(None, N, slots + 1, 6, hp.accept_t(), 99, out)   # more slots than the context has
    smp.close()


def test_serve_with_obs_beyond_max_b():
    """Observation-conditioned requests beyond the context's batch capacity (obs K/V buffers grow)."""
    wl = dict(inputs.WORKLOADS["pusht_xfmr"], precision=1)
    N, slots, K = 9, 3, 8
    big, *_ = hp.setup(wl, max_B=N, max_K=K)
    small, *_ = hp.setup(wl, max_B=slots, max_K=K)
    dobs = torch.tensor(inputs.make_obs(8, N, wl["To"], wl["Do"]), dtype=torch.float32, device="cuda")
    ref = torch.zeros(N, wl["H"], wl["A"], device="cuda"); out = torch.zeros_like(ref)
    big.sample_chunk(dobs, N, K, hp.accept_t(), 5, ref)
    small.serve(dobs, N, slots, K, hp.accept_t(), 5, out)
    assert torch.equal(out, ref)
    big.close(); small.close()


@pytest.mark.parametrize("arch", ["xfmr_bf16", "xfmr_fp32", "dit_bf16", "unet_bf16", "mlp_fp32"])
def test_compacted_rounds_give_the_same_bits_as_dense_rounds(arch, monkeypatch):
    """Each round lists the candidates that are still needed and the layer-by-layer forwards run on that list only.
    Rows are computed independently of one another, so the chunk must come out bit for bit as from the dense
    B x (K+1) layout (TSDP_NO_COMPACT), with the same counters, while fewer candidates are evaluated -- exactly as many
    as the acceptance kernel counts as useful base evaluations."""
    if arch == "xfmr_bf16":
        wl = hp.small_xfmr_workload(1, d=256, heads=4, layers=2, dd=128, dlayers=2, H=16, A=7, To=2, Do=16, gamma=0.05)
    elif arch == "xfmr_fp32":
        wl = hp.small_xfmr_workload(0, d=128, heads=4, layers=1, dd=128, dlayers=1, H=16, A=7, To=2, Do=16, gamma=0.05)
    elif arch == "dit_bf16":
        wl = dict(H=10, A=4, To=16, Do=8, T=100, precision=1, gamma=0.05,
                  base=dict(arch="dit", layers=2, d=128, heads=4), draft=dict(arch="dit", layers=1, d=128, heads=2))
    elif arch == "unet_bf16":
        wl = dict(H=16, A=10, To=2, Do=24, T=100, precision=1, gamma=0.05,
                  base=dict(arch="unet", layers=2, d=128, heads=8, temb=32), draft=dict(arch="xfmr", layers=1, d=128, heads=4))
    else:
        wl = dict(inputs.WORKLOADS["toy_mlp"])
    B, K, seed = 37, 6, 3
    Ks, Ss = inputs.markov_schedule(1, 60)
    Ks = [min(k, K) for k in Ks]
    res = []
    for dense in (True, False):
        if dense:
            monkeypatch.setenv("TSDP_NO_COMPACT", "1")
        else:
            monkeypatch.delenv("TSDP_NO_COMPACT")
        smp, *_ = hp.setup(wl, max_B=B, max_K=K, drafter=1, verifier=1)
        smp.set_schedule(Ks, [hp.accept_t(sigma_scale=s, bonus=(i % 3 != 0)) for i, s in enumerate(Ss)])
        obs = torch.tensor(inputs.make_obs(11, B, wl["To"], wl["Do"]), dtype=torch.float32, device="cuda")
        out = torch.zeros(B, wl["H"], wl["A"], device="cuda")
        smp.reset_stats()
        smp.sample_chunk(obs, B, K, hp.accept_t(), seed, out)
        st = smp.stats()
        # continuous batching on top: slots refill while others are still mid-chunk
        N = 3 * B + 5
        obs2 = torch.tensor(inputs.make_obs(12, N, wl["To"], wl["Do"]), dtype=torch.float32, device="cuda")
        out2 = torch.zeros(N, wl["H"], wl["A"], device="cuda")
        smp.serve(obs2, N, B, K, hp.accept_t(), seed + 1, out2)
        res.append((out.clone(), out2.clone(), st))
        smp.close()
    (o_d, o2_d, st_d), (o_c, o2_c, st_c) = res
    assert torch.equal(o_d, o_c) and torch.equal(o2_d, o2_c)
    for k in ("env_rounds", "base_evals", "draft_evals", "drafts_accepted", "rejections", "bonus_steps", "steps_advanced", "rounds"):
        assert st_d[k] == st_c[k], k
    assert np.array_equal(st_d["hist_accepted"], st_c["hist_accepted"])
    assert st_d["cand_computed"] == st_d["cand_dense"] == st_c["cand_dense"]
    assert st_c["cand_computed"] == st_c["base_evals"] < st_c["cand_dense"]


def test_no_kernel_writes_past_a_buffer():
    """Every device buffer of a context is followed by guard bytes; after whole chunks on every architecture pairing
    (ragged batch sizes, compacted rounds, continuous batching with buffers that had to grow, the cluster kernels at
    batch 1) all guards must be intact."""
    cases = [
        (hp.small_xfmr_workload(1, d=256, heads=4, layers=2, dd=128, dlayers=2, H=16, A=7, To=2, Do=16, gamma=0.05), 37, 6),
        (hp.small_xfmr_workload(1, d=128, heads=4, layers=2, dd=128, dlayers=1, H=7, A=3, To=3, Do=5, gamma=0.05), 5, 4),
        (dict(inputs.WORKLOADS["pusht_xfmr"], precision=1), 1, 8),
        (dict(H=10, A=4, To=16, Do=8, T=100, precision=1, gamma=0.05,
              base=dict(arch="dit", layers=2, d=128, heads=4), draft=dict(arch="dit", layers=1, d=128, heads=2)), 9, 5),
        (dict(H=16, A=10, To=2, Do=24, T=100, precision=1, gamma=0.05,
              base=dict(arch="unet", layers=2, d=128, heads=8, temb=32), draft=dict(arch="xfmr", layers=1, d=128, heads=4)), 11, 5),
        (dict(inputs.WORKLOADS["toy_mlp"]), 3, 4),
    ]
    for wl, B, K in cases:
        smp, *_ = hp.setup(wl, max_B=B, max_K=K)
        obs = torch.tensor(inputs.make_obs(11, B, wl["To"], wl["Do"]), dtype=torch.float32, device="cuda")
        out = torch.zeros(B, wl["H"], wl["A"], device="cuda")
        smp.sample_chunk(obs, B, K, hp.accept_t(), 3, out)
        N = 2 * B + 3
        obs2 = torch.tensor(inputs.make_obs(12, N, wl["To"], wl["Do"]), dtype=torch.float32, device="cuda")
        out2 = torch.zeros(N, wl["H"], wl["A"], device="cuda")
        smp.serve(obs2, N, B, K, hp.accept_t(bonus=0), 4, out2)
        assert smp.check_guards() >= 20
        assert torch.isfinite(out).all() and torch.isfinite(out2).all()
        smp.close()
