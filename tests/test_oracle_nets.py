"""Structural pins for the oracle's denoisers (their parity with the paper's trained networks is
unpinned: neither weights nor the exact layer layout are published)."""
import numpy as np
from scipy import special, stats

from oracle import ddpm, nets
from paper_2512_15773_b200 import inputs

S = ddpm.Schedule()


def _xfmr(seed=0, H=6, A=3, To=2, Do=5, d=16, heads=2, layers=2):
    p = inputs.make_xfmr_params(seed, H, A, To, Do, d, heads, layers, bf16=False)
    rng = np.random.default_rng(seed)
    return p, rng.normal(size=(H, A)), rng.normal(size=(To, Do))


def test_activations_against_library_definitions():
    v = np.linspace(-6, 6, 241)
    assert np.allclose(nets.silu(v), v * special.expit(v), atol=1e-14)
    assert np.max(np.abs(nets.gelu_tanh(v) - v * stats.norm.cdf(v))) < 1e-3     # tanh form of x Phi(x)
    assert np.allclose(nets.softmax(np.array([[1.0, 2.0, 3.0]])), special.softmax([[1.0, 2.0, 3.0]], axis=-1))
    h = np.random.default_rng(0).normal(size=(4, 32)) * 3 + 1
    y = nets.layer_norm(h, np.ones(32), np.zeros(32))
    assert np.allclose(y.mean(-1), 0, atol=1e-12) and np.allclose(y.var(-1), 1, atol=1e-4)


def test_self_attention_is_causal_and_candidates_are_independent():
    p, x, obs = _xfmr()
    e0 = nets.xfmr_eps(p, x, 40, obs)
    x2 = x.copy(); x2[4:] += 1.0                          # perturb late tokens only
    e1 = nets.xfmr_eps(p, x2, 40, obs)
    assert np.array_equal(e0[:4], e1[:4]) and not np.allclose(e0[4:], e1[4:])
    assert not np.allclose(e0, nets.xfmr_eps(p, x, 41, obs))         # the time token matters
    obs2 = obs.copy(); obs2[1] += 1.0
    assert not np.allclose(e0, nets.xfmr_eps(p, x, 40, obs2))        # the obs tokens matter


def test_zero_head_gives_bias_only():
    p, x, obs = _xfmr()
    p = dict(p); p["W_out"] = np.zeros_like(p["W_out"])
    assert np.allclose(nets.xfmr_eps(p, x, 3, obs), p["b_out"])
    m = inputs.make_mlp_params(0, 4, 2, 1, 5, 16, 2, temb=8)
    m["W"][-1] = np.zeros_like(m["W"][-1])
    assert np.allclose(nets.mlp_eps(m, np.ones((4, 2)), 3, np.ones((1, 5))).reshape(-1), m["b"][-1])


def test_single_token_single_key_case_by_hand():
    """H = 1, no obs tokens: both softmaxes are over one key, so attention is the identity on V and
    the block can be written without any attention code."""
    p, x, _ = _xfmr(H=1, To=0, layers=1, heads=1)
    obs = np.zeros((0, 5))
    L, d = p["layers"][0], p["d"]
    ln = lambda h, g, b: (h - h.mean()) / np.sqrt(h.var() + 1e-5) * g + b
    h = x[0] @ p["W_in"] + p["b_in"] + p["pos"][0]
    mem = ddpm.sinusoidal_embedding(7, d) + p["cpos"][0]
    v = (ln(h, L["ln1_g"], L["ln1_b"]) @ L["Wqkv"] + L["bqkv"])[2 * d:]
    h = h + v @ L["Wo"] + L["bo"]
    v2 = (mem @ L["Wkv2"] + L["bkv2"])[d:]
    h = h + v2 @ L["Wo2"] + L["bo2"]
    a = ln(h, L["ln3_g"], L["ln3_b"]) @ L["W1"] + L["b1"]
    h = h + (a * stats.norm.cdf(a)) @ L["W2"] + L["b2"]               # exact GELU: differs by < 1e-3
    ref = ln(h, p["lnf_g"], p["lnf_b"]) @ p["W_out"] + p["b_out"]
    assert np.allclose(nets.xfmr_eps(p, x, 7, obs)[0], ref, atol=5e-3)


def test_mlp_input_layout():
    m = inputs.make_mlp_params(1, 4, 2, 1, 5, 16, 1, temb=8)
    x, obs = np.arange(8.0).reshape(4, 2), np.arange(5.0).reshape(1, 5)
    inp = np.concatenate([x.reshape(-1), ddpm.sinusoidal_embedding(9, 8), obs.reshape(-1)])
    h = inp @ m["W"][0] + m["b"][0]
    ref = (h * special.expit(h)) @ m["W"][1] + m["b"][1]
    assert np.allclose(nets.mlp_eps(m, x, 9, obs).reshape(-1), ref, atol=1e-12)


def test_gaussian_denoiser_is_the_regression_of_eps_on_x():
    """E[eps | x_t] for x0 ~ N(m0, s0^2): checked by least squares on 2*10^6 forward samples."""
    rng = np.random.default_rng(0)
    p = inputs.make_gauss_params(0.7, 0.5)
    for t in (5, 50, 95):
        x0 = 0.7 + 0.5 * rng.normal(size=2_000_000)
        eps = rng.normal(size=x0.size)
        xt = np.sqrt(S.abar[t]) * x0 + np.sqrt(1 - S.abar[t]) * eps
        slope, icpt = np.polyfit(xt, eps, 1)
        got0, got1 = nets.gauss_eps(p, S, np.array([0.0]), t)[0], nets.gauss_eps(p, S, np.array([1.0]), t)[0]
        assert abs((got1 - got0) - slope) < 5e-3 and abs(got0 - icpt) < 5e-3


def test_bf16_rounding_of_inputs():
    a = np.array([1.0, 1.00390625, 1.001953125, 3.14159265, -2.7182818])
    r = inputs.bf16_round(a)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0          # 1+2^-8 ties to even, 1+2^-9 rounds down
    assert np.all(np.abs(r - a) <= np.abs(a) * 2.0 ** -8)
    u = r.astype(np.float32).view(np.uint32)
    assert np.all(u & 0xFFFF == 0)


# ----------------------------------------------------------------------------- DiT (structure only)
def _dit(seed=0, H=5, A=3, To=4, Do=6, d=16, heads=2, layers=2):
    p = inputs.make_dit_params(seed, H, A, To, Do, d, heads, layers, bf16=False)
    rng = np.random.default_rng(seed + 100)
    return p, rng.normal(size=(H, A)), rng.normal(size=(To, Do))


def test_dit_self_attention_is_bidirectional_and_context_enters_by_cross_attention_only():
    p, x, ctx = _dit()
    e0 = nets.dit_eps(p, x, 40, ctx)
    x2 = x.copy(); x2[-1] += 1.0                      # the LAST token changes ...
    assert np.abs(nets.dit_eps(p, x2, 40, ctx)[0] - e0[0]).max() > 1e-9      # ... and the first output moves
    q = dict(p, layers=[dict(L, Wo2=np.zeros_like(L["Wo2"]), bo2=np.zeros_like(L["bo2"])) for L in p["layers"]])
    assert np.array_equal(nets.dit_eps(q, x, 40, ctx), nets.dit_eps(q, x, 40, 3.0 * ctx))
    assert not np.allclose(nets.dit_eps(p, x, 40, 3.0 * ctx), e0)


def test_dit_zero_gates_make_a_block_the_identity_up_to_cross_attention():
    p, x, ctx = _dit(1)
    # gates 0 and no cross-attention output: every block is the identity, so the output is the final layer of the embedding
    Ls = []
    for L in p["layers"]:
        L = dict(L, Wo2=np.zeros_like(L["Wo2"]), bo2=np.zeros_like(L["bo2"]))
        W, b = L["Wmod"].copy(), L["bmod"].copy()
        d = p["d"]
        for g in (2, 5):
            W[:, g * d:(g + 1) * d] = 0.0; b[g * d:(g + 1) * d] = 0.0
        Ls.append(dict(L, Wmod=W, bmod=b))
    q = dict(p, layers=Ls)
    h = x @ p["W_in"] + p["b_in"] + p["pos"]
    sc = nets.silu(nets.dit_time_vector(p, 17))
    sf, kf = np.split(sc @ p["Wmodf"] + p["bmodf"], 2)
    ref = (nets.layer_norm_plain(h) * (1 + kf) + sf) @ p["W_out"] + p["b_out"]
    assert np.allclose(nets.dit_eps(q, x, 17, ctx), ref, atol=1e-12)


def test_dit_time_enters_through_modulation_only():
    p, x, ctx = _dit(2)
    q = dict(p, Wt2=np.zeros_like(p["Wt2"]))         # constant time vector: the timestep cannot matter
    assert np.array_equal(nets.dit_eps(q, x, 3, ctx), nets.dit_eps(q, x, 90, ctx))
    assert not np.allclose(nets.dit_eps(p, x, 3, ctx), nets.dit_eps(p, x, 90, ctx))


def test_layer_norm_plain_is_layer_norm_with_unit_gain():
    h = np.random.default_rng(0).normal(size=(4, 16))
    assert np.allclose(nets.layer_norm_plain(h), nets.layer_norm(h, np.ones(16), np.zeros(16)))
    assert np.allclose(nets.layer_norm_plain(h).mean(-1), 0) and np.allclose(nets.layer_norm_plain(h).var(-1), 1, atol=1e-4)


# ----------------------------------------------------------------------------- conv UNet (structure only)
def _unet(seed=0, H=8, A=3, To=2, Do=4, c=16, levels=2):
    p = inputs.make_unet_params(seed, H, A, To, Do, c, levels, groups=4, dt=8, bf16=False)
    rng = np.random.default_rng(seed + 7)
    return p, rng.normal(size=(H, A)), rng.normal(size=(To, Do))


def test_unet_primitives_against_library_routines():
    rng = np.random.default_rng(0)
    x, W, b = rng.normal(size=(9, 3)), rng.normal(size=(5, 3, 4)), rng.normal(size=4)
    y = nets.conv1d_k5(x, W, b)
    for co in range(4):        # each output channel = sum over input channels of a 'same' cross-correlation
        ref = sum(np.correlate(np.pad(x[:, ci], 2), W[:, ci, co], mode="valid") for ci in range(3)) + b[co]
        assert np.allclose(y[:, co], ref)
    v = rng.normal(size=100) * 5
    assert np.allclose(nets.mish(v), v * np.tanh(np.log(1 + np.exp(v))))
    z = rng.normal(size=(6, 8))
    gn = nets.group_norm(z, np.ones(8), np.zeros(8), 2)
    for g in range(2):
        blk = gn[:, 4 * g:4 * g + 4]
        assert abs(blk.mean()) < 1e-12 and abs(blk.var() - 1) < 1e-4


def test_unet_block_channel_plan_and_receptive_field():
    assert inputs.unet_block_channels(256, 3) == [(256, 256), (256, 256), (256, 512), (512, 512), (512, 1024), (1024, 1024),
                                                  (1024, 1024), (1024, 1024), (1536, 512), (512, 512), (768, 256), (256, 256)]
    p, x, obs = _unet()
    e0 = nets.unet_eps(p, x, 30, obs)
    assert e0.shape == x.shape
    x2 = x.copy(); x2[0] += 1.0                       # through pooling and the middle blocks every position sees every other
    assert np.abs(nets.unet_eps(p, x2, 30, obs)[-1] - e0[-1]).max() > 1e-12


def test_unet_conditioning_enters_through_film_only():
    p, x, obs = _unet(1)
    q = dict(p, blocks=[dict(R, Wf=np.zeros_like(R["Wf"])) for R in p["blocks"]])
    assert np.array_equal(nets.unet_eps(q, x, 5, obs), nets.unet_eps(q, x, 80, 2.0 * obs))
    assert not np.allclose(nets.unet_eps(p, x, 5, obs), nets.unet_eps(p, x, 80, obs))
    assert not np.allclose(nets.unet_eps(p, x, 5, obs), nets.unet_eps(p, x, 5, 2.0 * obs))
