"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle.

Holds data only: random weights, observations, workload shapes and the seeded K / sigma-scale
schedule that stands in for the RL scheduler.  None of the method's arithmetic lives here (no
DDPM table, no network forward, no acceptance rule, no counter-based noise generator), so both
the CUDA path and the oracle can draw their inputs from it without sharing an implementation.

The shapes are those of the paper's workloads (Diffusion Policy on Push-T / Robomimic style
tasks: horizon 16, low-dimensional actions, two observation steps; Sec. 4), the values are
synthetic: the paper's datasets, simulators and trained checkpoints are not available.
"""
import numpy as np


def bf16_round(a):
    """Round float values to the nearest bf16-representable value (ties to even), as float64."""
    f = np.asarray(a, dtype=np.float32).copy()
    u = f.view(np.uint32)
    u += np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    u &= np.uint32(0xFFFF0000)
    return f.astype(np.float64)


def _lin(rng, n_in, n_out, std, q):
    W = rng.normal(0.0, std, size=(n_in, n_out))
    b = rng.normal(0.0, 0.02, size=(n_out,))
    return q(W), q(b)


def make_gauss_params(m0, s0):
    return dict(arch="gauss", m0=float(m0), s0=float(s0))


def make_mlp_params(seed, H, A, To, Do, width, layers, temb=32, out_scale=1.0):
    """`layers` hidden layers of `width`; fp32-representable values."""
    rng = np.random.default_rng(seed)
    q = lambda a: np.asarray(a, dtype=np.float32).astype(np.float64)
    dims = [H * A + temb + To * Do] + [width] * layers + [H * A]
    Ws, bs = [], []
    for i in range(len(dims) - 1):
        W, b = _lin(rng, dims[i], dims[i + 1], 1.0 / np.sqrt(dims[i]), q)
        Ws.append(W); bs.append(b)
    Ws[-1] = q(Ws[-1] * out_scale); bs[-1] = q(bs[-1] * out_scale)
    return dict(arch="mlp", temb=temb, width=width, layers=layers, W=Ws, b=bs)


def make_xfmr_params(seed, H, A, To, Do, d, heads, layers, out_scale=1.0, bf16=True):
    """Random decoder-style transformer denoiser; values bf16-representable when bf16=True."""
    rng = np.random.default_rng(seed)
    q = bf16_round if bf16 else (lambda a: np.asarray(a, dtype=np.float32).astype(np.float64))
    p = dict(arch="xfmr", d=d, heads=heads, n_layers=layers)
    p["W_in"], p["b_in"] = _lin(rng, A, d, 1.0 / np.sqrt(A), q)
    p["pos"] = q(rng.normal(0.0, 0.02, size=(H, d)))
    p["W_obs"], p["b_obs"] = _lin(rng, Do, d, 1.0 / np.sqrt(Do), q)
    p["cpos"] = q(rng.normal(0.0, 0.02, size=(1 + To, d)))
    s = 1.0 / np.sqrt(d)
    Ls = []
    for _ in range(layers):
        L = {}
        for n in ("ln1", "ln2", "ln3"):
            L[n + "_g"] = q(1.0 + rng.normal(0.0, 0.02, size=(d,)))
            L[n + "_b"] = q(rng.normal(0.0, 0.02, size=(d,)))
        L["Wqkv"], L["bqkv"] = _lin(rng, d, 3 * d, s, q)
        L["Wo"], L["bo"] = _lin(rng, d, d, s, q)
        L["Wq2"], L["bq2"] = _lin(rng, d, d, s, q)
        L["Wkv2"], L["bkv2"] = _lin(rng, d, 2 * d, s, q)
        L["Wo2"], L["bo2"] = _lin(rng, d, d, s, q)
        L["W1"], L["b1"] = _lin(rng, d, 4 * d, s, q)
        L["W2"], L["b2"] = _lin(rng, 4 * d, d, 0.5 * s, q)
        Ls.append(L)
    p["layers"] = Ls
    p["lnf_g"] = q(1.0 + rng.normal(0.0, 0.02, size=(d,)))
    p["lnf_b"] = q(rng.normal(0.0, 0.02, size=(d,)))
    W, b = _lin(rng, d, A, s, q)
    p["W_out"], p["b_out"] = q(W * out_scale), q(b * out_scale)
    return p


def make_dit_params(seed, H, A, To, Do, d, heads, layers, out_scale=1.0, bf16=True):
    """Random adaptive-LayerNorm transformer (DiT-style) denoiser.  The modulation layers are given
    small weights so that the network starts near an un-modulated, gated-on state: gates get a bias
    of 1, shifts and scales a bias of 0."""
    rng = np.random.default_rng(seed)
    q = bf16_round if bf16 else (lambda a: np.asarray(a, dtype=np.float32).astype(np.float64))
    q32 = lambda a: np.asarray(a, dtype=np.float32).astype(np.float64)
    p = dict(arch="dit", d=d, heads=heads, n_layers=layers)
    p["W_in"], p["b_in"] = _lin(rng, A, d, 1.0 / np.sqrt(A), q)
    p["pos"] = q(rng.normal(0.0, 0.02, size=(H, d)))
    p["W_ctx"], p["b_ctx"] = _lin(rng, Do, d, 1.0 / np.sqrt(Do), q)
    p["cpos"] = q(rng.normal(0.0, 0.02, size=(To, d)))
    s = 1.0 / np.sqrt(d)
    # the time path runs in fp32 on the device (tables built at load): keep fp32-representable values
    p["Wt1"], p["bt1"] = _lin(rng, d, d, s, q32)
    p["Wt2"], p["bt2"] = _lin(rng, d, d, s, q32)
    Ls = []
    for _ in range(layers):
        L = {}
        W, b = _lin(rng, d, 6 * d, 0.3 * s, q32)
        b = b.copy(); b[2 * d:3 * d] += 1.0; b[5 * d:6 * d] += 1.0            # gates start at 1
        L["Wmod"], L["bmod"] = W, q32(b)
        L["lnc_g"] = q(1.0 + rng.normal(0.0, 0.02, size=(d,)))
        L["lnc_b"] = q(rng.normal(0.0, 0.02, size=(d,)))
        L["Wqkv"], L["bqkv"] = _lin(rng, d, 3 * d, s, q)
        L["Wo"], L["bo"] = _lin(rng, d, d, s, q)
        L["Wq2"], L["bq2"] = _lin(rng, d, d, s, q)
        L["Wkv2"], L["bkv2"] = _lin(rng, d, 2 * d, s, q)
        L["Wo2"], L["bo2"] = _lin(rng, d, d, s, q)
        L["W1"], L["b1"] = _lin(rng, d, 4 * d, s, q)
        L["W2"], L["b2"] = _lin(rng, 4 * d, d, 0.5 * s, q)
        Ls.append(L)
    p["layers"] = Ls
    p["Wmodf"], p["bmodf"] = _lin(rng, d, 2 * d, 0.3 * s, q32)
    W, b = _lin(rng, d, A, s, q)
    p["W_out"], p["b_out"] = q(W * out_scale), q(b * out_scale)
    return p


def unet_block_channels(c, levels):
    """(C_in, C_out) of the residual blocks of the conv UNet, in execution order."""
    ch = [c * 2 ** i for i in range(levels)]
    out, cin = [], c
    for lv in range(levels):
        out += [(cin, ch[lv]), (ch[lv], ch[lv])]
        cin = ch[lv]
    out += [(cin, cin), (cin, cin)]
    for lv in range(levels - 2, -1, -1):
        out += [(cin + ch[lv], ch[lv]), (ch[lv], ch[lv])]
        cin = ch[lv]
    return out


def make_unet_params(seed, H, A, To, Do, c, levels, groups=8, dt=256, out_scale=1.0, bf16=True):
    """Random 1-D conv UNet denoiser; conv / pointwise matrices bf16-representable when bf16=True, the
    time path and the FiLM layers (tabulated in fp32 on the device) fp32-representable."""
    rng = np.random.default_rng(seed)
    q = bf16_round if bf16 else (lambda a: np.asarray(a, dtype=np.float32).astype(np.float64))
    q32 = lambda a: np.asarray(a, dtype=np.float32).astype(np.float64)
    dc = dt + To * Do
    p = dict(arch="unet", c=c, levels=levels, groups=groups, dt=dt)
    p["W_in"], p["b_in"] = _lin(rng, A, c, 1.0 / np.sqrt(A), q32)
    p["Wt1"], p["bt1"] = _lin(rng, dt, 4 * dt, 1.0 / np.sqrt(dt), q32)
    p["Wt2"], p["bt2"] = _lin(rng, 4 * dt, dt, 0.5 / np.sqrt(dt), q32)

    def conv(cin, cout):
        return q(rng.normal(0.0, 1.0 / np.sqrt(5 * cin), size=(5, cin, cout))), q32(rng.normal(0.0, 0.02, size=(cout,)))

    blocks = []
    for cin, cout in unet_block_channels(c, levels):
        R = {}
        R["W1"], R["b1"] = conv(cin, cout)
        R["g1"], R["be1"] = q32(1.0 + rng.normal(0.0, 0.02, size=(cout,))), q32(rng.normal(0.0, 0.02, size=(cout,)))
        Wf, bf = _lin(rng, dc, 2 * cout, 0.3 / np.sqrt(dc), q32)
        bf = bf.copy(); bf[:cout] += 1.0                                   # FiLM starts near the identity
        R["Wf"], R["bf"] = Wf, q32(bf)
        R["W2"], R["b2"] = conv(cout, cout)
        R["g2"], R["be2"] = q32(1.0 + rng.normal(0.0, 0.02, size=(cout,))), q32(rng.normal(0.0, 0.02, size=(cout,)))
        if cin != cout:
            R["Wr"], R["br"] = _lin(rng, cin, cout, 1.0 / np.sqrt(cin), q)
        blocks.append(R)
    p["blocks"] = blocks
    p["Wh"], p["bh"] = conv(c, c)
    p["gh"], p["beh"] = q32(1.0 + rng.normal(0.0, 0.02, size=(c,))), q32(rng.normal(0.0, 0.02, size=(c,)))
    W, b = _lin(rng, c, A, 1.0 / np.sqrt(c), q32)
    p["W_out"], p["b_out"] = q32(W * out_scale), q32(b * out_scale)
    return p


def make_sched_params(seed, H, A, To, Do, scale=1.0):
    """Random weights of the scheduler network (three stream encoders 64 / 64 / 16, aggregate MLP
    64, 5 outputs); fp32-representable.  `scale` multiplies the output layer."""
    rng = np.random.default_rng(seed)
    q = lambda a: np.asarray(a, dtype=np.float32).astype(np.float64)
    p = dict(arch="sched")
    p["W_o"], p["b_o"] = _lin(rng, To * Do, 64, 1.0 / np.sqrt(max(To * Do, 1)), q)
    p["W_a"], p["b_a"] = _lin(rng, H * A, 64, 1.0 / np.sqrt(H * A), q)
    p["W_p"], p["b_p"] = _lin(rng, 1, 16, 1.0, q)
    p["W_1"], p["b_1"] = _lin(rng, 144, 64, 1.0 / 12.0, q)
    W, b = _lin(rng, 64, 5, 1.0 / 8.0, q)
    p["W_2"], p["b_2"] = q(W * scale), q(b * scale)
    return p


def make_obs(seed, B, To, Do):
    """Observation features ~ N(0,1), float32-representable, shape [B, To, Do]."""
    rng = np.random.default_rng(seed + 7919)
    return rng.normal(size=(B, To, Do)).astype(np.float32).astype(np.float64)


# ------------------------------------------------------------------------------- workloads
# Shapes of the named configurations.  `gamma` scales both output heads: random networks
# disagree far more than a distilled drafter does, so the heads are shrunk until the mean
# acceptance is near the rate the paper reports (about 85 %, App. A).
WORKLOADS = {
    "toy_mlp": dict(H=16, A=2, To=1, Do=20, T=100, precision=0,
                    base=dict(arch="mlp", layers=3, width=256), draft=dict(arch="mlp", layers=1, width=64),
                    B=1, K=4, gamma=0.05),
    "pusht_xfmr": dict(H=16, A=2, To=2, Do=20, T=100, precision=1,
                       base=dict(arch="xfmr", layers=8, d=256, heads=4),
                       draft=dict(arch="xfmr", layers=2, d=128, heads=4), B=1, K=8, gamma=0.05),
    "serving_xfmr": dict(H=16, A=7, To=2, Do=64, T=100, precision=1,
                         base=dict(arch="xfmr", layers=12, d=512, heads=8),
                         draft=dict(arch="xfmr", layers=2, d=256, heads=4), B=256, K=10, gamma=0.03),
    # Robomimic-shaped conv-UNet policy: 16 x 10 action chunk, 2 x 512 visual features, channels 256/512/1024
    "robomimic_unet": dict(H=16, A=10, To=2, Do=512, T=100, precision=1,
                           base=dict(arch="unet", layers=3, d=256, heads=8, temb=256),
                           draft=dict(arch="xfmr", layers=4, d=256, heads=4), B=32, K=8, gamma=0.03),
    # VLA-scale action expert: 50 x 14 action chunk, 256 context tokens of width 1024
    "vla_dit": dict(H=50, A=14, To=256, Do=1024, T=100, precision=1,
                    base=dict(arch="dit", layers=18, d=1024, heads=16),
                    draft=dict(arch="dit", layers=4, d=512, heads=8), B=64, K=16, gamma=0.012),
}


def make_net(seed, wl, which, gamma=None, bf16=None):
    """Parameter dict for the base (`which`='base') or drafter ('draft') of a workload."""
    n = wl[which]
    g = wl.get("gamma", 1.0) if gamma is None else gamma
    if n["arch"] == "mlp":
        return make_mlp_params(seed, wl["H"], wl["A"], wl["To"], wl["Do"], n["width"], n["layers"],
                               out_scale=g)
    if n["arch"] == "xfmr":
        use_bf16 = (wl["precision"] == 1) if bf16 is None else bf16
        return make_xfmr_params(seed, wl["H"], wl["A"], wl["To"], wl["Do"], n["d"], n["heads"],
                                n["layers"], out_scale=g, bf16=use_bf16)
    if n["arch"] == "unet":
        use_bf16 = (wl["precision"] == 1) if bf16 is None else bf16
        return make_unet_params(seed, wl["H"], wl["A"], wl["To"], wl["Do"], n["d"], n["layers"], groups=n.get("heads", 8),
                                dt=n.get("temb", 256), out_scale=g, bf16=use_bf16)
    if n["arch"] == "dit":
        use_bf16 = (wl["precision"] == 1) if bf16 is None else bf16
        return make_dit_params(seed, wl["H"], wl["A"], wl["To"], wl["Do"], n["d"], n["heads"], n["layers"],
                               out_scale=g, bf16=use_bf16)
    raise ValueError(n["arch"])


def markov_schedule(seed, n_rounds, p_stay=0.8):
    """Seeded 3-state chain {slow, medium, fast motion} standing in for the RL scheduler's
    per-round output: returns lists K[r], sigma_scale[r].  Faster motion => fewer accepted
    drafts in the paper (Fig. 4), hence shorter draft windows."""
    rng = np.random.default_rng(seed)
    k_rng = {0: (8, 10), 1: (4, 7), 2: (1, 3)}
    s_val = {0: 1.0, 1: 1.5, 2: 2.0}
    st, Ks, Ss = 0, [], []
    for _ in range(n_rounds):
        if rng.random() >= p_stay:
            st = (st + int(rng.integers(1, 3))) % 3
        lo, hi = k_rng[st]
        Ks.append(int(rng.integers(lo, hi + 1))); Ss.append(s_val[st])
    return Ks, Ss
