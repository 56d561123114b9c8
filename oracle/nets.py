"""The denoisers eps = M(x, tau; obs) in numpy fp64: closed-form Gaussian toy, MLP, transformer, DiT,
conv UNet.

The paper gives only the block counts (eight transformer blocks for the base policy, a single one for
the drafter, Sec. 4) and says that the drafter has the same input-output interface and shares the
encoder and scheduler (Sec. 3.2 "Draft Model Training").  Everything below that is more
specific than that is this library's own architecture definition; parity with the paper's trained
networks is UNPINNED (no weights or layer layout are published).  What is pinned is the wiring of that
definition: attention against a library routine and plain-loop restatements of a decoder block, an
adaptive-LayerNorm block and a 2-level UNet, closed forms for the modulation slices and the FiLM halves,
and structural invariants (causality, bidirectionality of the adaLN transformer, independence of candidates,
zero-head => zero output, the closed-form Gaussian denoiser against the analytic posterior mean).

Parameters are dicts of float64 arrays produced by the seeded input generators; a linear layer
y = x W + b stores W as [in, out].
"""
import numpy as np
from .ddpm import sinusoidal_embedding


# ----------------------------------------------------------------------------- Gaussian toy
def gauss_eps(p, sched, x, tau):
    """Optimal noise prediction when the data are iid N(m0, s0^2) per coordinate:

    E[eps | x_tau] = sqrt(1 - abar) (x - sqrt(abar) m0) / (abar s0^2 + 1 - abar)."""
    ab = sched.abar[tau]
    return np.sqrt(1.0 - ab) * (x - np.sqrt(ab) * p["m0"]) / (ab * p["s0"] ** 2 + 1.0 - ab)


# ----------------------------------------------------------------------------- MLP
def silu(v):
    return v / (1.0 + np.exp(-v))


def mlp_eps(p, x, tau, obs):
    """Input = [flattened latent | sinusoidal(tau, temb) | flattened obs]; `layers` hidden
    SiLU layers; linear head back to the latent shape."""
    temb = p["temb"]
    h = np.concatenate([x.reshape(-1), sinusoidal_embedding(tau, temb), obs.reshape(-1)])
    for W, b in zip(p["W"][:-1], p["b"][:-1]):
        h = silu(h @ W + b)
    return (h @ p["W"][-1] + p["b"][-1]).reshape(x.shape)


# ----------------------------------------------------------------------------- transformer
def layer_norm(h, g, b, eps=1e-5):
    m = h.mean(axis=-1, keepdims=True)
    v = ((h - m) ** 2).mean(axis=-1, keepdims=True)
    return (h - m) / np.sqrt(v + eps) * g + b


def gelu_tanh(v):
    return 0.5 * v * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (v + 0.044715 * v ** 3)))


def softmax(s):
    s = s - s.max(axis=-1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=-1, keepdims=True)


def attention(q, k, v, heads, causal):
    """Multi-head scaled dot-product attention; q [Nq,d], k,v [Nk,d]."""
    Nq, d = q.shape
    dh = d // heads
    out = np.empty_like(q)
    for h in range(heads):
        sl = slice(h * dh, (h + 1) * dh)
        s = q[:, sl] @ k[:, sl].T / np.sqrt(dh)
        if causal:
            s = np.where(np.tril(np.ones_like(s, dtype=bool)), s, -np.inf)
        out[:, sl] = softmax(s) @ v[:, sl]
    return out


def xfmr_eps(p, x, tau, obs):
    """Pre-LN decoder: tokens = latent rows [H, A] -> d; memory = [time token | obs tokens].

    h   = x W_in + b_in + pos
    mem = [sinusoidal(tau, d) ; obs W_obs + b_obs] + cpos
    per block:  h += SelfAttn_causal(LN1 h);  h += CrossAttn(LN2 h, mem);  h += MLP_gelu(LN3 h)
    eps = LN_f(h) W_out + b_out
    """
    d, heads = p["d"], p["heads"]
    h = x @ p["W_in"] + p["b_in"] + p["pos"]
    mem = np.vstack([sinusoidal_embedding(tau, d)[None, :], obs @ p["W_obs"] + p["b_obs"]]) + p["cpos"]
    for L in p["layers"]:
        a = layer_norm(h, L["ln1_g"], L["ln1_b"])
        qkv = a @ L["Wqkv"] + L["bqkv"]
        h = h + attention(qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:], heads, True) @ L["Wo"] + L["bo"]
        a = layer_norm(h, L["ln2_g"], L["ln2_b"])
        q = a @ L["Wq2"] + L["bq2"]
        kv = mem @ L["Wkv2"] + L["bkv2"]
        h = h + attention(q, kv[:, :d], kv[:, d:], heads, False) @ L["Wo2"] + L["bo2"]
        a = layer_norm(h, L["ln3_g"], L["ln3_b"])
        h = h + gelu_tanh(a @ L["W1"] + L["b1"]) @ L["W2"] + L["b2"]
    return layer_norm(h, p["lnf_g"], p["lnf_b"]) @ p["W_out"] + p["b_out"]


# ----------------------------------------------------------------------------- DiT
def layer_norm_plain(h, eps=1e-5):
    m = h.mean(axis=-1, keepdims=True)
    v = ((h - m) ** 2).mean(axis=-1, keepdims=True)
    return (h - m) / np.sqrt(v + eps)


def dit_time_vector(p, tau):
    """c(tau) = W_t2^T SiLU(W_t1^T sinusoidal(tau) + b_t1) + b_t2."""
    return silu(sinusoidal_embedding(tau, p["d"]) @ p["Wt1"] + p["bt1"]) @ p["Wt2"] + p["bt2"]


def dit_eps(p, x, tau, ctx):
    """Adaptive-LayerNorm transformer (the VLA-scale action expert of the largest configuration): the
    timestep enters every block as shift / scale / gate vectors; the context tokens enter through
    cross-attention; self-attention is bidirectional over the H action tokens.

    h    = x W_in + b_in + pos
    mem  = ctx W_ctx + b_ctx + cpos                                    [Tc, d]
    c    = time vector;  per block (s1, k1, g1, s2, k2, g2) = split(SiLU(c) W_mod + b_mod)
      h += g1 * ( SelfAttn( LN0(h) (1 + k1) + s1 ) W_o + b_o )
      h +=       CrossAttn( LN(h; lnc), mem ) W_o2 + b_o2
      h += g2 * ( GELU( (LN0(h) (1 + k2) + s2) W_1 + b_1 ) W_2 + b_2 )
    (sf, kf) = split(SiLU(c) W_modf + b_modf);   eps = (LN0(h) (1 + kf) + sf) W_out + b_out
    LN0 is LayerNorm without gain and bias."""
    d, heads = p["d"], p["heads"]
    h = x @ p["W_in"] + p["b_in"] + p["pos"]
    mem = ctx @ p["W_ctx"] + p["b_ctx"] + p["cpos"]
    sc = silu(dit_time_vector(p, tau))
    for L in p["layers"]:
        s1, k1, g1, s2, k2, g2 = np.split(sc @ L["Wmod"] + L["bmod"], 6)
        a = layer_norm_plain(h) * (1.0 + k1) + s1
        qkv = a @ L["Wqkv"] + L["bqkv"]
        h = h + g1 * (attention(qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:], heads, False) @ L["Wo"] + L["bo"])
        a = layer_norm(h, L["lnc_g"], L["lnc_b"])
        q = a @ L["Wq2"] + L["bq2"]
        kv = mem @ L["Wkv2"] + L["bkv2"]
        h = h + attention(q, kv[:, :d], kv[:, d:], heads, False) @ L["Wo2"] + L["bo2"]
        a = layer_norm_plain(h) * (1.0 + k2) + s2
        h = h + g2 * (gelu_tanh(a @ L["W1"] + L["b1"]) @ L["W2"] + L["b2"])
    sf, kf = np.split(sc @ p["Wmodf"] + p["bmodf"], 2)
    return (layer_norm_plain(h) * (1.0 + kf) + sf) @ p["W_out"] + p["b_out"]


# ----------------------------------------------------------------------------- conv UNet
def mish(v):
    return v * np.tanh(np.log1p(np.exp(-np.abs(v))) + np.maximum(v, 0.0))      # v tanh(softplus(v)), overflow-safe


def conv1d_k5(x, W, b):
    """x [L, C_in], W [5, C_in, C_out] (tap, in, out), zero padding 2:  y[l] = sum_j x[l + j - 2] W[j] + b."""
    L = x.shape[0]
    xp = np.vstack([np.zeros((2, x.shape[1])), x, np.zeros((2, x.shape[1]))])
    return sum(xp[j:j + L] @ W[j] for j in range(5)) + b


def group_norm(y, g, b, groups, eps=1e-5):
    """GroupNorm over (positions x channels-of-the-group) of one sample; y [L, C]."""
    L, C = y.shape
    yg = y.reshape(L, groups, C // groups)
    m = yg.mean(axis=(0, 2), keepdims=True)
    v = ((yg - m) ** 2).mean(axis=(0, 2), keepdims=True)
    return ((yg - m) / np.sqrt(v + eps)).reshape(L, C) * g + b


def unet_resblock(R, x, mcond, groups):
    """y = Mish(GN(conv5 x)); y = scale * y + bias (FiLM from Mish(cond)); y = Mish(GN(conv5 y)); out = y + res(x)."""
    y = mish(group_norm(conv1d_k5(x, R["W1"], R["b1"]), R["g1"], R["be1"], groups))
    film = mcond @ R["Wf"] + R["bf"]
    C = y.shape[1]
    y = film[:C] * y + film[C:]
    y = mish(group_norm(conv1d_k5(y, R["W2"], R["b2"]), R["g2"], R["be2"], groups))
    return y + (x @ R["Wr"] + R["br"] if "Wr" in R else x)


def unet_eps(p, x, tau, obs):
    """1-D temporal conv UNet over the H action positions (Robomimic-shaped configuration): channels
    c, 2c, 4c; two FiLM residual blocks per level, 2:1 mean pooling down, 2x repetition up, skip
    concatenation, two middle blocks; conditioning cond = [time vector | flattened obs].

    tvec = Mish(sin(tau) W_t1 + b_t1) W_t2 + b_t2;  every block's FiLM = Mish(cond) W_f + b_f."""
    groups = p["groups"]
    tvec = mish(sinusoidal_embedding(tau, p["dt"]) @ p["Wt1"] + p["bt1"]) @ p["Wt2"] + p["bt2"]
    mcond = mish(np.concatenate([tvec, obs.reshape(-1)]))
    rb = iter(p["blocks"])
    h = x @ p["W_in"] + p["b_in"]
    skips = []
    n_lv = p["levels"]
    for lv in range(n_lv):
        h = unet_resblock(next(rb), h, mcond, groups)
        h = unet_resblock(next(rb), h, mcond, groups)
        if lv < n_lv - 1:
            skips.append(h)
            h = 0.5 * (h[0::2] + h[1::2])
    h = unet_resblock(next(rb), h, mcond, groups)
    h = unet_resblock(next(rb), h, mcond, groups)
    for lv in range(n_lv - 2, -1, -1):
        h = np.concatenate([np.repeat(h, 2, axis=0), skips[lv]], axis=1)
        h = unet_resblock(next(rb), h, mcond, groups)
        h = unet_resblock(next(rb), h, mcond, groups)
    h = mish(group_norm(conv1d_k5(h, p["Wh"], p["bh"]), p["gh"], p["beh"], groups))
    return h @ p["W_out"] + p["b_out"]


def make_denoiser(p, sched):
    """Return eps(x [H,A], tau, obs [To,Do]) for a parameter dict with key 'arch'."""
    arch = p["arch"]
    if arch == "gauss":
        return lambda x, tau, obs: gauss_eps(p, sched, x, tau)
    if arch == "mlp":
        return lambda x, tau, obs: mlp_eps(p, x, tau, obs)
    if arch == "xfmr":
        return lambda x, tau, obs: xfmr_eps(p, x, tau, obs)
    if arch == "dit":
        return lambda x, tau, obs: dit_eps(p, x, tau, obs)
    if arch == "unet":
        return lambda x, tau, obs: unet_eps(p, x, tau, obs)
    raise ValueError(arch)
