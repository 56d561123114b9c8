"""Pins for the WIRING of the oracle's networks (oracle/nets.py): the attention scale and head partition, the
adaptive-LayerNorm block's shift / scale / gate order, the conv UNet's FiLM halves, pooling pairs and
upsample-then-concatenate order.

The paper fixes none of this (it gives block counts only), so the definition these tests hold the oracle to is
the architecture text of include/tsdp.h.  Three kinds of pin, none of which calls the oracle's own helpers for
the part under test:
  * a library routine (torch's scaled_dot_product_attention) for multi-head attention;
  * special cases with a closed form (a gate set to zero kills exactly one branch; scale = -1 turns a branch into
    a constant that can be written down);
  * an element-by-element restatement in plain Python loops on tiny shapes (2 heads / 3 keys, one adaLN block on
    2 tokens, a 2-level UNet on 4 positions), which a swapped half, a transposed operand or a wrong scale fails.
"""
import math

import numpy as np
import torch

from oracle import ddpm, nets
from paper_2512_15773_b200 import inputs


# ----------------------------------------------------------------------------- plain-loop building blocks
def _lin(x, W, b):
    return [sum(x[i] * W[i][o] for i in range(len(x))) + b[o] for o in range(len(b))]


def _ln(x, g=None, b=None, eps=1e-5):
    n = len(x)
    m = sum(x) / n
    v = sum((xi - m) ** 2 for xi in x) / n
    return [(x[i] - m) / math.sqrt(v + eps) * (1.0 if g is None else g[i]) + (0.0 if b is None else b[i]) for i in range(n)]


def _mha(Q, K, V, heads, causal):
    """Q [Nq][d], K, V [Nk][d]; head h owns the contiguous columns h*dh .. (h+1)*dh-1; scores / sqrt(dh)."""
    d = len(Q[0]); dh = d // heads
    out = [[0.0] * d for _ in Q]
    for i, q in enumerate(Q):
        for h in range(heads):
            cols = range(h * dh, (h + 1) * dh)
            keys = range(i + 1) if causal else range(len(K))
            sc = [sum(q[c] * K[j][c] for c in cols) / math.sqrt(dh) for j in keys]
            mx = max(sc)
            w = [math.exp(s - mx) for s in sc]
            z = sum(w)
            for c in cols:
                out[i][c] = sum(w[n] / z * V[j][c] for n, j in enumerate(keys))
    return out


def _silu(v):
    return v / (1.0 + math.exp(-v))


def _gelu(v):
    return 0.5 * v * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (v + 0.044715 * v ** 3)))


def _mish(v):
    return v * math.tanh(math.log1p(math.exp(v)))


# ----------------------------------------------------------------------------- attention
def test_attention_two_heads_three_keys_by_hand_and_against_torch():
    rng = np.random.default_rng(0)
    q, k, v = rng.normal(size=(2, 4)), rng.normal(size=(3, 4)), rng.normal(size=(3, 4))
    ref = np.array(_mha(q.tolist(), k.tolist(), v.tolist(), 2, False))
    assert np.allclose(nets.attention(q, k, v, 2, False), ref, atol=1e-12)
    # one head instead of two, or an unscaled score, must not pass
    assert not np.allclose(nets.attention(q, k, v, 1, False), ref, atol=1e-6)
    # the library routine: [heads, N, dh] layout, default scale 1/sqrt(dh)
    for heads, causal, Nq, Nk, d in ((2, False, 5, 3, 8), (4, True, 6, 6, 16), (1, True, 3, 3, 4)):
        q, k, v = rng.normal(size=(Nq, d)), rng.normal(size=(Nk, d)), rng.normal(size=(Nk, d))
        split = lambda a: torch.tensor(a).view(a.shape[0], heads, d // heads).transpose(0, 1)
        o = torch.nn.functional.scaled_dot_product_attention(split(q), split(k), split(v), is_causal=causal)
        assert np.allclose(nets.attention(q, k, v, heads, causal), o.transpose(0, 1).reshape(Nq, d).numpy(), atol=1e-12)


def test_decoder_block_two_heads_three_memory_tokens_by_hand():
    """One block of the decoder transformer, H = 3 tokens, memory = time token + 2 obs tokens, 2 heads, in loops."""
    H, A, To, Do, d, heads = 3, 2, 2, 3, 4, 2
    p = inputs.make_xfmr_params(5, H, A, To, Do, d, heads, 1, bf16=False)
    rng = np.random.default_rng(1)
    x, obs, tau = rng.normal(size=(H, A)), rng.normal(size=(To, Do)), 37
    L = {k_: np.asarray(v_).tolist() for k_, v_ in p["layers"][0].items()}
    P = {k_: np.asarray(v_).tolist() for k_, v_ in p.items() if k_ not in ("layers", "arch", "d", "heads", "n_layers")}
    h = [[a + b for a, b in zip(_lin(x[i].tolist(), P["W_in"], P["b_in"]), P["pos"][i])] for i in range(H)]
    half = d // 2
    temb = [math.sin(tau * 10000.0 ** (-i / half)) for i in range(half)] + [math.cos(tau * 10000.0 ** (-i / half)) for i in range(half)]
    mem = [temb] + [_lin(obs[j].tolist(), P["W_obs"], P["b_obs"]) for j in range(To)]
    mem = [[a + b for a, b in zip(mem[j], P["cpos"][j])] for j in range(1 + To)]
    qkv = [_lin(_ln(h[i], L["ln1_g"], L["ln1_b"]), L["Wqkv"], L["bqkv"]) for i in range(H)]
    att = _mha([r[:d] for r in qkv], [r[d:2 * d] for r in qkv], [r[2 * d:] for r in qkv], heads, True)
    h = [[a + b for a, b in zip(h[i], _lin(att[i], L["Wo"], L["bo"]))] for i in range(H)]
    q2 = [_lin(_ln(h[i], L["ln2_g"], L["ln2_b"]), L["Wq2"], L["bq2"]) for i in range(H)]
    kv = [_lin(mem[j], L["Wkv2"], L["bkv2"]) for j in range(1 + To)]
    att = _mha(q2, [r[:d] for r in kv], [r[d:] for r in kv], heads, False)
    h = [[a + b for a, b in zip(h[i], _lin(att[i], L["Wo2"], L["bo2"]))] for i in range(H)]
    for i in range(H):
        f = [_gelu(v) for v in _lin(_ln(h[i], L["ln3_g"], L["ln3_b"]), L["W1"], L["b1"])]
        h[i] = [a + b for a, b in zip(h[i], _lin(f, L["W2"], L["b2"]))]
    ref = np.array([_lin(_ln(h[i], P["lnf_g"], P["lnf_b"]), P["W_out"], P["b_out"]) for i in range(H)])
    assert np.allclose(nets.xfmr_eps(p, x, tau, obs), ref, atol=1e-11)


# ----------------------------------------------------------------------------- adaLN transformer
def _dit_small(seed=3, H=2, A=2, Tc=3, Do=3, d=4, heads=2):
    p = inputs.make_dit_params(seed, H, A, Tc, Do, d, heads, 1, bf16=False)
    rng = np.random.default_rng(seed + 50)
    return p, rng.normal(size=(H, A)), rng.normal(size=(Tc, Do))


def test_dit_block_with_nontrivial_gates_on_two_tokens_by_hand():
    p, x, ctx = _dit_small()
    H, d, heads, tau = 2, p["d"], p["heads"], 63
    L = {k_: np.asarray(v_).tolist() for k_, v_ in p["layers"][0].items()}
    P = {k_: np.asarray(v_).tolist() for k_, v_ in p.items() if k_ not in ("layers", "arch", "d", "heads", "n_layers")}
    half = d // 2
    temb = [math.sin(tau * 10000.0 ** (-i / half)) for i in range(half)] + [math.cos(tau * 10000.0 ** (-i / half)) for i in range(half)]
    c = _lin([_silu(v) for v in _lin(temb, P["Wt1"], P["bt1"])], P["Wt2"], P["bt2"])
    sc = [_silu(v) for v in c]
    mod = _lin(sc, L["Wmod"], L["bmod"])
    s1, k1, g1, s2, k2, g2 = (mod[i * d:(i + 1) * d] for i in range(6))       # shift1, scale1, gate1, shift2, scale2, gate2
    assert max(abs(v - 1.0) for v in g1) > 1e-3 and max(abs(v) for v in k1) > 1e-4        # the case is not a trivial one
    h = [[a + b for a, b in zip(_lin(x[i].tolist(), P["W_in"], P["b_in"]), P["pos"][i])] for i in range(H)]
    mem = [[a + b for a, b in zip(_lin(ctx[j].tolist(), P["W_ctx"], P["b_ctx"]), P["cpos"][j])] for j in range(len(ctx))]
    a = [[n * (1.0 + k1[i]) + s1[i] for i, n in enumerate(_ln(h[r]))] for r in range(H)]
    qkv = [_lin(a[r], L["Wqkv"], L["bqkv"]) for r in range(H)]
    att = _mha([r[:d] for r in qkv], [r[d:2 * d] for r in qkv], [r[2 * d:] for r in qkv], heads, False)
    h = [[h[r][i] + g1[i] * o for i, o in enumerate(_lin(att[r], L["Wo"], L["bo"]))] for r in range(H)]
    q2 = [_lin(_ln(h[r], L["lnc_g"], L["lnc_b"]), L["Wq2"], L["bq2"]) for r in range(H)]
    kv = [_lin(m, L["Wkv2"], L["bkv2"]) for m in mem]
    att = _mha(q2, [r[:d] for r in kv], [r[d:] for r in kv], heads, False)
    h = [[h[r][i] + o for i, o in enumerate(_lin(att[r], L["Wo2"], L["bo2"]))] for r in range(H)]
    for r in range(H):
        a = [n * (1.0 + k2[i]) + s2[i] for i, n in enumerate(_ln(h[r]))]
        f = [_gelu(v) for v in _lin(a, L["W1"], L["b1"])]
        h[r] = [h[r][i] + g2[i] * o for i, o in enumerate(_lin(f, L["W2"], L["b2"]))]
    modf = _lin(sc, P["Wmodf"], P["bmodf"])
    sf, kf = modf[:d], modf[d:]
    ref = np.array([_lin([n * (1.0 + kf[i]) + sf[i] for i, n in enumerate(_ln(h[r]))], P["W_out"], P["b_out"]) for r in range(H)])
    assert np.allclose(nets.dit_eps(p, x, tau, ctx), ref, atol=1e-11)


def test_dit_modulation_slices_each_do_their_own_job():
    """Constant modulation (W_mod = 0), one slice at a time.  gate = 0 removes exactly its branch; scale = -1 feeds
    the branch the shift alone, which turns it into a constant that is written out here."""
    p, x, ctx = _dit_small(4)
    d = p["d"]
    L0 = p["layers"][0]

    def with_bmod(**sl):       # slices: s1 k1 g1 s2 k2 g2, default (0, 0, 1, 0, 0, 1)
        b = np.concatenate([np.full(d, sl.get(n, dflt)) if np.isscalar(sl.get(n, dflt)) else sl[n]
                            for n, dflt in (("s1", 0.0), ("k1", 0.0), ("g1", 1.0), ("s2", 0.0), ("k2", 0.0), ("g2", 1.0))])
        return dict(p, layers=[dict(L0, Wmod=np.zeros_like(L0["Wmod"]), bmod=b)])

    def perturbed(q, *names):
        return dict(q, layers=[dict(q["layers"][0], **{n: q["layers"][0][n] * 1.7 + 0.1 for n in names})])

    e = lambda q: nets.dit_eps(q, x, 20, ctx)
    q = with_bmod(g1=0.0)       # self-attention branch gone, MLP branch alive
    assert np.array_equal(e(q), e(perturbed(q, "Wqkv", "Wo"))) and not np.allclose(e(q), e(perturbed(q, "W1")))
    q = with_bmod(g2=0.0)       # MLP branch gone, self-attention branch alive
    assert np.array_equal(e(q), e(perturbed(q, "W1", "W2"))) and not np.allclose(e(q), e(perturbed(q, "Wqkv")))
    # scale1 = -1, shift1 = s: every token's self-attention input is s, so the attention returns the value row of s
    s = np.linspace(-0.5, 0.7, d); g = np.linspace(0.3, 1.2, d)
    q = with_bmod(k1=-1.0, s1=s, g1=g, g2=0.0)
    L = q["layers"][0]
    h = x @ p["W_in"] + p["b_in"] + p["pos"]
    h = h + g * ((s @ L["Wqkv"] + L["bqkv"])[2 * d:] @ L["Wo"] + L["bo"])
    a = nets.layer_norm(h, L["lnc_g"], L["lnc_b"])
    mem = ctx @ p["W_ctx"] + p["b_ctx"] + p["cpos"]
    kv = mem @ L["Wkv2"] + L["bkv2"]
    att = torch.nn.functional.scaled_dot_product_attention(
        *(torch.tensor(m).view(m.shape[0], p["heads"], -1).transpose(0, 1) for m in (a @ L["Wq2"] + L["bq2"], kv[:, :d], kv[:, d:])))
    h = h + att.transpose(0, 1).reshape(h.shape).numpy() @ L["Wo2"] + L["bo2"]
    sf, kf = np.split(nets.silu(nets.dit_time_vector(p, 20)) @ p["Wmodf"] + p["bmodf"], 2)
    ref = (nets.layer_norm_plain(h) * (1 + kf) + sf) @ p["W_out"] + p["b_out"]
    assert np.allclose(e(q), ref, atol=1e-12)
    # scale2 = -1, shift2 = s: the MLP sees s on every token
    q = with_bmod(g1=0.0, k2=-1.0, s2=s, g2=g)
    L = q["layers"][0]
    h = x @ p["W_in"] + p["b_in"] + p["pos"]
    a = nets.layer_norm(h, L["lnc_g"], L["lnc_b"])
    att = torch.nn.functional.scaled_dot_product_attention(
        *(torch.tensor(m).view(m.shape[0], p["heads"], -1).transpose(0, 1) for m in (a @ L["Wq2"] + L["bq2"], kv[:, :d], kv[:, d:])))
    h = h + att.transpose(0, 1).reshape(h.shape).numpy() @ L["Wo2"] + L["bo2"]
    u = s @ L["W1"] + L["b1"]
    h = h + g * (np.array([_gelu(v) for v in u]) @ L["W2"] + L["b2"])
    ref = (nets.layer_norm_plain(h) * (1 + kf) + sf) @ p["W_out"] + p["b_out"]
    assert np.allclose(e(q), ref, atol=1e-12)


# ----------------------------------------------------------------------------- conv UNet
def _conv5(x, W, b):
    Lx, cout = len(x), len(b)
    out = []
    for l in range(Lx):
        row = list(b)
        for j in range(5):
            s = l + j - 2
            if 0 <= s < Lx:
                for ci, xv in enumerate(x[s]):
                    for co in range(cout):
                        row[co] += xv * W[j][ci][co]
        out.append(row)
    return out


def _gn(y, g, b, groups, eps=1e-5):
    Lx, C = len(y), len(y[0]); cg = C // groups
    out = [[0.0] * C for _ in range(Lx)]
    for gi in range(groups):
        vals = [y[l][c] for l in range(Lx) for c in range(gi * cg, (gi + 1) * cg)]
        m = sum(vals) / len(vals)
        v = sum((t - m) ** 2 for t in vals) / len(vals)
        for l in range(Lx):
            for c in range(gi * cg, (gi + 1) * cg):
                out[l][c] = (y[l][c] - m) / math.sqrt(v + eps) * g[c] + b[c]
    return out


def _resblock(R, x, mcond, groups):
    C = len(R["b1"])
    y = [[_mish(v) for v in row] for row in _gn(_conv5(x, R["W1"], R["b1"]), R["g1"], R["be1"], groups)]
    film = _lin(mcond, R["Wf"], R["bf"])
    y = [[film[c] * row[c] + film[C + c] for c in range(C)] for row in y]            # first C: scale, last C: bias
    y = [[_mish(v) for v in row] for row in _gn(_conv5(y, R["W2"], R["b2"]), R["g2"], R["be2"], groups)]
    res = [_lin(row, R["Wr"], R["br"]) for row in x] if "Wr" in R else x
    return [[a + b for a, b in zip(y[l], res[l])] for l in range(len(x))]


def test_two_level_unet_on_four_positions_by_hand():
    H, A, To, Do, c, dt, groups, tau = 4, 2, 1, 3, 4, 4, 2, 11
    p = inputs.make_unet_params(2, H, A, To, Do, c, 2, groups=groups, dt=dt, bf16=False)
    rng = np.random.default_rng(9)
    x, obs = rng.normal(size=(H, A)), rng.normal(size=(To, Do))
    P = {k_: np.asarray(v_).tolist() for k_, v_ in p.items() if k_ not in ("blocks", "arch", "c", "levels", "groups", "dt")}
    blocks = [{k_: np.asarray(v_).tolist() for k_, v_ in R.items()} for R in p["blocks"]]
    assert [(len(R["W1"][0]), len(R["b1"])) for R in blocks] == [(4, 4), (4, 4), (4, 8), (8, 8), (8, 8), (8, 8), (12, 4), (4, 4)]
    half = dt // 2
    temb = [math.sin(tau * 10000.0 ** (-i / half)) for i in range(half)] + [math.cos(tau * 10000.0 ** (-i / half)) for i in range(half)]
    tvec = _lin([_mish(v) for v in _lin(temb, P["Wt1"], P["bt1"])], P["Wt2"], P["bt2"])
    mcond = [_mish(v) for v in tvec + obs.reshape(-1).tolist()]                       # [time vector | flattened obs]
    h = [_lin(x[l].tolist(), P["W_in"], P["b_in"]) for l in range(H)]
    h = _resblock(blocks[1], _resblock(blocks[0], h, mcond, groups), mcond, groups)
    skip = h
    h = [[0.5 * (h[2 * l][ch] + h[2 * l + 1][ch]) for ch in range(c)] for l in range(H // 2)]      # pairs (0,1), (2,3)
    h = _resblock(blocks[3], _resblock(blocks[2], h, mcond, groups), mcond, groups)
    h = _resblock(blocks[5], _resblock(blocks[4], h, mcond, groups), mcond, groups)
    h = [h[l // 2] + skip[l] for l in range(H)]                                      # repeat each position twice, then [up | skip]
    h = _resblock(blocks[7], _resblock(blocks[6], h, mcond, groups), mcond, groups)
    h = [[_mish(v) for v in row] for row in _gn(_conv5(h, P["Wh"], P["bh"]), P["gh"], P["beh"], groups)]
    ref = np.array([_lin(row, P["W_out"], P["b_out"]) for row in h])
    assert np.allclose(nets.unet_eps(p, x, tau, obs), ref, atol=1e-10)


def test_film_halves_scale_first_then_bias():
    """FiLM = [scale | bias].  With the scale half zero the first convolution cannot matter; with scale 1, bias 0
    the block is two conv-GroupNorm-Mish stages plus the residual, written with the pinned primitives."""
    rng = np.random.default_rng(3)
    C, Lx, groups, dc = 8, 6, 2, 5
    R = dict(W1=rng.normal(size=(5, C, C)) * 0.2, b1=rng.normal(size=C) * 0.1, g1=np.ones(C), be1=np.zeros(C),
             Wf=np.zeros((dc, 2 * C)), bf=np.zeros(2 * C), W2=rng.normal(size=(5, C, C)) * 0.2, b2=rng.normal(size=C) * 0.1,
             g2=1 + 0.1 * rng.normal(size=C), be2=0.1 * rng.normal(size=C))
    x, mcond = rng.normal(size=(Lx, C)), rng.normal(size=dc)
    R["bf"] = np.concatenate([np.zeros(C), rng.normal(size=C)])                       # scale 0, bias b
    o = nets.unet_resblock(R, x, mcond, groups)
    assert np.array_equal(o, nets.unet_resblock(dict(R, W1=R["W1"] * 3.0), x, mcond, groups))
    const = np.tile(R["bf"][C:], (Lx, 1))
    assert np.allclose(o, nets.mish(nets.group_norm(nets.conv1d_k5(const, R["W2"], R["b2"]), R["g2"], R["be2"], groups)) + x)
    R["bf"] = np.concatenate([np.ones(C), np.zeros(C)])                               # scale 1, bias 0
    y = nets.mish(nets.group_norm(nets.conv1d_k5(x, R["W1"], R["b1"]), R["g1"], R["be1"], groups))
    y = nets.mish(nets.group_norm(nets.conv1d_k5(y, R["W2"], R["b2"]), R["g2"], R["be2"], groups))
    assert np.allclose(nets.unet_resblock(R, x, mcond, groups), y + x)
    assert not np.allclose(nets.unet_resblock(R, x, mcond, groups), nets.unet_resblock(dict(R, W1=R["W1"] * 3.0), x, mcond, groups))


def test_sinusoidal_embedding_layout():
    e = ddpm.sinusoidal_embedding(3, 8)
    assert np.allclose(e[:4], [math.sin(3 * 10000.0 ** (-i / 4)) for i in range(4)])
    assert np.allclose(e[4:], [math.cos(3 * 10000.0 ** (-i / 4)) for i in range(4)])
