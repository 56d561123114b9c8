"""The algebra behind the folded cross-attention sub-block of the CUDA path, checked on the CPU in fp64 against the
oracle's own (unfolded) definition of that sub-block.

With NK memory tokens whose keys k_j and values v_j do not depend on the token rows, the sub-block

    h + Attn(LN2(h) Wq2 + bq2, K, V) Wo2 + bo2

equals, per head hd (columns S of width dh),

    score_{hd,j} = xhat . kq_{j,hd} + c_{j,hd},       xhat = (h - mean) / sqrt(var + eps)
        kq_{j,hd}[i] = g2[i] sum_{c in S} Wq2[i, c] k_j[c] / sqrt(dh)
        c_{j,hd}     = sum_{c in S} (bq2[c] + sum_i b2[i] Wq2[i, c]) k_j[c] / sqrt(dh)
    out = sum_{hd,j} softmax_j(score)_{hd,j} u_{j,hd} + bo2,      u_{j,hd}[o] = sum_{c in S} v_j[c] Wo2[c, o]

The tables kq, c, u below are written from these formulas (not from the CUDA source); the reference side calls
oracle.nets.  A wrong scale, a bias dropped from c, or heads mixed in u fails the comparison."""
import numpy as np
import pytest

from oracle import nets


def _case(seed, d, heads, H, NK):
    rng = np.random.default_rng(seed)
    L = dict(ln2_g=rng.normal(1.0, 0.3, d), ln2_b=rng.normal(0.0, 0.3, d),
             Wq2=rng.normal(0.0, 1.0 / np.sqrt(d), (d, d)), bq2=rng.normal(0.0, 0.2, d),
             Wo2=rng.normal(0.0, 1.0 / np.sqrt(d), (d, d)), bo2=rng.normal(0.0, 0.2, d))
    h = rng.normal(0.3, 1.5, (H, d))
    k = rng.normal(0.0, 1.0, (NK, d))
    v = rng.normal(0.0, 1.0, (NK, d))
    return L, h, k, v


def _folded(L, h, k, v, heads):
    H, d = h.shape
    NK, dh = k.shape[0], d // heads
    kq = np.zeros((NK, heads, d)); cc = np.zeros((NK, heads)); u = np.zeros((NK, heads, d))
    wb = L["bq2"] + L["ln2_b"] @ L["Wq2"]
    for j in range(NK):
        for hd in range(heads):
            S = slice(hd * dh, (hd + 1) * dh)
            kq[j, hd] = L["ln2_g"] * (L["Wq2"][:, S] @ k[j, S]) / np.sqrt(dh)
            cc[j, hd] = wb[S] @ k[j, S] / np.sqrt(dh)
            u[j, hd] = v[j, S] @ L["Wo2"][S, :]
    xhat = nets.layer_norm_plain(h)
    score = np.einsum("ri,jhi->rhj", xhat, kq) + cc.T[None, :, :]          # [H, heads, NK]
    p = nets.softmax(score)
    return h + np.einsum("rhj,jho->ro", p, u) + L["bo2"]


@pytest.mark.parametrize("d,heads,H,NK", [(64, 4, 16, 3), (128, 8, 7, 1), (96, 2, 5, 4)])
def test_folded_cross_attention_equals_the_oracle_sub_block(d, heads, H, NK):
    L, h, k, v = _case(d + heads + NK, d, heads, H, NK)
    a = nets.layer_norm(h, L["ln2_g"], L["ln2_b"])
    ref = h + nets.attention(a @ L["Wq2"] + L["bq2"], k, v, heads, False) @ L["Wo2"] + L["bo2"]
    got = _folded(L, h, k, v, heads)
    assert np.max(np.abs(got - ref)) < 1e-11 * max(1.0, np.max(np.abs(ref)))


def test_a_dropped_layernorm_bias_term_would_be_seen():
    """The constant c carries the LayerNorm bias through Wq2; without it the result moves by far more than the tolerance."""
    L, h, k, v = _case(5, 64, 4, 16, 3)
    ref = _folded(L, h, k, v, 4)
    L2 = dict(L, ln2_b=np.zeros_like(L["ln2_b"]))
    assert np.max(np.abs(_folded(L2, h, k, v, 4) - ref)) > 1e-3
