"""Inference of the speculative-decoding scheduler (Sec. 3.3), numpy fp64.

What the paper fixes: the scheduler observes three streams -- the environment's object state, the
action chunk the policy produced last, and the task progress -- encodes each stream separately
(an MLP for state vectors), aggregates the features with an MLP, and outputs the speculative
parameters: the sigma scale, the acceptance threshold, and a draft-step count for each of the three
denoising stages (early high-noise, middle, late low-noise).  It is trained with PPO; only the
deterministic (mean) action is needed at inference.

What it does not fix, and this library defines: widths (64 / 64 / 16 -> 64 -> 5), tanh activations, the
squashing of the 5 raw outputs into parameter ranges, and the stage boundaries t >= 4T/5 (early),
t < T/5 (late).  PARITY UNPINNED against the paper (no architecture, weights or ranges are published);
pinned only by structure: zero weights give the mid-range parameters, the three streams enter through
their own encoders only, and the output ranges hold for any input.

    f_o = tanh(obs W_o + b_o)   f_a = tanh(act W_a + b_a)   f_p = tanh(progress W_p + b_p)
    g   = tanh([f_o | f_a | f_p] W_1 + b_1)
    y   = g W_2 + b_2                                   (5 raw outputs)
    sigma_scale = 1 + 2 sigmoid(y0)       in (1, 3)
    lambda      = sigmoid(y1)             in (0, 1)
    K_stage     = 1 + rint((K_max - 1) sigmoid(y_{2+stage})),  stage = early, mid, late
"""
import numpy as np

HID, PROG = 64, 16


def sigmoid(v):
    return 1.0 / (1.0 + np.exp(-v))


def raw_outputs(p, obs, prev_action, progress):
    f_o = np.tanh(obs.reshape(-1) @ p["W_o"] + p["b_o"])
    f_a = np.tanh(prev_action.reshape(-1) @ p["W_a"] + p["b_a"])
    f_p = np.tanh(np.array([progress], dtype=np.float64) @ p["W_p"] + p["b_p"])
    g = np.tanh(np.concatenate([f_o, f_a, f_p]) @ p["W_1"] + p["b_1"])
    return g @ p["W_2"] + p["b_2"]


def parameters(p, obs, prev_action, progress, K_max):
    """(sigma_scale, lambda, [K_early, K_mid, K_late], k_real) -- k_real are the unrounded draft
    counts, exposed so that a test can tell a rounding tie from a real disagreement."""
    y = raw_outputs(p, obs, prev_action, progress)
    k_real = 1.0 + (K_max - 1) * sigmoid(y[2:5])
    return 1.0 + 2.0 * sigmoid(y[0]), sigmoid(y[1]), [int(np.rint(k)) for k in k_real], k_real


def stage(t, T):
    """0 early (t >= 4T/5), 2 late (t < T/5), 1 in between; integer arithmetic."""
    if t >= (4 * T) // 5:
        return 0
    return 2 if t < T // 5 else 1


def process_reward(n_accept, n_draft, n_diffusion, R_final, T_max, dt):
    """Intermediate reward of one denoising cycle (Sec. 3.3, "Reward function"):

        r = (n_accept / n_draft + n_accept / n_diffusion) lambda,   lambda = (R_final / 4) / ceil(T_max / dt).

    n_accept accepted drafts, n_draft drafts proposed, n_diffusion diffusion steps of the cycle; T_max the
    task's step limit, dt the number of task steps between scheduler updates.  A ratio whose denominator
    is zero counts 0 (the paper does not say; K = 0 proposes no draft)."""
    lam = (R_final / 4.0) / float(-(-int(T_max) // int(dt)))
    a = n_accept / n_draft if n_draft > 0 else 0.0
    e = n_accept / n_diffusion if n_diffusion > 0 else 0.0
    return (a + e) * lam
