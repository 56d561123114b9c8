"""The speculative denoising round, the chunk sampler built from it, and vanilla DDPM.

Follows the paper in its own order and notation:
  Sec. 3.1 Eqs. (1)-(3)          likelihood-ratio test, first-rejection index j*.
  Sec. 3.1 reflection equations  accept x~ ~ r iff U <= min(1, s(x~)/r(x~)); otherwise reflect
                                 x~ - m_r across the hyperplane orthogonal to Delta = m_r - m_s.
  Sec. 3.2 Eq. (3)               drafter rollout with the shared scheduler S.
  Sec. 3.2 log-acceptance eq.    log alpha_i = -1/2 |d_i|^2 - <d_i, xi_i>, d_i = (mu^_i - mu_i)/sigma_i;
                                 p_i = min(1, exp(log alpha_i)); threshold rule p_i >= lambda.
  Sec. 3.2 last paragraph        chronological scan, commit the accepted prefix, reflect the first
                                 rejected draft.

Readings taken where the paper is silent or inconsistent:
  * timestep handed to a network = timestep of its input latent; draft k consumes draft k-1;
  * a round starts from the current latent x at timestep t; the base model is evaluated on the
    K_eff+1 latents x~_0..x~_{K_eff}; the last evaluation is a "bonus" base step, taken only when
    no draft was rejected (it is the paper's sequential x^(0) of the following round);
  * K_eff = min(K, t): the sigma_0 = 0 transition is never drafted;
  * mode 0: accept iff log alpha >= log U (lossless);  mode 1: accept iff min(0, log alpha) >= log lambda;
  * sigma_scale s >= 1 divides only the test statistic (d = (mu^ - mu)/(s sigma)); sampling and
    reflection use the true sigma_t (parity unpinned against the paper: no formula is given);
  * |Delta|^2 < 1e-30  =>  accepted.
"""
import numpy as np
from . import philox


class PhiloxNoise:
    """xi_tau, U_tau and x_T as pure functions of (seed, env, timestep, element)."""

    def __init__(self, seed):
        self.seed = seed

    def xi(self, env, tau, shape):
        return philox.xi(self.seed, env, tau, int(np.prod(shape))).reshape(shape)

    def u(self, env, tau):
        return philox.uniform(self.seed, env, tau)

    def x_init(self, env, shape):
        return philox.x_init(self.seed, env, int(np.prod(shape))).reshape(shape)


class Accept:
    def __init__(self, mode=0, lam=1.0, sigma_scale=1.0, bonus=True):
        self.mode, self.lam, self.sigma_scale, self.bonus = mode, lam, sigma_scale, bonus


def log_accept_ratio(mu_hat, mu, sigma, xi, sigma_scale=1.0):
    """log alpha = -1/2 |d|^2 - <d, xi>,  d = (mu^ - mu) / (s sigma), over the whole latent."""
    d = (mu_hat - mu) / (sigma_scale * sigma)
    return -0.5 * np.sum(d * d) - np.sum(d * xi)


def accepted(log_alpha, acc, log_u):
    """Decision for one draft.  mode 0: U <= min(1, alpha);  mode 1: p = min(1, alpha) >= lambda."""
    if acc.mode == 0:
        return log_alpha >= log_u
    return min(0.0, log_alpha) >= np.log(acc.lam)


def reflect(x_tilde, m_r, m_s):
    """x = m_s + (I - 2 e e^T)(x~ - m_r),  e = Delta/|Delta|,  Delta = m_r - m_s."""
    delta = (m_r - m_s).reshape(-1)
    e = delta / np.sqrt(np.sum(delta * delta))
    v = (x_tilde - m_r).reshape(-1)
    return m_s + (v - 2.0 * e * np.dot(e, v)).reshape(x_tilde.shape)


def first_rejection(acc_flags):
    """j* = min{ j in 1..L : draft j rejected }, or None when every draft is accepted."""
    for j, a in enumerate(acc_flags, start=1):
        if not a:
            return j
    return None


class FrozenTargetDraft:
    """Drafts without a drafter: every draft step of a round reuses the base model's output at the round's
    starting latent, eps^_k = eps_base(x, t) for k = 1..K (the "frozen target draft" of the prior work cited in
    Sec. 2.2, read as: the target's prediction is frozen over the window).  The first draft is then the base
    model's own reverse step, so its acceptance ratio is exactly 1; later ones drift from it.  Any draft mean
    leaves the sampler's law unchanged (Sec. 3.1), so this variant is lossless too.  A round costs one extra base
    evaluation (n_extra in the round's dump).  PARITY UNPINNED against that prior work (not in the paper);
    pinned by: first draft always accepted with log alpha = 0, K = 1 sample-identical to vanilla, and the
    Gaussian chain's marginal."""

    def __init__(self, base):
        self.base = base
        self.eps = None

    def begin_round(self, x, t, obs):
        self.eps = self.base(x, t, obs)

    def __call__(self, x, tau, obs):
        return self.eps


def spec_round(sched, base, drafter, noise, env, obs, x, t, K, acc, clip=0.0):
    """One speculative round for one environment.  Returns (x_new, t_new, dump)."""
    K_eff = min(K, t)
    shape = x.shape
    n_extra = 0
    if K_eff > 0 and hasattr(drafter, "begin_round"):      # drafter-free drafts: one base evaluation at the current latent
        drafter.begin_round(x, t, obs)
        n_extra = 1
    # --- draft rollout (Eq. (3)): x~_0 = x; draft k is the transition at tau = t-k+1
    x_t = [x]
    mu_hat, xis, eps_hats = [None], [None], [None]
    for k in range(1, K_eff + 1):
        tau = t - k + 1
        eps_hat = drafter(x_t[k - 1], tau, obs)
        xi_k = noise.xi(env, tau, shape)
        x_k, m_k = sched.step(x_t[k - 1], eps_hat, tau, xi_k, clip)
        x_t.append(x_k); mu_hat.append(m_k); xis.append(xi_k); eps_hats.append(eps_hat)
    # --- verification: base model on every candidate latent (one batched pass on the GPU)
    n_base = K_eff + 1 if (acc.bonus or K_eff == 0) else K_eff
    eps = [base(x_t[k], t - k, obs) for k in range(n_base)]
    mu = [None] + [sched.posterior_mean(x_t[k], eps[k], t - k, clip) for k in range(n_base)]
    # --- acceptance statistic and decisions, chronological
    log_alpha, flags = [], []
    for k in range(1, K_eff + 1):
        tau = t - k + 1
        delta2 = np.sum((mu_hat[k] - mu[k]) ** 2)
        la = log_accept_ratio(mu_hat[k], mu[k], sched.sigma[tau], xis[k], acc.sigma_scale)
        log_alpha.append(la)
        flags.append(bool(delta2 < 1e-30) or bool(accepted(la, acc, np.log(noise.u(env, tau)))))
    j = first_rejection(flags)
    # --- commit
    if j is not None:
        x_new = reflect(x_t[j], mu_hat[j], mu[j])
        t_new = t - j
    elif acc.bonus or K_eff == 0:
        tau = t - K_eff
        x_new = mu[K_eff + 1] + sched.sigma[tau] * noise.xi(env, tau, shape)
        t_new = t - K_eff - 1
    else:
        x_new, t_new = x_t[K_eff], t - K_eff
    dump = dict(K_eff=K_eff, x_tilde=x_t, mu_hat=mu_hat, eps_hat=eps_hats, xi=xis, eps=eps, mu=mu, log_alpha=log_alpha,
                flags=flags, jstar=(j if j is not None else K_eff + 1), n_base=n_base, n_extra=n_extra)
    return x_new, t_new, dump


def sample_chunk(sched, base, drafter, noise, env, obs, shape, K, acc, clip=0.0, schedule=None):
    """Rounds until t = -1.  `schedule(r, t)` may override (K, acc) for round r at timestep t.

    Returns (x, stats); stats counts rounds, base/drafter evaluations, drafts accepted, and the
    NFE ingredients the paper reports (Sec. 4 "Evaluation Metrics")."""
    x = noise.x_init(env, shape)
    t = sched.T - 1
    st = dict(rounds=0, base_evals=0, draft_evals=0, accepted=0, rejections=0, bonus=0, extra_base=0, draft_rounds=0,
              prefix=[], prop_hist=np.zeros(sched.T, int), test_hist=np.zeros(sched.T, int),
              acc_hist=np.zeros(sched.T, int))
    while t >= 0:
        K_r, acc_r = schedule(st["rounds"], t) if schedule else (K, acc)
        x, t_new, d = spec_round(sched, base, drafter, noise, env, obs, x, t, K_r, acc_r, clip)
        n_acc = min(d["jstar"] - 1, d["K_eff"])
        st["rounds"] += 1
        st["base_evals"] += d["n_base"]
        st["draft_evals"] += d["K_eff"]
        st["extra_base"] += d["n_extra"]
        st["draft_rounds"] += int(d["K_eff"] > 0)
        st["accepted"] += n_acc
        st["rejections"] += int(d["jstar"] <= d["K_eff"])
        st["bonus"] += int(d["jstar"] > d["K_eff"] and (t - t_new) == d["K_eff"] + 1)
        st["prefix"].append(n_acc)
        for k in range(1, d["K_eff"] + 1):
            st["prop_hist"][t - k + 1] += 1
            st["test_hist"][t - k + 1] += int(k <= d["jstar"])
            st["acc_hist"][t - k + 1] += int(k <= n_acc)
        t = t_new
    return x, st


def sample_vanilla(sched, base, noise, env, obs, shape, clip=0.0):
    """Plain ancestral DDPM sampling: T sequential base calls."""
    x = noise.x_init(env, shape)
    for t in range(sched.T - 1, -1, -1):
        x, _ = sched.step(x, base(x, t, obs), t, noise.xi(env, t, shape), clip)
    return x


class TableNoise:
    """The same streams as PhiloxNoise, evaluated once for a block of environments
    (philox.normals_table / uniform_table) and then looked up; used where a test runs many
    environments and the per-call overhead of the generator would dominate."""

    def __init__(self, seed, envs, T, n):
        self.env0 = int(envs[0])
        assert list(envs) == list(range(self.env0, self.env0 + len(envs)))
        self._xi = philox.normals_table(seed, envs, philox.STREAM_XI, range(T), n)
        self._init = philox.normals_table(seed, envs, philox.STREAM_INIT, [0], n)[:, 0]
        self._u = philox.uniform_table(seed, envs, T)

    def xi(self, env, tau, shape):
        return self._xi[env - self.env0, tau].reshape(shape)

    def u(self, env, tau):
        return float(self._u[env - self.env0, tau])

    def x_init(self, env, shape):
        return self._init[env - self.env0].reshape(shape)
