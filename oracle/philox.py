"""Philox4x32-10 counter-based generator and the noise/uniform streams built on it.

The paper fixes seeds but names no generator (Sec. 4 runs with fixed seeds; Sec. 3.2 keeps the
noise realisations of the drafter's rollout for the verification).  The reading used here: every random
number is a pure function of (seed, environment, stream, timestep, element), never of
the round structure, so a draft at timestep tau and a base step at tau draw the same
xi_tau.  Generator: Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11),
written from its published round function.
"""
import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = np.uint64(0x9E3779B9)
_W1 = np.uint64(0xBB67AE85)
_MASK = np.uint64(0xFFFFFFFF)
_SH = np.uint64(32)

STREAM_INIT = 0   # x_T ~ N(0, I)            (timestep code 0)
STREAM_XI = 1     # xi_tau of the transition taken at timestep tau
STREAM_U = 2      # U_tau of the acceptance test at timestep tau


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten Philox rounds on counter (c0..c3) with key (k0,k1); all 32-bit words.

    Inputs broadcast against each other; returns four uint64 arrays holding 32-bit
    values.  One round: (hi0,lo0) = M0*c0, (hi1,lo1) = M1*c2,
    new counter = (hi1^c1^k0, lo1, hi0^c3^k1, lo0); the key is bumped by the Weyl
    constants between rounds.
    """
    c0, c1, c2, c3, k0, k1 = [np.asarray(v, dtype=np.uint64) & _MASK
                              for v in (c0, c1, c2, c3, k0, k1)]
    c0, c1, c2, c3, k0, k1 = np.broadcast_arrays(c0, c1, c2, c3, k0, k1)
    for _ in range(10):
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _SH, p0 & _MASK
        hi1, lo1 = p1 >> _SH, p1 & _MASK
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + _W0) & _MASK
        k1 = (k1 + _W1) & _MASK
    return c0, c1, c2, c3


def bits_to_unit(n):
    """Map a 32-bit word to the open unit interval: ((n >> 9) + 0.5) * 2^-23.

    The value is exactly representable in fp32 and is never 0 or 1."""
    return ((np.asarray(n, dtype=np.uint64) >> np.uint64(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def _words(seed, env, stream, tcode, quads):
    k0 = np.uint64(seed & 0xFFFFFFFF)
    k1 = np.uint64((seed >> 32) & 0xFFFFFFFF)
    return philox4x32_10(quads, np.uint64(tcode), np.uint64(env), np.uint64(stream), k0, k1)


def normals(seed, env, stream, tcode, n):
    """n standard normals; element i comes from counter quad i//4, lane i%4.

    Lanes (0,1) and (2,3) of a quad are the cosine and sine branches of one Box-Muller
    pair: r = sqrt(-2 ln u_a), theta = 2 pi u_b."""
    nq = (n + 3) // 4
    w = _words(seed, env, stream, tcode, np.arange(nq, dtype=np.uint64))
    u = [bits_to_unit(x) for x in w]
    out = np.empty((nq, 4), dtype=np.float64)
    for pair in (0, 1):
        r = np.sqrt(-2.0 * np.log(u[2 * pair]))
        th = 2.0 * np.pi * u[2 * pair + 1]
        out[:, 2 * pair] = r * np.cos(th)
        out[:, 2 * pair + 1] = r * np.sin(th)
    return out.reshape(-1)[:n]


def xi(seed, env, tau, n):
    """Noise of the reverse transition taken at timestep tau (x_tau -> x_{tau-1})."""
    return normals(seed, env, STREAM_XI, tau, n)


def x_init(seed, env, n):
    """Initial latent x_T ~ N(0, I)."""
    return normals(seed, env, STREAM_INIT, 0, n)


def uniform(seed, env, tau):
    """U_tau of the acceptance test for the transition at timestep tau (lane 0 of quad 0)."""
    w = _words(seed, env, STREAM_U, tau, np.uint64(0))
    return float(bits_to_unit(w[0]))


def uniform_table(seed, envs, T):
    """U for every (env, tau): vectorised evaluation of `uniform`, shape [len(envs), T]."""
    envs = np.asarray(envs, dtype=np.uint64)[:, None]
    taus = np.arange(T, dtype=np.uint64)[None, :]
    k0 = np.uint64(seed & 0xFFFFFFFF)
    k1 = np.uint64((seed >> 32) & 0xFFFFFFFF)
    w = philox4x32_10(np.uint64(0), taus, envs, np.uint64(STREAM_U), k0, k1)
    return bits_to_unit(w[0])


def normals_table(seed, envs, stream, tcodes, n):
    """`normals` for every (env, tcode) at once: shape [len(envs), len(tcodes), n]."""
    envs = np.asarray(envs, dtype=np.uint64)[:, None, None]
    tc = np.asarray(tcodes, dtype=np.uint64)[None, :, None]
    nq = (n + 3) // 4
    quads = np.arange(nq, dtype=np.uint64)[None, None, :]
    k0 = np.uint64(seed & 0xFFFFFFFF)
    k1 = np.uint64((seed >> 32) & 0xFFFFFFFF)
    w = philox4x32_10(quads, tc, envs, np.uint64(stream), k0, k1)
    u = [bits_to_unit(x) for x in w]
    out = np.empty(u[0].shape + (4,), dtype=np.float64)
    for pair in (0, 1):
        r = np.sqrt(-2.0 * np.log(u[2 * pair]))
        th = 2.0 * np.pi * u[2 * pair + 1]
        out[..., 2 * pair] = r * np.cos(th)
        out[..., 2 * pair + 1] = r * np.sin(th)
    return out.reshape(out.shape[0], out.shape[1], -1)[:, :, :n]
