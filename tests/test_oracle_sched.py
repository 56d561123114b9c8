"""Pins of the scheduler-inference oracle: structure only (the paper publishes no architecture)."""
import numpy as np

from oracle import sched
from paper_2512_15773_b200 import inputs


def _case(seed=0, H=16, A=2, To=2, Do=20):
    rng = np.random.default_rng(seed)
    return (inputs.make_sched_params(seed, H, A, To, Do, scale=4.0), rng.normal(size=(To, Do)), rng.normal(size=(H, A)),
            float(rng.random()))


def test_zero_network_gives_mid_range_parameters():
    p, obs, act, prog = _case()
    z = {k: (np.zeros_like(v) if isinstance(v, np.ndarray) else v) for k, v in p.items()}
    s, lam, K, _ = sched.parameters(z, obs, act, prog, K_max=9)
    assert s == 2.0 and lam == 0.5 and K == [5, 5, 5]          # 1 + rint(8 * 0.5)


def test_ranges_hold_for_any_input():
    for seed in range(20):
        p, obs, act, prog = _case(seed)
        s, lam, K, _ = sched.parameters(p, 50.0 * obs, -30.0 * act, prog, K_max=10)
        assert 1.0 < s < 3.0 and 0.0 < lam < 1.0 and all(1 <= k <= 10 for k in K)


def test_each_stream_enters_through_its_own_encoder_only():
    p, obs, act, prog = _case(3)
    y = sched.raw_outputs(p, obs, act, prog)
    for name in ("W_o", "W_a", "W_p"):
        q = dict(p); q[name] = np.zeros_like(p[name])
        other = {"W_o": (2.0 * obs, act, prog), "W_a": (obs, -act, prog), "W_p": (obs, act, 1.0 - prog)}[name]
        # with a stream's encoder weights zeroed, changing that stream's input changes nothing
        assert np.array_equal(sched.raw_outputs(q, obs, act, prog), sched.raw_outputs(q, *other))
        assert not np.allclose(sched.raw_outputs(p, *other), y)


def test_one_unit_by_hand():
    # obs = [2], act = [3], progress = 0.5, every weight 0 except single paths set by hand
    p = dict(W_o=np.zeros((1, 64)), b_o=np.zeros(64), W_a=np.zeros((1, 64)), b_a=np.zeros(64), W_p=np.zeros((1, 16)),
             b_p=np.zeros(16), W_1=np.zeros((144, 64)), b_1=np.zeros(64), W_2=np.zeros((64, 5)), b_2=np.zeros(5))
    p["W_o"][0, 0] = 0.5; p["W_a"][0, 1] = -1.0; p["W_p"][0, 2] = 2.0
    p["W_1"][0, 0] = 1.0; p["W_1"][64 + 1, 0] = 1.0; p["W_1"][128 + 2, 0] = 1.0
    p["W_2"][0, 0] = 3.0; p["b_2"][1] = -1.0
    g0 = np.tanh(np.tanh(1.0) + np.tanh(-3.0) + np.tanh(1.0))
    y = sched.raw_outputs(p, np.array([[2.0]]), np.array([[3.0]]), 0.5)
    assert np.allclose(y, [3.0 * g0, -1.0, 0.0, 0.0, 0.0], atol=1e-15)
    s, lam, K, _ = sched.parameters(p, np.array([[2.0]]), np.array([[3.0]]), 0.5, K_max=7)
    assert abs(s - (1 + 2 / (1 + np.exp(-3.0 * g0)))) < 1e-15 and abs(lam - 1 / (1 + np.e)) < 1e-15 and K == [4, 4, 4]


def test_stage_boundaries():
    T = 100
    assert [sched.stage(t, T) for t in (99, 80, 79, 20, 19, 0)] == [0, 0, 1, 1, 2, 2]


# ---- intermediate reward (Sec. 3.3, "Reward function") ----

def test_process_reward_worked_values():
    # 80 of 100 drafts accepted in a 100-step cycle; R_final 100, 400 task steps, an update every 8: 50 updates,
    # lambda = 25 / 50 = 0.5, r = (0.8 + 0.8) 0.5
    assert abs(sched.process_reward(80, 100, 100, 100.0, 400, 8) - 0.8) < 1e-15
    # the update count is a ceiling: 401 steps need 51 updates
    assert abs(sched.process_reward(80, 100, 100, 100.0, 401, 8) - 1.6 * 25.0 / 51.0) < 1e-15
    # 60 of 75 drafts accepted: the two ratios differ (0.8 and 0.6)
    assert abs(sched.process_reward(60, 75, 100, 8.0, 10, 1) - 1.4 * 0.2) < 1e-15


def test_process_reward_accumulates_to_a_quarter_of_the_final_reward():
    # lambda is chosen so that cycles whose ratios sum to 1 add up, over the expected number of updates, to
    # R_final / 4 (the paper's stated purpose of the scaling factor)
    R, T_max, dt = 40.0, 300, 7
    n = -(-T_max // dt)
    total = sum(sched.process_reward(50, 100, 100, R, T_max, dt) for _ in range(n))
    assert abs(total - R / 4.0) < 1e-12


def test_process_reward_edge_cases_and_monotonicity():
    assert sched.process_reward(0, 0, 100, 10.0, 100, 10) == 0.0          # K = 0: nothing drafted
    assert sched.process_reward(0, 50, 100, 10.0, 100, 10) == 0.0
    r = [sched.process_reward(a, 90, 100, 10.0, 100, 10) for a in range(0, 91, 10)]
    assert all(b > a for a, b in zip(r, r[1:]))
    # fewer wasted drafts at the same number of accepted ones pays more
    assert sched.process_reward(60, 70, 100, 10.0, 100, 10) > sched.process_reward(60, 90, 100, 10.0, 100, 10)
