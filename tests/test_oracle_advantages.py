"""Pins for the oracle's TD/GAE pass with the absorbing failure transition (CPU only)."""
import numpy as np
import pytest
from scipy import signal

import oracle


def _ragged(rng, B, lo, hi, p_stop=0.35):
    lengths = rng.integers(lo, hi + 1, size=B).astype(np.int32)
    n = int(lengths.sum())
    rewards = rng.normal(0, 0.5, size=n)
    values = rng.normal(0, 0.5, size=n)
    stopped = (rng.random(B) < p_stop).astype(np.uint8)
    return rewards, values, lengths, stopped


def _split(a, lengths):
    return np.split(a, np.cumsum(lengths)[:-1])


@pytest.mark.parametrize("gamma,lam", [(1.0, 0.95), (0.99, 0.9), (1.0, 1.0), (0.9, 0.0)])
def test_recursion_equals_the_literal_sum(gamma, lam):
    r, v, L, s = _ragged(np.random.default_rng(0), 9, 1, 40)
    a = oracle.advantages(r, v, L, s, gamma, lam, -1.0)
    b = oracle.advantages(r, v, L, s, gamma, lam, -1.0, direct=True)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)


def test_brute_force_tiny_by_hand():
    # one stopped trajectory of 4 tokens, written out term by term (V_4 := 0, r_3 := r_fail)
    r = np.array([0.0, 0.0, 0.0, 0.7])          # 0.7 must be REPLACED by r_fail, not added to
    v = np.array([0.5, 0.4, 0.2, -0.1])
    g, l, rf = 0.9, 0.8, -1.0
    d = [0.0 + g * 0.4 - 0.5, 0.0 + g * 0.2 - 0.4, 0.0 + g * (-0.1) - 0.2, rf + 0.0 - (-0.1)]
    k = g * l
    want = [d[0] + k * d[1] + k**2 * d[2] + k**3 * d[3], d[1] + k * d[2] + k**2 * d[3], d[2] + k * d[3], d[3]]
    got = oracle.advantages(r, v, [4], [1], g, l, rf)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-15)
    # not stopped: the stored terminal reward is used
    d3 = 0.7 - (-0.1)
    got = oracle.advantages(r, v, [4], [0], g, l, rf)
    assert abs(got[3] - d3) < 1e-15 and abs(got[2] - (d[2] + k * d3)) < 1e-15


def test_monte_carlo_identity_at_gamma_lambda_one():
    # gamma = lambda = 1: A_t = (sum of remaining rewards) - V_t
    r, v, L, s = _ragged(np.random.default_rng(1), 12, 1, 300)
    got = _split(oracle.advantages(r, v, L, s, 1.0, 1.0, -1.0), L)
    for i, (ri, vi) in enumerate(zip(_split(r, L), _split(v, L))):
        ri = ri.copy()
        if s[i]:
            ri[-1] = -1.0
        ret = np.cumsum(ri[::-1])[::-1]
        np.testing.assert_allclose(got[i], ret - vi, rtol=0, atol=1e-10)


def test_lambda_zero_gives_td_errors():
    r, v, L, s = _ragged(np.random.default_rng(2), 7, 1, 50)
    got = _split(oracle.advantages(r, v, L, s, 0.97, 0.0, -2.0), L)
    for i, (ri, vi) in enumerate(zip(_split(r, L), _split(v, L))):
        ri = ri.copy()
        if s[i]:
            ri[-1] = -2.0
        v_next = np.r_[vi[1:], 0.0]
        np.testing.assert_allclose(got[i], ri + 0.97 * v_next - vi, rtol=0, atol=1e-14)


def test_matches_a_library_linear_filter():
    # A_t = delta_t + k A_{t+1} is a one-pole IIR filter run over the reversed TD errors
    gamma, lam = 0.995, 0.93
    r, v, L, s = _ragged(np.random.default_rng(3), 5, 100, 2000)
    got = _split(oracle.advantages(r, v, L, s, gamma, lam, -1.0), L)
    for i, (ri, vi) in enumerate(zip(_split(r, L), _split(v, L))):
        ri = ri.copy()
        if s[i]:
            ri[-1] = -1.0
        delta = ri + gamma * np.r_[vi[1:], 0.0] - vi
        want = signal.lfilter([1.0], [1.0, -gamma * lam], delta[::-1])[::-1]
        np.testing.assert_allclose(got[i], want, rtol=1e-11, atol=1e-11)


def test_absorbing_failure_special_cases():
    # stopped, zero rewards, constant value v, gamma = lambda = 1: A_t = r_fail - v for every t
    L = 37
    got = oracle.advantages(np.zeros(L), np.full(L, 0.3), [L], [1], 1.0, 1.0, -1.0)
    np.testing.assert_allclose(got, np.full(L, -1.3), rtol=0, atol=1e-12)
    # the last TD error is r_fail - V(s_Tstop): nothing is bootstrapped past the absorbing state
    r, v, Ls, s = _ragged(np.random.default_rng(4), 20, 1, 30, p_stop=1.0)
    a = _split(oracle.advantages(r, v, Ls, s, 0.99, 0.95, -1.0), Ls)
    for ai, vi in zip(a, _split(v, Ls)):
        assert abs(ai[-1] - (-1.0 - vi[-1])) < 1e-15
    # single-token trajectories
    got = oracle.advantages([0.25, 0.5], [0.1, 0.2], [1, 1], [0, 1], 0.9, 0.9, -1.0)
    np.testing.assert_allclose(got, [0.25 - 0.1, -1.0 - 0.2], rtol=0, atol=1e-15)
    # r_fail = 0 on a stopped row (the "no terminal penalty" variant) zeroes the terminal reward
    got = oracle.advantages([0.0, 0.9], [0.0, 0.0], [2], [1], 1.0, 1.0, 0.0)
    np.testing.assert_allclose(got, [0.0, 0.0], rtol=0, atol=0)


def test_trajectories_do_not_leak_into_each_other_and_empty_ones_are_skipped():
    rng = np.random.default_rng(5)
    r, v, L, s = _ragged(rng, 6, 1, 25)
    whole = _split(oracle.advantages(r, v, L, s, 1.0, 0.95, -1.0), L)
    for i, (ri, vi) in enumerate(zip(_split(r, L), _split(v, L))):
        alone = oracle.advantages(ri, vi, [L[i]], [s[i]], 1.0, 0.95, -1.0)
        np.testing.assert_array_equal(alone, whole[i])
    L2 = np.array([0, L[0], 0, 0, L[1], 0], dtype=np.int32)
    s2 = np.array([1, s[0], 1, 0, s[1], 1], dtype=np.uint8)
    n = L[0] + L[1]
    got = oracle.advantages(r[:n], v[:n], L2, s2, 1.0, 0.95, -1.0)
    np.testing.assert_array_equal(got, np.concatenate(whole[:2]))


def test_float32_threaded_entry_point_agrees():
    r, v, L, s = _ragged(np.random.default_rng(6), 33, 1, 400)
    r32, v32 = r.astype(np.float32), v.astype(np.float32)
    a = oracle.advantages(r32.astype(np.float64), v32.astype(np.float64), L, s, 1.0, 0.95, -1.0)
    b = oracle.advantages_f32(r32, v32, L, s, 1.0, 0.95, -1.0, n_threads=4)
    np.testing.assert_array_equal(a, b)


def test_padded_layout_is_the_literal_sum_row_by_row():
    # Eq. 5 written out for every row of a [B, t_max] batch on its own, padding filled with NaN
    rng = np.random.default_rng(5)
    B, t_max, gamma, lam, r_fail = 7, 23, 0.97, 0.9, -1.0
    L = np.array([0, 1, 23, 5, 22, 2, 11], dtype=np.int32)
    stopped = np.array([1, 1, 0, 1, 0, 0, 1], dtype=np.uint8)
    r = rng.normal(0, 0.5, size=(B, t_max)); v = rng.normal(0, 0.5, size=(B, t_max))
    pad = np.arange(t_max)[None, :] >= L[:, None]
    r[pad] = np.nan; v[pad] = np.nan
    got = oracle.advantages_padded(r, v, L, stopped, gamma, lam, r_fail)
    want = np.zeros((B, t_max))
    for i in range(B):
        n = int(L[i])
        rr = r[i, :n].copy()
        if n and stopped[i]:
            rr[n - 1] = r_fail                                   # Eq. 13 replaces the last reward
        vv = np.append(v[i, :n], 0.0)                            # nothing is bootstrapped past the last token
        delta = rr + gamma * vv[1:] - vv[:-1]                    # Eq. 4
        for t in range(n):
            want[i, t] = sum((gamma * lam) ** l * delta[t + l] for l in range(n - t))   # Eq. 5
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    assert np.all(got[pad] == 0.0)
