"""Pins for the oracle's decode-step function (CPU only).

Each test holds the oracle to something fixed outside it: a library routine, a closed
form, an invariant the paper states, a hand-worked example, or brute force.
"""
import math
import os

import numpy as np
import pytest
from scipy import special, stats

import oracle


def _rng(seed):
    return np.random.default_rng(seed)


def _peaked_logits(rng, n_rows, V, sd=2.0):
    x = rng.normal(0.0, sd, size=(n_rows, V))
    for r in range(n_rows):
        for _ in range(int(rng.integers(1, 4))):
            x[r, int(rng.integers(0, V))] += rng.uniform(6.0, 12.0)
    return x


# --------------------------------------------------------------------------- log-softmax


@pytest.mark.parametrize("temperature", [1.0, 0.6, 2.5])
def test_log_softmax_matches_library_and_normalises(temperature):
    x = _peaked_logits(_rng(1), 1, 5000)[0]
    got = oracle.log_softmax(x, temperature)
    want = special.log_softmax(x / temperature)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    assert abs(np.exp(got).sum() - 1.0) < 1e-12


def test_step_reports_the_log_prob_and_gap_of_its_token():
    # Eq. 6 the long way: two normalised log-probabilities, subtracted.
    rng = _rng(2)
    V = 3000
    x = _peaked_logits(rng, 6, V)
    for sampler in (oracle.SAMPLER_FLAT, oracle.SAMPLER_HIER):
        ro = oracle.Rollout(6, seed=17)
        p = oracle.make_params(temperature=0.8, sampler=sampler, warmup_complete=0)
        outs = ro.step(x, np.zeros(6), p)
        for r in range(6):
            lsm = special.log_softmax(x[r] / 0.8)
            tok = outs[r].token
            assert 0 <= tok < V
            assert abs(outs[r].logp - lsm[tok]) < 1e-11
            assert abs(outs[r].g - (lsm.max() - lsm[tok])) < 1e-11
            assert outs[r].g >= 0.0
            assert (outs[r].g == 0.0) == (x[r, tok] == x[r].max())
            assert abs(outs[r].max_x - (x[r] / 0.8).max()) < 1e-12
            assert abs(outs[r].log_s - (special.logsumexp(x[r] / 0.8) - (x[r] / 0.8).max())) < 1e-11


def test_shift_invariance():
    x = _peaked_logits(_rng(3), 4, 2500)
    for sampler in (oracle.SAMPLER_FLAT, oracle.SAMPLER_HIER):
        p = oracle.make_params(sampler=sampler)
        a = oracle.Rollout(4, seed=5).step(x, np.full(4, 0.5), p)
        b = oracle.Rollout(4, seed=5).step(x + 3.25, np.full(4, 0.5), p)   # 3.25 adds exactly in binary
        for r in range(4):
            assert a[r].token == b[r].token
            assert abs(a[r].g - b[r].g) < 1e-9 and abs(a[r].logp - b[r].logp) < 1e-9


# --------------------------------------------------------------------------- the sampler


def _token_counts(x_row, sampler, n_draws, seed, temperature=1.0):
    """Draw n_draws tokens from one row: every (slot, step) pair is an independent draw."""
    slots = 64
    steps = n_draws // slots
    ro = oracle.Rollout(slots, seed=seed)
    p = oracle.make_params(temperature=temperature, sampler=sampler, warmup_complete=0, t_max=10**9)
    rows = np.tile(x_row, (slots, 1))
    vals = np.zeros(slots)
    counts = np.zeros(x_row.size, dtype=np.int64)
    for _ in range(steps):
        outs = ro.step(rows, vals, p, n_threads=8)
        for r in range(slots):
            counts[outs[r].token] += 1
    return counts


def test_flat_sampler_draws_from_softmax_chi_square():
    x = np.array([1.2, -0.3, 0.0, 2.0, -1.5, 0.7, 0.1, -0.8])
    n = 200_000
    counts = _token_counts(x, oracle.SAMPLER_FLAT, n, seed=11, temperature=0.9)
    probs = special.softmax(x / 0.9)
    chi2, pval = stats.chisquare(counts, probs * counts.sum())
    assert pval > 1e-3, (chi2, pval)


def test_hierarchical_sampler_draws_from_softmax_chi_square():
    # 2100 ids = 3 blocks of 1024 (last one ragged) and 66 sub-blocks of 32 (last one ragged).
    rng = _rng(4)
    V = 2100
    x = rng.normal(0.0, 1.0, size=V)
    heavy = [3, 40, 1000, 1023, 1024, 1500, 2047, 2048, 2090, 2099]
    x[heavy] += np.linspace(3.0, 5.0, len(heavy))
    probs = special.softmax(x)
    n = 120_000
    counts = _token_counts(x, oracle.SAMPLER_HIER, n, seed=23)
    # bins: each heavy id on its own, the light ids pooled per sub-block group of 6 sub-blocks
    light = np.ones(V, bool)
    light[heavy] = False
    obs = [counts[i] for i in heavy]
    exp = [probs[i] * n for i in heavy]
    for lo in range(0, V, 192):
        sel = np.zeros(V, bool)
        sel[lo:lo + 192] = True
        sel &= light
        obs.append(counts[sel].sum())
        exp.append(probs[sel].sum() * n)
    obs, exp = np.array(obs, float), np.array(exp, float)
    assert exp.min() > 20
    chi2, pval = stats.chisquare(obs, exp * obs.sum() / exp.sum())
    assert pval > 1e-3, (chi2, pval)


def test_hierarchical_equals_flat_when_one_sub_block():
    # V <= 32: levels 2 and 1 have a single candidate, level 0 uses the flat sampler's draws.
    x = _peaked_logits(_rng(5), 16, 32, sd=1.0)
    a = oracle.Rollout(16, seed=9).step(x, np.zeros(16), oracle.make_params(sampler=oracle.SAMPLER_FLAT))
    b = oracle.Rollout(16, seed=9).step(x, np.zeros(16), oracle.make_params(sampler=oracle.SAMPLER_HIER))
    assert [o.token for o in a] == [o.token for o in b]


def test_flat_sampler_is_gumbel_argmax_brute_force():
    # brute force on V = 8: rebuild the perturbed scores from the exposed uniforms
    x = np.array([[0.5, 1.5, -0.2, 0.9, 0.0, 1.1, -1.0, 0.3]])
    ro = oracle.Rollout(3, seed=77, batch_id=2)
    p = oracle.make_params(temperature=0.7, warmup_complete=0)
    for step in range(4):
        out = ro.step(x, [0.0], p, row_ids=[2])[0]
        scores = [x[0, a] / 0.7 - math.log(-math.log(oracle.uniform(77, 2, 2, step, 0, a))) for a in range(8)]
        assert out.token == int(np.argmax(scores))
        top = sorted(scores)[-2:]
        assert abs(out.min_rel_gap - (top[1] - top[0]) / max(1.0, abs(top[0]), abs(top[1]))) < 1e-12


def test_hierarchical_sampler_follows_its_written_convention_brute_force():
    # level 2: blocks of 1024 ids, draw index = block number; level 1: sub-blocks of 32 ids,
    # draw index = id >> 5 (global); level 0: ids, draw index = id.  Rebuilt here with a
    # library log-sum-exp and the exposed uniforms.
    rng = _rng(14)
    V = 2100
    x = rng.normal(0, 2.0, size=(1, V))
    seed, batch, slot = 31, 3, 5
    ro = oracle.Rollout(8, seed=seed, batch_id=batch)
    p = oracle.make_params(temperature=1.3, sampler=oracle.SAMPLER_HIER, warmup_complete=0)

    def gum(step, level, index):
        return -math.log(-math.log(oracle.uniform(seed, batch, slot, step, level, index)))

    for step in range(6):
        out = ro.step(x, [0.0], p, row_ids=[slot])[0]
        xs = x[0] / 1.3
        blocks = [special.logsumexp(xs[b * 1024:(b + 1) * 1024]) + gum(step, 2, b) for b in range(3)]
        b = int(np.argmax(blocks))
        lo, hi = b * 1024, min(V, (b + 1) * 1024)
        subs = {j: special.logsumexp(xs[j * 32:min(V, (j + 1) * 32)]) + gum(step, 1, j)
                for j in range(lo // 32, (hi + 31) // 32)}
        j = max(subs, key=subs.get)
        ids = {a: xs[a] + gum(step, 0, a) for a in range(j * 32, min(V, (j + 1) * 32))}
        assert out.token == max(ids, key=ids.get)


def test_temperature_zero_is_greedy_first_argmax():
    x = np.array([[0.0, 3.0, 3.0, 1.0], [5.0, 1.0, 5.0, 5.0]])
    outs = oracle.Rollout(2, seed=1).step(x, [0.5, 0.5], oracle.make_params(temperature=0.0))
    assert [o.token for o in outs] == [1, 0]
    assert all(o.g == 0.0 and o.logp == 0.0 for o in outs)


def test_dominant_token_always_wins_and_low_temperature_tends_to_argmax():
    x = _rng(6).normal(size=(8, 500))
    x[:, 123] += 80.0   # Gumbel noise spans < 20, so nothing can overtake a +80 lead
    for sampler in (0, 1):
        outs = oracle.Rollout(8, seed=3).step(x, np.zeros(8), oracle.make_params(sampler=sampler))
        assert all(o.token == 123 and o.g == 0.0 for o in outs)
    y = _rng(7).normal(size=(8, 500))
    outs = oracle.Rollout(8, seed=3).step(y, np.zeros(8), oracle.make_params(temperature=1e-3))
    assert [o.token for o in outs] == list(y.argmax(axis=1))


def test_minus_infinity_logits_never_win():
    x = _rng(8).normal(size=(4, 100))
    x[:, ::2] = -np.inf
    for sampler in (0, 1):
        ro = oracle.Rollout(4, seed=2)
        for _ in range(20):
            outs = ro.step(x, np.zeros(4), oracle.make_params(sampler=sampler, warmup_complete=0))
            assert all(o.token % 2 == 1 for o in outs)


def test_unusable_rows_are_flagged_not_sampled():
    good = np.zeros(10)
    for bad_row in (np.full(10, -np.inf), np.r_[good[:5], np.nan, good[6:]], np.r_[good[:5], np.inf, good[6:]]):
        ro = oracle.Rollout(1, seed=0)
        out = ro.step(bad_row[None, :], [0.0], oracle.make_params())[0]
        assert out.bad == 1 and out.stop == 0 and out.token == 0
        assert ro.states[0].status == oracle.BAD and ro.states[0].t == 0 and ro.states[0].z == 0.0


# --------------------------------------------------------------------------- Eq. 9-11


def _forced(ro, x, v, p, tok):
    return ro.step(x, [v], p, forced_tokens=[tok])[0]


def test_worked_example_by_hand(golden_dir):
    rows = []
    with open(os.path.join(golden_dir, "worked_stop_example.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append([float(t) for t in line.split()])
    x = np.array([[math.log(4), math.log(2), 0, 0, 0, 0, 0, 0]], dtype=np.float64)
    tokens, values = [0, 1, 2, 1], [0.5, 0.5, 0.3, 0.1]
    p = oracle.make_params(mu_g=0.5, sigma2_g=0.25 - 1e-8, delta=1e-8, clip_c=1.5, alpha_s=0.5, beta=2.0, eps=0.2)
    ro = oracle.Rollout(1, seed=0)
    for step, g, gt, z, thr, stop in rows:
        out = _forced(ro, x, values[int(step)], p, tokens[int(step)])
        assert out.token == tokens[int(step)]
        assert abs(out.g - g) < 1e-12 and abs(out.g_tilde - gt) < 1e-9
        assert abs(out.z - z) < 1e-9 and abs(out.threshold - thr) < 1e-12
        assert out.stop == int(stop)
    st = ro.states[0]
    assert st.status == oracle.STOPPED and st.t_stop == 2 and st.t == 3   # stop-step token is kept
    # a finished trajectory is not advanced any further
    again = _forced(ro, x, 0.1, p, 1)
    assert again.token == -1 and again.stop == 0 and ro.states[0].t == 3


def test_identity_normalisation_and_clip():
    x = np.array([[2.0, 0.0, -1.0, -6.0]])
    p = oracle.make_params(mu_g=0.0, sigma2_g=1.0, delta=0.0, clip_c=1e30, alpha_s=0.0, warmup_complete=0)
    out = _forced(oracle.Rollout(1, 0), x, 0.0, p, 2)
    assert out.g == 3.0 and out.g_tilde == 3.0 and out.z == 3.0            # alpha_s = 0: z = g~
    p = oracle.make_params(mu_g=1.0, sigma2_g=3.0, delta=1.0, clip_c=2.5, alpha_s=0.0, warmup_complete=0)
    assert _forced(oracle.Rollout(1, 0), x, 0.0, p, 2).g_tilde == (3.0 - 1.0) / 2.0
    assert _forced(oracle.Rollout(1, 0), x, 0.0, p, 3).g_tilde == 2.5      # (8-1)/2 clipped from above
    p = oracle.make_params(mu_g=9.0, sigma2_g=1.0, delta=0.0, clip_c=2.5, alpha_s=0.0, warmup_complete=0)
    assert _forced(oracle.Rollout(1, 0), x, 0.0, p, 0).g_tilde == -2.5     # (0-9)/1 clipped from below


def test_smoothing_closed_form_and_bound():
    # constant g~ => z_t = g~ (1 - alpha^t); |z_t| <= c (1 - alpha^t)
    x = np.array([[1.0, 0.0, -2.0]])
    alpha, c = 0.9, 10.0
    p = oracle.make_params(mu_g=0.25, sigma2_g=0.5, delta=0.0, clip_c=c, alpha_s=alpha, warmup_complete=0)
    ro = oracle.Rollout(1, 0)
    gt = (3.0 - 0.25) / math.sqrt(0.5)
    for t in range(1, 60):
        out = _forced(ro, x, 0.0, p, 2)
        assert abs(out.z - gt * (1 - alpha**t)) < 1e-12
        assert abs(out.z) <= c * (1 - alpha**t) + 1e-15
    assert ro.states[0].n_tokens == 59
    assert abs(ro.states[0].sum_g - 59 * 3.0) < 1e-12 and abs(ro.states[0].sum_g2 - 59 * 9.0) < 1e-12


def test_stop_rule_strictness_gate_and_floor():
    x = np.array([[2.0, 0.5]])
    base = dict(mu_g=0.0, sigma2_g=1.0, delta=0.0, clip_c=100.0, alpha_s=0.0)   # z = g = 1.5 for token 1
    # z == threshold exactly: strict '>' does not fire
    assert _forced(oracle.Rollout(1, 0), x, 1.0, oracle.make_params(beta=1.5, eps=0.2, **base), 1).stop == 0
    assert _forced(oracle.Rollout(1, 0), x, 1.0, oracle.make_params(beta=1.4999, eps=0.2, **base), 1).stop == 1
    # value below the floor: threshold is beta * eps
    out = _forced(oracle.Rollout(1, 0), x, -0.7, oracle.make_params(beta=5.0, eps=0.2, **base), 1)
    assert out.threshold == 1.0 and out.stop == 1
    # warm-up gates the test but not the statistic
    ro = oracle.Rollout(1, 0)
    out = _forced(ro, x, 0.0, oracle.make_params(beta=0.1, eps=0.2, warmup_complete=0, **base), 1)
    assert out.stop == 0 and out.z == 1.5 and ro.states[0].status == oracle.ACTIVE
    # NaN value estimate never fires
    assert _forced(oracle.Rollout(1, 0), x, float("nan"), oracle.make_params(beta=0.1, **base), 1).stop == 0


def test_stop_is_monotone_in_beta_and_tokens_do_not_depend_on_it():
    rng = _rng(10)
    B, V, T = 6, 400, 60
    logits = rng.normal(0, 2.0, size=(T, B, V))
    values = rng.uniform(0.1, 0.9, size=(T, B))

    def run(beta):
        ro = oracle.Rollout(B, seed=4)
        p = oracle.make_params(mu_g=1.0, sigma2_g=1.0, beta=beta, t_max=T)
        toks = np.full((T, B), -1)
        for t in range(T):
            outs = ro.step(logits[t], values[t], p)
            toks[t] = [o.token for o in outs]
        stop_at = [ro.states[i].t_stop if ro.states[i].status == oracle.STOPPED else T for i in range(B)]
        return toks, stop_at

    toks_lo, stop_lo = run(0.5)
    toks_hi, stop_hi = run(2.0)
    assert any(s < T for s in stop_lo)
    for i in range(B):
        assert stop_hi[i] >= stop_lo[i]
        n = stop_lo[i] + 1 if stop_lo[i] < T else T
        assert np.array_equal(toks_lo[:n, i], toks_hi[:n, i])


def test_eos_wins_over_stop_and_horizon_ends_the_trajectory():
    x = np.array([[2.0, 0.5]])
    base = dict(mu_g=0.0, sigma2_g=1.0, delta=0.0, clip_c=100.0, alpha_s=0.0, beta=0.1)
    ro = oracle.Rollout(1, 0)
    out = _forced(ro, x, 1.0, oracle.make_params(eos_token=1, **base), 1)
    assert out.stop == 0 and ro.states[0].status == oracle.EOS and ro.states[0].t == 1
    ro = oracle.Rollout(1, 0)
    p = oracle.make_params(t_max=3, warmup_complete=0, **base)
    for t in range(3):
        out = _forced(ro, x, 1.0, p, 0)
        assert out.stop == 0
        assert ro.states[0].status == (oracle.TMAX if t == 2 else oracle.ACTIVE)
    assert ro.states[0].t == 3 and ro.states[0].t_stop == -1


def test_row_ids_route_rows_to_slots():
    x = _peaked_logits(_rng(12), 3, 200)
    p = oracle.make_params(warmup_complete=0)
    full = oracle.Rollout(8, seed=1)
    outs = full.step(x, np.zeros(3), p, row_ids=[6, 0, 3])
    for row, slot in enumerate([6, 0, 3]):
        single = oracle.Rollout(8, seed=1)
        o = single.step(x[row:row + 1], [0.0], p, row_ids=[slot])[0]
        assert o.token == outs[row].token and o.z == outs[row].z
        assert full.states[slot].t == 1
    assert full.states[1].t == 0


def test_float32_entry_point_agrees():
    x = _peaked_logits(_rng(13), 5, 700).astype(np.float32)
    p = oracle.make_params(temperature=0.6, sampler=oracle.SAMPLER_HIER)
    a = oracle.Rollout(5, seed=8).step(x, np.full(5, 0.4), p)
    b = oracle.Rollout(5, seed=8).step_f32(x, np.full(5, 0.4), p, n_threads=3)
    for r in range(5):
        assert (a[r].token, a[r].stop) == (b[r].token, b[r].stop)
        assert a[r].z == b[r].z and a[r].logp == b[r].logp


# --------------------------------------------------------------------------- batch boundary (Eq. 7-8, 12)


def test_end_batch_matches_numpy_statistics_and_the_controller_formula():
    # every regret value of a small rollout is collected by hand; the EMA targets are numpy's mean / population variance
    rng = _rng(40)
    B, V, T = 6, 400, 9
    ro = oracle.Rollout(B, seed=3)
    p = oracle.make_params(temperature=1.0, mu_g=0.5, sigma2_g=1.0, alpha_s=0.5, beta=0.8, eps=0.2, t_max=T)
    gs, stopped = [], set()
    for t in range(T):
        x = _peaked_logits(rng, B, V)
        outs = ro.step(x, rng.uniform(0.0, 1.0, size=B), p)
        for r in range(B):
            if outs[r].token >= 0:
                gs.append(outs[r].g)
            if outs[r].stop:
                stopped.add(r)
    assert 0 < len(stopped) < B
    gs = np.array(gs)
    mu, s2, beta, st = ro.end_batch(2.0, 3.0, 7.0, alpha_ema=0.9, eta_beta=0.1, tau=0.25, beta_min=0.0, beta_max=10.0)
    assert st[3] == len(gs) and st[4] == B and st[5] == len(stopped)
    assert abs(st[0] - gs.mean()) < 1e-12 and abs(st[1] - gs.var()) < 1e-12
    assert abs(mu - (0.9 * 2.0 + 0.1 * gs.mean())) < 1e-12
    assert abs(s2 - (0.9 * 3.0 + 0.1 * gs.var())) < 1e-12
    assert abs(beta - (7.0 + 0.1 * (len(stopped) / B - 0.25))) < 1e-12
    # first update: the statistics are the batch's own; the clip bounds hold
    mu, s2, beta, _ = ro.end_batch(2.0, 3.0, 7.0, eta_beta=100.0, tau=0.0, beta_max=7.5, first_update=True)
    assert abs(mu - gs.mean()) < 1e-12 and abs(s2 - gs.var()) < 1e-12 and beta == 7.5
    _, _, beta, _ = ro.end_batch(2.0, 3.0, 7.0, eta_beta=100.0, tau=1.0, beta_min=0.0)
    assert beta == 0.0
    # stop rate on target leaves beta alone; an empty batch changes nothing
    _, _, beta, _ = ro.end_batch(2.0, 3.0, 7.0, tau=len(stopped) / B)
    assert beta == 7.0
    assert oracle.Rollout(4, seed=1).end_batch(2.0, 3.0, 7.0)[:3] == (2.0, 3.0, 7.0)


# --------------------------------------------------------------------------- the ablation's stop rules (Sec. 6)


def _rollout_with(mode_kwargs, T=12, B=5, V=300, seed=50, values=None):
    rng = _rng(seed)
    ro = oracle.Rollout(B, seed=9)
    kw = dict(temperature=1.0, mu_g=0.5, sigma2_g=1.0, alpha_s=0.5, beta=0.8, eps=0.2, t_max=10**6)
    kw.update(mode_kwargs)
    p = oracle.make_params(**kw)
    hist = []
    for t in range(T):
        x = _peaked_logits(rng, B, V)
        v = rng.uniform(0.0, 1.0, size=B) if values is None else values[t]
        outs = ro.step(x, v, p)
        hist.append([(o.token, o.stop, o.z, float(v[r])) for r, o in enumerate(outs)])
    return ro, hist


def test_value_only_and_regret_only_rules_fire_exactly_on_their_inequality():
    for mode, tau in ((oracle.STOP_VALUE_ONLY, 0.3), (oracle.STOP_REGRET_ONLY, 0.4)):
        ro, hist = _rollout_with(dict(stop_mode=mode, tau=tau))
        fired = 0
        for step in hist:
            for tok, stop, z, v in step:
                if tok < 0:
                    continue                      # already ended
                want = (v < tau) if mode == oracle.STOP_VALUE_ONLY else (z > tau)
                assert bool(stop) == want
                fired += int(stop)
        assert fired > 0
    # the warm-up gate applies to every rule
    _, hist = _rollout_with(dict(stop_mode=oracle.STOP_VALUE_ONLY, tau=2.0, warmup_complete=0))
    assert not any(stop for step in hist for _, stop, _, _ in step)


def test_random_rule_has_the_requested_rate_and_does_not_disturb_the_sampler():
    _, base = _rollout_with(dict(stop_mode=oracle.STOP_ESPO, beta=1e9), T=6)
    _, never = _rollout_with(dict(stop_mode=oracle.STOP_RANDOM, p_random=0.0), T=6)
    _, always = _rollout_with(dict(stop_mode=oracle.STOP_RANDOM, p_random=1.0), T=6)
    assert [[t for t, _, _, _ in s] for s in base] == [[t for t, _, _, _ in s] for s in never]   # same tokens
    assert all(stop for _, stop, _, _ in always[0]) and all(t == -1 for t, _, _, _ in always[1])
    # rate: 4000 independent (slot, step 0) draws at p = 0.25
    B = 4000
    ro = oracle.Rollout(B, seed=123)
    p = oracle.make_params(stop_mode=oracle.STOP_RANDOM, p_random=0.25)
    outs = ro.step(np.zeros((B, 8)), np.zeros(B), p)
    k = sum(o.stop for o in outs)
    assert abs(k - 1000) < 5 * math.sqrt(B * 0.25 * 0.75)


def test_shadow_mode_records_the_first_firing_step_and_keeps_decoding():
    T = 12
    ro_a, hist_a = _rollout_with(dict(stop_mode=oracle.STOP_ESPO), T=T)
    ro_s, hist_s = _rollout_with(dict(stop_mode=oracle.STOP_ESPO, shadow=1), T=T)
    n_stopped = 0
    for r in range(ro_a.capacity):
        a, s = ro_a.states[r], ro_s.states[r]
        assert s.status == oracle.ACTIVE and s.t == T            # never ended
        assert s.t_stop == a.t_stop                               # same first firing step (or none)
        n_stopped += int(a.t_stop >= 0)
        upto = T if a.t_stop < 0 else a.t_stop + 1
        assert [h[r][0] for h in hist_s[:upto]] == [h[r][0] for h in hist_a[:upto]]   # same tokens until then
    assert 0 < n_stopped
    assert not any(stop for step in hist_s for _, stop, _, _ in step)


# --------------------------------------------------------------------------- policy entropy (analysis section)


def test_entropy_matches_library_and_closed_forms():
    rng = _rng(60)
    V = 700
    x = _peaked_logits(rng, 3, V)
    x[1, :] = 1.25                      # uniform: H = log V
    x[2, :] = -np.inf; x[2, 5] = 0.0    # one admissible id: H = 0
    for T in (1.0, 0.6):
        outs = oracle.Rollout(3, seed=2).step(x, np.zeros(3), oracle.make_params(temperature=T, warmup_complete=0))
        assert abs(outs[0].entropy - stats.entropy(special.softmax(x[0] / T))) < 1e-10
        assert abs(outs[1].entropy - math.log(V)) < 1e-10
        assert outs[2].entropy == 0.0 and outs[2].token == 5


# --------------------------------------------------------------------------- filtered sampling (top-p / top-k)


def _support_by_brute_force(x, temperature, top_p, top_k):
    """Token a stays iff the tokens strictly more probable than a weigh less than top_p and number fewer than top_k."""
    q = special.softmax(np.asarray(x, dtype=np.float64) / temperature)
    keep = np.zeros(q.size, dtype=bool)
    for a in range(q.size):
        above = x > x[a]
        keep[a] = (top_p >= 1.0 or q[above].sum() < top_p) and (top_k <= 0 or int(above.sum()) < top_k) and np.isfinite(x[a])
    return q, keep


@pytest.mark.parametrize("top_p,top_k", [(0.7, 0), (1.0, 3), (0.9, 4), (0.35, 0), (0.999, 0)])
def test_filtered_sampler_draws_from_the_renormalised_support(top_p, top_k):
    # ties on purpose: ids 1 and 6 share a logit, so do 2 and 7 -- equal tokens stay or go together
    x = np.array([1.2, 0.4, 0.0, 2.0, -1.5, 0.7, 0.4, 0.0, -np.inf, 1.9])
    temperature = 0.8
    q, keep = _support_by_brute_force(x, temperature, top_p, top_k)
    slots, steps = 64, 1500
    ro = oracle.Rollout(slots, seed=21)
    p = oracle.make_params(temperature=temperature, sampler=oracle.SAMPLER_FLAT, warmup_complete=0, t_max=10**9,
                           top_p=top_p, top_k=top_k)
    rows = np.tile(x, (slots, 1))
    counts = np.zeros(x.size, dtype=np.int64)
    for _ in range(steps):
        for o in ro.step(rows, np.zeros(slots), p, n_threads=8):
            counts[o.token] += 1
            assert o.kept == int(keep.sum())
            want_logp = np.log(q[o.token] / q[keep].sum())
            assert abs(o.logp - want_logp) < 1e-12 and abs(o.g - (x.max() - x[o.token]) / temperature) < 1e-12
    assert counts[~keep].sum() == 0                                   # nothing outside the support is ever drawn
    if keep.sum() > 1:
        chi2, pval = stats.chisquare(counts[keep], q[keep] / q[keep].sum() * counts.sum())
        assert pval > 1e-3, (chi2, pval)
    if (top_p, top_k) == (0.7, 0):
        assert list(np.nonzero(keep)[0]) == [0, 3, 9]                 # 0.37 + 0.33 < 0.7 <= 0.37 + 0.33 + 0.14
    if (top_p, top_k) == (1.0, 3):
        assert list(np.nonzero(keep)[0]) == [0, 3, 9]
    if (top_p, top_k) == (0.9, 4):
        assert list(np.nonzero(keep)[0]) == [0, 3, 5, 9]


def test_filters_that_keep_everything_change_nothing_and_top_k_one_is_the_argmax():
    rng = np.random.default_rng(3)
    x = rng.normal(0, 2, size=(6, 300))
    base = oracle.Rollout(6, seed=9).step(x, np.zeros(6), oracle.make_params(sampler=oracle.SAMPLER_FLAT))
    same = oracle.Rollout(6, seed=9).step(x, np.zeros(6), oracle.make_params(sampler=oracle.SAMPLER_FLAT, top_p=1.0, top_k=0))
    wide = oracle.Rollout(6, seed=9).step(x, np.zeros(6), oracle.make_params(sampler=oracle.SAMPLER_FLAT, top_p=1.0, top_k=300))
    one = oracle.Rollout(6, seed=9).step(x, np.zeros(6), oracle.make_params(sampler=oracle.SAMPLER_FLAT, top_k=1))
    tiny = oracle.Rollout(6, seed=9).step(x, np.zeros(6), oracle.make_params(sampler=oracle.SAMPLER_FLAT, top_p=1e-9))
    for r in range(6):
        assert base[r].token == same[r].token == wide[r].token and abs(base[r].logp - wide[r].logp) < 1e-12
        assert one[r].token == tiny[r].token == int(np.argmax(x[r])) and one[r].kept == 1
        assert abs(one[r].logp) < 1e-12 and one[r].g == 0.0           # the support is one token: probability 1, no regret
        assert np.isinf(one[r].filter_margin) and tiny[r].filter_margin < 1.0


def test_filter_margin_is_the_distance_of_the_nearest_decision_from_flipping():
    x = np.log(np.array([0.5, 0.3, 0.15, 0.05]))
    o = oracle.Rollout(1, seed=1).step(x[None, :], np.zeros(1), oracle.make_params(sampler=oracle.SAMPLER_FLAT, top_p=0.82))[0]
    # masses above the four tokens: 0, 0.5, 0.8, 0.95 -> kept 0, 1, 2; nearest decision: |0.8 - 0.82|
    assert o.kept == 3 and abs(o.filter_margin - 0.02) < 1e-12
