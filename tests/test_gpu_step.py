"""GPU parity of espo_step against the CPU oracle, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_29860_b200 as espo
from paper_2605_29860_b200 import synth
from parity_util import ParityRun, close

pytestmark = pytest.mark.gpu

SAMPLERS = [espo.ESPO_SAMPLER_HIER, espo.ESPO_SAMPLER_FLAT]


def _dev(a, dtype=None):
    t = torch.as_tensor(a)
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


# ---------------------------------------------------------------------------- tiny brute force


@pytest.mark.parametrize("sampler", SAMPLERS)
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_brute_force_v8_t4(sampler, dtype):
    rng = np.random.default_rng(0)
    B, V, T = 5, 8, 4
    p = espo.make_params(temperature=0.9, mu_g=0.4, sigma2_g=0.6, alpha_s=0.5, beta=1.0, eps=0.2, sampler=sampler)
    run = ParityRun(B, V, p, seed=123, batch_id=3)
    for t in range(T):
        x = _dev(rng.normal(0, 1.5, size=(B, V)), dtype)
        v = _dev(rng.uniform(-0.2, 0.9, size=B), torch.float32)
        run.step(x, v)
    assert run.stats.row_steps >= B
    run.close()


# ---------------------------------------------------------------------------- config 1 (tiny)


@pytest.mark.parametrize("sampler", SAMPLERS)
def test_tiny_config_every_row_every_step(sampler):
    # B=8, V=32000, fp32 logits N(0,2) + 1-3 boosted ids (+6..+12), temperature 1, V_phi random walk
    B, V = 8, 32000
    T = 256 if sampler == espo.ESPO_SAMPLER_HIER else 48
    # mu_g, sigma2_g: mean and variance of g measured on this input recipe (what the batch EMA would hold)
    p = espo.make_params(temperature=1.0, mu_g=4.4, sigma2_g=11.0, alpha_s=0.9, beta=1.5, eps=0.2, t_max=T,
                         sampler=sampler)
    vals = synth.value_walk(B, T, seed=0)
    run = ParityRun(B, V, p, seed=0)
    for t in range(T):
        x = synth.logits_batch(B, V, dtype=torch.float32, sd=2.0, n_peaks=3, peak_lo=6.0, peak_hi=12.0, zipf=False,
                               seed=1000 + t)
        run.step(x, vals[t].contiguous())
    st = run.stats
    assert st.row_steps > B * 40
    assert st.token_ties <= max(2, st.row_steps // 200), st
    if sampler == espo.ESPO_SAMPLER_HIER:
        assert st.stops >= 2 and st.tmax >= 2, st
    run.close()


# ---------------------------------------------------------------------------- config 2 (Qwen-7B-shaped)


@pytest.mark.parametrize("sampler", SAMPLERS)
def test_qwen_shaped_rows_with_failure_point(sampler):
    # B=64, V=152064, bf16 N(0,3) + 5 Zipf peaks, temperature 0.6, bf16 values; the peak ids are demoted
    # after an injected failure step so the regret rises and the rule fires.  The oracle follows 8 rows.
    B, V = 64, 152064
    T = 14 if sampler == espo.ESPO_SAMPLER_HIER else 5
    fail_at = torch.randint(2, 6, (B,), generator=torch.Generator().manual_seed(5))
    p = espo.make_params(temperature=0.6, mu_g=0.5, sigma2_g=1.0, alpha_s=0.9, beta=3.0, eps=0.2, sampler=sampler)
    vals = synth.value_walk(B, T, seed=2, dtype=torch.bfloat16)
    check = [0, 7, 13, 21, 34, 42, 55, 63]
    run = ParityRun(B, V, p, seed=42, batch_id=1, check_slots=check)
    for t in range(T):
        x = synth.logits_batch(B, V, dtype=torch.bfloat16, sd=3.0, seed=77 + t, demote_rows=(fail_at <= t))
        run.step(x, vals[t].contiguous())
    assert run.stats.row_steps >= len(check) * 3
    if sampler == espo.ESPO_SAMPLER_HIER:
        assert run.stats.stops >= 1
    run.close()


# ---------------------------------------------------------------------------- shapes and layouts


@pytest.mark.parametrize("sampler", SAMPLERS)
@pytest.mark.parametrize("V,dtype", [(1, torch.float32), (7, torch.bfloat16), (31, torch.float32),
                                     (33, torch.bfloat16), (1000, torch.bfloat16), (1024, torch.float32),
                                     (1025, torch.bfloat16), (8200, torch.float32), (8193, torch.bfloat16),
                                     (20011, torch.float32), (17000, torch.bfloat16)])
def test_ragged_vocab_sizes(V, dtype, sampler):
    rng = np.random.default_rng(V)
    B = 3
    p = espo.make_params(temperature=1.3, mu_g=1.0, sigma2_g=2.0, beta=1.5, sampler=sampler)
    run = ParityRun(B, V, p, seed=9)
    for t in range(3):
        x = _dev(rng.normal(0, 2.0, size=(B, V)), dtype)
        run.step(x, _dev(rng.uniform(0, 1, size=B), torch.float32))
    assert run.stats.row_steps == 3 * B or run.stats.stops > 0
    run.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_row_stride_row_ids_and_unaligned_base(dtype):
    rng = np.random.default_rng(3)
    cap, n, V = 16, 6, 5000
    p = espo.make_params(temperature=0.8, mu_g=1.0, sigma2_g=2.0, beta=50.0)
    ids = torch.tensor([11, 2, 7, 0, 15, 4], dtype=torch.int32).cuda()
    for shift in (0, 1):           # shift 1 breaks the 16-byte alignment -> element-wise loader
        run = ParityRun(cap, V, p, seed=31)
        for t in range(3):
            wide = _dev(rng.normal(0, 2.0, size=(n, V + 24 + shift)), dtype)
            x = wide[:, shift:shift + V]
            assert x.stride(0) == V + 24 + shift
            run.step(x, _dev(rng.uniform(0, 1, size=n), torch.float32), row_ids=ids)
        assert run.stats.row_steps == 3 * n
        t_host = run.view["t"].cpu().numpy()
        assert set(np.nonzero(t_host)[0]) == set(ids.cpu().tolist())
        run.close()


def test_results_do_not_depend_on_launch_shape_and_repeat_bit_exactly():
    B, V = 37, 152064
    x = synth.logits_batch(B, V, dtype=torch.bfloat16, seed=8)
    v = torch.rand(B, device="cuda")
    outs = []
    for warps, stages, ctas in [(0, 0, 0), (0, 0, 0), (31, 2, 1), (8, 4, 2), (5, 3, 3), (1, 12, 1), (15, 1, 2)]:
        for sampler in SAMPLERS:
            p = espo.make_params(temperature=1.0, mu_g=1.0, sigma2_g=2.0, beta=2.0, sampler=sampler)
            st = espo.espo_init_state(B, V, seed=5)
            espo.espo_set_launch_config(st, warps, stages, ctas)
            tok = torch.empty(B, dtype=torch.int32, device="cuda")
            stop = torch.empty(B, dtype=torch.uint8, device="cuda")
            for _ in range(2):
                espo.espo_step(x, v, st, p, tok, stop)
            view = espo.espo_state_view(st)
            outs.append((sampler, tok.cpu(), stop.cpu(), view["z"].cpu().clone(), view["logp"].cpu().clone()))
            assert espo.espo_state_status(st) == 0
            espo.espo_free_state(st)
    for sampler in SAMPLERS:
        group = [o for o in outs if o[0] == sampler]
        for o in group[1:]:
            for a, b in zip(o[1:], group[0][1:]):
                assert torch.equal(a, b)


def test_dependent_launch_changes_nothing():
    # espo_set_dependent_launch only lets the step kernel be set up early; several steps back to back (each the
    # programmatic dependent of the one before) must leave exactly what plain launches leave
    B, V, T = 300, 152064, 4
    p = espo.make_params(temperature=1.0, mu_g=1.0, sigma2_g=2.0, beta=2.0)
    xs = [synth.logits_batch(B, V, dtype=torch.bfloat16, seed=60 + t) for t in range(T)]
    v = torch.rand(B, device="cuda")
    outs = []
    for flag in (False, True):
        st = espo.espo_init_state(B, V, seed=11)
        espo.espo_set_dependent_launch(st, flag)
        toks = [torch.empty(B, dtype=torch.int32, device="cuda") for _ in range(T)]
        stop = torch.empty(B, dtype=torch.uint8, device="cuda")
        for t in range(T):
            espo.espo_step(xs[t], v, st, p, toks[t], stop)
        torch.cuda.synchronize()
        view = espo.espo_state_view(st)
        outs.append(([t.cpu() for t in toks], view["z"].cpu().clone(), view["logp"].cpu().clone(), view["t"].cpu().clone()))
        assert espo.espo_state_status(st) == 0
        espo.espo_free_state(st)
    for a, b in zip(outs[0][0], outs[1][0]):
        assert torch.equal(a, b)
    assert all(torch.equal(a, b) for a, b in zip(outs[0][1:], outs[1][1:]))
    assert int(outs[0][3].min()) >= 1


# ---------------------------------------------------------------------------- special rows and rules


@pytest.mark.parametrize("sampler", SAMPLERS)
def test_masked_ids_and_unusable_rows(sampler):
    rng = np.random.default_rng(4)
    B, V = 6, 3000
    x = rng.normal(0, 2.0, size=(B, V)).astype(np.float32)
    x[0, ::2] = -np.inf                 # masked ids never win
    x[1, :] = -np.inf                   # nothing finite: unusable
    x[2, 1234] = np.nan                 # NaN: unusable
    x[3, 77] = np.inf                   # +inf: unusable
    x[4, :2048] = -np.inf               # whole blocks masked
    p = espo.make_params(sampler=sampler, mu_g=1.0, sigma2_g=2.0, beta=100.0)
    run = ParityRun(B, V, p, seed=6)
    tok, _ = run.step(_dev(x), torch.full((B,), 0.5, device="cuda"))
    assert tok[0] % 2 == 1 and tok[4] >= 2048
    assert list(run.view["status"].cpu().numpy()) == [0, 4, 4, 4, 0, 0]
    assert espo.espo_state_status(run.state) & espo.ESPO_DEV_BAD_ROW
    tok, stp = run.step(_dev(x), torch.full((B,), 0.5, device="cuda"))   # dead rows are now ignored
    assert list(tok[1:4]) == [-1, -1, -1] and not stp.any()
    run.close()


@pytest.mark.parametrize("sampler", SAMPLERS)
def test_greedy_eos_horizon_warmup_and_nan_value(sampler):
    rng = np.random.default_rng(5)
    B, V = 4, 2500
    x = rng.normal(0, 1.0, size=(B, V)).astype(np.float32)
    x[0, 100] = x[0, 2000] = 9.0                 # tie: the first maximum wins under greedy decoding
    xg = _dev(x)
    # greedy
    run = ParityRun(B, V, espo.make_params(temperature=0.0, sampler=sampler, beta=100.0), seed=1)
    tok, _ = run.step(xg, torch.zeros(B, device="cuda"))
    assert tok[0] == 100 and list(tok) == list(x.argmax(axis=1))
    run.close()
    # EOS beats a stop on the same step; horizon; warm-up gate; NaN value never stops
    x2 = np.full((B, V), -30.0, dtype=np.float32)
    x2[:, 5] = 60.0                                # token 5 with certainty (a +90 lead); g = 0, so the
                                                   # regret signal comes from mu_g < 0: g~ = (0+5)/1
    base = dict(mu_g=-5.0, sigma2_g=1.0, alpha_s=0.0, beta=0.5, eps=0.2, sampler=sampler)
    run = ParityRun(B, V, espo.make_params(eos_token=5, **base), seed=2)
    tok, stp = run.step(_dev(x2), torch.full((B,), 0.3, device="cuda"))
    assert list(tok) == [5] * B and not stp.any()
    assert list(run.view["status"].cpu().numpy()) == [espo.ESPO_ROW_EOS] * B
    run.close()
    run = ParityRun(B, V, espo.make_params(t_max=2, warmup_complete=0, **base), seed=2)
    for _ in range(2):
        tok, stp = run.step(_dev(x2), torch.full((B,), 0.3, device="cuda"))
        assert not stp.any()
    assert list(run.view["status"].cpu().numpy()) == [espo.ESPO_ROW_TMAX] * B
    assert float(run.view["z"][0]) == 5.0          # z ran during warm-up: (0+5)/1, alpha_s = 0
    run.close()
    run = ParityRun(B, V, espo.make_params(**base), seed=2)
    vals = torch.tensor([0.3, float("nan"), 0.3, float("nan")], device="cuda")
    tok, stp = run.step(_dev(x2), vals)
    assert list(stp) == [1, 0, 1, 0]
    assert espo.espo_state_status(run.state) & espo.ESPO_DEV_NAN_VALUE
    assert list(run.view["t_stop"].cpu().numpy()) == [0, -1, 0, -1]
    run.close()


def test_compaction_and_shrinking_active_set():
    # rows leave the active set as they stop; the next step runs on the compacted rows only
    B, V, T = 48, 9000, 12
    p = espo.make_params(temperature=1.0, mu_g=0.5, sigma2_g=1.0, alpha_s=0.6, beta=1.0, eps=0.2)
    run = ParityRun(B, V, p, seed=10)
    ids = torch.arange(B, dtype=torch.int32, device="cuda")
    n_act = torch.zeros(1, dtype=torch.int32, device="cuda")
    n = B
    seen_shrink = False
    for t in range(T):
        x = synth.logits_batch(B, V, dtype=torch.bfloat16, sd=2.5, seed=300 + t)
        rows = ids[:n].long()
        vals = torch.rand(B, device="cuda", generator=torch.Generator("cuda").manual_seed(t))
        run.step(x[rows].contiguous(), vals[rows].contiguous(), row_ids=ids[:n].contiguous())
        espo.espo_compact_active(run.state, ids, n_act)
        status = run.view["status"].cpu().numpy()
        want = np.nonzero(status == espo.ESPO_ROW_ACTIVE)[0]
        n = int(n_act.item())
        assert n == len(want) and np.array_equal(ids[:n].cpu().numpy(), want)
        seen_shrink |= n < B
        if n == 0:
            break
    assert seen_shrink
    run.close()


@pytest.mark.parametrize("mode_kw", [dict(stop_mode=espo.ESPO_STOP_VALUE_ONLY, tau=0.3),
                                     dict(stop_mode=espo.ESPO_STOP_REGRET_ONLY, tau=0.35),
                                     dict(stop_mode=espo.ESPO_STOP_RANDOM, p_random=0.2),
                                     dict(stop_mode=espo.ESPO_STOP_ESPO, shadow=1),
                                     dict(stop_mode=espo.ESPO_STOP_RANDOM, p_random=0.3, shadow=1, warmup_complete=0)])
def test_ablation_stop_rules_and_shadow_mode(mode_kw):
    # the replacements of Eq. 11 studied in the ablation (value only, regret only, random) and the shadow mode
    B, V, T = 24, 5000, 10
    kw = dict(temperature=1.0, mu_g=0.5, sigma2_g=1.0, alpha_s=0.6, beta=1.0, eps=0.2)
    kw.update(mode_kw)
    p = espo.make_params(**kw)
    run = ParityRun(B, V, p, seed=33)
    for t in range(T):
        x = synth.logits_batch(B, V, dtype=torch.float32, sd=2.5, seed=900 + t)
        vals = torch.rand(B, device="cuda", generator=torch.Generator("cuda").manual_seed(70 + t))
        run.step(x, vals)
    st = run.stats
    t_stop = run.view["t_stop"].cpu().numpy()
    status = run.view["status"].cpu().numpy()
    if mode_kw.get("warmup_complete", 1) == 0:
        assert st.stops == 0 and (t_stop == -1).all()
    elif mode_kw.get("shadow"):
        assert st.stops == 0 and (status == espo.ESPO_ROW_ACTIVE).all() and (t_stop >= 0).any()
    else:
        assert st.stops > 0 and (status == espo.ESPO_ROW_STOPPED).sum() == st.stops
    bad = espo.make_params(stop_mode=9)
    with pytest.raises(espo.EspoError) as e:
        espo.espo_step(x, vals, run.state, bad, run.tokens, run.stop)
    assert e.value.code == espo.ESPO_ERR_BAD_PARAM
    run.close()


@pytest.mark.parametrize("V,dtype,temperature", [(152064, torch.bfloat16, 1.0), (152064, torch.bfloat16, 0.6),
                                                   (5000, torch.float32, 1.3), (1025, torch.bfloat16, 1.0)])
def test_policy_entropy_in_the_same_pass(V, dtype, temperature):
    B, T = 6, 3
    p = espo.make_params(temperature=temperature, mu_g=1.0, sigma2_g=2.0, beta=50.0, want_entropy=1)
    run = ParityRun(B, V, p, seed=17)
    for t in range(T):
        x = synth.logits_batch(B, V, dtype=dtype, sd=3.0 if t else 0.5, seed=40 + t)   # flat rows, then peaked ones
        if t == 1:
            x[0, : V // 2] = float("-inf")        # masked ids contribute nothing
        run.step(x, torch.full((B,), 0.5, device="cuda"))
    h = run.view["entropy"].cpu().numpy()
    assert (h >= 0).all() and (h <= np.log(V) + 1e-4).all()
    assert abs(float(run.view["sum_h"][1]) - sum_h_of(run, 1)) < 1e-3
    with pytest.raises(espo.EspoError) as e:
        espo.espo_step(x, torch.zeros(B, device="cuda"), run.state,
                       espo.make_params(want_entropy=1, sampler=espo.ESPO_SAMPLER_FLAT), run.tokens, run.stop)
    assert e.value.code == espo.ESPO_ERR_BAD_PARAM
    run.close()


@pytest.mark.parametrize("sampler", SAMPLERS)
@pytest.mark.parametrize("temperature", [0.05, 0.2, 3.0, 10.0])
def test_temperatures_far_from_one(temperature, sampler):
    # At T = 0.05 a logit is scaled by 20/ln 2 before the exponential, so the rounding of that scale times a block's
    # maximum is of the order 1e-5 in log pi unless the kernel takes it out; at T = 10 the row is nearly flat.
    B, T = 12, 3
    for V, dtype in ((152064, torch.bfloat16), (32000, torch.float32), (1000, torch.bfloat16)):
        p = espo.make_params(temperature=temperature, mu_g=1.0, sigma2_g=4.0, beta=2.0, eps=0.1, t_max=6,
                             sampler=sampler, want_entropy=int(sampler == espo.ESPO_SAMPLER_HIER))
        run = ParityRun(B, V, p, seed=int(temperature * 100) + V)
        for t in range(T):
            run.step(synth.logits_batch(B, V, dtype=dtype, sd=3.0, seed=t + int(temperature * 10)),
                     torch.rand(B, device="cuda", generator=torch.Generator("cuda").manual_seed(V + t)))
        assert run.stats.token_ties <= 2, (V, run.stats)
        run.close()


@pytest.mark.parametrize("sampler", SAMPLERS)
@pytest.mark.parametrize("offset,scale", [(1000.0, 1.0), (-5000.0, 1.0), (30000.0, 1.0), (200.0, 10.0)])
def test_rows_at_a_large_offset_or_scale(offset, scale, sampler):
    # log-softmax does not change when a row is shifted; the kernel's scaled exponent offsets must not either
    B = 8
    for V, dtype in ((152064, torch.float32), (5000, torch.bfloat16)):
        p = espo.make_params(temperature=0.3, mu_g=1.0, sigma2_g=4.0, beta=2.0, eps=0.1, t_max=6, sampler=sampler,
                             want_entropy=int(sampler == espo.ESPO_SAMPLER_HIER))
        run = ParityRun(B, V, p, seed=V)
        for t in range(2):
            x = synth.logits_batch(B, V, dtype=torch.float32, sd=3.0, seed=t + 3)
            run.step((x * scale + offset).to(dtype),
                     torch.rand(B, device="cuda", generator=torch.Generator("cuda").manual_seed(t)))
        assert run.stats.token_ties <= 2, (V, run.stats)
        run.close()


def sum_h_of(run, slot):
    return float(sum(run.entropy_log[slot]))


def test_end_batch_updates_statistics_and_beta_like_the_oracle():
    # a short rollout in which some rows stop, then the batch-boundary update (Eq. 7-8, 12) on both sides
    B, V, T = 40, 6000, 10
    p = espo.make_params(temperature=1.0, mu_g=0.5, sigma2_g=1.0, alpha_s=0.6, beta=1.0, eps=0.2)
    run = ParityRun(B + 3, V, p, seed=21)            # three slots never take part
    for t in range(T):
        x = synth.logits_batch(B, V, dtype=torch.bfloat16, sd=2.5, seed=700 + t)
        vals = torch.rand(B, device="cuda", generator=torch.Generator("cuda").manual_seed(50 + t))
        run.step(x, vals)
    assert run.stats.stops > 0 and not run.dropped
    for first in (False, True):
        q = espo.make_params(mu_g=2.0, sigma2_g=3.0, beta=7.0)
        st = espo.espo_end_batch(run.state, q, alpha_ema=0.9, eta_beta=0.5, tau=0.25, beta_min=0.0, beta_max=7.2,
                                 first_update=first)
        mu, s2, beta, ost = run.ro.end_batch(2.0, 3.0, 7.0, alpha_ema=0.9, eta_beta=0.5, tau=0.25, beta_min=0.0,
                                             beta_max=7.2, first_update=first)
        assert close(q.mu_g, mu) and close(q.sigma2_g, s2) and close(q.beta, beta)
        assert close(st["mean_g"], ost[0]) and close(st["var_g"], ost[1]) and close(st["stop_rate"], ost[2])
        assert (st["tokens"], st["trajectories"], st["stopped"]) == (int(ost[3]), B, int(ost[5]))
    with pytest.raises(espo.EspoError) as e:
        espo.espo_end_batch(run.state, p, alpha_ema=1.5)
    assert e.value.code == espo.ESPO_ERR_BAD_PARAM
    run.close()


def test_end_batch_over_two_states_equals_the_oracle_over_all_trajectories():
    # the rollout batch split over two states (as over two GPUs); each gives its six statistics, the merge pools them
    V, T = 5000, 8
    p = espo.make_params(temperature=1.0, mu_g=0.5, sigma2_g=1.0, alpha_s=0.6, beta=1.0, eps=0.2)
    whole = oracle.Rollout(50, seed=0)               # stands for all trajectories; slots 0..29 and 30..49
    parts = []
    for lo, n, seed in ((0, 30, 41), (30, 20, 42)):
        run = ParityRun(n, V, p, seed=seed)
        for t in range(T):
            x = synth.logits_batch(n, V, dtype=torch.bfloat16, sd=2.5, seed=800 + 10 * lo + t)
            run.step(x, torch.rand(n, device="cuda", generator=torch.Generator("cuda").manual_seed(lo + t)))
        assert not run.dropped
        for s_ in range(n):
            whole.states[lo + s_] = run.ro.states[s_]
        scratch = espo.make_params(mu_g=2.0, sigma2_g=3.0, beta=7.0)
        parts.append(espo.espo_end_batch(run.state, scratch, alpha_ema=0.9, eta_beta=0.5, tau=0.25, beta_max=7.2))
        run.close()
    for first in (False, True):
        q = espo.make_params(mu_g=2.0, sigma2_g=3.0, beta=7.0)
        st = espo.espo_end_batch_merge(parts, q, alpha_ema=0.9, eta_beta=0.5, tau=0.25, beta_min=0.0, beta_max=7.2,
                                       first_update=first)
        mu, s2, beta, ost = whole.end_batch(2.0, 3.0, 7.0, alpha_ema=0.9, eta_beta=0.5, tau=0.25, beta_min=0.0,
                                            beta_max=7.2, first_update=first)
        assert close(q.mu_g, mu) and close(q.sigma2_g, s2) and close(q.beta, beta)
        assert close(st["mean_g"], ost[0]) and close(st["var_g"], ost[1]) and close(st["stop_rate"], ost[2])
        assert (st["tokens"], st["trajectories"], st["stopped"]) == (int(ost[3]), 50, int(ost[5]))


def test_reset_state_starts_a_new_batch():
    B, V = 4, 4096
    p = espo.make_params(mu_g=1.0, sigma2_g=2.0, beta=100.0)
    x = synth.logits_batch(B, V, dtype=torch.float32, seed=1)
    v = torch.full((B,), 0.5, device="cuda")
    run = ParityRun(B, V, p, seed=77, batch_id=0)
    tok0, _ = run.step(x, v)
    run.close()
    st = espo.espo_init_state(B, V, seed=77, batch_id=5)
    tok = torch.empty(B, dtype=torch.int32, device="cuda")
    stop = torch.empty(B, dtype=torch.uint8, device="cuda")
    espo.espo_step(x, v, st, p, tok, stop)
    espo.espo_reset_state(st, 0)
    view = espo.espo_state_view(st)
    assert int(view["t"].sum()) == 0 and float(view["z"].abs().sum()) == 0.0 and int(view["t_stop"][0]) == -1
    espo.espo_step(x, v, st, p, tok, stop)
    assert np.array_equal(tok.cpu().numpy(), tok0)     # same seed, batch 0, step 0 -> same draws
    espo.espo_free_state(st)


def test_argument_errors():
    B, V = 4, 1024
    st = espo.espo_init_state(B, V, seed=1)
    x = torch.zeros(B, V, device="cuda")
    v = torch.zeros(B, device="cuda")
    tok = torch.empty(B, dtype=torch.int32, device="cuda")
    stop = torch.empty(B, dtype=torch.uint8, device="cuda")
    good = espo.make_params()
    for bad in (espo.make_params(temperature=-1.0), espo.make_params(alpha_s=1.0), espo.make_params(clip_c=0.0),
                espo.make_params(sigma2_g=0.0, delta=0.0), espo.make_params(t_max=0), espo.make_params(sampler=7)):
        with pytest.raises(espo.EspoError) as e:
            espo.espo_step(x, v, st, bad, tok, stop)
        assert e.value.code == espo.ESPO_ERR_BAD_PARAM
    with pytest.raises(espo.EspoError) as e:
        espo.espo_step(torch.zeros(B + 1, V, device="cuda"), torch.zeros(B + 1, device="cuda"), st, good,
                       torch.empty(B + 1, dtype=torch.int32, device="cuda"),
                       torch.empty(B + 1, dtype=torch.uint8, device="cuda"))
    assert e.value.code == espo.ESPO_ERR_CAPACITY
    espo.espo_step(x, v, st, good, tok, stop, n_rows=0)             # no-op
    bad_ids = torch.tensor([0, 1, 99, -3], dtype=torch.int32, device="cuda")
    espo.espo_step(x, v, st, good, tok, stop, row_ids=bad_ids)      # reported, not trapped
    assert espo.espo_state_status(st) & espo.ESPO_DEV_BAD_SLOT
    assert list(tok.cpu().numpy()[2:]) == [-1, -1]
    espo.espo_free_state(st)


# ---------------------------------------------------------------------------- full size, bench launch shape


@pytest.mark.parametrize("B", [512, 256])
def test_full_size_rollout_batch_sampled_rows_and_invariants(B):
    # The benchmark's workload: B x 152064 bf16, temperature 1, hierarchical sampler, default launch
    # shape.  The oracle checks a sample of rows one by one; every row is held to the invariants.
    V = 152064
    p = espo.make_params(temperature=1.0, mu_g=1.0, sigma2_g=2.0, alpha_s=0.9, beta=7.0, eps=0.2)
    check = sorted(set(np.random.default_rng(B).integers(0, B, size=10).tolist()) | {0, B - 1})
    run = ParityRun(B, V, p, seed=2024, check_slots=check)
    vals = synth.value_walk(B, 2, seed=4, dtype=torch.bfloat16)
    for t in range(2):
        x = synth.logits_batch(B, V, dtype=torch.bfloat16, sd=3.0, seed=900 + t)
        tok, stp = run.step(x, vals[t].contiguous())
        view = {k: a.cpu().numpy() for k, a in run.view.items()}
        assert (tok >= 0).all() and (tok < V).all()
        assert (view["g"] >= 0).all() and (view["logp"] <= 1e-6).all()
        assert (np.abs(view["z"]) <= p.clip_c * (1 - p.alpha_s ** (t + 1)) + 1e-6).all()
        # the regret is exactly the logit gap of the sampled token
        rows = torch.arange(B, device="cuda")
        gap = (x.float().max(dim=1).values - x[rows, torch.as_tensor(tok, device="cuda").long()].float()).cpu().numpy()
        assert np.allclose(view["g"], gap, rtol=1e-6, atol=1e-6)
    assert run.stats.row_steps == 2 * len(check)
    assert espo.espo_state_status(run.state) == 0
    run.close()
