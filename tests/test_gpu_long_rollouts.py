"""GPU parity of whole rollouts at the stated lengths of the Qwen-shaped configurations (needs a B200).

The short tests of test_gpu_step.py never see a trajectory state that is thousands of steps old: z near its fixed
point, a step counter of several thousand in the Philox counter, fp64 sums over thousands of regrets, rows that leave
through compaction late in a rollout.  Here the oracle follows a few rows (rows are independent, so a subset is a
valid check) through every step of:
  * config 2: B=64, V=152064, bf16 logits ~N(0,3) + 5 Zipf peaks, temperature 0.6, bf16 value walk, T = 4096 steps,
    an injected failure point per trajectory in [512, 4096] after which the peaks are demoted;
  * config 3: B=512 (64 prompts x 8 samples), the same rows at temperature 1, T = 8192 (the paper's T_max), with
    espo_compact_active feeding the slot list of every step and logits generated for the active rows only.
As the paper's warm-up does, the statistics mu_g, sigma_g^2 of Eq. 9 come from a first batch in which stopping is
disabled, through espo_end_batch(first_update=1) (Eq. 7-8).
"""
import numpy as np
import pytest
import torch

import paper_2605_29860_b200 as espo
from paper_2605_29860_b200 import synth
from parity_util import ParityRun

pytestmark = pytest.mark.gpu

V = 152064


def _calibrate(B, temperature, sampler, steps=24):
    """mu_g, sigma_g^2 of healthy rows: a rollout batch with the stop test disabled, then the batch-boundary update."""
    p0 = espo.make_params(temperature=temperature, warmup_complete=0, t_max=1 << 20, sampler=sampler)
    st = espo.espo_init_state(B, V, seed=40)
    tok = torch.empty(B, dtype=torch.int32, device="cuda")
    stop = torch.empty(B, dtype=torch.uint8, device="cuda")
    v = torch.full((B,), 0.5, device="cuda")
    for t in range(steps):
        espo.espo_step(synth.logits_batch(B, V, dtype=torch.bfloat16, sd=3.0, seed=5000 + t), v, st, p0, tok, stop)
    q = espo.make_params()
    stats = espo.espo_end_batch(st, q, first_update=True)
    espo.espo_free_state(st)
    assert stats["tokens"] == B * steps and stats["stopped"] == 0
    return q.mu_g, q.sigma2_g


@pytest.mark.parametrize("sampler,T", [(espo.ESPO_SAMPLER_HIER, 4096), (espo.ESPO_SAMPLER_FLAT, 320)])
def test_config2_full_length(sampler, T):
    B = 64
    check = [0, 9, 18, 27, 36, 45, 54, 63]
    lo = 512 if T >= 4096 else 64
    fail_at = torch.randint(lo, T + 1, (B,), generator=torch.Generator().manual_seed(5))
    fail_at[check[0]] = T          # two followed rows never fail inside the horizon ...
    fail_at[check[1]] = T
    fail_at[check[2]] = lo + 88    # ... and one fails early in the allowed range
    mu_g, sigma2_g = _calibrate(B, 0.6, sampler)
    p = espo.make_params(temperature=0.6, mu_g=mu_g, sigma2_g=sigma2_g, alpha_s=0.9, beta=7.0, eps=0.2, t_max=T,
                         sampler=sampler)
    vals = synth.value_walk(B, T, seed=2, dtype=torch.bfloat16)
    run = ParityRun(B, V, p, seed=42, batch_id=1, check_slots=check)
    for t in range(T):
        x = synth.logits_batch(B, V, dtype=torch.bfloat16, sd=3.0, seed=10_000 + t, demote_rows=(fail_at <= t))
        run.step(x, vals[t].contiguous())
    st = run.stats
    view = {k: a.cpu().numpy() for k, a in run.view.items()}
    followed = [s for s in check if s not in run.dropped]
    t_stop = view["t_stop"][followed]
    assert st.tmax >= 1, st                                   # a followed row reached the horizon
    assert (t_stop >= lo).sum() >= 1, (t_stop, st)            # a followed row stopped after its failure point
    assert st.token_ties <= max(2, st.row_steps // 2000), st
    assert len(run.dropped) <= 1, run.dropped
    assert espo.espo_state_status(run.state) == 0
    run.close()


def test_config3_full_length_with_compaction():
    B, T = 512, 8192
    rng = np.random.default_rng(3)
    check = sorted(rng.choice(B, size=16, replace=False).tolist())
    fail_at = torch.randint(512, 4097, (B,), generator=torch.Generator().manual_seed(6))
    fail_at[check[0]] = T          # followed rows that run to the horizon
    fail_at[check[1]] = T
    mu_g, sigma2_g = _calibrate(B, 1.0, espo.ESPO_SAMPLER_HIER, steps=8)
    # (at temperature 1 these rows are nearly flat with or without their peaks, so the regret signal is weak; beta is set
    # where a rollout batch loses most of its rows to the stop rule over the horizon and keeps some to the end)
    p = espo.make_params(temperature=1.0, mu_g=mu_g, sigma2_g=sigma2_g, alpha_s=0.9, beta=4.5, eps=0.2, t_max=T)
    run = ParityRun(B, V, p, seed=43, batch_id=2, check_slots=check)
    ids = torch.arange(B, dtype=torch.int32, device="cuda")
    n_act = torch.zeros(1, dtype=torch.int32, device="cuda")
    fail_dev = fail_at.cuda()
    # per-trajectory value walk, advanced on the device step by step (the recipe of synth.value_walk)
    gen = torch.Generator("cuda").manual_seed(8)
    v_cur = torch.empty(B, device="cuda").uniform_(0.2, 0.8, generator=gen)
    n = B
    sizes = []
    for t in range(T):
        if t:
            v_cur = (v_cur + torch.empty(B, device="cuda").normal_(0.0, 0.05, generator=gen)).clamp_(-1.0, 1.0)
        slots = ids[:n].long()
        x = synth.logits_batch(n, V, dtype=torch.bfloat16, sd=3.0, seed=20_000 + t, demote_rows=(fail_dev[slots] <= t))
        run.step(x, v_cur[slots].to(torch.bfloat16).contiguous(), row_ids=ids[:n].contiguous())
        espo.espo_compact_active(run.state, ids, n_act)
        n = int(n_act.item())
        sizes.append(n)
        if t % 128 == 0 or n < 8:
            want = np.nonzero(run.view["status"].cpu().numpy() == espo.ESPO_ROW_ACTIVE)[0]
            assert n == len(want) and np.array_equal(ids[:n].cpu().numpy(), want), f"compaction at step {t}"
        if n == 0:
            break
    st = run.stats
    status = run.view["status"].cpu().numpy()
    assert n == 0 and (status != espo.ESPO_ROW_ACTIVE).all()
    assert st.tmax >= 1 and st.stops >= 4, (st, sizes[::512])   # followed rows ended both ways
    assert (status == espo.ESPO_ROW_TMAX).sum() >= 2 and (status == espo.ESPO_ROW_STOPPED).sum() >= B // 2
    assert sizes[511] >= B // 2                               # most rows are still decoding at the first failure point
    assert st.token_ties <= max(2, st.row_steps // 2000), st
    assert len(run.dropped) <= 1, run.dropped
    assert espo.espo_state_status(run.state) == 0
    run.close()
