"""GPU parity of filtered sampling (top-p / top-k through espo_step) against the CPU oracle (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_29860_b200 as espo
from paper_2605_29860_b200 import synth
from parity_util import ParityRun, close, to_oracle_params

pytestmark = pytest.mark.gpu

MARGIN = 1e-5      # a keep/drop decision closer than this to flipping (in probability mass) may differ from the oracle's


def _run_filtered(B, V, dtype, params, steps, seed, make_logits):
    """Like ParityRun.step, with one more excuse for a token that differs: the edge of the support lies within MARGIN of
    top_p, so the two supports may differ by the groups at the edge.  (log pi is compared regardless: such groups weigh
    less than the tolerance.)"""
    st = espo.espo_init_state(B, V, seed=seed)
    ro = oracle.Rollout(B, seed=seed)
    op = to_oracle_params(params)
    view = espo.espo_state_view(st)
    tok = torch.empty(B, dtype=torch.int32, device="cuda"); stop = torch.empty(B, dtype=torch.uint8, device="cuda")
    checked = excused = ties = 0
    dropped = set()
    for t in range(steps):
        x = make_logits(t)
        v = torch.rand(B, generator=torch.Generator("cuda").manual_seed(1000 + t), device="cuda") * 1.2 - 0.1
        espo.espo_step(x, v, st, params, tok, stop)
        torch.cuda.synchronize()
        assert espo.espo_state_status(st) & ~espo.ESPO_DEV_BAD_ROW == 0      # one test row holds a NaN on purpose
        xs = x.float().cpu().numpy().astype(np.float64)
        before = [ro.snapshot(s) for s in range(B)]
        outs = ro.step(xs, v.cpu().numpy().astype(np.float64), op, n_threads=8)
        g, logp, z, status = (view[k].cpu().numpy() for k in ("g", "logp", "z", "status"))
        for r in range(B):
            if r in dropped or before[r].status != oracle.ACTIVE:
                continue
            o = outs[r]
            if o.bad:
                assert int(tok[r]) == 0 and int(status[r]) == espo.ESPO_ROW_BAD
                continue
            if int(tok[r]) != o.token:
                if o.filter_margin < MARGIN:                    # the supports may differ by the groups at the edge,
                    excused += 1; dropped.add(r); continue      # and one of those tokens may have won
                assert o.min_rel_gap < 1e-5, f"step {t} row {r}: token {int(tok[r])} != oracle {o.token} (kept {o.kept}, gap {o.min_rel_gap:.3e})"
                ties += 1; dropped.add(r); continue
            checked += 1
            assert close(float(g[r]), o.g) and close(float(logp[r]), o.logp) and close(float(z[r]), o.z), \
                f"step {t} row {r}: g {g[r]} vs {o.g}, logp {logp[r]} vs {o.logp}, z {z[r]} vs {o.z}"
            if int(stop[r]) != o.stop or int(status[r]) != ro.states[r].status:
                assert abs(o.z - o.threshold) < 1e-5
                dropped.add(r)
    espo.espo_free_state(st)
    return checked, excused, ties


@pytest.mark.parametrize("V,dtype,top_p,top_k", [(152064, torch.bfloat16, 0.7, 0), (152064, torch.bfloat16, 1.0, 50),
                                                 (152064, torch.bfloat16, 0.95, 20), (152064, torch.bfloat16, 0.9999, 0),
                                                 (50001, torch.bfloat16, 0.99, 0), (32000, torch.float32, 0.7, 0),
                                                 (152064, torch.float32, 0.999, 0), (152064, torch.bfloat16, 1.0, 5000),
                                                 (16391, torch.bfloat16, 0.97, 0), (16391, torch.bfloat16, 0.6, 0),
                                                 (32000, torch.float32, 0.999, 0), (5000, torch.float32, 1.0, 3),
                                                 (777, torch.bfloat16, 0.5, 0), (9, torch.float32, 0.8, 2)])
def test_filtered_step_matches_the_oracle(V, dtype, top_p, top_k):
    B, T = 20, 5
    p = espo.make_params(temperature=0.9, mu_g=2.0, sigma2_g=4.0, beta=1.5, eps=0.1, t_max=4, eos_token=3,
                         sampler=espo.ESPO_SAMPLER_FLAT, top_p=top_p, top_k=top_k)
    def logits(t):
        x = synth.logits_batch(B, V, dtype=dtype, sd=2.5, seed=40 + t)
        if t == 2 and V > 100:
            x[1, : V // 3] = float("-inf")                  # masked ids
            x[2, 7] = float("nan")                          # an unusable row
        return x
    checked, excused, ties = _run_filtered(B, V, dtype, p, T, seed=3, make_logits=logits)
    assert checked >= 2 * B and excused <= 3 and ties <= 2, (checked, excused, ties)


def test_support_is_respected_and_ties_stay_together():
    # a row with a handful of equal heavy tokens: top_k = 2 must keep all four of them (they tie), nothing else
    B, V = 64, 4096
    x = torch.full((B, V), -3.0, dtype=torch.bfloat16, device="cuda")
    heavy = [5, 1000, 2047, 4095]
    x[:, heavy] = 4.0
    p = espo.make_params(temperature=1.0, sampler=espo.ESPO_SAMPLER_FLAT, top_k=2, beta=1e9, t_max=10**6)
    st = espo.espo_init_state(B, V, seed=8)
    tok = torch.empty(B, dtype=torch.int32, device="cuda"); stop = torch.empty(B, dtype=torch.uint8, device="cuda")
    v = torch.zeros(B, device="cuda")
    seen = set()
    for _ in range(20):
        espo.espo_step(x, v, st, p, tok, stop)
        seen |= set(tok.cpu().tolist())
        lp = espo.espo_state_view(st)["logp"].cpu().numpy()
        assert np.allclose(lp, np.log(0.25), atol=1e-5)       # four equal tokens share the support
    assert seen == set(heavy)
    # no filter given (top_p = 0 from a zeroed struct, top_k = 0): the plain flat sampler
    q = espo.make_params(temperature=1.0, sampler=espo.ESPO_SAMPLER_FLAT, top_p=0.0, beta=1e9, t_max=10**6)
    st2 = espo.espo_init_state(B, V, seed=8); st3 = espo.espo_init_state(B, V, seed=8)
    t2 = torch.empty_like(tok); t3 = torch.empty_like(tok)
    espo.espo_step(x, v, st2, q, t2, stop)
    espo.espo_step(x, v, st3, espo.make_params(temperature=1.0, sampler=espo.ESPO_SAMPLER_FLAT, beta=1e9, t_max=10**6), t3, stop)
    torch.cuda.synchronize()
    assert torch.equal(t2, t3)
    with pytest.raises(espo.EspoError) as e:                  # the hierarchical sampler has no filtered form
        espo.espo_step(x, v, st2, espo.make_params(sampler=espo.ESPO_SAMPLER_HIER, top_p=0.7), t2, stop)
    assert e.value.code == espo.ESPO_ERR_BAD_PARAM
    for s in (st, st2, st3):
        espo.espo_free_state(s)


def test_more_tied_candidates_than_the_list_holds():
    # 10 000 equal logits at the top key of a sample-histogram bin: all of them lie above the candidate cut, the list
    # overflows, and the search runs over the whole row; top_k = 2 keeps exactly the tied tokens
    B, V, n_top = 8, 40000, 10000
    x = torch.full((B, V), -3.0, dtype=torch.bfloat16, device="cuda")
    g = torch.Generator().manual_seed(11)
    top_val = torch.tensor([0x408F], dtype=torch.int16).view(torch.bfloat16).item()     # 4.46875: low key bits 1111
    heavy = [torch.randperm(V, generator=g)[:n_top].cuda() for _ in range(B)]
    for r in range(B):
        x[r, heavy[r]] = top_val
    p = espo.make_params(temperature=1.0, sampler=espo.ESPO_SAMPLER_FLAT, top_k=2, beta=1e9, t_max=10**6)
    st = espo.espo_init_state(B, V, seed=21)
    tok = torch.empty(B, dtype=torch.int32, device="cuda"); stop = torch.empty(B, dtype=torch.uint8, device="cuda")
    v = torch.zeros(B, device="cuda")
    for _ in range(6):
        espo.espo_step(x, v, st, p, tok, stop)
        torch.cuda.synchronize()
        assert espo.espo_state_status(st) == 0
        lp = espo.espo_state_view(st)["logp"].cpu().numpy()
        assert np.allclose(lp, -np.log(n_top), atol=1e-5)
        for r in range(B):
            assert float(x[r, int(tok[r])]) == top_val
    espo.espo_free_state(st)


@pytest.mark.parametrize("V,dtype,top_p,top_k", [(152064, torch.bfloat16, 0.7, 0), (20480, torch.bfloat16, 0.9999, 0),
                                                 (16384, torch.float32, 0.6, 0), (50008, torch.bfloat16, 1.0, 40)])
def test_more_rows_than_ctas(V, dtype, top_p, top_k):
    # 330 rows on 296 CTAs: some CTAs work through two rows one after the other (shared-memory lists and histograms reused)
    B, T = 330, 3
    p = espo.make_params(temperature=0.9, mu_g=2.0, sigma2_g=4.0, beta=1.5, eps=0.1, t_max=4, eos_token=3,
                         sampler=espo.ESPO_SAMPLER_FLAT, top_p=top_p, top_k=top_k)
    def logits(t):
        x = synth.logits_batch(B, V, dtype=dtype, sd=2.5, seed=140 + t)
        if t == 1:
            x[1, : V // 3] = float("-inf")                  # masked ids
            x[2, 7] = float("nan")                          # an unusable row
            x[5, V - 1] = float("inf")                      # another one
        return x
    checked, excused, ties = _run_filtered(B, V, dtype, p, T, seed=13, make_logits=logits)
    assert checked >= 2 * B and excused <= 8 and ties <= 5, (checked, excused, ties)
