"""Seeded random configurations of every entry point against the CPU oracle (needs a B200): shapes, dtypes,
temperatures, masks, filters and shard counts drawn at random, so that combinations no hand-written case names are
still exercised.  Each case is small; the draws are fixed by the seed in the parametrisation."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_29860_b200 as espo
from paper_2605_29860_b200 import shard, synth
from parity_util import ParityRun
from test_gpu_filtered import _run_filtered
from test_gpu_vocab_shards import _sharded_launch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [11, 12])
def test_random_step_configurations(seed):
    rng = np.random.default_rng(seed)
    for it in range(20):
        V = int(rng.choice([1, 2, 33, 1024, 1025, 4097, 32000, 50257, 128256, 152064, 262144]))
        B = int(rng.integers(1, 40))
        dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
        sampler = int(rng.choice([espo.ESPO_SAMPLER_HIER, espo.ESPO_SAMPLER_FLAT]))
        temperature = float(rng.choice([0.05, 0.1, 0.5, 1.0, 2.0, 5.0]))
        p = espo.make_params(temperature=temperature, mu_g=1.0, sigma2_g=4.0, beta=float(rng.choice([0.5, 2.0, 50.0])),
                             eps=0.1, t_max=6, sampler=sampler,
                             want_entropy=int(sampler == espo.ESPO_SAMPLER_HIER and rng.random() < 0.5))
        run = ParityRun(B, V, p, seed=1000 * seed + it)
        sd = float(rng.choice([0.3, 3.0, 8.0]))
        for t in range(3):
            x = synth.logits_batch(B, V, dtype=dtype, sd=sd, seed=13 * it + t)
            if V > 4 and rng.random() < 0.5:                 # a masked stretch of ids in the first half of the rows
                lo = int(rng.integers(0, V - 1))
                hi = int(rng.integers(lo, V))
                x[: max(1, B // 2), lo:hi] = float("-inf")
            run.step(x, torch.rand(B, device="cuda", generator=torch.Generator("cuda").manual_seed(100 * it + t)))
        assert run.stats.token_ties <= 3, (it, V, B, temperature, sampler, run.stats)
        run.close()


@pytest.mark.parametrize("seed", [21])
def test_random_advantage_batches_padded_and_packed(seed):
    rng = np.random.default_rng(seed)
    for it in range(25):
        B = int(rng.integers(1, 400))
        t_max = int(rng.integers(1, 9000))
        g = torch.Generator("cuda").manual_seed(it)
        L = torch.randint(0, t_max + 1, (B,), generator=g, device="cuda").to(torch.int32)
        s = (torch.rand(B, generator=g, device="cuda") < 0.4).to(torch.uint8)
        r = torch.randn(B, t_max, generator=g, device="cuda")
        v = torch.randn(B, t_max, generator=g, device="cuda")
        pad = torch.arange(t_max, device="cuda")[None, :] >= L[:, None]
        r[pad] = float("nan")                                # padding is never read as a number
        v[pad] = float("inf")
        gamma = float(np.float32(rng.choice([1.0, 0.99, 0.9])))
        lam = float(np.float32(rng.choice([1.0, 0.95, 0.5, 0.0])))
        adv = torch.full((B, t_max), 3.0, device="cuda")
        ret = torch.full((B, t_max), 3.0, device="cuda")
        espo.espo_advantages_padded(r, v, L, s, gamma, lam, -1.0, adv, ret)
        ref = oracle.advantages_padded(r.cpu().numpy(), v.cpu().numpy(), L.cpu().numpy(), s.cpu().numpy(), gamma, lam, -1.0)
        got = adv.cpu().numpy().astype(np.float64)
        pad_h = pad.cpu().numpy()
        assert np.all(np.abs(got - ref) <= 1e-5 + 1e-4 * np.abs(ref)), ("padded", it, B, t_max, gamma, lam)
        assert np.all(got[pad_h] == 0) and np.all(ret.cpu().numpy()[pad_h] == 0)
        valid = ~pad
        rp, vp = r[valid].contiguous(), v[valid].contiguous()
        if rp.numel():                                       # the same trajectories packed, with the batch sums
            ap = torch.empty_like(rp)
            st = torch.zeros(2, dtype=torch.float64, device="cuda")
            espo.espo_advantages_stats(rp, vp, L, s, gamma, lam, -1.0, ap, st)
            refp = ref[~pad_h]
            assert np.all(np.abs(ap.cpu().numpy() - refp) <= 1e-5 + 1e-4 * np.abs(refp)), ("packed", it)
            assert abs(st[0].item() - refp.sum()) <= 1e-8 * np.abs(refp).sum() + 1e-9
    assert espo.espo_advantages_status() == 0


@pytest.mark.parametrize("seed", [31])
def test_random_filters_and_vocabulary_shards(seed):
    rng = np.random.default_rng(seed)
    for it in range(12):
        V = int(rng.choice([9, 100, 5000, 16384, 40000, 152064]))
        dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
        top_p = float(rng.choice([1.0, 0.3, 0.7, 0.9, 0.99]))
        top_k = int(rng.choice([0, 1, 5, 64, 1000]))
        if top_p >= 1.0 and top_k == 0:
            top_k = 3
        p = espo.make_params(temperature=float(rng.choice([0.7, 1.0, 1.3])), mu_g=2.0, sigma2_g=4.0, beta=2.0, t_max=6,
                             sampler=espo.ESPO_SAMPLER_FLAT, top_p=top_p, top_k=top_k)
        sd = float(rng.choice([0.5, 2.5, 4.0]))
        checked, excused, ties = _run_filtered(
            12, V, dtype, p, 4, seed=100 + it,
            make_logits=lambda t: synth.logits_batch(12, V, dtype=dtype, sd=sd, seed=7 * it + t))
        assert checked >= 20 and excused <= 6 and ties <= 3, (it, V, top_p, top_k, checked, excused, ties)
    for it in range(6):
        V = int(rng.choice([300, 5000, 40000, 152064]))
        world = int(rng.choice([1, 2, 3, 8]))
        p = espo.make_params(temperature=0.9, mu_g=2.0, sigma2_g=4.0, beta=1.5, eps=0.1, t_max=5,
                             sampler=espo.ESPO_SAMPLER_FLAT)
        run = ParityRun(10, V, p, seed=50 + it)
        run.launch = _sharded_launch(shard.vocab_shards(V, world))
        for t in range(4):
            run.step(synth.logits_batch(10, V, dtype=torch.bfloat16, sd=3.0, seed=11 * it + t),
                     torch.rand(10, device="cuda", generator=torch.Generator("cuda").manual_seed(it + t)))
        run.close()
