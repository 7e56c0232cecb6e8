"""GPU parity of the vocabulary-sharded step (espo_step_partial + espo_step_merge) against the CPU oracle's samplers
on the whole rows, through the C ABI (needs a B200).  The flat sampler's draws belong to token ids, so any cut works;
the hierarchical sampler's belong to blocks of 1024 ids of the whole vocabulary, so its shards start on one.  The shards of a step are run one after the other on the
one GPU, which is what N tensor-parallel ranks compute side by side."""
import numpy as np
import pytest
import torch

import paper_2605_29860_b200 as espo
from paper_2605_29860_b200 import shard, synth
from parity_util import ParityRun

pytestmark = pytest.mark.gpu


def _sharded_launch(cuts):
    """A replacement for espo_step: one espo_step_partial per (offset, size) in ``cuts``, then espo_step_merge."""
    def launch(run, logits, values, row_ids, n):
        parts = torch.full((len(cuts), n, 8), float("nan"), dtype=torch.float32, device="cuda")
        for k, (lo, size) in enumerate(cuts):
            if size == 0:                                  # a rank without a shard still contributes: "nothing here"
                parts[k, :, 0] = float("-inf"); parts[k, :, 1] = 0.0; parts[k, :, 2] = float("-inf")
                parts[k, :, 3] = torch.tensor(-1, dtype=torch.int32).view(torch.float32)
                parts[k, :, 4:] = 0.0
                continue
            espo.espo_step_partial(logits[:n, lo:lo + size], lo, run.state, run.params, parts[k], row_ids=row_ids, n_rows=n)
        espo.espo_step_merge(parts, values, run.state, run.params, run.tokens, run.stop, row_ids=row_ids, n_rows=n)
    return launch


@pytest.mark.parametrize("sampler", [espo.ESPO_SAMPLER_FLAT, espo.ESPO_SAMPLER_HIER])
@pytest.mark.parametrize("V,world,dtype", [(152064, 8, torch.bfloat16), (152064, 2, torch.float32), (32000, 3, torch.bfloat16),
                                           (5000, 4, torch.float32), (300, 8, torch.bfloat16)])
def test_sharded_step_matches_the_oracle_on_whole_rows(V, world, dtype, sampler):
    B, T = 24, 6
    p = espo.make_params(temperature=0.8, mu_g=2.0, sigma2_g=4.0, beta=1.5, eps=0.1, t_max=5, eos_token=7,
                         sampler=sampler)
    run = ParityRun(B, V, p, seed=77, batch_id=2)
    run.launch = _sharded_launch(shard.vocab_shards(V, world, multiple=1024 if sampler == espo.ESPO_SAMPLER_HIER else 128))
    for t in range(T):
        x = synth.logits_batch(B, V, dtype=dtype, sd=3.0, seed=900 + t)
        if t == 1:
            x[3, : V // 2] = float("-inf")                 # a row whose first shards hold no finite logit
            x[4, 5] = float("nan")                         # a row one shard must flag
        v = torch.rand(B, generator=torch.Generator("cuda").manual_seed(t), device="cuda") * 1.2 - 0.1
        run.step(x, v)
    assert run.stats.row_steps >= 3 * B and run.stats.stops + run.stats.eos + run.stats.tmax > 0
    run.close()


def test_cut_does_not_change_the_tokens_and_greedy_takes_the_first_maximum():
    B, V = 16, 40000
    x = synth.logits_batch(B, V, dtype=torch.bfloat16, sd=3.0, seed=5)
    x[:, 123] = x.max() + 1; x[:, 30123] = x[:, 123]       # two equal maxima in different shards
    v = torch.full((B,), 0.5, device="cuda")
    outs = []
    for cuts, temp in (([(0, V)], 1.0), (shard.vocab_shards(V, 4), 1.0), ([(0, 4), (4, 1020), (1024, V - 1024)], 1.0),
                       (shard.vocab_shards(V, 4), 0.0)):
        p = espo.make_params(temperature=temp, mu_g=2.0, sigma2_g=4.0, beta=50.0, t_max=100, sampler=espo.ESPO_SAMPLER_FLAT)
        st = espo.espo_init_state(B, V, seed=11)
        tok = torch.empty(B, dtype=torch.int32, device="cuda"); stop = torch.empty(B, dtype=torch.uint8, device="cuda")
        parts = torch.empty(len(cuts), B, 8, dtype=torch.float32, device="cuda")
        for k, (lo, size) in enumerate(cuts):
            espo.espo_step_partial(x[:, lo:lo + size], lo, st, p, parts[k])
        espo.espo_step_merge(parts, v, st, p, tok, stop)
        ref_tok = torch.empty(B, dtype=torch.int32, device="cuda")
        st2 = espo.espo_init_state(B, V, seed=11)
        espo.espo_step(x, v, st2, p, ref_tok, stop)          # the unsharded flat sampler on the same state
        torch.cuda.synchronize()
        assert torch.equal(tok, ref_tok)
        g1, g2 = espo.espo_state_view(st)["g"].clone(), espo.espo_state_view(st2)["g"].clone()
        assert torch.allclose(g1, g2, rtol=1e-4, atol=1e-5)
        outs.append(tok.clone())
        espo.espo_free_state(st); espo.espo_free_state(st2)
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])
    assert torch.all(outs[3] == 123)                        # greedy: the lowest id among equal maxima, across shards


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_hierarchical_shards_give_the_unsharded_tokens(dtype):
    # the block-level draws are indexed by the block's number in the whole vocabulary, so 1, 2, 3 and 8 shards cut at
    # multiples of 1024 ids sample exactly the token of espo_step with the hierarchical sampler
    B, V = 40, 152064
    v = torch.rand(B, device="cuda")
    p = espo.make_params(temperature=0.9, mu_g=2.0, sigma2_g=4.0, beta=2.0, t_max=100, sampler=espo.ESPO_SAMPLER_HIER)
    stop = torch.empty(B, dtype=torch.uint8, device="cuda")
    for step_seed in (5, 6):
        x = synth.logits_batch(B, V, dtype=dtype, sd=3.0, seed=step_seed)
        st2 = espo.espo_init_state(B, V, seed=11)
        ref_tok = torch.empty(B, dtype=torch.int32, device="cuda")
        espo.espo_step(x, v, st2, p, ref_tok, stop)
        ref = {k: a.clone() for k, a in espo.espo_state_view(st2).items()}
        for world in (1, 2, 3, 8):
            cuts = shard.vocab_shards(V, world, multiple=1024)
            st = espo.espo_init_state(B, V, seed=11)
            tok = torch.empty(B, dtype=torch.int32, device="cuda")
            parts = torch.empty(len(cuts), B, 8, dtype=torch.float32, device="cuda")
            for k, (lo, size) in enumerate(cuts):
                espo.espo_step_partial(x[:, lo:lo + size], lo, st, p, parts[k])
            espo.espo_step_merge(parts, v, st, p, tok, stop)
            torch.cuda.synchronize()
            assert torch.equal(tok, ref_tok), world
            got = espo.espo_state_view(st)
            assert torch.equal(got["g"], ref["g"]) and torch.equal(got["status"], ref["status"])
            assert torch.allclose(got["logp"], ref["logp"], rtol=1e-4, atol=1e-5)
            assert espo.espo_state_status(st) == 0
            espo.espo_free_state(st)
        espo.espo_free_state(st2)


def test_argument_errors_of_the_sharded_calls():
    st = espo.espo_init_state(4, 4096, seed=1)
    x = torch.zeros(4, 2048, dtype=torch.bfloat16, device="cuda")
    parts = torch.zeros(1, 4, 8, dtype=torch.float32, device="cuda")
    flat = espo.make_params(sampler=espo.ESPO_SAMPLER_FLAT)
    hier = espo.make_params(sampler=espo.ESPO_SAMPLER_HIER)
    for kwargs, code in ((dict(off=2, p=flat), espo.ESPO_ERR_BAD_SHAPE), (dict(off=4096, p=flat), espo.ESPO_ERR_BAD_SHAPE),
                         (dict(off=512, p=hier), espo.ESPO_ERR_BAD_PARAM),        # not on a block of 1024 ids
                         (dict(off=0, p=espo.make_params(sampler=espo.ESPO_SAMPLER_HIER, temperature=0.0)), espo.ESPO_ERR_BAD_PARAM),
                         (dict(off=0, p=espo.make_params(sampler=espo.ESPO_SAMPLER_HIER, want_entropy=1)), espo.ESPO_ERR_BAD_PARAM)):
        with pytest.raises(espo.EspoError) as e:
            espo.espo_step_partial(x, kwargs["off"], st, kwargs["p"], parts[0])
        assert e.value.code == code
    with pytest.raises(espo.EspoError) as e:
        espo.espo_step_merge(parts, torch.zeros(4, device="cuda"), st, espo.make_params(want_entropy=1),
                             torch.empty(4, dtype=torch.int32, device="cuda"), torch.empty(4, dtype=torch.uint8, device="cuda"))
    assert e.value.code == espo.ESPO_ERR_BAD_PARAM
    espo.espo_free_state(st)


def test_sharded_step_with_row_ids_and_a_partial_batch():
    # 7 of 12 slots take part, in scrambled order; the sharded route must treat slots exactly like espo_step does
    cap, V = 12, 9000
    ids = torch.tensor([9, 2, 11, 0, 5, 7, 3], dtype=torch.int32, device="cuda")
    p = espo.make_params(temperature=1.1, mu_g=2.0, sigma2_g=4.0, beta=1.0, eps=0.1, t_max=50, sampler=espo.ESPO_SAMPLER_FLAT)
    run = ParityRun(cap, V, p, seed=31)
    run.launch = _sharded_launch(shard.vocab_shards(V, 3))
    for t in range(5):
        x = synth.logits_batch(ids.numel(), V, dtype=torch.float32, sd=2.0, seed=60 + t)
        run.step(x, torch.rand(ids.numel(), device="cuda"), row_ids=ids)
    view = espo.espo_state_view(run.state)
    untouched = [s for s in range(cap) if s not in set(ids.cpu().tolist())]
    assert torch.all(view["t"][untouched] == 0) and run.stats.row_steps >= 20
    run.close()
