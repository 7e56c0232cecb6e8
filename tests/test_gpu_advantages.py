"""GPU parity of espo_advantages against the CPU oracle, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_29860_b200 as espo
from paper_2605_29860_b200 import synth

pytestmark = pytest.mark.gpu


def _check(rewards, values, lengths, stopped, gamma, lam, r_fail):
    total = rewards.numel()
    adv = torch.full((max(total, 1),), float("nan"), device="cuda")
    espo.espo_advantages(rewards, values, lengths, stopped, gamma, lam, r_fail, adv, total_tokens=total)
    torch.cuda.synchronize()
    assert espo.espo_advantages_status() == 0
    ref = oracle.advantages(rewards.cpu().numpy(), values.cpu().numpy(), lengths.cpu().numpy(),
                            stopped.cpu().numpy(), gamma, lam, r_fail)
    got = adv[:total].cpu().numpy().astype(np.float64)
    err = np.abs(got - ref)
    tol = 1e-5 + 1e-4 * np.abs(ref)
    bad = np.nonzero(~(err <= tol))[0]
    assert bad.size == 0, f"{bad.size} of {total} advantages off; first at {bad[:5]}: gpu {got[bad[:5]]} ref {ref[bad[:5]]}"
    return float(err.max()) if total else 0.0


@pytest.mark.parametrize("lam", [0.95, 1.0])
def test_config5_ragged_batch(lam):
    # B=1024, lengths U[256,16384], 35% stopped (terminal r_fail=-1), others Bernoulli terminal reward
    r, v, L, s = synth.ragged_trajectories(1024, seed=0)
    assert r.numel() > 8_000_000
    _check(r, v, L, s, 1.0, lam, -1.0)


@pytest.mark.parametrize("gamma,lam", [(0.99, 0.9), (1.0, 0.0), (0.0, 0.5)])
def test_discount_variants(gamma, lam):
    r, v, L, s = synth.ragged_trajectories(200, len_lo=1, len_hi=5000, seed=1)
    _check(r, v, L, s, gamma, lam, -1.0)


@pytest.mark.parametrize("lengths", [[1], [2048], [2047], [2049], [4096, 4096], [1] * 5000, [0, 3, 0, 0, 2050, 0],
                                     [70000], [2048, 1, 2047, 4097, 5], [3, 2045, 2048, 2048, 1],
                                     # around the kernel's 3072-token chunks and its 4-token range granularity
                                     [2], [3], [5], [3071], [3072], [3073], [3072, 3072], [3070, 3, 3071, 6145], [6143, 1, 0, 7],
                                     # thousands of one- and two-token trajectories: more ends in a chunk than one round
                                     # of the flag-setting warp covers, over several CTAs' ranges
                                     [1] * 40001, [2, 1] * 9000 + [30000, 1, 1],
                                     # one trajectory crossing many CTAs' ranges (each looks ahead to its end, or as
                                     # far as the weights matter), then short ones
                                     [1_500_002, 7, 1, 4099]])
def test_edge_lengths(lengths):
    g = torch.Generator("cuda").manual_seed(len(lengths) + sum(lengths))
    L = torch.tensor(lengths, dtype=torch.int32, device="cuda")
    total = int(sum(lengths))
    r = torch.randn(total, device="cuda", generator=g) * 0.5
    v = torch.randn(total, device="cuda", generator=g) * 0.5
    s = (torch.rand(len(lengths), device="cuda", generator=g) < 0.5).to(torch.uint8)
    _check(r, v, L, s, 1.0, 1.0, -1.0)
    _check(r, v, L, s, 0.98, 0.97, -0.5)


def test_replace_not_add_and_repeat_calls_bit_identical():
    r, v, L, s = synth.ragged_trajectories(64, len_lo=1, len_hi=9000, seed=3)
    last = (torch.cumsum(L.long(), 0) - 1)
    r[last] = 0.7                       # a stopped trajectory's stored last reward must be replaced
    _check(r, v, L, s, 1.0, 0.95, -1.0)
    outs = []
    for _ in range(3):
        adv = torch.empty_like(r)
        espo.espo_advantages(r, v, L, s, 1.0, 0.95, -1.0, adv)
        outs.append(adv.clone())
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])


def test_inconsistent_lengths_are_reported_not_trapped():
    r, v, L, s = synth.ragged_trajectories(16, len_lo=10, len_hi=100, seed=4)
    adv = torch.empty_like(r)
    espo.espo_advantages(r, v, L, s, 1.0, 0.95, -1.0, adv, total_tokens=r.numel() - 3)
    torch.cuda.synchronize()
    assert espo.espo_advantages_status() & espo.ESPO_DEV_BAD_LENGTHS
    assert espo.espo_advantages_status() == 0            # reading clears it
    with pytest.raises(espo.EspoError) as e:
        espo.espo_advantages(r[1:], v[1:], L, s, 1.0, 0.95, -1.0, adv[1:], total_tokens=8)
    assert e.value.code == espo.ESPO_ERR_ALIGN


def test_reserve_then_smaller_calls():
    espo.espo_advantages_reserve(2048, 20_000_000)
    for seed in (5, 6):
        r, v, L, s = synth.ragged_trajectories(300, len_lo=1, len_hi=3000, seed=seed)
        _check(r, v, L, s, 1.0, 0.95, -1.0)


def test_returns_are_written_in_the_same_pass():
    # value targets A_t + V_t; with gamma = lambda = 1 they are the reward-to-go with the failure transition applied
    r, v, L, s = synth.ragged_trajectories(300, len_lo=1, len_hi=9000, seed=8)
    adv, ret = torch.empty_like(r), torch.empty_like(r)
    for gamma, lam in ((1.0, 1.0), (0.99, 0.95)):
        espo.espo_advantages_returns(r, v, L, s, gamma, lam, -1.0, adv, ret)
        torch.cuda.synchronize()
        ref = oracle.advantages(r.cpu().numpy(), v.cpu().numpy(), L.cpu().numpy(), s.cpu().numpy(), gamma, lam, -1.0)
        want = ref + v.cpu().numpy().astype(np.float64)
        got = ret.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - want) <= 1e-5 + 1e-4 * np.abs(want))
        assert np.all(np.abs(adv.cpu().numpy() - ref) <= 1e-5 + 1e-4 * np.abs(ref))
        if gamma == 1.0 and lam == 1.0:
            rr = r.cpu().numpy().astype(np.float64)
            off = np.concatenate([[0], np.cumsum(L.cpu().numpy().astype(np.int64))])
            for i in (0, 7, 150, 299):
                seg = rr[off[i]:off[i + 1]].copy()
                if seg.size and s[i]:
                    seg[-1] = -1.0
                togo = np.cumsum(seg[::-1])[::-1]
                assert np.allclose(got[off[i]:off[i + 1]], togo, rtol=1e-4, atol=1e-5)
    assert espo.espo_advantages_status() == 0


def test_batch_sums_come_out_of_the_same_pass():
    # sum A and sum A^2 over all tokens, as a trainer needs them to normalise a batch of advantages
    for seed, B, hi in ((9, 300, 9000), (10, 1024, 16384), (11, 3, 5)):
        r, v, L, s = synth.ragged_trajectories(B, len_lo=1, len_hi=hi, seed=seed)
        adv, ret = torch.empty_like(r), torch.empty_like(r)
        stats = torch.full((2,), float("nan"), dtype=torch.float64, device="cuda")
        espo.espo_advantages_stats(r, v, L, s, 1.0, 0.95, -1.0, adv, stats, returns_out=ret)
        torch.cuda.synchronize()
        assert espo.espo_advantages_status() == 0
        # the C ABI takes lambda as float32: the oracle gets the same number
        ref = oracle.advantages(r.cpu().numpy(), v.cpu().numpy(), L.cpu().numpy(), s.cpu().numpy(), 1.0,
                                float(np.float32(0.95)), -1.0)
        got = stats.cpu().numpy()
        assert abs(got[0] - ref.sum()) <= 1e-9 * np.abs(ref).sum() + 1e-12
        assert abs(got[1] - (ref * ref).sum()) <= 1e-9 * (ref * ref).sum() + 1e-12
        assert np.all(np.abs(adv.cpu().numpy() - ref) <= 1e-5 + 1e-4 * np.abs(ref))
        assert np.all(np.abs(ret.cpu().numpy() - (ref + v.cpu().numpy())) <= 1e-5 + 1e-4 * np.abs(ref + v.cpu().numpy()))
        # a second call: bit-identical sums, and the plain entry point still gives the same advantages
        stats2 = torch.zeros(2, dtype=torch.float64, device="cuda")
        adv2 = torch.empty_like(r)
        espo.espo_advantages_stats(r, v, L, s, 1.0, 0.95, -1.0, adv2, stats2)
        adv3 = torch.empty_like(r)
        espo.espo_advantages(r, v, L, s, 1.0, 0.95, -1.0, adv3)
        torch.cuda.synchronize()
        assert torch.equal(stats, stats2) and torch.equal(adv, adv2) and torch.equal(adv, adv3)
    empty = torch.full((2,), 7.0, dtype=torch.float64, device="cuda")
    z = torch.empty(0, device="cuda")
    espo.espo_advantages_stats(z, z, torch.empty(0, dtype=torch.int32, device="cuda"),
                               torch.empty(0, dtype=torch.uint8, device="cuda"), 1.0, 0.95, -1.0, z, empty)
    torch.cuda.synchronize()
    assert empty.tolist() == [0.0, 0.0]


@pytest.mark.parametrize("B,t_max,lo", [(64, 4096, 1), (300, 1000, 0), (1000, 37, 0), (3, 20000, 15000), (1, 5, 5), (5, 1, 0),
                                        (40, 3072, 3072), (17, 6145, 0)])
def test_padded_layout(B, t_max, lo):
    # [B, t_max] batch; the padding holds NaN on the way in and must come back as 0
    g = torch.Generator("cuda").manual_seed(B * 131 + t_max)
    L = torch.randint(lo, t_max + 1, (B,), generator=g, device="cuda", dtype=torch.int64).to(torch.int32)
    s = (torch.rand(B, generator=g, device="cuda") < 0.4).to(torch.uint8)
    r = torch.randn(B, t_max, generator=g, device="cuda") * 0.5
    v = torch.randn(B, t_max, generator=g, device="cuda") * 0.5
    pad = torch.arange(t_max, device="cuda")[None, :] >= L[:, None]
    r[pad] = float("nan"); v[pad] = float("nan")
    for gamma, lam in ((1.0, 1.0), (0.99, 0.95)):
        adv = torch.full((B, t_max), 7.0, device="cuda"); ret = torch.full((B, t_max), 7.0, device="cuda")
        espo.espo_advantages_padded(r, v, L, s, gamma, lam, -1.0, adv, ret)
        adv2 = torch.full((B, t_max), 7.0, device="cuda")
        espo.espo_advantages_padded(r, v, L, s, gamma, lam, -1.0, adv2)
        torch.cuda.synchronize()
        assert espo.espo_advantages_status() == 0
        ref = oracle.advantages_padded(r.cpu().numpy(), v.cpu().numpy(), L.cpu().numpy(), s.cpu().numpy(),
                                       float(np.float32(gamma)), float(np.float32(lam)), -1.0)
        got = adv.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref) <= 1e-5 + 1e-4 * np.abs(ref))
        assert torch.equal(adv, adv2)
        assert np.all(got[pad.cpu().numpy()] == 0.0)
        want_ret = ref + np.where(pad.cpu().numpy(), 0.0, np.nan_to_num(v.cpu().numpy().astype(np.float64)))
        got_ret = ret.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got_ret - want_ret) <= 1e-5 + 1e-4 * np.abs(want_ret))
        assert np.all(got_ret[pad.cpu().numpy()] == 0.0)
    # a length outside [0, t_max] is reported, not trapped
    bad = L.clone(); bad[0] = t_max + 3
    espo.espo_advantages_padded(torch.nan_to_num(r), torch.nan_to_num(v), bad, s, 1.0, 0.95, -1.0, adv)
    torch.cuda.synchronize()
    assert espo.espo_advantages_status() & espo.ESPO_DEV_BAD_LENGTHS


def test_a_broken_trajectory_does_not_reach_its_neighbours():
    # NaN and infinities inside one trajectory: every other trajectory comes out as if it were not there
    r, v, L, s = synth.ragged_trajectories(200, len_lo=1, len_hi=3000, seed=12)
    off = torch.cumsum(L.long(), 0) - L.long()
    for bad, val in ((17, float("nan")), (90, float("inf")), (150, float("-inf"))):
        v[off[bad] + L[bad].long() // 2] = val
        r[off[bad]] = val
    adv = torch.empty_like(r)
    espo.espo_advantages(r, v, L, s, 1.0, 0.95, -1.0, adv)
    torch.cuda.synchronize()
    ref = oracle.advantages(r.cpu().numpy(), v.cpu().numpy(), L.cpu().numpy(), s.cpu().numpy(), 1.0, float(np.float32(0.95)), -1.0)
    got = adv.cpu().numpy().astype(np.float64)
    finite = np.isfinite(ref)
    assert finite.sum() > 0.95 * ref.size                      # the oracle keeps the damage inside the three trajectories
    assert np.all(np.abs(got[finite] - ref[finite]) <= 1e-5 + 1e-4 * np.abs(ref[finite]))
    assert not np.any(np.isfinite(got[~finite]))               # and what is broken stays broken
