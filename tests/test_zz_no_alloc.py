"""espo_advantages_noalloc against espo_advantages and against the CPU oracle, through the C ABI (needs a B200).

The entry point exists for processes that cannot allocate device memory once they are running --
a rollout worker whose serving engine took all free memory for its own pools, or a loop that
cannot tolerate cudaMalloc's device-wide synchronisation -- so its scratch is a fixed array
inside the library.  That array is shared by every call and keeps the previous call's contents,
which is what the second call of each pair below runs into.  This file is named so that pytest
collects it last.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_29860_b200 as espo
from paper_2605_29860_b200 import synth

pytestmark = pytest.mark.gpu

ATOL, RTOL = 1e-5, 1e-4     # the tolerance of the advantage parity tests


def _both(r, v, L, s, gamma, lam, r_fail, status):
    ref = torch.empty_like(r)
    got = torch.full_like(r, float("nan"))
    espo.espo_advantages(r, v, L, s, gamma, lam, r_fail, ref)
    espo.espo_advantages_noalloc(r, v, L, s, gamma, lam, r_fail, got, status_out=status)
    torch.cuda.synchronize()
    ref, got = ref.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
    bad = np.nonzero(~(np.abs(got - ref) <= ATOL + RTOL * np.abs(ref)))[0]
    assert bad.size == 0, f"{bad.size} of {ref.size} differ, first at {bad[:5]}: {got[bad[:5]]} vs {ref[bad[:5]]}"
    # and against the CPU oracle (Eq. 4-5, 13 in float64), the checker of every other advantage test;
    # the C ABI takes gamma, lambda and r_fail as float32, so the oracle gets the same numbers
    f32 = lambda x: float(np.float32(x))
    want = oracle.advantages(r.cpu().numpy(), v.cpu().numpy(), L.cpu().numpy(), s.cpu().numpy(), f32(gamma), f32(lam),
                             f32(r_fail))
    bad = np.nonzero(~(np.abs(got - want) <= ATOL + RTOL * np.abs(want)))[0]
    assert bad.size == 0, f"{bad.size} of {want.size} differ from the oracle, first at {bad[:5]}: {got[bad[:5]]} vs {want[bad[:5]]}"


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # a large ragged batch, then a smaller one with other lengths, parameters and chunk boundaries:
    # the second call finds the first call's descriptors, offsets and tickets in the scratch
    r, v, L, s = synth.ragged_trajectories(1024, len_lo=256, len_hi=16384, seed=11)
    assert r.numel() <= espo.ESPO_NOALLOC_MAX_TOKENS
    _both(r, v, L, s, 1.0, 0.95, -1.0, status)
    r, v, L, s = synth.ragged_trajectories(333, len_lo=1, len_hi=7000, seed=12)
    _both(r, v, L, s, 0.99, 1.0, -0.5, status)
    _both(r, v, L, s, 1.0, 1.0, -1.0, None)          # status word inside the scratch
    assert int(status.item()) == 0
    assert espo.espo_advantages_status() == 0


def test_sizes_beyond_the_fixed_scratch_are_refused():
    L = torch.ones(espo.ESPO_NOALLOC_MAX_B + 1, dtype=torch.int32, device="cuda")
    x = torch.zeros(espo.ESPO_NOALLOC_MAX_B + 1, device="cuda")
    s = torch.zeros(espo.ESPO_NOALLOC_MAX_B + 1, dtype=torch.uint8, device="cuda")
    with pytest.raises(espo.EspoError) as e:
        espo.espo_advantages_noalloc(x, x, L, s, 1.0, 0.95, -1.0, torch.empty_like(x))
    assert e.value.code == espo.ESPO_ERR_CAPACITY
    big = torch.zeros(espo.ESPO_NOALLOC_MAX_TOKENS + 1, device="cuda")
    Lb = torch.tensor([espo.ESPO_NOALLOC_MAX_TOKENS, 1], dtype=torch.int32, device="cuda")
    with pytest.raises(espo.EspoError) as e:
        espo.espo_advantages_noalloc(big, big, Lb, s[:2], 1.0, 0.95, -1.0, torch.empty_like(big))
    assert e.value.code == espo.ESPO_ERR_CAPACITY
    del big
    # inconsistent lengths are reported through the caller's status word, not trapped
    r, v, L, s = synth.ragged_trajectories(16, len_lo=10, len_hi=100, seed=4)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    espo.espo_advantages_noalloc(r, v, L, s, 1.0, 0.95, -1.0, torch.empty_like(r), status_out=status,
                                 total_tokens=r.numel() - 3)
    torch.cuda.synchronize()
    assert int(status.item()) & espo.ESPO_DEV_BAD_LENGTHS
