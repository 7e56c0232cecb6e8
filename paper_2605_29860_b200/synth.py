"""Seeded synthetic inputs shaped like the paper's workloads.

The paper's rollouts (DeepSeek-R1-Distill-Qwen policies decoding DAPO-Math-17k prompts) are
not available offline; these generators stand in for them: LLM-shaped logit rows (a broad
Gaussian body plus a few strongly boosted ids), critic values that drift as a clipped random
walk, and ragged trajectory batches for the advantage pass.  This module holds no part of
the method's arithmetic; both the CUDA path and the CPU oracle consume its outputs as bits.
"""
from __future__ import annotations

import torch


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def logits_batch(n_rows: int, V: int, *, dtype=torch.bfloat16, sd: float = 3.0, n_peaks: int = 5,
                 peak_lo: float = 8.0, peak_hi: float = 15.0, zipf: bool = True, seed: int = 0,
                 device="cuda", demote_rows: torch.Tensor | None = None, row_stride: int | None = None) -> torch.Tensor:
    """[n_rows, V] logits ~ N(0, sd) with ``n_peaks`` boosted ids per row.

    zipf=True : the j-th peak (j = 1..n_peaks) is boosted by peak_lo + (peak_hi-peak_lo)/j
                (the "Zipf-weighted top-k peaks (+8..+15)" of the Qwen-shaped configs);
    zipf=False: boosts are uniform in [peak_lo, peak_hi] and the number of peaks per row is
                uniform in 1..n_peaks (the tiny config's "1-3 boosted tokens (+6..+12)").
    Rows flagged in ``demote_rows`` (bool [n_rows]) get every boost flattened to +4: the
    "failure point after which the peak token is demoted so regret rises".
    ``row_stride`` > V returns a strided view into a wider buffer.
    """
    g = _gen(seed, device)
    stride = V if row_stride is None else int(row_stride)
    buf = torch.empty(n_rows, stride, dtype=torch.float32, device=device)
    buf.normal_(0.0, sd, generator=g)
    x = buf[:, :V]
    ids = torch.randint(0, V, (n_rows, n_peaks), generator=g, device=device)
    if zipf:
        j = torch.arange(1, n_peaks + 1, device=device, dtype=torch.float32)
        boost = (peak_lo + (peak_hi - peak_lo) / j).expand(n_rows, n_peaks).clone()
    else:
        boost = torch.empty(n_rows, n_peaks, device=device).uniform_(peak_lo, peak_hi, generator=g)
        k = torch.randint(1, n_peaks + 1, (n_rows, 1), generator=g, device=device)
        boost = boost * (torch.arange(n_peaks, device=device)[None, :] < k)
    if demote_rows is not None:
        boost = torch.where(demote_rows[:, None].to(device), torch.full_like(boost, 4.0) * (boost > 0), boost)
    x.scatter_add_(1, ids, boost)
    return buf.to(dtype)[:, :V]


def value_walk(n_traj: int, T: int, *, step_sd: float = 0.05, lo: float = -1.0, hi: float = 1.0, seed: int = 0,
               device="cuda", dtype=torch.float32) -> torch.Tensor:
    """[T, n_traj] critic values: per-trajectory Gaussian random walk from U[0.2, 0.8], clipped to [lo, hi]."""
    g = _gen(seed, device)
    start = torch.empty(n_traj, device=device).uniform_(0.2, 0.8, generator=g)
    steps = torch.empty(T, n_traj, device=device).normal_(0.0, step_sd, generator=g)
    steps[0] = 0.0
    # the running walk is clipped at every step (not its final sum)
    out = torch.empty_like(steps)
    cur = start.clone()
    for t in range(T):
        cur = (cur + steps[t]).clamp_(lo, hi)
        out[t] = cur
    return out.to(dtype)


def ragged_trajectories(B: int, *, len_lo: int = 256, len_hi: int = 16384, p_stopped: float = 0.35, sd: float = 0.5,
                        seed: int = 0, device="cuda"):
    """Packed ragged batch for the advantage pass.

    lengths ~ U{len_lo..len_hi}; ``p_stopped`` of the trajectories are flagged stopped (their
    stored last reward is 0, as the failure transition prescribes; the kernel substitutes
    r_fail); the others end with a Bernoulli(0.5) reward in {0, 1}; every other reward and all
    values are N(0, sd).  Returns (rewards, values, lengths int32, stopped uint8).
    """
    g = _gen(seed, device)
    lengths = torch.randint(len_lo, len_hi + 1, (B,), generator=g, device=device, dtype=torch.int64)
    total = int(lengths.sum().item())
    rewards = torch.empty(total, device=device).normal_(0.0, sd, generator=g)
    values = torch.empty(total, device=device).normal_(0.0, sd, generator=g)
    stopped = (torch.rand(B, generator=g, device=device) < p_stopped)
    last = torch.cumsum(lengths, 0) - 1
    has = lengths > 0
    term = (torch.rand(B, generator=g, device=device) < 0.5).float()
    rewards[last[has]] = torch.where(stopped[has], torch.zeros_like(term[has]), term[has])
    return rewards, values, lengths.to(torch.int32), stopped.to(torch.uint8)
