"""Shared harness of the GPU parity tests: drives the CUDA library and the CPU oracle over
the same seeded inputs and compares them under the stated rules.

Rules (from the benchmark spec of this build):
  * sampled token ids are bit-exact, except where the oracle's two best perturbed scores of
    some argmax it took lie within 1e-5 relative -- those are counted, and the oracle is
    re-run for that row with the library's token so that later steps stay comparable;
  * g, g~, z, log pi(a_t): |gpu - ref| <= 1e-5 + 1e-4 |ref|;
  * stop decisions identical, except where the rule in force was decided within 1e-5 of its
    threshold at the step where they differ: |z - beta*max(V, eps)| for Eq. 11, |z - tau| for the
    regret-only rule.  The value-only rule (V < tau) and the random rule (u < p_random) compare
    numbers that both sides hold exactly (input bits, a 24-bit uniform), so they are never excused.
    Excused cases are counted, and the row is dropped from later comparison.
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

import oracle
import paper_2605_29860_b200 as espo

TIE_REL = 1e-5
ATOL, RTOL = 1e-5, 1e-4
MARGIN = 1e-5


@dataclasses.dataclass
class ParityStats:
    row_steps: int = 0
    token_ties: int = 0        # excused token mismatches (near-tie in the oracle)
    stop_margins: int = 0      # excused stop mismatches (threshold margin < 1e-5)
    stops: int = 0
    eos: int = 0
    tmax: int = 0
    max_err: float = 0.0


def to_oracle_params(p: espo.espo_params) -> oracle.Params:
    return oracle.make_params(temperature=p.temperature, mu_g=p.mu_g, sigma2_g=p.sigma2_g, delta=p.delta,
                              clip_c=p.clip_c, alpha_s=p.alpha_s, beta=p.beta, eps=p.eps,
                              warmup_complete=p.warmup_complete, t_max=p.t_max, eos_token=p.eos_token,
                              sampler=p.sampler, stop_mode=p.stop_mode, shadow=p.shadow, tau=p.tau, p_random=p.p_random,
                              top_p=(p.top_p if 0.0 < p.top_p < 1.0 else 1.0), top_k=p.top_k)


def close(gpu: float, ref: float) -> bool:
    if np.isnan(gpu) or np.isnan(ref):
        return False
    return abs(gpu - ref) <= ATOL + RTOL * abs(ref)


def stop_margin(op: "oracle.Params", o) -> float:
    """Distance of the oracle's stop decision from its threshold, for the rule in force."""
    if op.stop_mode == oracle.STOP_ESPO:
        return abs(o.z - o.threshold)              # Eq. 11
    if op.stop_mode == oracle.STOP_REGRET_ONLY:
        return abs(o.z - op.tau)
    return float("inf")                            # value-only and random: exact on both sides


class ParityRun:
    """One rollout batch advanced in lock-step on the GPU library and on the oracle."""

    def __init__(self, capacity: int, V: int, params: espo.espo_params, seed: int, batch_id: int = 0,
                 check_slots=None):
        self.capacity, self.V, self.params = capacity, V, params
        self.state = espo.espo_init_state(capacity, V, seed, batch_id)
        self.ro = oracle.Rollout(capacity, seed, batch_id)
        self.op = to_oracle_params(params)
        self.view = espo.espo_state_view(self.state)
        self.tokens = torch.empty(capacity, dtype=torch.int32, device="cuda")
        self.stop = torch.empty(capacity, dtype=torch.uint8, device="cuda")
        self.stats = ParityStats()
        # slots the oracle follows (rows are independent, so a subset is a valid check)
        self.check = set(range(capacity)) if check_slots is None else set(int(s) for s in check_slots)
        self.dropped = set()
        self.entropy_log = {}      # slot -> oracle entropies of its steps (when params.want_entropy)
        self.launch = None         # callable(run, logits, values, row_ids, n) replacing espo_step

    def step(self, logits: torch.Tensor, values: torch.Tensor, row_ids: torch.Tensor | None = None):
        n = logits.shape[0]
        if self.launch is None:
            espo.espo_step(logits, values, self.state, self.params, self.tokens, self.stop, row_ids=row_ids, n_rows=n)
        else:      # another route to the same step (the vocabulary-sharded pair of calls)
            self.launch(self, logits, values, row_ids, n)
        torch.cuda.synchronize()
        slots = np.arange(n) if row_ids is None else row_ids[:n].cpu().numpy()
        tok = self.tokens[:n].cpu().numpy()
        stp = self.stop[:n].cpu().numpy()
        v = {k: a.cpu().numpy() for k, a in self.view.items()}
        rows = [r for r in range(n) if int(slots[r]) in self.check and int(slots[r]) not in self.dropped]
        if not rows:
            return tok, stp
        x = logits[rows].float().cpu().numpy().astype(np.float64)
        vals = values[:n][rows].float().cpu().numpy().astype(np.float64)
        sl = np.array([slots[r] for r in rows], dtype=np.int32)
        before = [self.ro.snapshot(int(s)) for s in sl]
        outs = self.ro.step(x, vals, self.op, row_ids=sl, n_threads=8)
        for i, r in enumerate(rows):
            s = int(sl[i])
            o = outs[i]
            was_active = before[i].status == oracle.ACTIVE
            if not was_active:
                assert tok[r] == -1 and stp[r] == 0, f"row {r}: finished slot {s} must be ignored"
                continue
            self.stats.row_steps += 1
            if o.bad:
                assert tok[r] == 0 and stp[r] == 0 and v["status"][s] == espo.ESPO_ROW_BAD, f"row {r}: bad-row handling"
                continue
            if tok[r] != o.token:
                assert o.min_rel_gap < TIE_REL, (
                    f"row {r} slot {s} t={before[i].t}: token {tok[r]} != oracle {o.token}, "
                    f"oracle top-two relative gap {o.min_rel_gap:.3e} is not a near-tie")
                assert 0 <= tok[r] < self.V
                self.stats.token_ties += 1
                self.ro.restore(s, before[i])
                o = self.ro.step(x[i:i + 1], vals[i:i + 1], self.op, row_ids=sl[i:i + 1], forced_tokens=[int(tok[r])])[0]
            for name, ref in (("g", o.g), ("g_tilde", o.g_tilde), ("z", o.z), ("logp", o.logp)):
                got = float(v[name][s])
                assert close(got, ref), f"row {r} slot {s} t={before[i].t}: {name} gpu={got!r} oracle={ref!r}"
                self.stats.max_err = max(self.stats.max_err, abs(got - ref))
            if self.params.want_entropy:
                got = float(v["entropy"][s])
                assert close(got, o.entropy), f"row {r} slot {s} t={before[i].t}: entropy gpu={got!r} oracle={o.entropy!r}"
                self.entropy_log.setdefault(s, []).append(o.entropy)
            ost = self.ro.states[s]
            if int(stp[r]) != o.stop or int(v["status"][s]) != ost.status:
                margin = stop_margin(self.op, o)
                assert margin < MARGIN, (
                    f"row {r} slot {s} t={before[i].t}: stop gpu={stp[r]} status={v['status'][s]} vs oracle "
                    f"stop={o.stop} status={ost.status}; margin {margin:.3e}")
                self.stats.stop_margins += 1
                self.dropped.add(s)
                continue
            assert int(v["t"][s]) == ost.t and int(v["t_stop"][s]) == ost.t_stop, f"row {r}: t / t_stop"
            assert abs(float(v["sum_g"][s]) - ost.sum_g) <= 1e-4 * max(1.0, abs(ost.sum_g)), f"row {r}: sum_g"
            assert abs(float(v["sum_g2"][s]) - ost.sum_g2) <= 1e-4 * max(1.0, abs(ost.sum_g2)), f"row {r}: sum_g2"
            self.stats.stops += int(o.stop)
            self.stats.eos += int(ost.status == oracle.EOS)
            self.stats.tmax += int(ost.status == oracle.TMAX)
        return tok, stp

    def close(self):
        espo.espo_free_state(self.state)
