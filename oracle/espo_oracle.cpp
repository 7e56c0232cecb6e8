// ESPO reference oracle: a plain, slow, double-precision CPU statement of the
// per-decode-step early-stopping rule and of the truncated-trajectory GAE pass.
//
// THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the tests, the smoke check
// and the benchmark's CPU-baseline leg may load it.  It shares no source, header,
// table or helper with the CUDA library; the two were written separately from
// the same written definitions.
//
// What follows the paper, and where:
//   * surrogate regret  g_t = max_a log pi(a|s_t) - log pi(a_t|s_t)   (Sec. 4.1, Eq. 6)
//   * normalised signal g~_t = clip((g_t - mu_g)/sqrt(sigma_g^2 + delta), -c, c)  (Sec. 4.2, Eq. 9)
//   * smoothed cumulative regret z_t = a_s z_{t-1} + (1-a_s) g~_t, z_0 = 0        (Sec. 4.2, Eq. 10)
//   * value-gated stop  z_t > beta * max(V_phi(s_t), eps), only after warm-up     (Sec. 4.3, Eq. 11; Algorithm 1)
//   * failure transition r_{T_stop} = r_fail, nothing bootstrapped past the end   (Sec. 4.4, Eq. 13)
//   * batch statistics  mu_g, sigma_g^2: EMA of the batch mean / variance of g    (Sec. 4.2, Eq. 7-8)
//   * threshold control beta <- clip(beta + eta (rho_stop - tau), b_min, b_max)   (Sec. 4.3, Eq. 12)
//   * TD error and GAE  delta_t = r_t + gamma V(s_{t+1}) - V(s_t),
//                       A_t = sum_l (gamma lambda)^l delta_{t+l}                  (Sec. 3, Eq. 4-5)
//
// What the paper leaves open and this file fixes (the same written convention the
// CUDA library follows):
//   * "sample a_t ~ pi" is done by Gumbel-max with a counter-based Philox4x32-10
//     generator (Salmon et al., SC'11): key = (seed low, seed high), counter =
//     (index >> 2, step t, trajectory slot, (batch_id << 2) | level), the draw for
//     `index` is output word (index & 3); k = word >> 9, u = (2k+1) / 2^24,
//     G = -log(-log u).
//   * sampler 0 ("flat"): a_t = argmax_a (x_a + G_a), level 0, index a; lowest id
//     wins exact ties.
//   * sampler 1 ("hierarchical"): the same Gumbel-max applied level by level, which
//     is the same distribution because the maximum of independent Gumbel-shifted
//     scores over a group is itself Gumbel-shifted by the group's log-sum-exp:
//       level 2 picks a block of 1024 consecutive ids by argmax_b (LSE_b + G), index b;
//       level 1 picks a sub-block of 32 ids inside it by argmax_j (LSE_j + G), index
//               = global sub-block number (id >> 5);
//       level 0 picks the id inside that sub-block by argmax_a (x_a + G_a), index a
//               (the same draws the flat sampler would use for those ids).
//   * x_a = logit_a / temperature; pi is the temperature-scaled distribution that is
//     actually sampled from.  temperature == 0 means greedy: a_t = first argmax,
//     g_t = 0, log pi(a_t) = 0.
//   * a sampled EOS ends the trajectory naturally even if the test would also fire.
//   * filtered sampling (flat sampler; the paper's evaluation decodes with top-p 0.7 and says no more): a token
//     stays in the support iff the tokens strictly more probable than it weigh less than top_p and number fewer
//     than top_k, so tokens of equal probability stay or go together; the token is the Gumbel-max over the
//     support with the flat sampler's draws; log pi(a_t) is taken under the renormalised support, the regret
//     of Eq. 6 is unchanged (the normaliser cancels and the most probable token is always in the support).
//
//   * r_fail REPLACES the stored last reward of a stopped trajectory (Eq. 13 sets it).
//
// Five of these readings are fixed by nothing the paper prints, and no test can hold them to
// anything but this file's own statement -- for them parity is "parity unpinned" by the paper:
// which distribution pi is in Eq. 6 (temperature-scaled here), the values of delta and c in
// Eq. 9 (run-time parameters), EOS taking precedence over a stop on the same step,
// r_fail replacing (not adding to) the stored reward, and how ties at the edge of a top-p / top-k support are cut
// (kept together here).  Everything else is pinned by the tests
// (known-answer vectors, library routines, closed forms, invariants, brute force).
//
// Everything is brute force over the vocabulary, one row at a time, no blocking or
// reordering beyond what the definitions above state.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw 2011): ten rounds of two 32x32->64
// multiplies, with the key advanced by the Weyl constants between rounds.
// ---------------------------------------------------------------------------
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  const uint64_t mul_a = 0xD2511F53ull, mul_b = 0xCD9E8D57ull;
  const uint32_t weyl_a = 0x9E3779B9u, weyl_b = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) { k0 += weyl_a; k1 += weyl_b; }
    const uint64_t pa = mul_a * (uint64_t)c0;
    const uint64_t pb = mul_b * (uint64_t)c2;
    const uint32_t n0 = (uint32_t)(pb >> 32) ^ c1 ^ k0;
    const uint32_t n1 = (uint32_t)pb;
    const uint32_t n2 = (uint32_t)(pa >> 32) ^ c3 ^ k1;
    const uint32_t n3 = (uint32_t)pa;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

struct DrawKey {
  uint64_t seed;
  uint64_t batch_id;
  uint32_t slot;
  uint32_t step;
};

// The open-interval uniform attached to (level, index): 23 random bits k, u = (2k+1)/2^24.
double uniform_for(const DrawKey& dk, int level, uint64_t index) {
  uint32_t ctr[4] = {(uint32_t)(index >> 2), dk.step, dk.slot,
                     (uint32_t)((dk.batch_id << 2) | (uint64_t)level)};
  uint32_t key[2] = {(uint32_t)(dk.seed & 0xffffffffull), (uint32_t)(dk.seed >> 32)};
  uint32_t w[4];
  philox4x32_10(ctr, key, w);
  const uint32_t k = w[index & 3] >> 9;
  return (2.0 * (double)k + 1.0) / 16777216.0;
}

double gumbel_for(const DrawKey& dk, int level, uint64_t index) {
  return -std::log(-std::log(uniform_for(dk, level, index)));
}

const double NEG_INF = -std::numeric_limits<double>::infinity();

// log sum_a exp(x_a) over [lo, hi); -inf for an empty or all -inf range.
double log_sum_exp(const double* x, int64_t lo, int64_t hi) {
  double m = NEG_INF;
  for (int64_t a = lo; a < hi; ++a) if (x[a] > m) m = x[a];
  if (m == NEG_INF) return NEG_INF;
  double s = 0.0;
  for (int64_t a = lo; a < hi; ++a) s += std::exp(x[a] - m);
  return m + std::log(s);
}

// Relative gap between the best and second-best perturbed score of one argmax.
// The scale has a floor of 1 because the scores are only defined up to a common
// shift of the logits, so a gap relative to a score near zero means nothing.
double relative_gap(double best, double second) {
  if (second == NEG_INF) return std::numeric_limits<double>::infinity();
  double scale = std::fmax(1.0, std::fmax(std::fabs(best), std::fabs(second)));
  return (best - second) / scale;
}

struct ArgmaxResult {
  int64_t index;    // winner (lowest index on exact ties), -1 if no finite candidate
  double best;      // its perturbed score
  double second;    // runner-up's perturbed score
  int64_t runner;   // runner-up index
};

template <class ScoreFn>
ArgmaxResult perturbed_argmax(int64_t lo, int64_t hi, ScoreFn score) {
  ArgmaxResult r{-1, NEG_INF, NEG_INF, -1};
  for (int64_t i = lo; i < hi; ++i) {
    const double s = score(i);
    if (s > r.best) {
      r.second = r.best; r.runner = r.index;
      r.best = s; r.index = i;
    } else if (s > r.second) {
      r.second = s; r.runner = i;
    }
  }
  return r;
}

}  // namespace

extern "C" {

// ---- plain-data records shared with the Python loader (ctypes mirrors them) ----

struct espo_oracle_params {
  double temperature;
  double mu_g, sigma2_g, delta, clip_c;   // Eq. 9 (frozen for the whole rollout batch)
  double alpha_s;                          // Eq. 10
  double beta, eps;                        // Eq. 11
  int32_t warmup_complete;                 // Algorithm 1: the test is gated, z is not
  int32_t t_max;                           // horizon T_max
  int32_t eos_token;                       // -1: none
  int32_t sampler;                         // 0 flat, 1 hierarchical
  // Stop rules of the ablation study (Sec. 6): 0 the method's rule (Eq. 11); 1 value only, V_phi(s_t) < tau;
  // 2 regret only, z_t > tau; 3 random, with probability p_random per step.  shadow != 0: the first step at
  // which the rule holds is recorded in t_stop but the trajectory is not ended (the analysis' "Original" curves).
  int32_t stop_mode;
  int32_t shadow;
  double tau;
  double p_random;
  // Filtered sampling (flat sampler only; the paper's evaluation samples with top-p 0.7).  With pi the temperature-
  // scaled softmax, token a stays in the support iff the mass of the tokens strictly more probable than a is below
  // top_p (top_p >= 1: no filter) and fewer than top_k tokens are strictly more probable than a (top_k <= 0: no
  // filter).  Tokens of equal probability are therefore kept or dropped together, whatever their ids.
  double top_p;
  int32_t top_k;
  int32_t pad_;
};

enum { ORACLE_ACTIVE = 0, ORACLE_STOPPED = 1, ORACLE_EOS = 2, ORACLE_TMAX = 3, ORACLE_BAD = 4 };

struct espo_oracle_row_state {
  double z;          // smoothed cumulative regret
  double sum_g;      // running sums over this trajectory's tokens (for the batch statistics of Eq. 7-8)
  double sum_g2;
  int64_t n_tokens;
  int32_t t;         // tokens generated so far
  int32_t status;
  int32_t t_stop;    // index of the stop step, -1 if none
  int32_t pad_;
};

struct espo_oracle_step_out {
  double g, g_tilde, z, logp;
  double max_x, log_s;           // max_a x_a and log sum_a exp(x_a - max_x)
  double min_rel_gap;            // smallest top-two relative gap over the argmaxes taken
  double threshold;              // beta * max(V, eps)
  double entropy;                // H(pi(.|s_t)) = -sum_a pi(a) log pi(a), the quantity tracked in the analysis section
  int32_t token;
  int32_t stop;
  int32_t runner_up;             // token that the closest argmax would have produced instead (-1 unknown)
  int32_t bad;                   // 1: row had NaN / +inf / no finite logit
  // filtered sampling only: size of the support, and how far the nearest keep/drop decision was from flipping
  // (distance of the mass above the last kept and above the first dropped value from top_p; inf without top-p)
  double filter_margin;
  int64_t kept;
};

void espo_oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  philox4x32_10(ctr, key, out);
}

double espo_oracle_uniform(uint64_t seed, uint64_t batch_id, uint32_t slot, uint32_t step,
                           int level, uint64_t index) {
  DrawKey dk{seed, batch_id, slot, step};
  return uniform_for(dk, level, index);
}

void espo_oracle_init_row(espo_oracle_row_state* st) {
  std::memset(st, 0, sizeof(*st));
  st->t_stop = -1;
  st->status = ORACLE_ACTIVE;
}

// Full log-softmax of one row (used by the pins): out[a] = x_a - max - log s.
void espo_oracle_log_softmax(const double* logits, int64_t V, double temperature, double* out) {
  std::vector<double> x(V);
  for (int64_t a = 0; a < V; ++a) x[a] = logits[a] / temperature;
  const double lse = log_sum_exp(x.data(), 0, V);
  for (int64_t a = 0; a < V; ++a) out[a] = x[a] - lse;
}

// One pass of Algorithm 1's loop body for one trajectory.
//   logits        [V] the row, already widened exactly to double
//   value         V_phi(s_t) for the same position
//   forced_token  >= 0: skip the draw and take this token (used to re-align the
//                 oracle after a counted near-tie); -1: sample
// A row that is not ACTIVE is left untouched (token -1, stop 0).
void espo_oracle_step_row(const double* logits, int64_t V, double value,
                          uint64_t seed, uint64_t batch_id, uint32_t slot,
                          const espo_oracle_params* p, int32_t forced_token,
                          espo_oracle_row_state* st, espo_oracle_step_out* out) {
  std::memset(out, 0, sizeof(*out));
  out->token = -1;
  out->runner_up = -1;
  out->min_rel_gap = std::numeric_limits<double>::infinity();
  if (st->status != ORACLE_ACTIVE) return;

  // Row screening: NaN or +inf anywhere, or nothing finite, makes the row unusable.
  bool any_finite = false, poisoned = false;
  for (int64_t a = 0; a < V; ++a) {
    const double l = logits[a];
    if (std::isnan(l) || l == std::numeric_limits<double>::infinity()) poisoned = true;
    else if (l != NEG_INF) any_finite = true;
  }
  if (poisoned || !any_finite) {
    out->bad = 1;
    out->token = 0;
    st->status = ORACLE_BAD;
    return;
  }

  const bool greedy = (p->temperature == 0.0);
  std::vector<double> x(V);
  for (int64_t a = 0; a < V; ++a) x[a] = greedy ? logits[a] : logits[a] / p->temperature;

  double m = NEG_INF;
  int64_t first_argmax = 0;
  for (int64_t a = 0; a < V; ++a) if (x[a] > m) { m = x[a]; first_argmax = a; }
  double s = 0.0;
  for (int64_t a = 0; a < V; ++a) s += std::exp(x[a] - m);
  out->max_x = m;
  out->log_s = std::log(s);
  {
    // entropy of the sampling distribution, term by term (0 log 0 = 0 for masked ids)
    double h = 0.0;
    for (int64_t a = 0; a < V; ++a) {
      const double lp = x[a] - m - out->log_s;
      if (lp > NEG_INF) h -= std::exp(lp) * lp;
    }
    out->entropy = greedy ? 0.0 : h;
  }

  const DrawKey dk{seed, batch_id, slot, (uint32_t)st->t};
  int64_t token = -1;
  double filtered_log_s = out->log_s;   // log of the support's mass relative to exp(m); the whole row without a filter
  out->filter_margin = std::numeric_limits<double>::infinity();
  out->kept = V;
  if (forced_token >= 0) {
    token = forced_token;
  } else if (greedy) {
    token = first_argmax;
  } else if (p->sampler == 0 && (p->top_k > 0 || p->top_p < 1.0)) {
    // ---- support of the filtered distribution, from its definition: ids ordered by decreasing probability,
    //      groups of equal probability taken as a whole ----
    std::vector<int64_t> order(V);
    for (int64_t a = 0; a < V; ++a) order[a] = a;
    std::sort(order.begin(), order.end(), [&](int64_t a, int64_t b) { return x[a] > x[b] || (x[a] == x[b] && a < b); });
    std::vector<char> keep(V, 0);
    double mass_above = 0.0;        // probability of everything strictly more probable than the current group
    int64_t count_above = 0;
    double margin = std::numeric_limits<double>::infinity();
    int64_t kept = 0;
    for (int64_t i = 0; i < V;) {
      int64_t j = i;
      double group = 0.0;
      while (j < V && x[order[j]] == x[order[i]]) { group += std::exp(x[order[j]] - m) / s; ++j; }
      const bool in_p = (p->top_p >= 1.0) || (mass_above < p->top_p);
      const bool in_k = (p->top_k <= 0) || (count_above < p->top_k);
      if (p->top_p < 1.0 && x[order[i]] > NEG_INF) margin = std::fmin(margin, std::fabs(mass_above - p->top_p));
      if (!(in_p && in_k)) break;   // every later group has at least this much above it
      for (int64_t q = i; q < j; ++q) if (x[order[q]] > NEG_INF) { keep[order[q]] = 1; ++kept; }
      mass_above += group;
      count_above += j - i;
      i = j;
    }
    out->filter_margin = margin;
    out->kept = kept;
    double s_kept = 0.0;
    for (int64_t a = 0; a < V; ++a) if (keep[a]) s_kept += std::exp(x[a] - m);
    filtered_log_s = std::log(s_kept);
    ArgmaxResult r = perturbed_argmax(0, V, [&](int64_t a) { return keep[a] ? x[a] + gumbel_for(dk, 0, (uint64_t)a) : NEG_INF; });
    token = r.index;
    out->min_rel_gap = relative_gap(r.best, r.second);
    out->runner_up = (int32_t)r.runner;
  } else if (p->sampler == 0) {
    ArgmaxResult r = perturbed_argmax(0, V, [&](int64_t a) { return x[a] + gumbel_for(dk, 0, (uint64_t)a); });
    token = r.index;
    out->min_rel_gap = relative_gap(r.best, r.second);
    out->runner_up = (int32_t)r.runner;
  } else {
    const int64_t BLOCK = 1024, SUB = 32;
    const int64_t n_blocks = (V + BLOCK - 1) / BLOCK;
    ArgmaxResult rb = perturbed_argmax(0, n_blocks, [&](int64_t b) {
      const int64_t lo = b * BLOCK, hi = std::min<int64_t>(V, lo + BLOCK);
      return log_sum_exp(x.data(), lo, hi) + gumbel_for(dk, 2, (uint64_t)b);
    });
    const int64_t b_lo = rb.index * BLOCK, b_hi = std::min<int64_t>(V, b_lo + BLOCK);
    const int64_t j_lo = b_lo / SUB, j_hi = (b_hi + SUB - 1) / SUB;
    ArgmaxResult rj = perturbed_argmax(j_lo, j_hi, [&](int64_t j) {
      const int64_t lo = j * SUB, hi = std::min<int64_t>(V, lo + SUB);
      return log_sum_exp(x.data(), lo, hi) + gumbel_for(dk, 1, (uint64_t)j);
    });
    const int64_t a_lo = rj.index * SUB, a_hi = std::min<int64_t>(V, a_lo + SUB);
    ArgmaxResult ra = perturbed_argmax(a_lo, a_hi, [&](int64_t a) { return x[a] + gumbel_for(dk, 0, (uint64_t)a); });
    token = ra.index;
    const double gb = relative_gap(rb.best, rb.second);
    const double gj = relative_gap(rj.best, rj.second);
    const double ga = relative_gap(ra.best, ra.second);
    out->min_rel_gap = std::fmin(gb, std::fmin(gj, ga));
    if (ga <= gb && ga <= gj) out->runner_up = (int32_t)ra.runner;
  }

  // Eq. 6: the normaliser cancels in the difference of the two log-probabilities.
  const double x_tok = x[token];
  const double g = greedy ? 0.0 : (m - x_tok);
  const double logp = greedy ? 0.0 : (x_tok - m - filtered_log_s);   // under the distribution the token was drawn from

  // Eq. 9 with the frozen batch statistics.
  double gt = (g - p->mu_g) / std::sqrt(p->sigma2_g + p->delta);
  if (gt > p->clip_c) gt = p->clip_c;
  if (gt < -p->clip_c) gt = -p->clip_c;

  // Eq. 10: updated on every step, warm-up or not (Algorithm 1 updates z before the gated test).
  const double z = p->alpha_s * st->z + (1.0 - p->alpha_s) * gt;

  // Eq. 11, strict inequality; a NaN value estimate never stops.  The ablation's rules replace the inequality.
  const double thr = p->beta * std::fmax(value, p->eps);
  bool rule = false;
  if (p->stop_mode == 0) rule = !std::isnan(value) && (z > thr);
  else if (p->stop_mode == 1) rule = !std::isnan(value) && (value < p->tau);
  else if (p->stop_mode == 2) rule = (z > p->tau);
  else rule = (uniform_for(dk, 3, 0) < p->p_random);       // one more draw of the step's Philox stream: level 3, index 0
  const bool fires = (p->warmup_complete != 0) && rule;

  st->z = z;
  st->sum_g += g;
  st->sum_g2 += g * g;
  st->n_tokens += 1;
  const int32_t t_now = st->t;
  st->t = t_now + 1;

  int32_t stop = 0;
  if (p->eos_token >= 0 && token == p->eos_token) {
    st->status = ORACLE_EOS;
  } else if (fires && p->shadow) {
    if (st->t_stop < 0) st->t_stop = t_now;                // remembered, not acted upon
    if (st->t >= p->t_max) st->status = ORACLE_TMAX;
  } else if (fires) {
    st->status = ORACLE_STOPPED;
    st->t_stop = t_now;
    stop = 1;
  } else if (st->t >= p->t_max) {
    st->status = ORACLE_TMAX;
  }

  out->g = g; out->g_tilde = gt; out->z = z; out->logp = logp;
  out->threshold = thr;
  out->token = (int32_t)token;
  out->stop = stop;
}

// The same step over n_rows independent rows, rows split over n_threads host threads.
//   logits   [n_rows, V] doubles, row-major
//   row_ids  [n_rows] trajectory slot of each row, or null for identity
//   states   indexed by slot;  outs indexed by row
void espo_oracle_step_batch(const double* logits, int64_t V, const double* values,
                            const int32_t* row_ids, int32_t n_rows,
                            uint64_t seed, uint64_t batch_id,
                            const espo_oracle_params* p, const int32_t* forced_tokens,
                            espo_oracle_row_state* states, espo_oracle_step_out* outs,
                            int32_t n_threads) {
  auto work = [&](int32_t r0, int32_t r1) {
    for (int32_t r = r0; r < r1; ++r) {
      const int32_t slot = row_ids ? row_ids[r] : r;
      espo_oracle_step_row(logits + (int64_t)r * V, V, values[r], seed, batch_id, (uint32_t)slot, p,
                           forced_tokens ? forced_tokens[r] : -1, &states[slot], &outs[r]);
    }
  };
  if (n_threads <= 1 || n_rows <= 1) { work(0, n_rows); return; }
  if (n_threads > n_rows) n_threads = n_rows;
  std::vector<std::thread> pool;
  for (int32_t k = 0; k < n_threads; ++k) {
    const int32_t r0 = (int32_t)((int64_t)n_rows * k / n_threads);
    const int32_t r1 = (int32_t)((int64_t)n_rows * (k + 1) / n_threads);
    pool.emplace_back(work, r0, r1);
  }
  for (auto& th : pool) th.join();
}

// Same as above for float32 rows widened on the fly (lets the timed CPU baseline
// run without a [n_rows, V] double copy of a large batch).  Widening is exact.
void espo_oracle_step_batch_f32(const float* logits, int64_t V, const double* values,
                                const int32_t* row_ids, int32_t n_rows,
                                uint64_t seed, uint64_t batch_id,
                                const espo_oracle_params* p,
                                espo_oracle_row_state* states, espo_oracle_step_out* outs,
                                int32_t n_threads) {
  auto work = [&](int32_t r0, int32_t r1) {
    std::vector<double> row(V);
    for (int32_t r = r0; r < r1; ++r) {
      const float* src = logits + (int64_t)r * V;
      for (int64_t a = 0; a < V; ++a) row[a] = (double)src[a];
      const int32_t slot = row_ids ? row_ids[r] : r;
      espo_oracle_step_row(row.data(), V, values[r], seed, batch_id, (uint32_t)slot, p, -1,
                           &states[slot], &outs[r]);
    }
  };
  if (n_threads <= 1 || n_rows <= 1) { work(0, n_rows); return; }
  if (n_threads > n_rows) n_threads = n_rows;
  std::vector<std::thread> pool;
  for (int32_t k = 0; k < n_threads; ++k) {
    const int32_t r0 = (int32_t)((int64_t)n_rows * k / n_threads);
    const int32_t r1 = (int32_t)((int64_t)n_rows * (k + 1) / n_threads);
    pool.emplace_back(work, r0, r1);
  }
  for (auto& th : pool) th.join();
}

// ---------------------------------------------------------------------------
// Advantages over ragged, truncated trajectories (Eq. 4-5 with the failure
// transition of Eq. 13).  Trajectory i owns tokens [off_i, off_i + L_i) of the
// packed arrays, off = exclusive prefix sum of lengths.
//   r'_t = rewards[t], except r'_{L-1} = r_fail when stopped[i] (replaces, not adds)
//   V_L := 0 for every trajectory: nothing is bootstrapped past its last token
//   delta_t = r'_t + gamma V_{t+1} - V_t
// ---------------------------------------------------------------------------

// Literal Eq. 5: A_t = sum_{l=0}^{L-1-t} (gamma*lambda)^l delta_{t+l}.  O(L^2).
void espo_oracle_advantages_direct(const double* rewards, const double* values,
                                   const int32_t* lengths, const uint8_t* stopped, int32_t B,
                                   double gamma, double lambda, double r_fail, double* adv_out) {
  int64_t off = 0;
  for (int32_t i = 0; i < B; ++i) {
    const int64_t L = lengths[i];
    std::vector<double> delta(L > 0 ? L : 0);
    for (int64_t t = 0; t < L; ++t) {
      double r = rewards[off + t];
      if (t == L - 1 && stopped[i]) r = r_fail;
      const double v_next = (t + 1 < L) ? values[off + t + 1] : 0.0;
      delta[t] = r + gamma * v_next - values[off + t];
    }
    for (int64_t t = 0; t < L; ++t) {
      double acc = 0.0;
      for (int64_t l = 0; t + l < L; ++l) acc += std::pow(gamma * lambda, (double)l) * delta[t + l];
      adv_out[off + t] = acc;
    }
    off += L;
  }
}

// The equivalent backward recursion A_t = delta_t + gamma*lambda*A_{t+1}, A_L = 0.  O(L).
void espo_oracle_advantages(const double* rewards, const double* values,
                            const int32_t* lengths, const uint8_t* stopped, int32_t B,
                            double gamma, double lambda, double r_fail, double* adv_out) {
  int64_t off = 0;
  for (int32_t i = 0; i < B; ++i) {
    const int64_t L = lengths[i];
    double a_next = 0.0, v_next = 0.0;
    for (int64_t t = L - 1; t >= 0; --t) {
      double r = rewards[off + t];
      if (t == L - 1 && stopped[i]) r = r_fail;
      const double delta = r + gamma * v_next - values[off + t];
      a_next = delta + gamma * lambda * a_next;
      adv_out[off + t] = a_next;
      v_next = values[off + t];
    }
    off += L;
  }
}

// float32 inputs widened on the fly, trajectories split over host threads (timed CPU baseline).
void espo_oracle_advantages_f32(const float* rewards, const float* values,
                                const int32_t* lengths, const uint8_t* stopped, int32_t B,
                                double gamma, double lambda, double r_fail, double* adv_out,
                                int32_t n_threads) {
  std::vector<int64_t> off(B + 1, 0);
  for (int32_t i = 0; i < B; ++i) off[i + 1] = off[i] + lengths[i];
  auto work = [&](int32_t i0, int32_t i1) {
    for (int32_t i = i0; i < i1; ++i) {
      const int64_t L = lengths[i], o = off[i];
      double a_next = 0.0, v_next = 0.0;
      for (int64_t t = L - 1; t >= 0; --t) {
        double r = (double)rewards[o + t];
        if (t == L - 1 && stopped[i]) r = r_fail;
        const double v = (double)values[o + t];
        const double delta = r + gamma * v_next - v;
        a_next = delta + gamma * lambda * a_next;
        adv_out[o + t] = a_next;
        v_next = v;
      }
    }
  };
  if (n_threads <= 1 || B <= 1) { work(0, B); return; }
  if (n_threads > B) n_threads = B;
  std::vector<std::thread> pool;
  for (int32_t k = 0; k < n_threads; ++k)
    pool.emplace_back(work, (int32_t)((int64_t)B * k / n_threads), (int32_t)((int64_t)B * (k + 1) / n_threads));
  for (auto& th : pool) th.join();
}

// ---------------------------------------------------------------------------
// Batch boundary (Sec. 4.2, Eq. 7-8; Sec. 4.3, Eq. 12).  After a rollout batch:
//   g_B      = every regret value generated in the batch (all tokens of all
//              trajectories that took part, stop-step tokens included)
//   mu_g     <- a_ema mu_g     + (1 - a_ema) mean(g_B)
//   sigma_g2 <- a_ema sigma_g2 + (1 - a_ema) Var(g_B)        (population variance)
//   beta     <- clip(beta + eta_beta (rho_stop - tau), beta_min, beta_max)
// rho_stop = stopped trajectories / trajectories that took part (t > 0).  With
// first_update != 0 the statistics are set to the batch values (nothing to average with
// yet).  An empty batch changes nothing.  out6 = {mean, var, rho_stop, tokens, trajectories,
// stopped}.
// ---------------------------------------------------------------------------
void espo_oracle_end_batch(const espo_oracle_row_state* states, int32_t n_slots,
                           double alpha_ema, double eta_beta, double tau, double beta_min, double beta_max,
                           int32_t first_update, double* mu_g, double* sigma2_g, double* beta, double* out6) {
  double sg = 0.0, sg2 = 0.0;
  int64_t n_tok = 0, n_traj = 0, n_stop = 0;
  for (int32_t i = 0; i < n_slots; ++i) {
    if (states[i].t <= 0) continue;
    sg += states[i].sum_g;
    sg2 += states[i].sum_g2;
    n_tok += states[i].n_tokens;
    n_traj += 1;
    if (states[i].status == ORACLE_STOPPED) n_stop += 1;
  }
  double mean = 0.0, var = 0.0, rho = 0.0;
  if (n_tok > 0) {
    mean = sg / (double)n_tok;
    var = sg2 / (double)n_tok - mean * mean;
    if (var < 0.0) var = 0.0;
    rho = (double)n_stop / (double)n_traj;
    if (first_update) { *mu_g = mean; *sigma2_g = var; }
    else {
      *mu_g = alpha_ema * (*mu_g) + (1.0 - alpha_ema) * mean;
      *sigma2_g = alpha_ema * (*sigma2_g) + (1.0 - alpha_ema) * var;
    }
    double b = *beta + eta_beta * (rho - tau);
    if (b < beta_min) b = beta_min;
    if (b > beta_max) b = beta_max;
    *beta = b;
  }
  if (out6) { out6[0] = mean; out6[1] = var; out6[2] = rho; out6[3] = (double)n_tok; out6[4] = (double)n_traj; out6[5] = (double)n_stop; }
}

}  // extern "C"
