// ESPO decode-step kernel for sm_100a and the C entry points around it.
//
// One launch performs, for every logit row of the batch, the body of the rollout loop
// (Algorithm 1): log-softmax statistics, Gumbel-max sampling, the surrogate regret of
// Eq. 6, its normalisation (Eq. 9) and smoothing (Eq. 10), the value-gated stop test
// (Eq. 11) and the per-trajectory bookkeeping.
//
// Shape of the kernel
//   * The [n_rows, V] logits are a sequence of n_rows * ceil(V/1024) blocks of 1024 ids.  A
//     persistent grid (a multiple of the SM count) splits that sequence into equal contiguous
//     ranges, so every SM streams the same number of bytes whatever n_rows is.
//   * Inside a CTA every streaming warp owns a private ring of shared-memory stages, one block
//     each.  Its lane 0 fetches the warp's next blocks with bulk asynchronous copies (TMA
//     without a tensor map) that complete on the stage's mbarrier; the warp reduces a block
//     to (max logit, sum of exp) -- plus, for the flat sampler, the block's best perturbed
//     score -- writes that record to a per-row table in global memory and refills the stage.
//     Warps never wait for one another.
//   * A row may be spread over several CTAs.  The warps of a CTA count the blocks they have
//     contributed to a row in shared memory; when the CTA's share of the row is complete the
//     row is posted to a small queue.  The CTA's finalizer warp (and, once they run out of
//     blocks, the streaming warps) take rows from the queue, add the CTA's share to the
//     row's ticket in global memory, and whoever completes the ticket merges the block
//     records in a fixed order (so results do not depend on the grid), draws the token,
//     applies Eq. 6, 9, 10, 11 and writes the outputs and the trajectory state.
//   * A CTA walks its range starting with the row it shares with the next CTA, then the row it
//     shares with the previous one, then its whole rows: shared rows complete early in the
//     launch instead of all at its end.
//   * Every wait in the kernel is bounded; a wait that runs out sets ESPO_DEV_TIMEOUT.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <new>

#include "espo.h"
#include "espo_device.cuh"
#include "espo_host.h"
#include "espo_step_common.cuh"
#include "espo_step_hier.cuh"

namespace espo {

// All perturbed scores below are "x/T + G" on the absolute scale of the logits, with the
// Gumbel written through its exponential draw E = -ln u:  G = -ln E, and for a group with
// log-sum-exp  m/T + ln s  the score is  m/T + ln(s / E).
template <int ES, int SAMPLER>
__device__ __noinline__ void finalize_row(const StepArgs& a, int row, int lane, const RowPre pre, const void* rec_row,
                                          bool rec_local, bool no_ticket, const float* noise) {
  const float NINF = __int_as_float(0xff800000);
  // only the flat sampler's kernels serve vocabulary shards
  const bool partial = (SAMPLER == ESPO_SAMPLER_FLAT) && a.partial_out != nullptr;
  const int slot = pre.slot;
  // A vocabulary shard reports instead of acting: `flags` tells the merge what happened (bit 0: the shard's part of
  // the row held NaN or +inf; bit 1: nothing was computed because the slot is bad or the trajectory has ended).
  auto report = [&](unsigned flags) {
    if (lane == 0) {
      espo_partial pr;
      pr.m = NINF; pr.s = 0.f; pr.best = NINF; pr.best_id = -1; pr.x_best = NINF; pr.flags = flags; pr.reserved[0] = 0u; pr.reserved[1] = 0u;
      a.partial_out[row] = pr;
      if (!no_ticket) a.ticket[row] = 0;
    }
  };
  if (slot < 0) { if (partial) report(2u); else mark_row(a, row, 0, lane, -1, ESPO_DEV_BAD_SLOT, -1, no_ticket); return; }
  if (pre.status != ESPO_ROW_ACTIVE) {   // finished: untouched
    if (partial) report(2u); else mark_row(a, row, slot, lane, -1, 0u, -1, no_ticket);
    return;
  }
  const int t_now = pre.t_now;
  const unsigned char* row_base = a.logits + (size_t)row * a.row_stride_bytes;
  const DrawStream ds{a.key0, a.key1, (uint32_t)t_now, (uint32_t)slot, a.batch_bits};

  // ---- one pass over the row's block records (m_b, s_b, third, fourth); lane l takes blocks l, l+32, ...
  //      HIER: the block's perturbed score is m_b/T + ln s_b - ln E_b; `noise` (may be null) holds ln E_b
  //      for every block of the row, prepared ahead of time by the CTA's finalizer warp;
  //      FLAT: third = best perturbed score inside the block relative to m_b/T, fourth = its id.
  //      Running (max, sum) per lane gives S = sum_b s_b exp((m_b - M)/T). ----
  float best = NINF;          // best perturbed score among this lane's blocks (greedy: largest block maximum)
  int best_i = -1;            // HIER / greedy: block number; FLAT: token id
  bool poisoned = false;
  float run_m = NINF, run_s = 0.f, run_u = 0.f;   // sums of e and of e*t over this lane's blocks, relative to run_m
  // The pass is one warp's latency chain for every row, so it is written without data-dependent branches: the five
  // records of a lane are loaded, summed and scored as five independent strands.
  constexpr int kPerLane = 5;                   // records a lane holds at once (covers V <= 163840 in one go)
  for (int base = 0; base < a.nblk; base += 32 * kPerLane) {
    float4 r[kPerLane];
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
      const int b = base + 32 * i + lane;
      // shared-memory table or global records written by other CTAs: one generic load that bypasses L1 serves both
      r[i] = (b < a.nblk) ? ld_volatile_f4(static_cast<const float4*>(rec_row) + b) : make_float4(NINF, 0.f, NINF, __int_as_float(-1));
    }
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
      // The block's exponents were all off by dlt = fl(-m_b*k2) + m_b*k2 (reduce_block), which the fused
      // multiply-add returns exactly: s_b and u_b carry a factor 2^dlt (and u_b the shift dlt*s_b), taken out here.
      // dlt is half an ulp of m_b*k2 at most: 1e-5 for logits of some tens at low temperature, more for rows that
      // sit at a large offset.
      const float dlt = fmaf(r[i].x, a.k2, -r[i].x * a.k2);
      if (r[i].y > 0.f && !isinf(r[i].y)) {
        const float f = ex2_approx(-dlt);
        const float s_c = r[i].y * f;
        if (SAMPLER == ESPO_SAMPLER_HIER) r[i].z = fmaf(r[i].z, f, -dlt * s_c);
        r[i].y = s_c;
      }
    }
    float lm = run_m;
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
      poisoned |= !(r[i].y >= 0.0f) || isinf(r[i].y);   // NaN or inf sum: the block held NaN or +inf
      lm = (r[i].y > 0.f) ? fmaxf(lm, r[i].x) : lm;
    }
    // sum of s_b 2^((m_b - lm) k2), independent terms; the carried sums are rescaled once.  Moving the reference
    // from R to R' turns (S, U) into f (S, U + (R - R') k2 S) with f = 2^((R - R') k2).
    float acc = run_s, accu = run_u;
    if (run_m != lm && run_s > 0.f) {
      const float dt = (run_m - lm) * a.k2, f = ex2_approx(dt);
      accu = f * fmaf(dt, run_s, run_u);
      acc = f * run_s;
    }
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
      const bool ok = r[i].y > 0.f;
      const float dt = ok ? (r[i].x - lm) * a.k2 : 0.f, f = ex2_approx(dt);
      acc = ok ? fmaf(r[i].y, f, acc) : acc;
      if (SAMPLER == ESPO_SAMPLER_HIER) accu = ok ? fmaf(f, fmaf(dt, r[i].y, r[i].z), accu) : accu;
    }
    run_m = lm; run_s = acc; run_u = accu;
    if (a.greedy) {
#pragma unroll
      for (int i = 0; i < kPerLane; ++i) {
        const bool take = (r[i].y > 0.f) && (r[i].x > best);          // lowest block holding the maximum
        best = take ? r[i].x : best;
        best_i = take ? base + 32 * i + lane : best_i;
      }
    } else if (SAMPLER == ESPO_SAMPLER_FLAT) {
#pragma unroll
      for (int i = 0; i < kPerLane; ++i) {
        const float sc = fmaf(r[i].x, a.inv_temp, r[i].z);            // the block's best, moved to the absolute scale
        const int id = __float_as_int(r[i].w);
        const bool take = (r[i].y > 0.f) && id >= 0 && (best_i < 0 || sc > best);
        best = take ? sc : best;
        best_i = take ? id : best_i;
      }
    } else {
      float ln_e[kPerLane];
      if (noise) {
#pragma unroll
        for (int i = 0; i < kPerLane; ++i) {
          const int b = base + 32 * i + lane;
          ln_e[i] = (b < a.nblk) ? noise[b] : 0.f;
        }
      } else {
        // the finalizer warp had not prepared this row's block-level noise: draw it here (kept as a loop: it is rare)
#pragma unroll 1
        for (int i = 0; i < kPerLane; ++i) {
          const int b = base + 32 * i + lane;
          const float e = (b < a.nblk) ? ln_expo(expo_at(ds, 2u, (uint32_t)b)) : 0.f;
#pragma unroll
          for (int j = 0; j < kPerLane; ++j) if (j == i) ln_e[j] = e;
        }
      }
#pragma unroll
      for (int i = 0; i < kPerLane; ++i) {
        const float sc = fmaf(r[i].x, a.inv_temp, log_sum(r[i].y) - ln_e[i]);
        const bool take = (r[i].y > 0.f) && (best_i < 0 || sc > best);
        best = take ? sc : best;
        best_i = take ? base + 32 * i + lane : best_i;
      }
    }
  }
  {
    const float mm = warp_max(run_m);
    if (run_m != mm) {
      if (run_s > 0.f) {
        const float dt = (run_m - mm) * a.k2, f = ex2_approx(dt);
        run_u = f * fmaf(dt, run_s, run_u);
        run_s *= f;
      } else {
        run_s = 0.f; run_u = 0.f;     // a lane without blocks (run_m = -inf)
      }
    }
    run_m = mm;
    run_s = warp_sum(run_s);
    if (a.want_entropy) run_u = warp_sum(run_u);
  }
  const float M = run_m, S = run_s;
  const float log_S = logf(S);   // needed at the very end; started before the loads below
  // (a shard may hold no finite logit at all; a whole row may not)
  poisoned = __any_sync(kFullMask, poisoned) || M == __int_as_float(0x7f800000) || M != M;
  poisoned = poisoned || (!partial && (!(M > NINF) || isinf(M)));
  if (poisoned) { if (partial) report(1u); else mark_row(a, row, slot, lane, 0, ESPO_DEV_BAD_ROW, ESPO_ROW_BAD, no_ticket); return; }
  warp_argmax(best, best_i);
  if (best_i < 0) {   // nothing to pick from
    if (partial) report(0u); else mark_row(a, row, slot, lane, 0, ESPO_DEV_BAD_ROW, ESPO_ROW_BAD, no_ticket);
    return;
  }

  int token;
  float l_tok;
  if (a.greedy || SAMPLER == ESPO_SAMPLER_HIER) {
    // ---- look inside the chosen block: lane j owns sub-block j (32 consecutive ids) ----
    const int blk_lo = best_i * kBlockIds;
    const int sub_lo = blk_lo + lane * kSubIds;
    const int n_here = min(kSubIds, a.V - sub_lo);    // <= 0: sub-block lies beyond V
    float x[kSubIds];
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(row_base) & 15u) == 0) && (n_here == kSubIds);
    if (vec_ok) {
      const uint4* vp = reinterpret_cast<const uint4*>(row_base + (size_t)sub_lo * ES);
      if (ES == 2) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint4 q = __ldg(vp + i);
          const uint32_t ww[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
          for (int k = 0; k < 4; ++k) { x[8 * i + 2 * k] = bf16_lo(ww[k]); x[8 * i + 2 * k + 1] = bf16_hi(ww[k]); }
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint4 q = __ldg(vp + i);
          x[4 * i] = __uint_as_float(q.x); x[4 * i + 1] = __uint_as_float(q.y);
          x[4 * i + 2] = __uint_as_float(q.z); x[4 * i + 3] = __uint_as_float(q.w);
        }
      }
    } else {
#pragma unroll
      for (int i = 0; i < kSubIds; ++i) x[i] = (i < n_here) ? load_logit<ES>(row_base, sub_lo + i) : NINF;
    }

    // the sub-block's noise does not depend on the data: drawn while the loads above are in flight
    const float ln_e1 = a.greedy ? 0.f : ln_expo(expo_at(ds, 1u, (uint32_t)(sub_lo >> 5)));   // index = global sub-block number
    if (a.greedy) {
      // first id equal to the maximum
      int first = -1;
#pragma unroll
      for (int i = kSubIds - 1; i >= 0; --i) if (x[i] == M) first = sub_lo + i;
      float key = 0.f;
      warp_argmax(key, first);           // equal keys: lowest id wins
      token = max(first, blk_lo);
      l_tok = M;
    } else {
      float m_j = NINF;
#pragma unroll
      for (int i = 0; i < kSubIds; ++i) m_j = fmaxf(m_j, x[i]);
      float sc = NINF;
      int j = -1;
      if (m_j > NINF) {
        const float s_j = sum_exp2_32(x, m_j, a.k2);
        sc = fmaf(m_j, a.inv_temp, log_sum(s_j) - ln_e1);
        j = sub_lo >> 5;
      }
      warp_argmax(sc, j);
      const int sub_pick = max(j, blk_lo >> 5);        // j < 0 cannot happen: the block has a finite id
      // ---- ids of the chosen sub-block: lane e takes id 32*sub_pick + e ----
      const int id = sub_pick * kSubIds + lane;
      const float mine = (id < a.V) ? load_logit<ES>(row_base, id) : NINF;   // the lines are in L1 since the loads above
      float sc0 = NINF;
      int cand = -1;
      if (id < a.V && mine > NINF) { sc0 = fmaf(mine, a.inv_temp, -ln_expo(expo_at(ds, 0u, (uint32_t)id))); cand = id; }
      warp_argmax(sc0, cand);
      token = max(cand, sub_pick * kSubIds);           // cand < 0 cannot happen for a sub-block with a finite id
      l_tok = __shfl_sync(kFullMask, mine, token & 31);
    }
  } else {
    token = best_i;                                             // a global id
    l_tok = load_logit<ES>(row_base, token - a.vocab_offset);
  }
  if (a.greedy || SAMPLER == ESPO_SAMPLER_HIER) token += a.vocab_offset;

  if (partial) {
    // a vocabulary shard: leave what the merge needs and do not touch the state
    if (lane == 0) {
      espo_partial pr;
      pr.m = M; pr.s = S; pr.best = best; pr.best_id = token; pr.x_best = l_tok; pr.flags = 0u; pr.reserved[0] = 0u; pr.reserved[1] = 0u;
      a.partial_out[row] = pr;
      if (!no_ticket) a.ticket[row] = 0;   // ready for the next launch
    }
    return;
  }
  if (lane == 0) commit_row(a, row, pre, ds, M, S, log_S, run_u, l_tok, token, no_ticket);
}

// -------------------------------------------------------------------------------------------
// The kernel.
// -------------------------------------------------------------------------------------------

// Take rows from the CTA's queue until none are left: add the CTA's share to the row's ticket
// and finalize the row if that completed it.  Entry h is claimed before it is waited for, so
// each entry is handled by exactly one warp.
// Shared-memory tables a CTA keeps about the rows its range touches (indexed by local row).
struct RowTables {
  volatile int* queue;     // [queue_cap] local rows whose share of this CTA is complete, in completion order
  volatile int* ready;     // [queue_cap] 1: pre[k] (and noise row k, if k < noise_rows) are filled in
  RowPre* pre;             // [queue_cap]
  float* noise;            // [noise_rows][nblk] ln E of the block-level draws (hierarchical sampler)
  unsigned char* lrec;     // [local_rows][nblk] records of rows that lie wholly inside the range
};

// Take rows from the CTA's queue until none are left: add the CTA's share to the row's ticket
// and finalize the row if that completed it.  Entry h is claimed before it is waited for, so
// each entry is handled by exactly one warp.
template <int ES, int SAMPLER>
__device__ void drain_queue(const StepArgs& a, const CtaRange& cr, StepCtrl* ctrl, const RowTables& tb, int lane) {
  constexpr int kRecBytes = 16;
  volatile int* abort_flag = &ctrl->abort_flag;
  for (;;) {
    int h = 0;
    if (lane == 0) h = atomicAdd(&ctrl->head, 1);
    h = __shfl_sync(kFullMask, h, 0);
    if (h >= cr.n_local) return;
    int k = -1;
    if (lane == 0) {
      for (uint32_t it = 0; it < kPollSpinLimit; ++it) {
        k = tb.queue[h];
        if (k >= 0 || *abort_flag) break;
        __nanosleep(32);
      }
      if (k < 0 && !*abort_flag) { atomicOr(a.dev_status, ESPO_DEV_TIMEOUT); *abort_flag = 1; }
      __threadfence_block();                             // what the posting warp published before the entry
    }
    k = __shfl_sync(kFullMask, k, 0);
    if (k < 0) return;
    const int row = (int)(cr.r_first + k);
    // the row's state and noise: from the tables if the finalizer warp got that far, else fetched here
    const bool have = tb.ready[k] != 0;
    __threadfence_block();
    const RowPre pre = have ? tb.pre[k] : prefetch_row(a, row);
    const float* noise = (have && SAMPLER == ESPO_SAMPLER_HIER && !a.greedy && k < a.noise_rows)
                             ? tb.noise + (size_t)k * a.nblk : nullptr;
    const int li = cr.local_index(k, a.local_rows);
    if (li >= 0) {
      // every record of the row was written by this CTA, into its shared-memory table
      __syncwarp();
      finalize_row<ES, SAMPLER>(a, row, lane, pre, tb.lrec + (size_t)li * a.nblk * kRecBytes, true, true, noise);
      continue;
    }
    const unsigned share = (unsigned)cr.share(k);
    if (share == (unsigned)a.nblk) {
      // the row lies wholly inside this CTA's range but did not fit the shared-memory table: its records are in
      // global memory, all written by this CTA, so no other CTA has to be heard from
      __syncwarp();
      finalize_row<ES, SAMPLER>(a, row, lane, pre,
                                reinterpret_cast<const unsigned char*>(a.records) + (size_t)row * a.nblk * kRecBytes, false,
                                true, noise);
      continue;
    }
    unsigned old = 0;
    if (lane == 0) old = atom_add_acq_rel_gpu(a.ticket + row, share);   // the CTA's records before its ticket
    old = __shfl_sync(kFullMask, old, 0);
    __syncwarp();
    if (old + share == (unsigned)a.nblk)                 // this CTA completed the row
      finalize_row<ES, SAMPLER>(a, row, lane, pre,
                                reinterpret_cast<const unsigned char*>(a.records) + (size_t)row * a.nblk * kRecBytes, false,
                                false, noise);
  }
}

// The finalizer warp's first job, while the streaming warps fetch their first blocks: read the
// state of every row the range touches and draw the block-level noise of those rows.
template <int SAMPLER>
__device__ void prepare_rows(const StepArgs& a, const CtaRange& cr, const RowTables& tb, int lane, int first, int step) {
  for (int k = first; k < cr.n_local; k += step) {
    const int row = (int)(cr.r_first + k);
    const RowPre pre = prefetch_row(a, row);
    if (lane == 0) tb.pre[k] = pre;
    if (SAMPLER == ESPO_SAMPLER_HIER && !a.greedy && k < a.noise_rows && pre.slot >= 0 && pre.status == ESPO_ROW_ACTIVE) {
      const DrawStream ds{a.key0, a.key1, (uint32_t)pre.t_now, (uint32_t)pre.slot, a.batch_bits};
      // lane l draws for blocks 4l..4l+3 of every group of 128: one Philox call serves four blocks
      for (int c0 = 0; c0 < a.nblk; c0 += 128) {
        const int b0 = c0 + 4 * lane;
        if (b0 >= a.nblk) continue;
        const uint4 rnd = philox4x32_10((uint32_t)b0 >> 2, ds.step, ds.slot, ds.batch_bits | 2u, ds.k0, ds.k1);
        const uint32_t wd[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (b0 + i < a.nblk) tb.noise[(size_t)k * a.nblk + b0 + i] = ln_expo(expo_from_word(wd[i]));
      }
    }
    __syncwarp();
    if (lane == 0) { __threadfence_block(); tb.ready[k] = 1; }
  }
}

template <int ES, int SAMPLER, bool BULK>
__global__ void __launch_bounds__(kMaxStepThreads, 1) espo_step_kernel(const __grid_constant__ StepArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int W = a.warps, S = a.stages;
  unsigned char* ring = smem;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)W * S * a.stage_bytes);
  int2* metas = reinterpret_cast<int2*>(bars + W * S);
  StepCtrl* ctrl = reinterpret_cast<StepCtrl*>(metas + W * S);
  volatile int* cnt = reinterpret_cast<volatile int*>(ctrl + 1);
  RowTables tb;
  tb.queue = cnt + a.queue_cap;
  tb.ready = tb.queue + a.queue_cap;
  {
    // 16-byte aligned tables after the int arrays
    size_t off = (size_t)W * S * (a.stage_bytes + 16) + sizeof(StepCtrl) + 3 * sizeof(int) * (size_t)a.queue_cap;
    off = (off + 15) & ~(size_t)15;
    tb.pre = reinterpret_cast<RowPre*>(smem + off);
    off += sizeof(RowPre) * (size_t)a.queue_cap;
    tb.noise = reinterpret_cast<float*>(smem + off);
    off += ((sizeof(float) * (size_t)a.noise_rows * a.nblk) + 15) & ~(size_t)15;
    tb.lrec = smem + off;
  }
  volatile int* queue = tb.queue;
  unsigned char* lrec = tb.lrec;
  constexpr int kRecBytes = 16;
  volatile int* abort_flag = &ctrl->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  CtaRange cr;
  {
    const long long g0 = (long long)blockIdx.x * a.total_blocks / gridDim.x;
    const long long g1 = (long long)(blockIdx.x + 1) * a.total_blocks / gridDim.x;
    cr.nblk = a.nblk;
    cr.r_first = g0 / a.nblk;
    cr.b0 = (int)(g0 - cr.r_first * a.nblk);
    cr.n = (int)(g1 - g0);
    const long long r_last = (g1 - 1) / a.nblk;
    cr.n_local = (int)(r_last - cr.r_first) + 1;
    const long long last_start = r_last * a.nblk;       // the walk starts where the last row's part starts
    cr.off = (last_start > g0) ? (int)(last_start - g0) : 0;
  }

  if (threadIdx.x == 0) { ctrl->head = 0; ctrl->posted = 0; ctrl->abort_flag = 0; ctrl->pad = 0; }
  for (int i = threadIdx.x; i < a.queue_cap; i += blockDim.x) { cnt[i] = 0; tb.queue[i] = -1; tb.ready[i] = 0; }
  if (warp < W && lane == 0) {
    for (int s = 0; s < S; ++s) mbar_init(&bars[warp * S + s], 1);
    mbar_init_fence();
  }
  __syncwarp();
  // A streaming warp needs only its own barriers to start fetching; the CTA-wide tables set up above are first
  // touched after the rendezvous (A) that follows the first fetches.

  if (warp < W) {
    // ------------------------------------------------------------------ streaming warps
    unsigned char* my_ring = ring + (size_t)warp * S * a.stage_bytes;
    uint64_t* my_bar = bars + warp * S;
    int2* my_meta = metas + warp * S;            // (local row, block) of the block each stage holds
    // The warps take turns of C consecutive positions of the CTA's walk: warp w owns the runs w, w + W, w + 2W, ...
    // (C = 1 for long rows; short rows use longer runs so that a warp reports to a row once per run, not per block).
    const int C = a.run_len;
    int n_my = 0;
    {
      const int n_runs = (cr.n + C - 1) / C;
      if (n_runs > warp) {
        const int mine = (n_runs - warp + W - 1) / W;            // runs owned by this warp
        n_my = mine * C;
        if ((n_runs - 1) % W == warp) n_my -= n_runs * C - cr.n;  // the walk's last run may be short
      }
    }
    constexpr int kBlockBytes = kBlockIds * ES;

    // Where the warp's next block to fetch lies.  The cursor moves by one block inside a run and by (W-1)C+1
    // between runs, and only divides when the walk wraps around the end of the range.
    int fq, f_lrow, f_blk, f_run = 0;
    const unsigned char* f_ptr;
    auto seek = [&](int q) {
      fq = q;
      const int li = cr.b0 + q;
      f_lrow = li / cr.nblk;
      f_blk = li - f_lrow * cr.nblk;
      f_ptr = a.logits + (size_t)(cr.r_first + f_lrow) * a.row_stride_bytes + (size_t)f_blk * kBlockBytes;
    };
    auto advance = [&]() {
      int step = 1;
      if (++f_run == C) { f_run = 0; step = (W - 1) * C + 1; }
      if (fq + step >= cr.n) { seek(fq + step - cr.n); return; }
      fq += step;
      f_blk += step;
      f_ptr += (size_t)step * kBlockBytes;
      while (f_blk >= cr.nblk) {
        f_blk -= cr.nblk;
        ++f_lrow;
        f_ptr += a.row_stride_bytes - (int64_t)cr.nblk * kBlockBytes;
      }
    };
    {
      int q = warp * C + cr.off;
      if (q >= cr.n) q -= cr.n;
      seek(n_my > 0 ? q : 0);
    }
    auto issue = [&](int s) {   // lane 0: fetch the block under the cursor into stage s
      const uint32_t bytes = (uint32_t)min(kBlockIds, a.V - f_blk * kBlockIds) * ES;
      my_meta[s] = make_int2(f_lrow, f_blk);
      fence_proxy_async();             // the warp's reads of this stage come before the copy's writes
      mbar_arrive_expect_tx(&my_bar[s], bytes);
      bulk_copy_g2s(my_ring + (size_t)s * a.stage_bytes, f_ptr, bytes, &my_bar[s]);
    };
    int fetched = 0;
    if (BULK) {
      for (; fetched < S && fetched < n_my; ++fetched) {
        if (lane == 0) issue(fetched);
        advance();
      }
    }
    cta_rendezvous(blockDim.x);   // (A) the queue, counters and tables are initialised

    int cur_k = -1;
    unsigned mine = 0;
    void* rec_row = nullptr;
    DrawStream ds{a.key0, a.key1, 0u, 0u, a.batch_bits};
    auto flush = [&]() {
      if (lane == 0 && mine > 0) {
        __threadfence_block();                                   // this warp's records before its count
        const int old = atomicAdd(const_cast<int*>(cnt) + cur_k, (int)mine);
        if (old + (int)mine == cr.share(cur_k)) {                // the CTA's share of the row is complete
          __threadfence_block();
          const int qi = atomicAdd(&ctrl->posted, 1);
          if (qi < a.queue_cap) queue[qi] = cur_k;
          else atomicOr(a.dev_status, ESPO_DEV_TIMEOUT);         // cannot happen: the host sizes the queue
        }
      }
      mine = 0;
    };

    int s = 0;
    uint32_t parity = 0;
    int done = 0;
    bool gave_up = false;
    for (; done < n_my; ++done) {
      unsigned char* stage = my_ring + (size_t)s * a.stage_bytes;
      int lrow, blk;
      if (BULK) {
        if (!mbar_wait_bounded(&my_bar[s], parity, abort_flag)) { gave_up = true; break; }
        const int2 mt = my_meta[s];
        lrow = mt.x; blk = mt.y;
      } else {
        lrow = f_lrow; blk = f_blk;
      }
      const int nvalid = min(kBlockIds, a.V - blk * kBlockIds);
      if (!BULK) {
        // element-wise loader for rows that are not 16-byte aligned
        if (ES == 2) {
          const unsigned short* sp = reinterpret_cast<const unsigned short*>(f_ptr);
          unsigned short* dp = reinterpret_cast<unsigned short*>(stage);
          for (int i = lane; i < nvalid; i += 32) dp[i] = __ldg(sp + i);
        } else {
          const float* sp = reinterpret_cast<const float*>(f_ptr);
          float* dp = reinterpret_cast<float*>(stage);
          for (int i = lane; i < nvalid; i += 32) dp[i] = __ldg(sp + i);
        }
        advance();
        __syncwarp();
      }
      if (lrow != cur_k) {
        flush();
        cur_k = lrow;
        const int li = cr.local_index(lrow, a.local_rows);
        rec_row = (li >= 0) ? static_cast<void*>(lrec + (size_t)li * a.nblk * kRecBytes)
                            : static_cast<void*>(reinterpret_cast<unsigned char*>(a.records) +
                                                 (size_t)(cr.r_first + lrow) * a.nblk * kRecBytes);
        if (SAMPLER == ESPO_SAMPLER_FLAT) {
          // the flat sampler perturbs every id, so the streaming warps need the row's draw stream
          const int row = (int)(cr.r_first + lrow);
          int slot = a.row_ids ? __ldg(a.row_ids + row) : row;
          slot = min(max(slot, 0), a.capacity - 1);              // a bad slot is reported by the finalizer
          ds.slot = (uint32_t)slot;
          ds.step = (uint32_t)a.t[slot];
        }
      }
      reduce_block<ES, SAMPLER>(a, stage, lane, nvalid, rec_row, blk, ds);
      ++mine;
      __syncwarp();
      if (BULK) {
        if (fetched < n_my) {
          if (lane == 0) issue(s);
          advance();
          ++fetched;
        }
        if (++s == S) { s = 0; parity ^= 1u; }
      }
    }
    if (gave_up) {
      if (lane == 0) { atomicOr(a.dev_status, ESPO_DEV_TIMEOUT); *abort_flag = 1; }
      // copies still in flight target this CTA's shared memory: give each one more bounded wait
      for (int i = done; BULK && i < fetched; ++i) {
        (void)mbar_wait_bounded(&my_bar[s], parity, nullptr);
        if (++s == S) { s = 0; parity ^= 1u; }
      }
    } else {
      flush();
    }
  }
  // The finalizer warp comes here at once; streaming warps join when they run out of blocks.
  if (warp >= W) {
    cta_rendezvous(blockDim.x);   // (A)
    prepare_rows<SAMPLER>(a, cr, tb, lane, warp - W, a.fin_warps);   // the finalizer warps share the rows
  }
  drain_queue<ES, SAMPLER>(a, cr, ctrl, tb, lane);
}

// -------------------------------------------------------------------------------------------
// Vocabulary shards: one thread per row merges the shards' partial results and commits the row.
// -------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(64) espo_merge_kernel(const __grid_constant__ StepArgs a) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= a.n_rows) return;
  const float NINF = __int_as_float(0xff800000);
  const RowPre pre = prefetch_row(a, row);
  if (pre.slot < 0) { mark_row(a, row, 0, 0, -1, ESPO_DEV_BAD_SLOT, -1, true); return; }
  if (pre.status != ESPO_ROW_ACTIVE) { mark_row(a, row, pre.slot, 0, -1, 0u, -1, true); return; }   // finished: untouched
  // one pass over the shards: running maximum with the sum rescaled whenever the maximum moves
  float M = NINF, S = 0.f, best = NINF, x_best = NINF;
  int best_id = -1;
  bool poisoned = false;
#pragma unroll 4
  for (int k = 0; k < a.n_shards; ++k) {
    const espo_partial pr = a.partials[(long long)k * a.shard_stride + row];
    poisoned |= (pr.flags & 1u) != 0u || !(pr.s >= 0.f) || isinf(pr.s);
    if (pr.s > 0.f) {
      const float Mn = fmaxf(M, pr.m);
      S = S * ex2_approx((M - Mn) * a.k2) + pr.s * ex2_approx((pr.m - Mn) * a.k2);   // M = -inf: S is 0 and stays 0
      M = Mn;
    }
    if (pr.best_id >= 0 && (best_id < 0 || pr.best > best || (pr.best == best && pr.best_id < best_id))) {
      best = pr.best; best_id = pr.best_id; x_best = pr.x_best;      // equal scores: the lowest id wins
    }
  }
  poisoned |= !(M > NINF) || isinf(M);
  if (poisoned) { mark_row(a, row, pre.slot, 0, 0, ESPO_DEV_BAD_ROW, ESPO_ROW_BAD, true); return; }
  if (best_id < 0) { mark_row(a, row, pre.slot, 0, 0, ESPO_DEV_BAD_ROW, ESPO_ROW_BAD, true); return; }
  const DrawStream ds{a.key0, a.key1, (uint32_t)pre.t_now, (uint32_t)pre.slot, a.batch_bits};
  commit_row(a, row, pre, ds, M, S, logf(S), 0.f, x_best, best_id, true);
}

// -------------------------------------------------------------------------------------------
// Filtered sampling (top-p / top-k, flat sampler).  A token stays in the support iff the tokens strictly more
// probable than it weigh less than top_p and number fewer than top_k, so the support is "every logit >= tau" for
// one threshold tau, which a radix search over the logits' bit patterns finds exactly: one pass per 8-bit digit (two
// for bfloat16, four for float32), each a histogram of (count, probability mass) over the 256 values of the digit
// among the logits that share the digits found so far.  Masses are summed as 2^-40 fixed point, so the sums do
// not depend on the order of the additions and a repeated call takes the same decisions.  One CTA of 512 threads works
// on a row at a time, two CTAs share an SM (one's search and sampling fill the gaps of the other's pass); the row is
// read once from HBM (maximum, candidates) and then, where the candidates do not suffice, from L2 (digit passes,
// sampling pass).
// -------------------------------------------------------------------------------------------
constexpr int kFiltThreads = 512;                  // two CTAs per SM: one's search and sampling overlap the other's pass over its row
constexpr int kFiltWarps = kFiltThreads / 32;
constexpr int kFiltSeg = 400;                      // candidate-list entries per warp
constexpr int kFiltCopies = 4;                     // copies of the digit histogram for a candidate list (four warps share one)
constexpr int kFiltRing = 4;                       // 16-byte pieces a thread keeps in flight during the pass over the row
constexpr size_t kFiltRingBytes = (size_t)kFiltRing * kFiltThreads * 16;
constexpr int kFiltCells = 16;                     // whole-row passes: copies of every histogram bin (lanes l and l + 16 share one)
constexpr size_t kFiltLaneHist = (size_t)4 * 256 * kFiltCells * sizeof(unsigned);   // (3 mass limbs + count) x 256 bins x cells
static_assert(kFiltRingBytes >= (size_t)kFiltCopies * 256 * sizeof(uint4), "the histograms reuse the ring's memory");
static_assert(kFiltRingBytes >= kFiltLaneHist / 2 && (size_t)kFiltWarps * kFiltSeg * sizeof(uint2) >= kFiltLaneHist / 2,
              "the per-lane histograms reuse the ring's and the candidate list's memory");
constexpr size_t kFiltSmemBytes = kFiltRingBytes +
                                  256 * (sizeof(unsigned long long) + sizeof(unsigned)) + 192 * sizeof(float) +
                                  (size_t)kFiltWarps * kFiltSeg * (sizeof(uint2) + sizeof(unsigned)) + 128;

// A probability mass e in [0, 1] as an integer count of 2^-40 (exact for a float; two 32-bit conversions).
__device__ __forceinline__ unsigned long long filt_fixed(float e) {
  const unsigned hi = __float2uint_rz(e * 65536.f);                       // e's first 16 binary places
  const float rest = fmaf(-(float)hi, 1.52587890625e-05f, e);             // exact: the places that follow
  return ((unsigned long long)hi << 24) + __float2uint_rz(rest * 1099511627776.f);
}

// Monotone key of a logit's bit pattern (larger logit, larger key); -0 and +0 share a key.
template <int ES>
__device__ __forceinline__ uint32_t filt_key(uint32_t bits) {
  if (ES == 2) {
    if (bits == 0x8000u) bits = 0u;
    return (bits & 0x8000u) ? (~bits & 0xffffu) : (bits | 0x8000u);
  }
  if (bits == 0x80000000u) bits = 0u;
  return (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
}

struct FiltCross {
  int bin;                       // first bin, from 255 down, after which a limit is reached; -1: none
  int last;                      // lowest non-empty bin, -1: all empty
  unsigned long long m, last_m;  // mass above `bin` / above `last`
  unsigned c, last_c;            // count above `bin` / above `last`
};

// Walks 256 bins of (mass, count) from the top, starting from (acc_m, acc_c) above them, and finds the first bin
// after which the mass reaches pf or the count reaches kf.  Called by one whole warp: lane l owns bins 255-8l .. 248-8l.
__device__ __forceinline__ FiltCross filt_cross(const unsigned long long* mass, const unsigned* cnt, unsigned long long acc_m,
                                                unsigned acc_c, unsigned long long pf, unsigned long long kf, int lane) {
  unsigned long long lm = 0ull;
  unsigned lc = 0u;
#pragma unroll
  for (int i = 0; i < 8; ++i) { lm += mass ? mass[255 - 8 * lane - i] : 0ull; lc += cnt[255 - 8 * lane - i]; }
  unsigned long long pm = lm;
  unsigned pc = lc;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long um = __shfl_up_sync(kFullMask, pm, o);
    const unsigned uc = __shfl_up_sync(kFullMask, pc, o);
    if (lane >= o) { pm += um; pc += uc; }
  }
  unsigned long long cm = acc_m + pm - lm;     // above this lane's bins
  unsigned cc = acc_c + pc - lc;
  FiltCross r{-1, -1, 0ull, 0ull, 0u, 0u};
  for (int i = 0; i < 8; ++i) {
    const int b = 255 - 8 * lane - i;
    const unsigned n = cnt[b];
    if (n == 0u) continue;
    const unsigned long long mb = mass ? mass[b] : 0ull;
    r.last = b; r.last_m = cm; r.last_c = cc;
    if (r.bin < 0 && (cm + mb >= pf || (unsigned long long)cc + n >= kf)) { r.bin = b; r.m = cm; r.c = cc; }
    cm += mb; cc += n;
  }
  const unsigned hit = __ballot_sync(kFullMask, r.bin >= 0), any = __ballot_sync(kFullMask, r.last >= 0);
  const int fl = hit ? __ffs(hit) - 1 : 0, ll = any ? 31 - __clz(any) : 0;
  FiltCross out;
  out.bin = hit ? __shfl_sync(kFullMask, r.bin, fl) : -1;
  out.m = __shfl_sync(kFullMask, r.m, fl);
  out.c = __shfl_sync(kFullMask, r.c, fl);
  out.last = any ? __shfl_sync(kFullMask, r.last, ll) : -1;
  out.last_m = __shfl_sync(kFullMask, r.last_m, ll);
  out.last_c = __shfl_sync(kFullMask, r.last_c, ll);
  return out;
}

template <int ES>
__global__ void __launch_bounds__(kFiltThreads, 2) espo_filtered_kernel(const __grid_constant__ StepArgs a) {
  extern __shared__ __align__(16) unsigned char fsm[];
  // digit histograms: per bin the mass as three limbs of 14 + 13 + 13 bits (32-bit shared-memory atomics are native,
  // 64-bit ones are not; a copy sees fewer than 2^18 logits per pass, so no limb overflows) and the count
  uint4* whist = reinterpret_cast<uint4*>(fsm);                                          // [copies][256]
  unsigned char* ring = fsm;                             // the row pass's landing slots (the histograms are idle then)
  unsigned long long* bmass = reinterpret_cast<unsigned long long*>(fsm + kFiltRingBytes);   // [256] all copies together
  unsigned* bcnt = reinterpret_cast<unsigned*>(bmass + 256);                             // [256]
  float* red_f = reinterpret_cast<float*>(bcnt + 256);                                   // [32] scores / sums
  int* red_i = reinterpret_cast<int*>(red_f + 32);                                       // [32] ids, flags
  unsigned long long* red_u = reinterpret_cast<unsigned long long*>(red_i + 32);         // [2][32] integer sums
  uint2* cand = reinterpret_cast<uint2*>(red_u + 64);                                    // [warps][kFiltSeg] (id, bits)
  unsigned* glist = reinterpret_cast<unsigned*>(cand + kFiltWarps * kFiltSeg);           // [warps][kFiltSeg] first ids of groups with a candidate
  unsigned* sbin = reinterpret_cast<unsigned*>(whist);                                   // 4096 sample bins (before the digit passes)
  // whole-row digit passes: one copy of every bin per lane, the four limbs in arrays of their own; they reuse the
  // ring's and the candidate list's memory, both idle by then
  unsigned* lh0 = reinterpret_cast<unsigned*>(fsm);
  unsigned* lh1 = lh0 + 256 * kFiltCells;
  unsigned* lh2 = reinterpret_cast<unsigned*>(cand);
  unsigned* lh3 = lh2 + 256 * kFiltCells;
  __shared__ RowPre pre_s;
  __shared__ unsigned long long sh_acc_mass, sh_kept_mass;
  __shared__ unsigned sh_acc_cnt, sh_prefix, sh_cut_a;
  __shared__ int sh_found, sh_overflow;
  __shared__ unsigned seg_n[kFiltWarps], seg_g[kFiltWarps];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float NINF = __int_as_float(0xff800000);
  constexpr int VEC = 16 / ES;

  for (int row = blockIdx.x; row < a.n_rows; row += gridDim.x) {
    __syncthreads();                                         // the previous row's shared values are no longer read
    // Thread 0 asks for the row's state now and hands it over at the barrier after the sampling phase, so that the
    // loads (a chain of two or three) are under way while the CTA samples the row.
    RowPre pre_r;
    if (tid == 0) { pre_r = prefetch_row(a, row); sh_overflow = 0; sh_cut_a = 0u; }
    if (tid < kFiltWarps) { seg_n[tid] = 0u; seg_g[tid] = 0u; }
    for (int i = tid; i < 4096; i += kFiltThreads) sbin[i] = 0u;
    __syncthreads();

    const unsigned char* row_base = a.logits + (size_t)row * a.row_stride_bytes;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(row_base) & 15u) == 0;
    // Walks the row (from L2 after the first pass): fnv(first id, four 32-bit words) for every whole 16-byte piece of an
    // aligned row, fns(id, raw bits) for the logits that are left (all of them if the row is not 16-byte aligned).
    auto for_each_piece = [&](auto&& fnv, auto&& fns) {
      const int v_main = vec_ok ? (a.V / VEC) * VEC : 0;
      constexpr int kInFlight = 4;                           // loads a thread issues before it looks at the first
      for (int base0 = tid * VEC; base0 < v_main; base0 += kInFlight * kFiltThreads * VEC) {
        uint4 q[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
          const int base = base0 + u * kFiltThreads * VEC;
          q[u] = (base < v_main) ? __ldg(reinterpret_cast<const uint4*>(row_base + (size_t)base * ES)) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
          const int base = base0 + u * kFiltThreads * VEC;
          if (base >= v_main) break;
          const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
          fnv(base, w);
        }
      }
      for (int id = v_main + tid; id < a.V; id += kFiltThreads) {
        const uint32_t bits = (ES == 2) ? (uint32_t)__ldg(reinterpret_cast<const unsigned short*>(row_base) + id)
                                        : __ldg(reinterpret_cast<const uint32_t*>(row_base) + id);
        fns(id, bits);
      }
    };
    // Calls fn(id, raw bits) for every logit of the row.
    auto for_each = [&](auto&& fn) {
      for_each_piece([&](int base, const uint32_t (&w)[4]) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (ES == 2) { fn(base + 2 * j, w[j] & 0xffffu); fn(base + 2 * j + 1, w[j] >> 16); }
          else fn(base + j, w[j]);
        }
      }, fn);
    };
    auto value_of = [&](uint32_t bits) -> float { return __uint_as_float(ES == 2 ? bits << 16 : bits); };
    // The pass over the whole row works on groups of VEC consecutive logits, already as floats: fn(first id,
    // values); positions past the row's end read as -inf, which no pass counts.
    auto for_each_group = [&](auto&& fn) {
      const int v_main = vec_ok ? (a.V / VEC) * VEC : 0;
      // Every thread copies its own 16-byte pieces of the row (piece number g * threads + tid) into its own slots of
      // a ring in shared memory, kFiltRing - 1 pieces ahead of the one it works on, so that the loads of the whole
      // CTA keep the memory pipe full while the arithmetic runs; no other thread reads the slots: no barrier.
      const int n_vec = v_main / VEC;
      const int n_mine = n_vec > tid ? (n_vec - tid + kFiltThreads - 1) / kFiltThreads : 0;
      const int n_warp = __shfl_sync(kFullMask, n_mine, 0);          // lane 0 has the most pieces: the warp calls fn together
      const uint32_t slot0 = smem_addr(ring) + (uint32_t)tid * 16u;
      const unsigned char* src0 = row_base + (size_t)tid * 16;
      auto issue = [&](int g) {
        if (g < n_mine)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot0 + (uint32_t)(g % kFiltRing) * (kFiltThreads * 16u)),
                       "l"(src0 + (size_t)g * (kFiltThreads * 16)) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");       // one group per piece, empty past the end
      };
      for (int g = 0; g < kFiltRing - 1; ++g) issue(g);
      for (int g = 0; g < n_warp; ++g) {
        issue(g + kFiltRing - 1);                                   // into the slot read one turn ago
        asm volatile("cp.async.wait_group %0;" ::"n"(kFiltRing - 1) : "memory");
        uint4 q = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);   // -inf in either format: no piece left
        if (ES == 4) q = make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
        if (g < n_mine) q = *reinterpret_cast<const uint4*>(ring + (size_t)(g % kFiltRing) * (kFiltThreads * 16) + (size_t)tid * 16);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
        float x[VEC];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (ES == 2) { x[2 * j] = __uint_as_float(w[j] << 16); x[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u); }
          else x[j] = __uint_as_float(w[j]);
        }
        fn((g * kFiltThreads + tid) * VEC, x);
      }
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      for (int base_w = v_main + (tid - lane) * VEC; base_w < a.V; base_w += kFiltThreads * VEC) {   // the same trips for a warp
        const int base = base_w + lane * VEC;
        float x[VEC];
#pragma unroll
        for (int j = 0; j < VEC; ++j) x[j] = (base + j < a.V) ? load_logit<ES>(row_base, base + j) : NINF;
        fn(base, x);
      }
    };
    auto bits_of = [&](float x) -> uint32_t { return ES == 2 ? __float_as_uint(x) >> 16 : __float_as_uint(x); };

    // ---- candidate cut.  A histogram of the whole row would put nearly every logit into a handful of bins, and
    //      shared-memory atomics on one address serialise.  So 4096 logits (16 stretches of 256 spread over the row)
    //      are sampled into a histogram over the upper 12 bits of their keys, and the cut is the key above which
    //      about 64 samples lie -- about 2400 logits of the row.  The pass over the row lists the logits above the cut;
    //      if they already reach top_p or top_k they contain the whole support and the search below runs over the
    //      list, otherwise (or if the list overflows) it runs over the whole row again. ----
    if (a.V >= 16384) {
      constexpr int kStretch = 256, kStretches = 16;
#pragma unroll
      for (int j = 0; j < kStretch * kStretches / kFiltThreads; ++j) {
        const int n = tid + j * kFiltThreads;                // sample number
        const int id = (int)((long long)(n / kStretch) * a.V / kStretches) + (n % kStretch);
        atomicAdd(sbin + (filt_key<ES>(bits_of(load_logit<ES>(row_base, id))) >> (8 * ES - 12)), 1u);
      }
      __syncthreads();
      if (tid < 256) {                                       // groups of 16 bins
        unsigned t = 0u;
        for (int i = 0; i < 16; ++i) t += sbin[tid * 16 + i];
        bcnt[tid] = t;
      }
      __syncthreads();
      if (warp == 0) {
        const unsigned long long want = 64ull;
        const FiltCross g = filt_cross(nullptr, bcnt, 0ull, 0u, ~0ull, want, lane);
        if (lane == 0 && g.bin >= 0) {
          // the bin in which the count is reached, and inside it the share of its keys (from the top) that the
          // missing samples are of the bin's samples: a bin is half a unit wide for logits between 4 and 8, and its
          // lower edge would admit up to twice the wanted number
          constexpr int kLow = 8 * ES - 12;                  // key bits below a bin
          unsigned cum = g.c;
          unsigned long long cut = (unsigned long long)(g.bin * 16) << kLow;
          for (int i = 15; i >= 0; --i) {
            const unsigned c = sbin[g.bin * 16 + i];
            cum += c;
            if (cum >= want) {
              const unsigned long long r = want - (cum - c);                          // 1 .. c samples of this bin
              const unsigned long long take = ((r << kLow) + c - 1) / c;              // 1 .. 2^kLow keys
              cut = ((unsigned long long)(g.bin * 16 + i + 1) << kLow) - take;
              break;
            }
          }
          sh_cut_a = (unsigned)cut;
        }
      }
    }
    if (tid == 0) pre_s = pre_r;
    __syncthreads();
    const RowPre pre = pre_s;
    if (pre.slot < 0) { mark_row(a, row, 0, tid, -1, ESPO_DEV_BAD_SLOT, -1, true); continue; }
    if (pre.status != ESPO_ROW_ACTIVE) { mark_row(a, row, pre.slot, tid, -1, 0u, -1, true); continue; }   // finished: untouched
    const uint32_t cut_a = sh_cut_a;
    // the cut as a logit: keys are monotone in the value, so key >= cut_a is x >= cut_x
    const uint32_t key_top = (ES == 2) ? 0x8000u : 0x80000000u;
    const float cut_x = (cut_a == 0u) ? __int_as_float(0x7f800000)
                                      : value_of((cut_a & key_top) ? (cut_a & ~key_top) : (~cut_a & (ES == 2 ? 0xffffu : 0xffffffffu)));

    // ---- the pass over the row (from HBM): the largest logit and the row's mass sum_a exp((x_a - M)/T), kept per
    //      lane relative to the warp's running maximum; NaN or +inf anywhere makes the row unusable (either turns a
    //      lane's sum into NaN or the maximum into +inf); logits at or above the cut go onto the list. ----
    float m = NINF, s_t = 0.f;
    uint2* my_seg = cand + warp * kFiltSeg;
    unsigned* my_groups = glist + warp * kFiltSeg;
    // The warp keeps one running maximum mw for all of its lanes (a trip's maximum comes from one redux), so that the
    // exponents are one packed multiply-add x*k2 + c0 with c0 = -mw*k2 and the sums packed adds; c0 is rounded once
    // per value of mw, which leaves every term of that stretch with the common factor 2^dl, dl = c0 + mw*k2 (exact
    // as a fused multiply-add), taken out when mw moves and at the end.
    float mw = NINF, c0 = 0.f;
    float2 acc = make_float2(0.f, 0.f);
    bool nan_seen = false;
    for_each_group([&](int base, const float (&x)[VEC]) {
      float vm = x[0];
#pragma unroll
      for (int j = 1; j < VEC; ++j) vm = fmaxf(vm, x[j]);
      const float wmax = warp_max(vm);
      if (wmax > mw) {                                       // the same in every lane
        if (mw > NINF) {
          const float dl = fmaf(mw, a.k2, c0);
          const float sc = ex2_approx(fmaf(mw - wmax, a.k2, -dl));   // to the new maximum, the old stretch's factor out
          acc.x *= sc; acc.y *= sc;
        }
        mw = wmax;
        c0 = -mw * a.k2;
      }
      if (mw > NINF) {
        const float2 k2v = make_float2(a.k2, a.k2), c0v = make_float2(c0, c0);
#pragma unroll
        for (int j = 0; j < VEC / 2; ++j) {                  // NaN stays NaN; +inf makes mw +inf, then NaN or 0
          const float2 t = __ffma2_rn(make_float2(x[2 * j], x[2 * j + 1]), k2v, c0v);
          acc = __fadd2_rn(acc, make_float2(ex2_approx(t.x), ex2_approx(t.y)));
        }
      } else {
#pragma unroll
        for (int j = 0; j < VEC; ++j) nan_seen = nan_seen || (x[j] != x[j]);   // a NaN among logits that are all -inf so far
      }
      // About one logit in 50 lies above the cut, so in nearly every trip some lane of the warp has one, and what the
      // lane does about it the whole warp waits for: the pass only notes the group on the warp's list of groups
      // (measured: faster than listing the logits here, and than bit masks in registers scanned afterwards).
      if (vm >= cut_x) {
        const unsigned at = atomicAdd(&seg_g[warp], 1u);
        if (at < (unsigned)kFiltSeg) my_groups[at] = (unsigned)base;
        else sh_overflow = 1;
      }
    });
    m = mw;
    s_t = (acc.x + acc.y) * ex2_approx(-fmaf(mw, a.k2, c0));
    if (!(mw > NINF)) s_t = 0.f;
    if (nan_seen) s_t = __int_as_float(0x7fc00000);
    // ---- the noted groups, read again (L2, a few per lane), give the list of candidates ----
    __syncwarp();
    {
      const unsigned n_g = min(seg_g[warp], (unsigned)kFiltSeg);
      const int v_main = vec_ok ? (a.V / VEC) * VEC : 0;
      constexpr int kAhead = 4;                              // groups a lane asks for before it takes the first apart
      for (unsigned i0 = lane; i0 < n_g; i0 += 32 * kAhead) {
        int base[kAhead];
        uint4 q[kAhead];
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
          const unsigned i = i0 + 32u * u;
          base[u] = i < n_g ? (int)my_groups[i] : -1;
          q[u] = make_uint4(0u, 0u, 0u, 0u);
          if (base[u] >= 0 && base[u] + VEC <= v_main)       // a whole 16-byte piece of an aligned row
            q[u] = __ldg(reinterpret_cast<const uint4*>(row_base + (size_t)base[u] * ES));
        }
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
          if (base[u] < 0) continue;
          float x[VEC];
          if (base[u] + VEC <= v_main) {
            const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (ES == 2) { x[2 * j] = __uint_as_float(w[j] << 16); x[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u); }
              else x[j] = __uint_as_float(w[j]);
            }
          } else {
#pragma unroll
            for (int j = 0; j < VEC; ++j) x[j] = (base[u] + j < a.V) ? load_logit<ES>(row_base, base[u] + j) : NINF;
          }
          unsigned n_c = 0u;
#pragma unroll
          for (int j = 0; j < VEC; ++j) n_c += (x[j] >= cut_x) ? 1u : 0u;
          unsigned at = atomicAdd(&seg_n[warp], n_c);
#pragma unroll
          for (int j = 0; j < VEC; ++j) {
            if (!(x[j] >= cut_x)) continue;
            if (at < (unsigned)kFiltSeg) my_seg[at] = make_uint2((unsigned)(base[u] + j), bits_of(x[j]));
            else sh_overflow = 1;
            ++at;
          }
        }
      }
    }
    bool poisoned = (s_t != s_t) || (m == __int_as_float(0x7f800000));
    const float wm = warp_max(m);
    poisoned = __any_sync(kFullMask, poisoned);
    if (lane == 0) { red_f[warp] = wm; red_i[warp] = poisoned; }
    __syncthreads();
    static_assert(kFiltWarps <= 32, "one lane per warp's partial result");
    const bool has_part = lane < kFiltWarps;
    const float M = warp_max(has_part ? red_f[lane] : NINF); // every warp folds the warps' partial results by itself
    poisoned = __any_sync(kFullMask, has_part && red_i[lane] != 0);
    if (poisoned || !(M > NINF)) { mark_row(a, row, pre.slot, tid, 0, ESPO_DEV_BAD_ROW, ESPO_ROW_BAD, true); continue; }
    float tot_f = (m > NINF) ? s_t * ex2_approx((m - M) * a.k2) : 0.f;
    tot_f = warp_sum(tot_f);                                 // fixed order: the same bits on every call

    // ---- what the list holds: exact integer sums of mass and count ----
    unsigned long long m_a = 0ull;
    unsigned c_a = 0u;
    if (cut_a != 0u && sh_overflow == 0) {
      const unsigned n = seg_n[warp];
      for (unsigned i = lane; i < n; i += 32) { m_a += filt_fixed(ex2_approx((value_of(my_seg[i].y) - M) * a.k2)); ++c_a; }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) { m_a += __shfl_xor_sync(kFullMask, m_a, o); c_a += __shfl_xor_sync(kFullMask, c_a, o); }
    __syncthreads();
    if (lane == 0) { red_f[warp] = tot_f; red_u[warp] = m_a; red_u[32 + warp] = c_a; }
    __syncthreads();
    double tot = has_part ? (double)red_f[lane] : 0.0;                        // butterfly: the same tree, hence the same bits, in every lane and call
    unsigned long long ma = has_part ? red_u[lane] : 0ull, ca = has_part ? red_u[32 + lane] : 0ull;   // integer sums: the order does not matter
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      tot += __shfl_xor_sync(kFullMask, tot, o);
      ma += __shfl_xor_sync(kFullMask, ma, o);
      ca += __shfl_xor_sync(kFullMask, ca, o);
    }
    const unsigned long long total = (unsigned long long)(tot * 1099511627776.0);
    const unsigned long long pf = (a.top_p < 1.f) ? (unsigned long long)((double)total * (double)a.top_p) : ~0ull;   // top_p of the row's mass
    const unsigned long long kf = a.top_k > 0 ? (unsigned long long)a.top_k : ~0ull;
    const bool use_list = cut_a != 0u && (ma >= pf || ca >= kf) && sh_overflow == 0;
    const bool cut_active = use_list;

    // ---- whole-row search: a first bid for the sampling pass.  The list did not reach top_p or top_k, so each of its
    //      logits has less than top_p of the mass and fewer than top_k logits above it: all of them stay, and the best
    //      of their scores is a lower bound of the row's best score (the list's memory is reused below). ----
    const DrawStream ds{a.key0, a.key1, (uint32_t)pre.t_now, (uint32_t)pre.slot, a.batch_bits};
    float seed_b = NINF;
    int seed_id = -1;
    if (!use_list && cut_a != 0u && sh_overflow == 0) {
      const unsigned n = seg_n[warp];
      for (unsigned i = lane; i < n; i += 32) {
        const uint2 c = my_seg[i];
        const float x = value_of(c.y);
        if (!(x > NINF)) continue;
        const float sc = fmaf(x - M, a.inv_temp, gumbel_at(ds, 0u, c.x));
        if (sc > seed_b || (sc == seed_b && (int)c.x < seed_id)) { seed_b = sc; seed_id = (int)c.x; }
      }
      warp_argmax(seed_b, seed_id);
      __syncthreads();                                       // red_f of the sums above is no longer read
      if (lane == 0) { red_f[warp] = seed_b; red_i[warp] = seed_id; }
      __syncthreads();
      seed_b = has_part ? red_f[lane] : NINF; seed_id = has_part ? red_i[lane] : -1;
      warp_argmax(seed_b, seed_id);                          // the same pair in every thread
    }

    // ---- digit passes: find the threshold key.  The keys that take part lie between key_lo (the cut, or 0) and
    //      the key of the largest logit; only the bits in which that range varies are searched, 8 at a time from the
    //      top, so the logits of a list (a narrow range of values) spread over the bins of a single pass or two. ----
    const uint32_t key_lo = use_list ? cut_a : 0u;
    const uint32_t span = filt_key<ES>(bits_of(M)) - key_lo;
    const int n_digits = span == 0u ? 1 : (32 - __clz(span) + 7) / 8;
    if (tid == 0) { sh_acc_mass = 0ull; sh_acc_cnt = 0u; sh_prefix = 0u; sh_kept_mass = total; sh_found = 0; }
    for (int d = 0; d < n_digits; ++d) {
      const int shift = 8 * (n_digits - 1 - d);
      if (use_list) {
        // a short list: four copies of the histogram, one per group of four warps
        constexpr int copies = kFiltCopies;
        for (int i = tid; i < copies * 256; i += kFiltThreads) whist[i] = make_uint4(0u, 0u, 0u, 0u);
        __syncthreads();
        const uint32_t prefix = sh_prefix;                   // the digits above this one, as found so far
        unsigned* my_hist = reinterpret_cast<unsigned*>(whist + (warp % copies) * 256);
        const unsigned n = seg_n[warp];
        for (unsigned i = lane; i < n; i += 32) {
          const uint32_t bits = my_seg[i].y;
          const uint32_t key = filt_key<ES>(bits) - key_lo;  // every candidate's key is at least key_lo
          if (d > 0 && (key >> (shift + 8)) != prefix) continue;
          const unsigned long long fx = filt_fixed(ex2_approx((value_of(bits) - M) * a.k2));
          unsigned* h = my_hist + 4u * ((key >> shift) & 255u);
          atomicAdd(h, (unsigned)(fx >> 26));                // 14 bits (an e of exactly 1 gives 2^14)
          atomicAdd(h + 1, (unsigned)(fx >> 13) & 0x1fffu);
          atomicAdd(h + 2, (unsigned)fx & 0x1fffu);
          atomicAdd(h + 3, 1u);
        }
        __syncthreads();
        if (tid < 256) {
          unsigned long long tm = 0ull;
          unsigned tc = 0u;
          for (int w = 0; w < copies; ++w) {
            const uint4 h = whist[w * 256 + tid];
            tm += ((unsigned long long)h.x << 26) + ((unsigned long long)h.y << 13) + h.z;
            tc += h.w;
          }
          bmass[tid] = tm; bcnt[tid] = tc;
        }
      } else {
        // The whole row: nearly all of its logits fall into a handful of bins, and atomics of one warp on one address
        // take turns.  So every bin has kFiltCells copies, picked by the lane (cell = bin * 16 + lane % 16: lanes l and
        // l + 16 share a cell, the others hit banks of their own whatever their bins); a cell sees V / 16 logits, and
        // V <= 2^21 keeps the 14-bit limb's sum below 2^31.
        for (int i = tid; i < (int)(kFiltLaneHist / 2 / sizeof(uint4)); i += kFiltThreads) {
          reinterpret_cast<uint4*>(lh0)[i] = make_uint4(0u, 0u, 0u, 0u);
          reinterpret_cast<uint4*>(lh2)[i] = make_uint4(0u, 0u, 0u, 0u);
        }
        __syncthreads();
        const uint32_t prefix = sh_prefix;
        for_each([&](int, uint32_t bits) {
          const uint32_t key = filt_key<ES>(bits);
          if (d > 0 && (key >> (shift + 8)) != prefix) return;
          const unsigned long long fx = filt_fixed(ex2_approx((value_of(bits) - M) * a.k2));
          const unsigned cell = ((key >> shift) & 255u) * (unsigned)kFiltCells + ((unsigned)lane & (kFiltCells - 1));
          atomicAdd(lh0 + cell, (unsigned)(fx >> 26));
          atomicAdd(lh1 + cell, (unsigned)(fx >> 13) & 0x1fffu);
          atomicAdd(lh2 + cell, (unsigned)fx & 0x1fffu);
          atomicAdd(lh3 + cell, 1u);
        });
        __syncthreads();
        if (tid < 256) {
          unsigned long long t0 = 0ull, t1 = 0ull, t2 = 0ull;
          unsigned tc = 0u;
          for (int w = 0; w < kFiltCells; ++w) {
            const unsigned cell = (unsigned)tid * kFiltCells + ((unsigned)(w + tid) & (kFiltCells - 1));   // the lanes of a warp spread over the banks
            t0 += lh0[cell]; t1 += lh1[cell]; t2 += lh2[cell]; tc += lh3[cell];
          }
          bmass[tid] = (t0 << 26) + (t1 << 13) + t2; bcnt[tid] = tc;
        }
      }
      __syncthreads();
      if (warp == 0 && (d == 0 || sh_found)) {
        // Every value of a bin has at least the running mass and count above it; the first bin after which one of
        // the two limits is reached holds the last value that stays.
        const FiltCross x = filt_cross(bmass, bcnt, sh_acc_mass, sh_acc_cnt, pf, kf, lane);
        int boundary = x.bin;
        unsigned long long cum_m = x.m;
        unsigned cum_c = x.c;
        // a cut was enough, or an upper digit found a boundary: the boundary lies among what was histogrammed (exact
        // sums make this branch unreachable; it keeps the search well-defined regardless)
        if (boundary < 0 && (d > 0 || cut_active) && x.last >= 0) { boundary = x.last; cum_m = x.last_m; cum_c = x.last_c; }
        if (lane == 0) {
          if (boundary >= 0) {
            sh_found = 1;
            sh_acc_mass = cum_m; sh_acc_cnt = cum_c;
            sh_prefix = (sh_prefix << 8) | (unsigned)boundary;
            if (d == n_digits - 1) sh_kept_mass = cum_m + bmass[boundary];   // the boundary value itself stays
          } else {
            sh_found = 0;                                    // neither limit is reached: the whole row stays
          }
        }
      }
      __syncthreads();
      if (!sh_found) break;                                  // the same for every thread: read after the barrier
    }
    const bool filtered = sh_found != 0;
    const uint32_t tau_key = filtered ? key_lo + sh_prefix : 0u;   // keep everything unless a boundary was found
    const unsigned long long kept_mass = sh_kept_mass;

    // ---- sampling pass: Gumbel-max over the support with the flat sampler's draws ----
    float best = seed_b;
    int best_id = seed_id;
    auto offer = [&](int id, uint32_t bits) {
      if (filt_key<ES>(bits) < tau_key) return;
      const float x = value_of(bits);
      if (!(x > NINF)) return;
      const float sc = fmaf(x - M, a.inv_temp, gumbel_at(ds, 0u, (uint32_t)id));
      if (sc > best || (sc == best && id < best_id)) { best = sc; best_id = id; }
    };
    // Four logits whose ids share a Philox counter (id0 is a multiple of 4): one generator call for those that stay.
    // A logit whose score without noise lies 6 or more under the thread's best needs a Gumbel above 6 to matter; the
    // draws up to kGumbelBelow6 give less than 5.9001, so they are dropped on the integer and the two logarithms
    // are taken for one draw in 365 only (the margin of 0.1 covers the rounding of every term many times over).
    constexpr uint32_t kGumbelBelow6 = 8365658u;             // (2k+1)/2^24 <= exp(-exp(-5.9)) for the 23-bit draw k
    auto offer4 = [&](int id0, const uint32_t (&b)[4]) {
      bool in[4];
      bool any = false;
#pragma unroll
      for (int j = 0; j < 4; ++j) { in[j] = filt_key<ES>(b[j]) >= tau_key && value_of(b[j]) > NINF; any = any || in[j]; }
      if (!any) return;
      const uint4 rnd = philox4x32_10((uint32_t)id0 >> 2, ds.step, ds.slot, ds.batch_bits | 0u, ds.k0, ds.k1);
      const uint32_t word[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (!in[j]) continue;
        const float bare = (value_of(b[j]) - M) * a.inv_temp;
        if (best - bare >= 6.f && (word[j] >> 9) <= kGumbelBelow6) continue;
        const float sc = fmaf(value_of(b[j]) - M, a.inv_temp, gumbel_from_word(word[j]));
        if (sc > best || (sc == best && id0 + j < best_id)) { best = sc; best_id = id0 + j; }
      }
    };
    if (use_list) {
      const unsigned n = seg_n[warp];
      for (unsigned i = lane; i < n; i += 32) { const uint2 c = my_seg[i]; offer((int)c.x, c.y); }
    } else {
      for_each_piece([&](int base, const uint32_t (&w)[4]) {
        if (ES == 2) {
          const uint32_t lo[4] = {w[0] & 0xffffu, w[0] >> 16, w[1] & 0xffffu, w[1] >> 16};
          const uint32_t hi[4] = {w[2] & 0xffffu, w[2] >> 16, w[3] & 0xffffu, w[3] >> 16};
          offer4(base, lo);
          offer4(base + 4, hi);
        } else {
          offer4(base, w);
        }
      }, offer);
    }
    warp_argmax(best, best_id);
    __syncthreads();                                         // red_f / red_i of the sums above are no longer read
    if (lane == 0) { red_f[warp] = best; red_i[warp] = best_id; }
    __syncthreads();
    if (warp == 0) {
      float b = has_part ? red_f[lane] : NINF;
      int tok = has_part ? red_i[lane] : -1;
      warp_argmax(b, tok);                                   // largest score, the smaller id among equal ones, -1 if none
      if (lane == 0) {
        if (tok < 0) {
          mark_row(a, row, pre.slot, 0, 0, ESPO_DEV_BAD_ROW, ESPO_ROW_BAD, true);
        } else {
          const float l_tok = load_logit<ES>(row_base, tok);
          const float S = (float)((double)kept_mass * (1.0 / 1099511627776.0));
          commit_row(a, row, pre, ds, M, S, logf(S), 0.f, l_tok, tok, true);
        }
      }
    }
  }
}

}  // namespace espo

// ===========================================================================================
// Host side: state, launch, compaction.
// ===========================================================================================

struct espo_state {
  int device, capacity, V, nblk, sm_count, max_smem;
  uint64_t seed, batch_id;
  int cfg_warps, cfg_stages, cfg_ctas_per_sm;   // 0 = library default
  int dependent_launch;                         // espo_set_dependent_launch
  void* arena;
  size_t arena_bytes;
  float *z, *g, *g_tilde, *logp;
  int32_t *t, *t_stop;
  uint8_t* status;
  double *sum_g, *sum_g2;
  float* entropy;
  double* sum_h;
  float4* records;
  unsigned *ticket, *dev_status;
  double* batch_out;   // [9] result of espo_end_batch
};

namespace espo {

__global__ void espo_compact_kernel(const uint8_t* __restrict__ status, int capacity, int32_t* __restrict__ out,
                                    int32_t* __restrict__ n_out) {
  __shared__ int warp_total[32];
  __shared__ int base;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // (launched as a programmatic dependent when the state asks for it: the step before has completed after the wait;
  // the kernel after this one may be set up meanwhile)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (threadIdx.x == 0) base = 0;
  __syncthreads();
  for (int start = 0; start < capacity; start += blockDim.x) {
    const int i = start + threadIdx.x;
    const bool active = (i < capacity) && (status[i] == ESPO_ROW_ACTIVE);
    const unsigned bal = __ballot_sync(kFullMask, active);
    const int rank = __popc(bal & ((1u << lane) - 1u));
    if (lane == 0) warp_total[warp] = __popc(bal);
    __syncthreads();
    int before = 0;
    for (int w = 0; w < warp; ++w) before += warp_total[w];
    if (active) out[base + before + rank] = i;
    __syncthreads();
    if (threadIdx.x == 0) {
      int tot = 0;
      for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += warp_total[w];
      base += tot;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) *n_out = base;
}

// Batch boundary (Eq. 7-8, 12): reduces the per-slot sums over the slots that took part (t > 0) and applies the
// EMA and the proportional controller.  One CTA; out = {mu_g, sigma2_g, beta, mean, var, rho_stop, tokens,
// trajectories, stopped trajectories}.
struct EndBatchArgs {
  const double *sum_g, *sum_g2;
  const int32_t* t;
  const uint8_t* status;
  int capacity;
  double mu_g, sigma2_g, beta, alpha_ema, eta_beta, tau, beta_min, beta_max;
  int first_update;
  double* out;
};

__global__ void __launch_bounds__(1024) espo_end_batch_kernel(const EndBatchArgs e) {
  __shared__ double red[5][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double acc[5] = {0.0, 0.0, 0.0, 0.0, 0.0};   // sum g, sum g^2, tokens, trajectories, stopped
  for (int i = threadIdx.x; i < e.capacity; i += blockDim.x) {
    const int ti = e.t[i];
    if (ti > 0) {
      acc[0] += e.sum_g[i]; acc[1] += e.sum_g2[i]; acc[2] += (double)ti; acc[3] += 1.0;
      if (e.status[i] == ESPO_ROW_STOPPED) acc[4] += 1.0;
    }
  }
#pragma unroll
  for (int k = 0; k < 5; ++k) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc[k] += __shfl_xor_sync(kFullMask, acc[k], o);
    if (lane == 0) red[k][warp] = acc[k];
  }
  __syncthreads();
  if (warp == 0) {
#pragma unroll
    for (int k = 0; k < 5; ++k) {
      double v = (lane < (int)(blockDim.x >> 5)) ? red[k][lane] : 0.0;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
      acc[k] = v;
    }
    if (lane == 0) {
      double mu = e.mu_g, s2 = e.sigma2_g, beta = e.beta, mean = 0.0, var = 0.0, rho = 0.0;
      if (acc[2] > 0.0) {
        mean = acc[0] / acc[2];
        var = fmax(acc[1] / acc[2] - mean * mean, 0.0);
        rho = acc[4] / acc[3];
        if (e.first_update) { mu = mean; s2 = var; }
        else {
          mu = e.alpha_ema * mu + (1.0 - e.alpha_ema) * mean;
          s2 = e.alpha_ema * s2 + (1.0 - e.alpha_ema) * var;
        }
        beta = fmin(fmax(beta + e.eta_beta * (rho - e.tau), e.beta_min), e.beta_max);
      }
      e.out[0] = mu; e.out[1] = s2; e.out[2] = beta; e.out[3] = mean; e.out[4] = var; e.out[5] = rho;
      e.out[6] = acc[2]; e.out[7] = acc[3]; e.out[8] = acc[4];
    }
  }
}

using StepKernel = void (*)(const StepArgs);

static StepKernel pick_kernel(int es, int sampler, bool bulk) {
  if (es == 2) {
    if (sampler == ESPO_SAMPLER_FLAT) return bulk ? espo_step_kernel<2, 0, true> : espo_step_kernel<2, 0, false>;
    return bulk ? espo_step_kernel<2, 1, true> : espo_step_kernel<2, 1, false>;
  }
  if (sampler == ESPO_SAMPLER_FLAT) return bulk ? espo_step_kernel<4, 0, true> : espo_step_kernel<4, 0, false>;
  return bulk ? espo_step_kernel<4, 1, true> : espo_step_kernel<4, 1, false>;
}

static int reset_arrays(espo_state* st, cudaStream_t stream) {
  ESPO_CUDA_TRY(cudaMemsetAsync(st->arena, 0, st->arena_bytes, stream));
  ESPO_CUDA_TRY(cudaMemsetAsync(st->t_stop, 0xFF, sizeof(int32_t) * (size_t)st->capacity, stream));   // -1
  return ESPO_OK;
}

}  // namespace espo

extern "C" {

int espo_init_state(espo_state** out, int32_t capacity, int32_t V, uint64_t seed, uint64_t batch_id, void* stream) {
  using namespace espo;
  if (!out) return ESPO_ERR_NULL;
  *out = nullptr;
  if (capacity < 1 || V < 1) return ESPO_ERR_BAD_SHAPE;
  if (batch_id >= (1ull << 30)) return ESPO_ERR_BAD_PARAM;
  espo_state* st = new (std::nothrow) espo_state();
  if (!st) return ESPO_ERR_CAPACITY;
  memset(st, 0, sizeof(*st));
  cudaError_t e = cudaGetDevice(&st->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&st->sm_count, cudaDevAttrMultiProcessorCount, st->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&st->max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, st->device);
  if (e != cudaSuccess) { delete st; return record_cuda_error(e); }
  st->capacity = capacity;
  st->V = V;
  st->nblk = (V + kBlockIds - 1) / kBlockIds;
  st->seed = seed;
  st->batch_id = batch_id;

  const size_t cap = (size_t)capacity;
  size_t off = 0;
  auto carve = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t o_z = carve(4 * cap), o_g = carve(4 * cap), o_gt = carve(4 * cap), o_lp = carve(4 * cap);
  const size_t o_t = carve(4 * cap), o_ts = carve(4 * cap), o_st = carve(cap);
  const size_t o_sg = carve(8 * cap), o_sg2 = carve(8 * cap), o_h = carve(4 * cap), o_sh = carve(8 * cap);
  const size_t o_rec = carve(sizeof(float4) * cap * (size_t)st->nblk);
  const size_t o_tk = carve(4 * cap), o_ds = carve(4), o_bo = carve(8 * 9);
  st->arena_bytes = off;
  e = cudaMalloc(&st->arena, st->arena_bytes);
  if (e != cudaSuccess) { delete st; return record_cuda_error(e); }
  unsigned char* base = static_cast<unsigned char*>(st->arena);
  st->z = (float*)(base + o_z); st->g = (float*)(base + o_g); st->g_tilde = (float*)(base + o_gt);
  st->logp = (float*)(base + o_lp); st->t = (int32_t*)(base + o_t); st->t_stop = (int32_t*)(base + o_ts);
  st->status = (uint8_t*)(base + o_st); st->sum_g = (double*)(base + o_sg); st->sum_g2 = (double*)(base + o_sg2);
  st->entropy = (float*)(base + o_h); st->sum_h = (double*)(base + o_sh);
  st->records = (float4*)(base + o_rec); st->ticket = (unsigned*)(base + o_tk); st->dev_status = (unsigned*)(base + o_ds);
  st->batch_out = (double*)(base + o_bo);

  for (int es = 2; es <= 4; es += 2)
    for (int sm = 0; sm < 2; ++sm)
      for (int b = 0; b < 2; ++b) {
        e = cudaFuncSetAttribute((const void*)pick_kernel(es, sm, b != 0), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 st->max_smem);
        if (e != cudaSuccess) { cudaFree(st->arena); delete st; return record_cuda_error(e); }
      }
  // (the attribute belongs to the device that is current, so it is set for every state rather than once per process)
  {
    const void* hk[4] = {(const void*)espo_step_hier_kernel<2, true>, (const void*)espo_step_hier_kernel<2, false>,
                         (const void*)espo_step_hier_kernel<4, true>, (const void*)espo_step_hier_kernel<4, false>};
    for (int i = 0; i < 4 && e == cudaSuccess; ++i)
      e = cudaFuncSetAttribute(hk[i], cudaFuncAttributeMaxDynamicSharedMemorySize, st->max_smem);
    if (e != cudaSuccess) { cudaFree(st->arena); delete st; return record_cuda_error(e); }
  }
  e = cudaFuncSetAttribute((const void*)espo_filtered_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFiltSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute((const void*)espo_filtered_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFiltSmemBytes);
  if (e != cudaSuccess) { cudaFree(st->arena); delete st; return record_cuda_error(e); }
  int rc = reset_arrays(st, (cudaStream_t)stream);
  if (rc != ESPO_OK) { cudaFree(st->arena); delete st; return rc; }
  *out = st;
  return ESPO_OK;
}

int espo_reset_state(espo_state* st, uint64_t batch_id, void* stream) {
  if (!st) return ESPO_ERR_NULL;
  if (batch_id >= (1ull << 30)) return ESPO_ERR_BAD_PARAM;
  st->batch_id = batch_id;
  return espo::reset_arrays(st, (cudaStream_t)stream);
}

void espo_free_state(espo_state* st) {
  if (!st) return;
  cudaDeviceSynchronize();
  cudaFree(st->arena);
  delete st;
}

int espo_set_launch_config(espo_state* st, int32_t consumer_warps, int32_t stages, int32_t ctas_per_sm) {
  if (!st) return ESPO_ERR_NULL;
  if (consumer_warps < 0 || consumer_warps > espo::kMaxConsumerWarps || stages < 0 || stages > 64 || ctas_per_sm < 0 ||
      ctas_per_sm > 8)
    return ESPO_ERR_BAD_PARAM;
  st->cfg_warps = consumer_warps;
  st->cfg_stages = stages;
  st->cfg_ctas_per_sm = ctas_per_sm;
  return ESPO_OK;
}

int espo_set_dependent_launch(espo_state* st, int32_t enable) {
  if (!st) return ESPO_ERR_NULL;
  st->dependent_launch = enable != 0;
  return ESPO_OK;
}

// Checks the frozen parameters and digests them into the kernel's arguments (everything but shapes and pointers).
static int fill_params(espo::StepArgs& a, const espo_state* st, const espo_params* p) {
  using namespace espo;
  if (!(p->temperature >= 0.f) || isinf(p->temperature)) return ESPO_ERR_BAD_PARAM;
  if (!(p->sigma2_g >= 0.f) || !(p->sigma2_g + p->delta > 0.f) || !(p->clip_c > 0.f)) return ESPO_ERR_BAD_PARAM;
  if (!(p->alpha_s >= 0.f && p->alpha_s < 1.f) || p->t_max < 1) return ESPO_ERR_BAD_PARAM;
  if (p->sampler != ESPO_SAMPLER_FLAT && p->sampler != ESPO_SAMPLER_HIER) return ESPO_ERR_BAD_PARAM;
  if (isnan(p->mu_g) || isnan(p->beta) || isnan(p->eps)) return ESPO_ERR_BAD_PARAM;
  if (p->stop_mode < ESPO_STOP_ESPO || p->stop_mode > ESPO_STOP_RANDOM || isnan(p->tau) ||
      !(p->p_random >= 0.f && p->p_random <= 1.f))
    return ESPO_ERR_BAD_PARAM;
  if (p->want_entropy && p->sampler != ESPO_SAMPLER_HIER) return ESPO_ERR_BAD_PARAM;   // the flat sampler's records are full
  if (isnan(p->top_p) || p->top_k < 0) return ESPO_ERR_BAD_PARAM;
  a.top_p = (p->top_p > 0.f && p->top_p < 1.f) ? p->top_p : 1.f;
  a.top_k = p->top_k;
  a.capacity = st->capacity;
  a.z = st->z; a.g = st->g; a.g_tilde = st->g_tilde; a.logp = st->logp;
  a.t = st->t; a.t_stop = st->t_stop; a.status = st->status; a.sum_g = st->sum_g; a.sum_g2 = st->sum_g2; a.entropy = st->entropy; a.sum_h = st->sum_h;
  a.records = st->records; a.ticket = st->ticket; a.dev_status = st->dev_status;
  a.greedy = (p->temperature == 0.f);
  const double inv_t = a.greedy ? 1.0 : 1.0 / (double)p->temperature;
  a.inv_temp = (float)inv_t;
  a.k2 = (float)(inv_t * 1.4426950408889634074);
  a.mu_g = p->mu_g;
  a.inv_sigma = (float)(1.0 / sqrt((double)p->sigma2_g + (double)p->delta));
  a.clip_c = p->clip_c;
  a.alpha_s = p->alpha_s;
  a.one_minus_alpha = 1.0f - p->alpha_s;
  a.beta = p->beta; a.eps = p->eps;
  a.warmup_complete = p->warmup_complete; a.t_max = p->t_max; a.eos_token = p->eos_token;
  a.want_entropy = p->want_entropy != 0;
  a.stop_mode = p->stop_mode; a.shadow = p->shadow != 0; a.tau = p->tau; a.p_random = p->p_random;
  a.key0 = (uint32_t)(st->seed & 0xffffffffull);
  a.key1 = (uint32_t)(st->seed >> 32);
  a.batch_bits = (uint32_t)(st->batch_id << 2);
  return ESPO_OK;
}

// Launch of the hierarchical sampler's kernel: shape of the grid and layout of its shared-memory tables.  Returns 1
// (nothing launched) when a CTA's range holds more blocks than its record table can: espo_step_kernel takes those.
static int launch_hier(espo::StepArgs& a, const espo_state* st, int es, bool bulk, cudaStream_t stream) {
  using namespace espo;
  const int ctas_per_sm = st->cfg_ctas_per_sm ? st->cfg_ctas_per_sm : 1;
  const int max_warps = (kMaxStepThreads / 32 < 64 / ctas_per_sm) ? kMaxStepThreads / 32 : 64 / ctas_per_sm;
  // Finalizer warps: one follows a row for about 3.5 us on top of the row's streaming time, and an SM streams a row
  // in row_bytes / ~43 GB/s; short rows need several.
  const double row_us = (double)a.V * es / 43e3;
  int fin = (int)ceil(3.5 / (row_us * ctas_per_sm)) + 1;     // one more: a row shared with another CTA takes longer
  fin = fin < 2 ? 2 : (fin > 4 ? 4 : fin);
  if (fin > max_warps - 1) fin = max_warps - 1 < 1 ? 1 : max_warps - 1;
  // (fp32 logits: 14 streaming + 2 finalizer warps are four per scheduler; 15 + 2 measured 0.5-1.5 % slower)
  int warps = st->cfg_warps ? st->cfg_warps : (es == 2 ? 31 : 14);
  int stages = st->cfg_stages ? st->cfg_stages : 2;
  if (warps + fin > max_warps) warps = max_warps - fin;
  if (warps < 1) warps = 1;
  if (a.total_blocks >= (1ll << 31)) return 1;
  long long grid = (long long)st->sm_count * ctas_per_sm;
  if (grid > a.total_blocks) grid = a.total_blocks;
  a.blk_base = (int)(a.total_blocks / grid);
  a.blk_rem = (int)(a.total_blocks % grid);
  const long long blocks_per_cta = (a.total_blocks + grid - 1) / grid;
  if (!st->cfg_warps && es == 2) {
    // The launch ends when the warp with the most blocks ends, and the warps share the SM's transcendental pipe, so
    // the sweep costs blocks per warp (rounded up) x warps block times of about 0.046 us: a range of 516 blocks costs
    // 30 warps 18 x 30 = 540 of them and 26 warps 20 x 26 = 520 (measured at B=512, V=152064: 30.5 against 29.9 us).
    // Warps are taken away four at a time, so that the SM's four schedulers keep equal numbers (28 or 24 streaming
    // warps measured worse than either neighbour).  Every warp less costs about 0.5 % of streaming throughput
    // (latency hiding: at B=2048 thirty warps win) and saves 0.04 us of fixed time per launch, 0.1 us when the
    // launch is a programmatic dependent (fitted to launches of 64 to 2048 rows: 22 warps win below 256 rows).
    const long long per_warp_fixed = st->dependent_launch ? 2174 : 870;    // in units of 1/1000 block time
    int best_w = warps;
    long long best_cost = -1;
    for (int w = warps; w >= warps - 8 && w >= 8; w -= 4) {
      const long long cost = (blocks_per_cta + w - 1) / w * w * (1000 + 5 * (warps - w)) + per_warp_fixed * w;
      if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_w = w; }
    }
    warps = best_w;
  }
  if (blocks_per_cta < warps) warps = (int)blocks_per_cta;
  const long long rows = blocks_per_cta / a.nblk + 2;      // rows a CTA's range can touch
  if (rows > kMaxQueue) return 1;
  a.queue_cap = (int)rows;
  // block-level noise of the rows the range touches (at most 16 KB; rows past the table have theirs drawn when needed)
  long long noise_rows = rows;
  if ((size_t)noise_rows * a.nblk * 4 > 16384) noise_rows = (long long)(16384 / ((size_t)a.nblk * 4));
  a.noise_rows = (int)noise_rows;
  a.local_rows = 0;
  const size_t budget = (size_t)st->max_smem / ctas_per_sm - (ctas_per_sm > 1 ? 1024 : 0);
  size_t total = 0;
  auto lay_out = [&](int w, int sg) {
    size_t off = (size_t)w * sg * a.stage_bytes;
    auto take = [&](size_t bytes) { off = (off + 15) & ~(size_t)15; const size_t o = off; off += bytes; return (int)o; };
    a.h_bars = take((size_t)w * sg * 8);
    a.h_meta = take((size_t)w * sg * 8);
    a.h_ctrl = take(16);
    a.h_ready = take(4 * (size_t)rows);
    a.h_pre = take(sizeof(RowPre) * (size_t)rows);
    a.h_noise = take((size_t)a.noise_rows * a.nblk * 4);
    a.h_lrec = take((size_t)blocks_per_cta * sizeof(float4));       // one record per block of the range
    a.h_fscratch = take((size_t)fin * a.stage_bytes);
    total = (off + 15) & ~(size_t)15;
    return total;
  };
  while (stages > 1 && lay_out(warps, stages) > budget) --stages;
  while (warps > 1 && lay_out(warps, stages) > budget) --warps;
  const long long per_warp = (blocks_per_cta + warps - 1) / warps;
  if (per_warp < stages) stages = (int)per_warp;
  if (lay_out(warps, stages) > budget) return 1;
  a.warps = warps;
  a.fin_warps = fin;
  a.stages = stages;
  a.run_len = (a.nblk >= 64) ? 1 : (a.nblk >= 32 ? 4 : (a.nblk >= 8 ? 2 : 1));
  for (int i = 0; i < 2; ++i) {
    const int n_runs = (a.blk_base + i + a.run_len - 1) / a.run_len;
    a.runs_q[i] = n_runs / warps;
    a.runs_r[i] = n_runs % warps;
  }
  auto k = (es == 2) ? (bulk ? espo_step_hier_kernel<2, true> : espo_step_hier_kernel<2, false>)
                     : (bulk ? espo_step_hier_kernel<4, true> : espo_step_hier_kernel<4, false>);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)(warps + fin) * 32u);
  cfg.dynamicSmemBytes = total;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may be set up while the kernel before it winds down
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  if (st->dependent_launch) { cfg.attrs = attr; cfg.numAttrs = 1; }
  ESPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, k, a));
  return ESPO_OK;
}

// One launch of the step kernel over rows of `v_eff` logits whose first id is `vocab_offset`: the whole vocabulary
// (espo_step) or one shard of it (espo_step_partial, which passes `partial_out`).
static int step_launch(const void* logits, int32_t logits_dtype, int64_t row_stride, const void* values, int32_t values_dtype,
                       const int32_t* row_ids, int32_t n_rows, espo_state* st, const espo_params* p, int32_t* tokens_out,
                       uint8_t* stop_out, int32_t v_eff, int32_t vocab_offset, espo_partial* partial_out, void* stream) {
  using namespace espo;
  if (!st || !p) return ESPO_ERR_NULL;
  if (n_rows < 0) return ESPO_ERR_BAD_SHAPE;
  if (n_rows > st->capacity) return ESPO_ERR_CAPACITY;
  if ((logits_dtype != ESPO_F32 && logits_dtype != ESPO_BF16) || (values_dtype != ESPO_F32 && values_dtype != ESPO_BF16))
    return ESPO_ERR_BAD_DTYPE;
  StepArgs a;
  memset(&a, 0, sizeof(a));
  {
    const int rc = fill_params(a, st, p);
    if (rc != ESPO_OK) return rc;
  }
  if (n_rows == 0) return ESPO_OK;
  {
    int dev = -1;
    ESPO_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != st->device) return ESPO_ERR_BAD_PARAM;      // the state lives on the device that was current at its creation
  }
  if (!logits) return ESPO_ERR_NULL;
  if (!partial_out && (!values || !tokens_out || !stop_out)) return ESPO_ERR_NULL;
  if (row_stride < v_eff) return ESPO_ERR_BAD_SHAPE;
  const int nblk_eff = (v_eff + kBlockIds - 1) / kBlockIds;
  const int es = (logits_dtype == ESPO_BF16) ? 2 : 4;
  const int ves = (values_dtype == ESPO_BF16) ? 2 : 4;
  if (((uintptr_t)logits % es) || ((uintptr_t)values % ves) || ((uintptr_t)tokens_out % 4) ||
      (row_ids && ((uintptr_t)row_ids % 4)) || ((uintptr_t)partial_out % 16))
    return ESPO_ERR_ALIGN;

  a.vocab_offset = vocab_offset;
  a.partial_out = partial_out;
  a.logits = static_cast<const unsigned char*>(logits);
  a.row_stride_bytes = row_stride * es;
  a.values = values;
  a.values_bf16 = (values_dtype == ESPO_BF16);
  a.row_ids = row_ids;
  a.n_rows = n_rows; a.V = v_eff;
  a.nblk = nblk_eff;
  a.total_blocks = (long long)n_rows * nblk_eff;
  a.stage_bytes = kBlockIds * es;
  a.tokens_out = tokens_out; a.stop_out = stop_out;

  if (!a.greedy && (a.top_p < 1.f || a.top_k > 0)) {
    // filtered sampling: its own kernel, one CTA per row at a time, two CTAs per SM
    if (p->sampler != ESPO_SAMPLER_FLAT || partial_out) return ESPO_ERR_BAD_PARAM;
    if (v_eff > (1 << 21)) return ESPO_ERR_CAPACITY;       // the histogram limbs are sized for rows up to 2^21 logits
    auto fk = (es == 2) ? espo_filtered_kernel<2> : espo_filtered_kernel<4>;
    const int fgrid = n_rows < 2 * st->sm_count ? n_rows : 2 * st->sm_count;
    fk<<<(unsigned)fgrid, kFiltThreads, kFiltSmemBytes, (cudaStream_t)stream>>>(a);
    ESPO_CUDA_TRY(cudaGetLastError());
    return ESPO_OK;
  }
  const bool bulk = ((uintptr_t)logits % 16 == 0) && (a.row_stride_bytes % 16 == 0) && (((size_t)v_eff * es) % 16 == 0);
  if (p->sampler == ESPO_SAMPLER_HIER && !a.greedy) {
    const int rc = launch_hier(a, st, es, bulk, (cudaStream_t)stream);
    if (rc != 1) return rc;
    if (partial_out) return ESPO_ERR_CAPACITY;     // only that kernel serves shards of the hierarchical sampler
  }
  // Launch shape: ctas_per_sm CTAs of `warps` streaming warps (+1 finalizer warp), `stages` blocks in flight per warp.
  int ctas_per_sm = st->cfg_ctas_per_sm ? st->cfg_ctas_per_sm : 1;
  // Finalizer warps per CTA: one row takes a warp about 5 us to finalize, and an SM streams a row in
  // row_bytes / ~43 GB/s; short rows need several finalizers to keep up with the streaming warps.
  const double row_us = (double)v_eff * es / 43e3;
  int fin = (int)ceil(5.0 / (row_us * ctas_per_sm));
  fin = fin < 1 ? 1 : (fin > 8 ? 8 : fin);
  const int max_warps = (kMaxStepThreads / 32 < 64 / ctas_per_sm) ? kMaxStepThreads / 32 : 64 / ctas_per_sm;
  int warps = st->cfg_warps ? st->cfg_warps : (es == 2 ? 31 : 15);
  int stages = st->cfg_stages ? st->cfg_stages : 2;
  if (warps + fin > max_warps) warps = max_warps - fin;
  if (warps < 1) { warps = 1; fin = (fin < max_warps - 1) ? fin : (max_warps - 1 < 1 ? 1 : max_warps - 1); }
  long long grid = (long long)st->sm_count * ctas_per_sm;
  if (grid > a.total_blocks) grid = a.total_blocks;
  const long long blocks_per_cta = (a.total_blocks + grid - 1) / grid;
  if (blocks_per_cta < warps) warps = (int)blocks_per_cta;
  const long long qcap = blocks_per_cta / a.nblk + 2;
  if (qcap > kMaxQueue) return ESPO_ERR_CAPACITY;
  a.queue_cap = (int)qcap;
  // shared-memory table for the records of rows that one CTA reduces alone (at most 40 KB of it)
  const size_t rec_bytes = (size_t)a.nblk * 16;
  long long local_rows = blocks_per_cta / a.nblk + 1;
  if ((size_t)local_rows * rec_bytes > 40960) local_rows = (long long)(40960 / rec_bytes);
  a.local_rows = (int)local_rows;
  // ... and one for the block-level noise of the rows the range touches (at most 16 KB)
  long long noise_rows = a.queue_cap;
  if ((size_t)noise_rows * a.nblk * 4 > 16384) noise_rows = (long long)(16384 / ((size_t)a.nblk * 4));
  a.noise_rows = (int)noise_rows;
  const size_t fixed = sizeof(StepCtrl) + 3 * sizeof(int) * (size_t)a.queue_cap + 16 + sizeof(RowPre) * (size_t)a.queue_cap +
                       (((size_t)a.noise_rows * a.nblk * 4 + 15) & ~(size_t)15) + (size_t)a.local_rows * rec_bytes;
  const size_t budget = (size_t)st->max_smem / ctas_per_sm - (ctas_per_sm > 1 ? 1024 : 0);
  auto footprint = [&](int w, int sg) { return (size_t)w * sg * (a.stage_bytes + 16) + fixed; };
  while (stages > 1 && footprint(warps, stages) > budget) --stages;
  while (warps > 1 && footprint(warps, stages) > budget) --warps;
  const long long per_warp = (blocks_per_cta + warps - 1) / warps;
  if (per_warp < stages) stages = (int)per_warp;
  a.warps = warps;
  a.fin_warps = fin;
  a.run_len = (nblk_eff >= 64) ? 1 : (nblk_eff >= 32 ? 4 : (nblk_eff >= 8 ? 2 : 1));
  a.stages = stages;
  const size_t smem = footprint(warps, stages);
  if (smem > (size_t)st->max_smem) return ESPO_ERR_CAPACITY;

  StepKernel k = pick_kernel(es, p->sampler, bulk);
  k<<<(unsigned)grid, (unsigned)(warps + fin) * 32u, smem, (cudaStream_t)stream>>>(a);
  ESPO_CUDA_TRY(cudaGetLastError());
  return ESPO_OK;
}

int espo_step(const void* logits, int32_t logits_dtype, int64_t row_stride, const void* values, int32_t values_dtype,
              const int32_t* row_ids, int32_t n_rows, espo_state* st, const espo_params* p, int32_t* tokens_out,
              uint8_t* stop_out, void* stream) {
  if (!st) return ESPO_ERR_NULL;
  return step_launch(logits, logits_dtype, row_stride, values, values_dtype, row_ids, n_rows, st, p, tokens_out, stop_out,
                     st->V, 0, nullptr, stream);
}

int espo_step_partial(const void* logits_shard, int32_t logits_dtype, int64_t row_stride, int32_t v_shard,
                      int32_t vocab_offset, const int32_t* row_ids, int32_t n_rows, espo_state* st, const espo_params* p,
                      espo_partial* partial_out, void* stream) {
  if (!st || !p) return ESPO_ERR_NULL;
  if (v_shard < 1 || vocab_offset < 0 || (vocab_offset & 3) || (long long)vocab_offset + v_shard > st->V) return ESPO_ERR_BAD_SHAPE;
  if (p->sampler == ESPO_SAMPLER_HIER) {
    // the hierarchical sampler's draws belong to blocks of 1024 ids of the whole vocabulary: a shard starts on one
    if ((vocab_offset & 1023) || p->want_entropy || !(p->temperature > 0.f)) return ESPO_ERR_BAD_PARAM;
  } else if (p->sampler != ESPO_SAMPLER_FLAT) {
    return ESPO_ERR_BAD_PARAM;
  }
  if (n_rows > 0 && !partial_out) return ESPO_ERR_NULL;
  return step_launch(logits_shard, logits_dtype, row_stride, nullptr, ESPO_F32, row_ids, n_rows, st, p, nullptr, nullptr,
                     v_shard, vocab_offset, partial_out, stream);
}

int espo_step_merge(const espo_partial* partials, int32_t n_shards, int64_t shard_stride, const void* values,
                    int32_t values_dtype, const int32_t* row_ids, int32_t n_rows, espo_state* st, const espo_params* p,
                    int32_t* tokens_out, uint8_t* stop_out, void* stream) {
  using namespace espo;
  if (!st || !p) return ESPO_ERR_NULL;
  if (n_rows < 0 || n_shards < 1 || shard_stride < n_rows) return ESPO_ERR_BAD_SHAPE;
  if (n_rows > st->capacity) return ESPO_ERR_CAPACITY;
  if (values_dtype != ESPO_F32 && values_dtype != ESPO_BF16) return ESPO_ERR_BAD_DTYPE;
  StepArgs a;
  memset(&a, 0, sizeof(a));
  {
    const int rc = fill_params(a, st, p);
    if (rc != ESPO_OK) return rc;
  }
  if (p->want_entropy) return ESPO_ERR_BAD_PARAM;      // the partials do not carry the entropy sums
  if (n_rows == 0) return ESPO_OK;
  if (!partials || !values || !tokens_out || !stop_out) return ESPO_ERR_NULL;
  const int ves = (values_dtype == ESPO_BF16) ? 2 : 4;
  if (((uintptr_t)partials % 16) || ((uintptr_t)values % ves) || ((uintptr_t)tokens_out % 4) || (row_ids && ((uintptr_t)row_ids % 4)))
    return ESPO_ERR_ALIGN;
  a.values = values;
  a.values_bf16 = (values_dtype == ESPO_BF16);
  a.row_ids = row_ids;
  a.n_rows = n_rows; a.V = st->V;
  a.partials = partials; a.n_shards = n_shards; a.shard_stride = shard_stride;
  a.tokens_out = tokens_out; a.stop_out = stop_out;
  espo_merge_kernel<<<(unsigned)((n_rows + 63) / 64), 64, 0, (cudaStream_t)stream>>>(a);
  ESPO_CUDA_TRY(cudaGetLastError());
  return ESPO_OK;
}

int espo_end_batch_merge(const double* stats, int32_t n_parts, float alpha_ema, float eta_beta, float tau, float beta_min,
                         float beta_max, int32_t first_update, espo_params* params_inout, double* stats_out) {
  if (!stats || !params_inout) return ESPO_ERR_NULL;
  if (n_parts < 1) return ESPO_ERR_BAD_SHAPE;
  if (!(alpha_ema >= 0.f && alpha_ema <= 1.f) || isnan(eta_beta) || isnan(tau) || isnan(beta_min) || isnan(beta_max) ||
      beta_min > beta_max || isnan(params_inout->mu_g) || isnan(params_inout->sigma2_g) || isnan(params_inout->beta))
    return ESPO_ERR_BAD_PARAM;
  // pooled first and second moments of g over all parts, from each part's mean, variance and token count
  double n = 0.0, s1 = 0.0, s2 = 0.0, traj = 0.0, stopped = 0.0;
  for (int i = 0; i < n_parts; ++i) {
    const double* p = stats + 6 * (size_t)i;
    if (!(p[3] >= 0.0) || !(p[4] >= 0.0) || !(p[5] >= 0.0) || isnan(p[0]) || isnan(p[1])) return ESPO_ERR_BAD_PARAM;
    n += p[3];
    s1 += p[3] * p[0];
    s2 += p[3] * (p[1] + p[0] * p[0]);
    traj += p[4];
    stopped += p[5];
  }
  double mean = 0.0, var = 0.0, rho = 0.0;
  if (n > 0.0) {
    mean = s1 / n;
    var = fmax(s2 / n - mean * mean, 0.0);
    rho = traj > 0.0 ? stopped / traj : 0.0;
    double mu = params_inout->mu_g, sg = params_inout->sigma2_g, beta = params_inout->beta;
    if (first_update) { mu = mean; sg = var; }
    else {
      mu = (double)alpha_ema * mu + (1.0 - (double)alpha_ema) * mean;        // Eq. 7
      sg = (double)alpha_ema * sg + (1.0 - (double)alpha_ema) * var;         // Eq. 8
    }
    beta = fmin(fmax(beta + (double)eta_beta * (rho - (double)tau), (double)beta_min), (double)beta_max);   // Eq. 12
    params_inout->mu_g = (float)mu;
    params_inout->sigma2_g = (float)sg;
    params_inout->beta = (float)beta;
  }
  if (stats_out) {
    stats_out[0] = mean; stats_out[1] = var; stats_out[2] = rho; stats_out[3] = n; stats_out[4] = traj; stats_out[5] = stopped;
  }
  return ESPO_OK;
}

int espo_state_view(espo_state* st, const float** z, const float** g, const float** g_tilde, const float** logp,
                    const int32_t** t, const uint8_t** status, const int32_t** t_stop, const double** sum_g,
                    const double** sum_g2, const float** entropy, const double** sum_h) {
  if (!st) return ESPO_ERR_NULL;
  if (z) *z = st->z;
  if (g) *g = st->g;
  if (g_tilde) *g_tilde = st->g_tilde;
  if (logp) *logp = st->logp;
  if (t) *t = st->t;
  if (status) *status = st->status;
  if (t_stop) *t_stop = st->t_stop;
  if (sum_g) *sum_g = st->sum_g;
  if (sum_g2) *sum_g2 = st->sum_g2;
  if (entropy) *entropy = st->entropy;
  if (sum_h) *sum_h = st->sum_h;
  return ESPO_OK;
}

int espo_compact_active(espo_state* st, int32_t* row_ids_out, int32_t* n_active_out, void* stream) {
  if (!st || !row_ids_out || !n_active_out) return ESPO_ERR_NULL;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(1);
  cfg.blockDim = dim3(1024);
  cfg.stream = (cudaStream_t)stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  if (st->dependent_launch) { cfg.attrs = attr; cfg.numAttrs = 1; }
  ESPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, espo::espo_compact_kernel, (const uint8_t*)st->status, st->capacity, row_ids_out, n_active_out));
  return ESPO_OK;
}

int espo_end_batch(espo_state* st, float alpha_ema, float eta_beta, float tau, float beta_min, float beta_max,
                   int32_t first_update, espo_params* params_inout, double* stats_out, void* stream) {
  if (!st || !params_inout) return ESPO_ERR_NULL;
  if (!(alpha_ema >= 0.f && alpha_ema <= 1.f) || isnan(eta_beta) || isnan(tau) || isnan(beta_min) || isnan(beta_max) ||
      beta_min > beta_max || isnan(params_inout->mu_g) || isnan(params_inout->sigma2_g) || isnan(params_inout->beta))
    return ESPO_ERR_BAD_PARAM;
  espo::EndBatchArgs e;
  e.sum_g = st->sum_g; e.sum_g2 = st->sum_g2; e.t = st->t; e.status = st->status; e.capacity = st->capacity;
  e.mu_g = params_inout->mu_g; e.sigma2_g = params_inout->sigma2_g; e.beta = params_inout->beta;
  e.alpha_ema = alpha_ema; e.eta_beta = eta_beta; e.tau = tau; e.beta_min = beta_min; e.beta_max = beta_max;
  e.first_update = first_update != 0;
  e.out = st->batch_out;
  cudaStream_t s = (cudaStream_t)stream;
  espo::espo_end_batch_kernel<<<1, 1024, 0, s>>>(e);
  ESPO_CUDA_TRY(cudaGetLastError());
  double host[9];
  ESPO_CUDA_TRY(cudaMemcpyAsync(host, st->batch_out, sizeof(host), cudaMemcpyDeviceToHost, s));
  ESPO_CUDA_TRY(cudaStreamSynchronize(s));
  params_inout->mu_g = (float)host[0];
  params_inout->sigma2_g = (float)host[1];
  params_inout->beta = (float)host[2];
  if (stats_out) {
    stats_out[0] = host[3]; stats_out[1] = host[4]; stats_out[2] = host[5];
    stats_out[3] = host[6]; stats_out[4] = host[7]; stats_out[5] = host[8];
  }
  return ESPO_OK;
}

int espo_state_status(espo_state* st, uint32_t* host_out, void* stream) {
  if (!st || !host_out) return ESPO_ERR_NULL;
  ESPO_CUDA_TRY(cudaMemcpyAsync(host_out, st->dev_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  ESPO_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
  return ESPO_OK;
}

}  // extern "C"
