// ESPO decode-step kernel for the hierarchical sampler (sm_100a).
//
// The sweep is that of espo_step_kernel (a persistent grid splits the sequence of 1024-id blocks into equal
// contiguous ranges; every streaming warp owns a private ring of shared-memory stages filled by bulk copies), with
// the work divided so that the streaming warps do nothing but reduce blocks and the rest overlaps the sweep:
//   * A streaming warp reduces a block to (max, sum of exp, entropy sum) and its lane 0 stores that record, with a
//     presence mark, into a shared-memory table indexed by the block's position in the CTA's range -- one 16-byte
//     store, no fence, no counter: the loop is bound by instruction issue, and everything else was measured to cost
//     more there than anywhere else.
//   * The finalizer warps follow the rows in the order the CTA streams them.  For a row that lies wholly inside the
//     CTA's range they consume its records as they appear: lane l takes blocks l, l+32, ... in increasing order,
//     takes the rounding offset of the block's exponents out, forms the block's perturbed score
//     m_b/T + ln s_b - ln E_b (block-level noise drawn ahead of time) and folds the block into the lane's running
//     (max, sum, entropy sum, best score).  Once half of the row is in, whenever the best block so far changes
//     they also resolve the sub-block and id levels inside it ahead of time (the block comes back from L2 into a
//     scratch buffer).  When the last record appears, what is left is the cross-lane merge, the winner's token if
//     the last records changed it, Eq. 6, 9, 10, 11 and the state update.
//   * The part of a row that another CTA also works on is copied to global memory when it is complete, the CTA's
//     share is added to the row's global ticket, and whoever completes the ticket runs the same per-lane fold over
//     the whole row's records.
// The per-lane fold visits a lane's blocks in a fixed order and the lanes are merged in a fixed order, so results
// do not depend on the launch shape or on the order in which records appear.  Every wait is bounded; a wait that
// runs out sets ESPO_DEV_TIMEOUT.
#pragma once

#include "espo_step_common.cuh"

namespace espo {

// Shared-memory tables of a CTA; "rows" are the rows its range touches, indexed by local row.
struct HierTables {
  volatile int* ready;     // [rows] 1: pre[k] (and noise row k, if k < noise_rows) are filled in
  RowPre* pre;             // [rows] slot, state and critic value of the row
  float* noise;            // [noise_rows][nblk] ln E of the block-level draws
  float4* lrec;            // [blocks of the range] (m_b, s_b, u_b, mark) by position in the CTA's range; mark 0: not there yet
};

__device__ __forceinline__ HierTables hier_tables(const StepArgs& a, unsigned char* smem) {
  HierTables tb;
  tb.ready = reinterpret_cast<volatile int*>(smem + a.h_ready);
  tb.pre = reinterpret_cast<RowPre*>(smem + a.h_pre);
  tb.noise = reinterpret_cast<float*>(smem + a.h_noise);
  tb.lrec = reinterpret_cast<float4*>(smem + a.h_lrec);
  return tb;
}

// (max, sum of 2^((x - max) k2), sum of e * t) of one 1024-id block held in a shared-memory stage; every lane gets
// the results.  The exponents are x*k2 + c0 with c0 = -max*k2 rounded once, so all of them are off by the rounding
// error of that product; the caller takes the common factor out.
template <int ES>
__device__ __forceinline__ void hier_reduce_block(const StepArgs& a, const unsigned char* blk, int lane, int nvalid,
                                                  float& m_b, float& s_b, float& u_b) {
  BlockVals<ES> bv;
  bv.load(blk, lane, nvalid);
  m_b = warp_max(bv.lane_max());
  const float ref = (m_b == __int_as_float(0xff800000)) ? 0.0f : m_b;   // an all -inf block sums to 0
  const float2 k2v = make_float2(a.k2, a.k2);
  const float c0 = -ref * a.k2;
  const float2 c0v = make_float2(c0, c0);
  float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
  u_b = 0.f;
  if (a.want_entropy) {
    float2 ua = make_float2(0.f, 0.f);
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      float2 t = __ffma2_rn(bv.pair(j), k2v, c0v);
      const float2 e = make_float2(ex2_approx(t.x), ex2_approx(t.y));
      if (e.x == 0.f) t.x = 0.f;   // masked ids (t = -inf): 0 * -inf is not a number
      if (e.y == 0.f) t.y = 0.f;
      ua = __ffma2_rn(e, t, ua);
      if (j & 1) acc1 = __fadd2_rn(acc1, e); else acc0 = __fadd2_rn(acc0, e);
    }
    u_b = warp_sum(ua.x + ua.y);
  } else {
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const float2 t = __ffma2_rn(bv.pair(j), k2v, c0v);
      const float2 e = make_float2(ex2_approx(t.x), ex2_approx(t.y));
      if (j & 1) acc1 = __fadd2_rn(acc1, e); else acc0 = __fadd2_rn(acc0, e);
    }
  }
  s_b = warp_sum((acc0.x + acc0.y) + (acc1.x + acc1.y));
}

// One logit of the block held in a stage, by its position in the block; positions at or beyond nvalid read as -inf.
template <int ES>
__device__ __forceinline__ float stage_logit(const unsigned char* stage, int pos, int nvalid) {
  if (pos >= nvalid) return __int_as_float(0xff800000);
  if (ES == 2) return __uint_as_float((uint32_t)reinterpret_cast<const unsigned short*>(stage)[pos] << 16);
  return reinterpret_cast<const float*>(stage)[pos];
}

// The sub-block and id levels of the sampler inside block `blk` of a row, taken from a shared-memory copy of the
// block (levels 1 and 0 of the row's draw stream): lane j scores sub-block j (32 consecutive ids) by its
// log-sum-exp plus Gumbel noise, then lane e scores id e of the winning sub-block.  Every lane returns the token
// (a row-relative id) and its logit.  The block must hold a finite logit.  Written to need few registers: the 32
// logits of a lane's sub-block are read twice (maximum, then sum) instead of being kept.
template <int ES>
__device__ __forceinline__ void hier_descend_stage(const StepArgs& a, const unsigned char* stage, int nvalid, int blk,
                                                   uint32_t slot, uint32_t step, int lane, int& token, float& l_tok) {
  // `blk` is the block's number in the whole vocabulary (a vocabulary shard starts at a multiple of 1024 ids): the
  // draws belong to global sub-block and token numbers, and the token returned is a global id.
  const float NINF = __int_as_float(0xff800000);
  const DrawStream ds{a.key0, a.key1, step, slot, a.batch_bits};
  constexpr int kVecsPerSub = kSubIds * ES / 16;     // 16-byte vectors of a sub-block: 4 (bfloat16) or 8 (float32)
  const uint4* sp = reinterpret_cast<const uint4*>(stage) + lane * kVecsPerSub;
  float m_j = NINF;
  float s_j = 0.f;
  if (nvalid == kBlockIds) {
    if (ES == 2) {
      uint32_t mm = 0xFF80FF80u;
#pragma unroll
      for (int i = 0; i < kVecsPerSub; ++i) {
        const uint4 q = sp[i];
        mm = bf16x2_max(bf16x2_max(mm, q.x), bf16x2_max(bf16x2_max(q.y, q.z), q.w));
      }
      m_j = fmaxf(bf16_lo(mm), bf16_hi(mm));
    } else {
#pragma unroll
      for (int i = 0; i < kVecsPerSub; ++i) {
        const uint4 q = sp[i];
        m_j = fmaxf(fmaxf(m_j, __uint_as_float(q.x)), fmaxf(fmaxf(__uint_as_float(q.y), __uint_as_float(q.z)), __uint_as_float(q.w)));
      }
    }
    if (m_j > NINF) {
      // sum over the 32 values of 2^((x - m_j) k2), two per packed multiply-add, pair i into accumulator i & 1
      const float c0 = -m_j * a.k2;
      const float2 k2v = make_float2(a.k2, a.k2), c0v = make_float2(c0, c0);
      float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
      for (int i = 0; i < kVecsPerSub; ++i) {
        const uint4 q = sp[i];
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
        if (ES == 2) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float2 t = __ffma2_rn(make_float2(bf16_lo(w[k]), bf16_hi(w[k])), k2v, c0v);
            const float2 e = make_float2(ex2_approx(t.x), ex2_approx(t.y));
            if (k & 1) acc1 = __fadd2_rn(acc1, e); else acc0 = __fadd2_rn(acc0, e);
          }
        } else {
#pragma unroll
          for (int k = 0; k < 2; ++k) {
            const float2 t = __ffma2_rn(make_float2(__uint_as_float(w[2 * k]), __uint_as_float(w[2 * k + 1])), k2v, c0v);
            const float2 e = make_float2(ex2_approx(t.x), ex2_approx(t.y));
            if ((2 * i + k) & 1) acc1 = __fadd2_rn(acc1, e); else acc0 = __fadd2_rn(acc0, e);
          }
        }
      }
      // every exponent is off by the rounding error of m_j*k2: one factor takes it out
      s_j = ((acc0.x + acc0.y) + (acc1.x + acc1.y)) * ex2_approx(-fmaf(m_j, a.k2, c0));
    }
  } else {
    // the row's ragged last block: element by element
    const int p0 = lane * kSubIds;
#pragma unroll 1
    for (int i = 0; i < kSubIds; ++i) m_j = fmaxf(m_j, stage_logit<ES>(stage, p0 + i, nvalid));
    if (m_j > NINF) {
      const float c0 = -m_j * a.k2;
      float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll 1
      for (int i = 0; i < kSubIds / 2; ++i) {
        const float2 t = __ffma2_rn(make_float2(stage_logit<ES>(stage, p0 + 2 * i, nvalid), stage_logit<ES>(stage, p0 + 2 * i + 1, nvalid)),
                                    make_float2(a.k2, a.k2), make_float2(c0, c0));
        const float2 e = make_float2(ex2_approx(t.x), ex2_approx(t.y));
        if (i & 1) acc1 = __fadd2_rn(acc1, e); else acc0 = __fadd2_rn(acc0, e);
      }
      s_j = ((acc0.x + acc0.y) + (acc1.x + acc1.y)) * ex2_approx(-fmaf(m_j, a.k2, c0));
    }
  }
  float sc = NINF;
  int j = -1;
  if (m_j > NINF) {
    const int gsub = blk * (kBlockIds / kSubIds) + lane;           // the row's sub-block number
    sc = fmaf(m_j, a.inv_temp, log_sum(s_j) - ln_expo(expo_at(ds, 1u, (uint32_t)gsub)));
    j = lane;
  }
  warp_argmax(sc, j);
  const int sub_pick = max(j, 0);                  // j < 0 cannot happen: the block has a finite id
  // ---- ids of the chosen sub-block: lane e takes position 32*sub_pick + e of the block ----
  const int pos = sub_pick * kSubIds + lane;
  const float mine = stage_logit<ES>(stage, pos, nvalid);
  float sc0 = NINF;
  int cand = -1;
  if (mine > NINF) {
    sc0 = fmaf(mine, a.inv_temp, -ln_expo(expo_at(ds, 0u, (uint32_t)(blk * kBlockIds + pos))));
    cand = pos;
  }
  warp_argmax(sc0, cand);
  const int pick = max(cand, sub_pick * kSubIds);  // cand < 0 cannot happen for a sub-block with a finite id
  token = blk * kBlockIds + pick;
  l_tok = __shfl_sync(kFullMask, mine, pick & 31);
}

// The same two levels for a block that has no shared-memory copy (rows past the candidate buffers): the block is
// brought from global memory (it was streamed moments ago: L2) into the calling warp's scratch first.
template <int ES>
__device__ __forceinline__ void hier_fetch_block(const StepArgs& a, const unsigned char* row_base, int blk, int nvalid,
                                                 unsigned char* scratch, int lane) {
  const unsigned char* src = row_base + (size_t)blk * kBlockIds * ES;
  if ((reinterpret_cast<uintptr_t>(src) & 15u) == 0 && nvalid == kBlockIds) {
    const uint4* s4 = reinterpret_cast<const uint4*>(src);
    uint4* d4 = reinterpret_cast<uint4*>(scratch);
#pragma unroll
    for (int i = 0; i < kBlockIds * ES / 16 / 32; ++i) d4[i * 32 + lane] = __ldg(s4 + i * 32 + lane);
  } else if (ES == 2) {
    for (int i = lane; i < nvalid; i += 32) reinterpret_cast<unsigned short*>(scratch)[i] = __ldg(reinterpret_cast<const unsigned short*>(src) + i);
  } else {
    for (int i = lane; i < nvalid; i += 32) reinterpret_cast<uint32_t*>(scratch)[i] = __ldg(reinterpret_cast<const uint32_t*>(src) + i);
  }
  __syncwarp();
}

// What a lane has folded of its blocks of a row so far.
struct LaneAcc {
  float run_m, run_s, run_u;   // running maximum; sums of e and of e*t relative to it
  float best;                  // best perturbed block score, and the block that has it (the lower one of equal scores)
  int best_b;
  bool poisoned;               // some block held NaN or +inf
};

__device__ __forceinline__ LaneAcc lane_acc_init() {
  LaneAcc c;
  c.run_m = __int_as_float(0xff800000); c.run_s = 0.f; c.run_u = 0.f;
  c.best = __int_as_float(0xff800000); c.best_b = -1; c.poisoned = false;
  return c;
}

// Folds the record r = (m_b, s_b, u_b, mark) of block b into the lane's running values; ln_e is ln E_b of the block's
// draw.  Both ways of finishing a row (as records appear; all at once from global memory) go through here with the
// same blocks per lane in the same order, so they produce the same bits.
__device__ __forceinline__ void lane_fold(const StepArgs& a, LaneAcc& c, float4 r, int b, float ln_e) {
  const float NINF = __int_as_float(0xff800000);
  c.poisoned |= !(r.y >= 0.0f) || isinf(r.y);      // NaN or inf sum: the block held NaN or +inf
  if (!(r.y > 0.f) || isinf(r.y)) return;          // nothing finite in the block
  // The block's exponents were all off by dlt = fl(-m_b*k2) + m_b*k2 (hier_reduce_block), which the fused
  // multiply-add returns exactly: s_b and u_b carry a factor 2^dlt (and u_b the shift dlt*s_b), taken out here.
  // |dlt| is half an ulp of m_b*k2 (below 2^-9 even for rows at an offset of 30 000), so 2^-dlt is 1 + x + x^2/2
  // with x = -dlt ln 2 to better than 1e-9: this warp shares the transcendental pipe with the streaming warps,
  // whose exponentials keep it full, and every use of it here waits in that queue.
  const float dlt = fmaf(r.x, a.k2, -r.x * a.k2);
  const float x = -dlt * 0.6931471805599453f;
  const float f = fmaf(x, fmaf(x, 0.5f, 1.0f), 1.0f);
  const float s_c = r.y * f;
  const float u_c = fmaf(r.z, f, -dlt * s_c);
  // Moving the reference from R to R' turns (S, U) into g (S, U + (R - R') k2 S) with g = 2^((R - R') k2).  Of the
  // running sums and the block only the one with the smaller maximum moves: one exponential.
  const bool up = (r.x > c.run_m);                       // the block raises the maximum (always true for the first one)
  const float nm = up ? r.x : c.run_m;
  const float d = (c.run_s > 0.f) ? -fabsf(c.run_m - r.x) * a.k2 : 0.f;
  const float g = ex2_approx(d);
  const float d1 = up ? d : 0.f, f1 = up ? g : 1.0f;     // applied to the running sums
  const float d2 = up ? 0.f : d, f2 = up ? 1.0f : g;     // applied to the block
  c.run_u = fmaf(f1, fmaf(d1, c.run_s, c.run_u), f2 * fmaf(d2, s_c, u_c));
  c.run_s = fmaf(f1, c.run_s, f2 * s_c);
  c.run_m = nm;
  const float sc = fmaf(r.x, a.inv_temp, log_sum(s_c) - ln_e);
  if (sc > c.best || c.best_b < 0) { c.best = sc; c.best_b = b; }
  (void)NINF;
}

// The token inside block `blk` of a row whose block is no longer in shared memory: the block comes back from global
// memory (L2) into `scratch`, then the sub-block and id levels are resolved there.
template <int ES>
__device__ __forceinline__ void hier_resolve(const StepArgs& a, int row, int blk, const RowPre& pre, unsigned char* scratch,
                                             int lane, int& token, float& l_tok) {
  const int nvalid = min(kBlockIds, a.V - blk * kBlockIds);
  hier_fetch_block<ES>(a, a.logits + (size_t)row * a.row_stride_bytes, blk, nvalid, scratch, lane);
  hier_descend_stage<ES>(a, scratch, nvalid, blk + (a.vocab_offset >> 10), (uint32_t)pre.slot, (uint32_t)pre.t_now, lane, token, l_tok);
  __syncwarp();
}

// What a vocabulary shard leaves about a row instead of acting on it (espo_step_partial): flags bit 0: the shard's
// part of the row held NaN or +inf; bit 1: nothing was computed because the slot is bad or the trajectory has ended.
__device__ __forceinline__ void hier_report(const StepArgs& a, int row, int lane, float m, float s, float best, int token,
                                            float l_tok, unsigned flags, bool no_ticket) {
  if (lane == 0) {
    espo_partial pr;
    pr.m = m; pr.s = s; pr.best = best; pr.best_id = token; pr.x_best = l_tok; pr.flags = flags;
    pr.reserved[0] = 0u; pr.reserved[1] = 0u;
    a.partial_out[row] = pr;
    if (!no_ticket) a.ticket[row] = 0;   // ready for the next launch
  }
}

// A row whose slot is bad or whose trajectory has ended: untouched, token -1.
__device__ __forceinline__ void hier_skip_row(const StepArgs& a, int row, int lane, const RowPre& pre, bool no_ticket) {
  const float NINF = __int_as_float(0xff800000);
  if (a.partial_out) hier_report(a, row, lane, NINF, 0.f, NINF, -1, NINF, 2u, no_ticket);
  else if (pre.slot < 0) mark_row(a, row, 0, lane, -1, ESPO_DEV_BAD_SLOT, -1, no_ticket);
  else mark_row(a, row, pre.slot, lane, -1, 0u, -1, no_ticket);
}

// The end of a row: merges the lanes' running values in a fixed order and commits the row (Eq. 6, 9, 10, 11).
// (c_blk, c_token, c_ltok): the token already resolved inside block c_blk (-1: none); resolved here if the winning
// block is another one.
template <int ES>
__device__ __noinline__ void hier_commit(const StepArgs& a, int row, int lane, const RowPre pre, LaneAcc c, int c_blk,
                                         int c_token, float c_ltok, unsigned char* scratch, bool no_ticket) {
  const float NINF = __int_as_float(0xff800000);
  const int slot = pre.slot;
  float best = c.best;
  int best_b = c.best_b;
  warp_argmax(best, best_b);
  const bool poisoned = __any_sync(kFullMask, c.poisoned);
  if (!poisoned && best_b >= 0 && best_b != c_blk) hier_resolve<ES>(a, row, best_b, pre, scratch, lane, c_token, c_ltok);
  float run_m = c.run_m, run_s = c.run_s, run_u = c.run_u;
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
  if (a.partial_out) {
    // a vocabulary shard: leave what the merge needs and do not touch the state (a shard may hold no finite logit)
    if (poisoned || M == __int_as_float(0x7f800000) || M != M) hier_report(a, row, lane, NINF, 0.f, NINF, -1, NINF, 1u, no_ticket);
    else if (best_b < 0) hier_report(a, row, lane, NINF, 0.f, NINF, -1, NINF, 0u, no_ticket);
    else hier_report(a, row, lane, M, S, best, c_token, c_ltok, 0u, no_ticket);
    return;
  }
  if (poisoned || best_b < 0 || M == __int_as_float(0x7f800000) || M != M || !(M > NINF) || isinf(M)) {
    mark_row(a, row, slot, lane, 0, ESPO_DEV_BAD_ROW, ESPO_ROW_BAD, no_ticket);
    return;
  }
  const DrawStream ds{a.key0, a.key1, (uint32_t)pre.t_now, (uint32_t)slot, a.batch_bits};
  if (lane == 0) commit_row(a, row, pre, ds, M, S, logf(S), run_u, c_ltok, c_token, no_ticket);
}

__device__ __forceinline__ int hier_walk_row(const CtaRange& cr, int idx) {
  // the walk starts with the range's last row when that row is shared with the next CTA
  return cr.off > 0 ? (idx == 0 ? cr.n_local - 1 : idx - 1) : idx;
}

// The preparation pass, run by the finalizer warps while the streaming warps fetch their first blocks: read the
// state of every row the range touches (lane-parallel over rows, in the order of the walk) and draw the block-level
// noise of those rows (lane-parallel over groups of four blocks: one Philox call serves four).  The first group's
// loads are issued by the caller before the CTA's first rendezvous (`first_pre`), ahead of the bulk copies' traffic.
__device__ __forceinline__ void hier_prepare_rows(const StepArgs& a, const CtaRange& cr, const HierTables& tb, int lane,
                                                  int first, int step, const RowPre& first_pre) {
  // the draws belong to block numbers of the whole vocabulary (a shard's first block is number boff); one Philox
  // call serves the four blocks 4 gq .. 4 gq + 3
  const int boff = a.vocab_offset >> 10;
  const int gq0 = boff >> 2;
  const int nq = ((boff + a.nblk - 1) >> 2) - gq0 + 1;
  for (int g0 = first * 32; g0 < cr.n_local; g0 += step * 32) {
    const int n_g = min(32, cr.n_local - g0);
    if (lane < n_g) {
      const int k = hier_walk_row(cr, g0 + lane);
      tb.pre[k] = (g0 == first * 32) ? first_pre : prefetch_row(a, (int)(cr.r_first + k));
    }
    __syncwarp();
    const int items = n_g * nq;
    for (int it = lane; it < items; it += 32) {
      const int r = it / nq, q = it - r * nq;
      const int k = hier_walk_row(cr, g0 + r);
      if (k >= a.noise_rows) continue;
      const int slot = tb.pre[k].slot, status = tb.pre[k].status, t_now = tb.pre[k].t_now;
      if (slot < 0 || status != ESPO_ROW_ACTIVE) continue;
      const uint4 rnd = philox4x32_10((uint32_t)(gq0 + q), (uint32_t)t_now, (uint32_t)slot, a.batch_bits | 2u, a.key0, a.key1);
      const uint32_t wd[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int b = 4 * (gq0 + q) + i - boff;
        if (b >= 0 && b < a.nblk) tb.noise[(size_t)k * a.nblk + b] = ln_expo(expo_from_word(wd[i]));
      }
    }
    __syncwarp();
    __threadfence_block();
    if (lane < n_g) tb.ready[hier_walk_row(cr, g0 + lane)] = 1;
  }
}

// What a finalizer warp does after the preparation pass (and a streaming warp once it has run out of blocks): take the
// next row of the CTA's walk that nobody follows yet, follow it to its end, repeat.
template <int ES>
__device__ void hier_follow_rows(const StepArgs& a, const CtaRange& cr, const HierTables& tb, volatile int* abort_flag,
                                 int* next_row, unsigned char* scratch, int lane) {
  const float NINF = __int_as_float(0xff800000);
  auto give_up = [&]() { if (lane == 0 && !*abort_flag) { atomicOr(a.dev_status, ESPO_DEV_TIMEOUT); *abort_flag = 1; } };
  for (;;) {
    // rows are handed out in the order of the CTA's walk, to whichever warp is free
    int idx = 0;
    if (lane == 0) idx = atomicAdd(next_row, 1);
    idx = __shfl_sync(kFullMask, idx, 0);
    if (idx >= cr.n_local) return;
    const int k = hier_walk_row(cr, idx);
    const int row = (int)(cr.r_first + k);
    // ---- the row's state (another finalizer warp may be the one that prepares it) ----
    {
      int ok = 1;
      if (lane == 0) {
        uint32_t it = 0;
        while (tb.ready[k] == 0) {
          if (*abort_flag || ++it >= kPollSpinLimit) { ok = 0; break; }
          __nanosleep(40);
        }
        __threadfence_block();
      }
      ok = __shfl_sync(kFullMask, ok, 0);
      __syncwarp();
      if (!ok) { give_up(); return; }
    }
    const RowPre pre = tb.pre[k];
    const bool live = pre.slot >= 0 && pre.status == ESPO_ROW_ACTIVE;
    const int share = cr.share(k);
    const int b_lo = max(k * cr.nblk, cr.b0) - k * cr.nblk;         // first block of the row that is this CTA's
    const float4* rec = tb.lrec + (k * cr.nblk - cr.b0);            // rec[b] for the CTA's blocks b of the row
    const float* nz = (k < a.noise_rows) ? tb.noise + (size_t)k * a.nblk : nullptr;
    const DrawStream ds{a.key0, a.key1, (uint32_t)pre.t_now, (uint32_t)pre.slot, a.batch_bits};
    auto noise_at = [&](int b) { return nz ? nz[b] : ln_expo(expo_at(ds, 2u, (uint32_t)(b + (a.vocab_offset >> 10)))); };
    const bool whole = share == a.nblk;
    if (!live) {
      // a row that takes no part needs no records: a whole row is answered at once, a shared one by whoever
      // completes its ticket (every CTA sees the same state, so all of them come here)
      if (whole) {
        hier_skip_row(a, row, lane, pre, true);
      } else {
        unsigned old = 0;
        if (lane == 0) old = atom_add_acq_rel_gpu(a.ticket + row, (unsigned)share);
        old = __shfl_sync(kFullMask, old, 0);
        if (old + (unsigned)share == (unsigned)a.nblk) hier_skip_row(a, row, lane, pre, false);
      }
      continue;
    }
    if (whole) {
      // ---- fold the records round by round as they appear: in round j lane l takes block 32 j + l, once all blocks
      //      of the round are there (they are reduced within one turn of the streaming warps, about 1.5 us; folding
      //      them one by one would run the whole warp for one lane's sake) ----
      LaneAcc acc = lane_acc_init();
      int c_blk = -1, c_token = 0;
      float c_ltok = NINF;
      const int n_rounds = (a.nblk + 31) >> 5;
      for (int j = 0; j < n_rounds; ++j) {
        const int b = 32 * j + lane;
        float4 r = make_float4(0.f, 0.f, 0.f, 1.f);
        uint32_t idle = 0;
        for (;;) {
          if (b < a.nblk) r = ld_volatile_f4(rec + b);
          if (__all_sync(kFullMask, r.w != 0.f)) break;
          if (*abort_flag || ++idle >= kPollSpinLimit) { give_up(); return; }
          __nanosleep(j + 1 == n_rounds ? 30 : 250);     // only the row's last round is waited for closely
        }
        if (b < a.nblk) lane_fold(a, acc, r, b, noise_at(b));
        // in the rows that end the CTA's walk (the launch waits for them), once half of the row is in, resolve the
        // token inside the best block so far ahead of time
        if (idx + 2 >= cr.n_local && j + 1 < n_rounds && 2 * (j + 1) >= n_rounds) {
          float best = acc.best;
          int best_b = acc.best_b;
          warp_argmax(best, best_b);
          if (best_b >= 0 && best_b != c_blk && !__any_sync(kFullMask, acc.poisoned)) {
            hier_resolve<ES>(a, row, best_b, pre, scratch, lane, c_token, c_ltok);
            c_blk = best_b;
          }
        }
      }
      hier_commit<ES>(a, row, lane, pre, acc, c_blk, c_token, c_ltok, scratch, true);
      continue;
    }
    // ---- a row shared with other CTAs: wait for this CTA's records, copy them to global memory, add the share to
    //      the row's ticket; whoever completes it folds the whole row ----
    for (int b = b_lo + lane; __any_sync(kFullMask, b < b_lo + share); b += 32) {
      uint32_t idle = 0;
      for (;;) {
        const bool there = (b >= b_lo + share) || ld_volatile_f4(rec + b).w != 0.f;
        if (__all_sync(kFullMask, there)) break;
        if (*abort_flag || ++idle >= kPollSpinLimit) { give_up(); return; }
        __nanosleep(b - lane + 32 >= b_lo + share ? 30 : 250);
      }
    }
    float4* rec_g = a.records + (size_t)row * a.nblk;
    for (int b = b_lo + lane; b < b_lo + share; b += 32) rec_g[b] = rec[b];
    __syncwarp();
    unsigned old = 0;
    if (lane == 0) old = atom_add_acq_rel_gpu(a.ticket + row, (unsigned)share);   // the CTA's records before its ticket
    old = __shfl_sync(kFullMask, old, 0);
    __syncwarp();
    if (old + (unsigned)share != (unsigned)a.nblk) continue;
    // this CTA completed the row: the same fold over all of its records, five of a lane's blocks at a time
    LaneAcc acc = lane_acc_init();
    constexpr int kPerLane = 5;
    for (int base = 0; base < a.nblk; base += 32 * kPerLane) {
      float4 r[kPerLane];
#pragma unroll
      for (int i = 0; i < kPerLane; ++i) {
        const int b = base + 32 * i + lane;
        r[i] = (b < a.nblk) ? ld_volatile_f4(rec_g + b) : make_float4(NINF, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int i = 0; i < kPerLane; ++i) {
        const int b = base + 32 * i + lane;
        if (b < a.nblk) lane_fold(a, acc, r[i], b, noise_at(b));
      }
    }
    hier_commit<ES>(a, row, lane, pre, acc, -1, 0, NINF, scratch, false);
  }
}

template <int ES, bool BULK>
__global__ void __launch_bounds__(kMaxStepThreads, 1) espo_step_hier_kernel(const __grid_constant__ StepArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int W = a.warps, S = a.stages;
  unsigned char* ring = smem;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + a.h_bars);
  int2* metas = reinterpret_cast<int2*>(smem + a.h_meta);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + a.h_ctrl);
  int* next_row = reinterpret_cast<int*>(smem + a.h_ctrl) + 1;      // rows of the walk handed out so far
  const HierTables tb = hier_tables(a, smem);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // The next kernel in the stream may be set up now (if it was launched as a programmatic dependent); this one reads
  // or writes no global memory before the wait below.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // The CTA's range: the first `blk_rem` CTAs take blk_base + 1 blocks, the others blk_base (fewer than 2^31 blocks in
  // all: 32-bit arithmetic, a launch starts with cold instruction and constant caches and every subroutine counts).
  CtaRange cr;
  const int big = (int)blockIdx.x < a.blk_rem;
  {
    const unsigned g0 = blockIdx.x * (unsigned)a.blk_base + (unsigned)min((int)blockIdx.x, a.blk_rem);
    cr.nblk = a.nblk;
    cr.n = a.blk_base + big;
    const unsigned r_first = g0 / (unsigned)a.nblk;
    cr.r_first = r_first;
    cr.b0 = (int)(g0 - r_first * (unsigned)a.nblk);
    const int last = cr.b0 + cr.n - 1;                  // the range's last block, counted from block 0 of its first row
    const int k_last = last / a.nblk;
    cr.n_local = k_last + 1;
    cr.off = k_last > 0 ? k_last * a.nblk - cr.b0 : 0;  // the walk starts where the last row's part starts
  }

  if (warp >= W) {
    // ------------------------------------------------------------------ finalizer warps
    // the state of the first rows of the walk is asked for before anything else, ahead of the streaming warps' traffic
    asm volatile("griddepcontrol.wait;" ::: "memory");     // the kernel before this one has completed
    RowPre first_pre;
    {
      const int idx = (warp - W) * 32 + lane;
      first_pre = prefetch_row(a, (int)(cr.r_first + hier_walk_row(cr, idx < cr.n_local ? idx : 0)));
    }
    for (int i = threadIdx.x - W * 32; i < a.queue_cap; i += (blockDim.x - W * 32)) tb.ready[i] = 0;
    // (B): the streaming warps have cleared the record table and the control words; they do not wait here
    asm volatile("bar.sync 2, %0;" ::"r"(blockDim.x) : "memory");
    hier_prepare_rows(a, cr, tb, lane, warp - W, a.fin_warps, first_pre);
    hier_follow_rows<ES>(a, cr, tb, abort_flag, next_row, smem + a.h_fscratch + (size_t)(warp - W) * a.stage_bytes, lane);
    return;
  }

  // -------------------------------------------------------------------- streaming warps
  if (threadIdx.x == 0) { *abort_flag = 0; *next_row = 0; }
  if (lane == 0) {
    for (int s = 0; s < S; ++s) mbar_init(&bars[warp * S + s], 1);
    mbar_init_fence();
  }
  __syncwarp();
  unsigned char* my_ring = ring + (size_t)warp * S * a.stage_bytes;
  uint64_t* my_bar = bars + warp * S;
  int2* my_meta = metas + warp * S;            // (position in the range, block of its row) of the block each stage holds
  // The warps take turns of C consecutive positions of the CTA's walk: warp w owns the runs w, w + W, w + 2W, ...
  const int C = a.run_len;
  int n_my;
  {
    // runs of the walk = runs_q * W + runs_r (divided on the host, for either size of range)
    const int q = a.runs_q[big], r = a.runs_r[big];
    n_my = (q + (warp < r ? 1 : 0)) * C;
    const int last_owner = r ? r - 1 : W - 1;                   // the walk's last run may be short
    if (warp == last_owner && n_my > 0) n_my -= (q * W + r) * C - cr.n;
  }
  constexpr int kBlockBytes = kBlockIds * ES;

  // Where the warp's next block to fetch lies: position fq of the range, block f_blk of its row.  The cursor moves by
  // one block inside a run and by (W-1)C+1 between runs, and only divides when the walk wraps around the range's end.
  int fq, f_blk, f_run = 0;
  const unsigned char* f_ptr;
  auto seek = [&](int q) {
    fq = q;
    const int li = cr.b0 + q;
    const int lrow = (int)((unsigned)li / (unsigned)cr.nblk);
    f_blk = li - lrow * cr.nblk;
    f_ptr = a.logits + (size_t)(cr.r_first + lrow) * a.row_stride_bytes + (size_t)f_blk * kBlockBytes;
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
    my_meta[s] = make_int2(fq, f_blk);
    fence_proxy_async();             // the warp's reads of this stage come before the copy's writes
    mbar_arrive_expect_tx(&my_bar[s], bytes);
    bulk_copy_g2s(my_ring + (size_t)s * a.stage_bytes, f_ptr, bytes, &my_bar[s]);
  };
  int fetched = 0;
  asm volatile("griddepcontrol.wait;" ::: "memory");       // the kernel before this one has completed
  if (BULK) {
    for (; fetched < S && fetched < n_my; ++fetched) {
      if (lane == 0) issue(fetched);
      advance();
    }
  }
  for (int i = threadIdx.x; i < cr.n; i += W * 32) tb.lrec[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  // (A) among the streaming warps: the record table is cleared before anybody writes a record; (B) tells the
  // finalizer warps so without waiting for them (they start with loads from global memory)
  asm volatile("bar.sync 1, %0;" ::"r"(W * 32) : "memory");
  asm volatile("bar.arrive 2, %0;" ::"r"(blockDim.x) : "memory");

  int s = 0;
  uint32_t parity = 0;
  int done = 0;
  bool gave_up = false;
  for (; done < n_my; ++done) {
    unsigned char* stage = my_ring + (size_t)s * a.stage_bytes;
    int q, blk;
    if (BULK) {
      if (!mbar_wait_bounded(&my_bar[s], parity, abort_flag)) { gave_up = true; break; }
      const int2 mt = my_meta[s];
      q = mt.x; blk = mt.y;
    } else {
      q = fq; blk = f_blk;
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
    float m_b, s_b, u_b;
    hier_reduce_block<ES>(a, stage, lane, nvalid, m_b, s_b, u_b);
    if (lane == 0) tb.lrec[q] = make_float4(m_b, s_b, u_b, 1.0f);     // one 16-byte store: the mark comes with the values
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
    return;
  }
  // A streaming warp that has run out of blocks follows rows that nobody has taken yet; the first stage of its ring
  // (all of its copies have landed) is its scratch.
  hier_follow_rows<ES>(a, cr, tb, abort_flag, next_row, my_ring, lane);
}

}  // namespace espo
