// Pieces shared by the ESPO decode-step kernels: the kernel argument block, the reduction of one 1024-id block held in
// shared memory, what a warp reads about a row before it finishes it, and the per-row commit (Eq. 6, 9, 10, 11).
#pragma once

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "espo.h"
#include "espo_device.cuh"

namespace espo {

constexpr int kMaxStepThreads = 1024;
constexpr int kMaxConsumerWarps = kMaxStepThreads / 32 - 1;   // at least one more warp is a finalizer
constexpr int kMaxQueue = 4096;

struct StepArgs {
  // inputs
  const unsigned char* logits;
  int64_t row_stride_bytes;
  const void* values;
  int values_bf16;
  const int32_t* row_ids;
  int n_rows, V, capacity;
  // tiling
  int nblk;                 // 1024-id blocks per row
  long long total_blocks;   // n_rows * nblk
  int warps, fin_warps, stages, stage_bytes, queue_cap;   // streaming warps, finalizer warps, ring depth
  int run_len;              // consecutive blocks a streaming warp takes per turn (1 unless rows are short)
  int local_rows;           // rows whose block records fit in the CTA's shared-memory table (0: none)
  int noise_rows;           // rows whose block-level noise fits in the CTA's shared-memory table
  // trajectory state (indexed by slot)
  float *z, *g, *g_tilde, *logp;
  int32_t *t, *t_stop;
  uint8_t* status;
  double *sum_g, *sum_g2;
  float* entropy;       // per slot: H(pi(.|s_t)) of the latest step (only written when want_entropy)
  double* sum_h;        // per slot: running sum of those
  // scratch (indexed by row of this call)
  float4* records;      // [capacity * nblk] block records
  unsigned* ticket;     // [capacity] blocks of the row reduced so far
  unsigned* dev_status; // sticky ESPO_DEV_* bits
  // shared-memory layout of the hierarchical kernel: byte offsets of its tables, laid out by the host
  int h_bars, h_meta, h_ctrl, h_ready, h_pre, h_noise, h_lrec, h_fscratch;
  int blk_base, blk_rem;      // blocks per CTA: the first blk_rem CTAs take blk_base + 1, the others blk_base
  int runs_q[2], runs_r[2];   // runs of run_len blocks in a range of blk_base (+1) blocks, divided by the streaming warps
  // frozen parameters, pre-digested on the host
  float inv_temp;       // 1/temperature (1 when greedy)
  float k2;             // inv_temp * log2(e)
  int greedy;
  float mu_g, inv_sigma, clip_c, alpha_s, one_minus_alpha, beta, eps;
  int warmup_complete, t_max, eos_token;
  int stop_mode, shadow, want_entropy;
  float tau, p_random;
  float top_p;          // filtered sampling: < 1 keeps a nucleus (>= 1: off)
  int top_k;            // filtered sampling: > 0 keeps the k most probable (0: off)
  uint32_t key0, key1, batch_bits;
  // outputs
  int32_t* tokens_out;
  uint8_t* stop_out;
  // vocabulary shards (espo_step_partial / espo_step_merge)
  int vocab_offset;              // global id of the shard's first logit (0 for a whole row)
  espo_partial* partial_out;     // not null: write the row's partial result here instead of updating the state
  const espo_partial* partials;  // merge: [n_shards][shard_stride] partial results
  int n_shards;
  long long shard_stride;
};

struct StepCtrl {
  int head;         // queue entries claimed so far
  int posted;       // queue entries posted so far
  int abort_flag;   // a bounded wait ran out somewhere in this CTA
  int pad;
};

// -------------------------------------------------------------------------------------------
// Reduction of one 1024-id block held in a shared-memory stage.  Lane l owns the 16-byte
// vectors l, l+32, l+64, ... of the block, so the warp reads consecutive 512-byte lines.
// -------------------------------------------------------------------------------------------

template <int ES>
struct BlockVals;

template <>
struct BlockVals<2> {   // bfloat16: 4 vectors of 8 ids per lane
  static constexpr int kVecs = 4, kPerVec = 8;
  uint32_t w[16];
  __device__ __forceinline__ void load(const unsigned char* blk, int lane, int nvalid) {
    const uint4* sp = reinterpret_cast<const uint4*>(blk);
    if (nvalid == kBlockIds) {       // warp-uniform: every block but a row's ragged last one
#pragma unroll
      for (int i = 0; i < kVecs; ++i) {
        const uint4 q = sp[i * 32 + lane];
        w[4 * i + 0] = q.x; w[4 * i + 1] = q.y; w[4 * i + 2] = q.z; w[4 * i + 3] = q.w;
      }
    } else {                         // ids at or beyond nvalid read as -inf
#pragma unroll
      for (int i = 0; i < kVecs; ++i) {
        const int first = (i * 32 + lane) * kPerVec;
        uint4 q = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
        if (first < nvalid) q = sp[i * 32 + lane];   // the stage is a full block long; the excess is masked below
        uint32_t ww[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (first + 2 * k >= nvalid) ww[k] = (ww[k] & 0xffff0000u) | 0x0000FF80u;
          if (first + 2 * k + 1 >= nvalid) ww[k] = (ww[k] & 0x0000ffffu) | 0xFF800000u;
          w[4 * i + k] = ww[k];
        }
      }
    }
  }
  __device__ __forceinline__ float lane_max() const {
    uint32_t m = w[0];
#pragma unroll
    for (int i = 1; i < 16; ++i) m = bf16x2_max(m, w[i]);
    return fmaxf(bf16_lo(m), bf16_hi(m));
  }
  __device__ __forceinline__ float val(int j) const { return (j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]); }
  __device__ __forceinline__ float2 pair(int j) const { return make_float2(bf16_lo(w[j]), bf16_hi(w[j])); }
};

template <>
struct BlockVals<4> {   // float32: 8 vectors of 4 ids per lane
  static constexpr int kVecs = 8, kPerVec = 4;
  float f[32];
  __device__ __forceinline__ void load(const unsigned char* blk, int lane, int nvalid) {
    const float4* sp = reinterpret_cast<const float4*>(blk);
    const float ninf = __int_as_float(0xff800000);
    if (nvalid == kBlockIds) {       // warp-uniform: every block but a row's ragged last one
#pragma unroll
      for (int i = 0; i < kVecs; ++i) {
        const float4 q = sp[i * 32 + lane];
        f[4 * i + 0] = q.x; f[4 * i + 1] = q.y; f[4 * i + 2] = q.z; f[4 * i + 3] = q.w;
      }
    } else {                         // ids at or beyond nvalid read as -inf
#pragma unroll
      for (int i = 0; i < kVecs; ++i) {
        const int first = (i * 32 + lane) * kPerVec;
        float4 q = make_float4(ninf, ninf, ninf, ninf);
        if (first < nvalid) q = sp[i * 32 + lane];   // the stage is a full block long; the excess is masked below
        f[4 * i + 0] = q.x;
        f[4 * i + 1] = (first + 1 < nvalid) ? q.y : ninf;
        f[4 * i + 2] = (first + 2 < nvalid) ? q.z : ninf;
        f[4 * i + 3] = (first + 3 < nvalid) ? q.w : ninf;
      }
    }
  }
  __device__ __forceinline__ float lane_max() const {
    float m = f[0];
#pragma unroll
    for (int i = 1; i < 32; ++i) m = fmaxf(m, f[i]);
    return m;
  }
  __device__ __forceinline__ float val(int j) const { return f[j]; }
  __device__ __forceinline__ float2 pair(int j) const { return make_float2(f[2 * j], f[2 * j + 1]); }
};

// Position inside the block of the j-th value a lane holds.
template <int ES>
__device__ __forceinline__ int id_in_block(int j, int lane) {
  constexpr int P = BlockVals<ES>::kPerVec;
  return ((j / P) * 32 + lane) * P + (j % P);
}

template <int ES, int SAMPLER>
__device__ __forceinline__ void reduce_block(const StepArgs& a, const unsigned char* blk, int lane, int nvalid,
                                             void* rec_row, int block, const DrawStream& ds) {
  BlockVals<ES> bv;
  bv.load(blk, lane, nvalid);
  const float m_b = warp_max(bv.lane_max());
  const float ref = (m_b == __int_as_float(0xff800000)) ? 0.0f : m_b;   // an all -inf block sums to 0
  // sum of 2^((x - ref) * k2): two ids per packed fp32 multiply-add and add, one exponential each
  const float2 k2v = make_float2(a.k2, a.k2);
  const float c0 = -ref * a.k2;
  const float2 c0v = make_float2(c0, c0);
  float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
  float u_b = 0.f;   // sum of e * t with t = (x - ref) k2 <= 0, e = 2^t: what the entropy needs besides the sum of e
  if (SAMPLER == ESPO_SAMPLER_HIER && a.want_entropy) {
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
  // (The exponents were x*k2 + c0 with c0 = -ref*k2 rounded once, so every one of them is off by the same
  // dlt = c0 + ref*k2, the rounding error of that product: up to 1e-5 at low temperatures.  The warp that reads the
  // record takes the common factor 2^dlt out again; see finalize_row.)
  const float s_b = warp_sum((acc0.x + acc0.y) + (acc1.x + acc1.y));

  if (SAMPLER == ESPO_SAMPLER_FLAT) {
    // one Philox block serves 4 consecutive ids; a lane's vector starts at a multiple of 4
    float best = __int_as_float(0xff800000);
    int best_id = -1;
#pragma unroll
    for (int q = 0; q < 32 / 4; ++q) {
      const int first = a.vocab_offset + block * kBlockIds + id_in_block<ES>(4 * q, lane);   // global id, a multiple of 4
      const uint4 rnd = philox4x32_10((uint32_t)first >> 2, ds.step, ds.slot, ds.batch_bits | 0u, ds.k0, ds.k1);
      const uint32_t wd[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float sc = (bv.val(4 * q + e) - ref) * a.inv_temp + gumbel_from_word(wd[e]);
        if (sc > best) { best = sc; best_id = first + e; }
      }
    }
    warp_argmax(best, best_id);
    if (lane == 0) static_cast<float4*>(rec_row)[block] = make_float4(m_b, s_b, best, __int_as_float(best_id));
  } else {
    if (lane == 0) static_cast<float4*>(rec_row)[block] = make_float4(m_b, s_b, u_b, 0.f);
  }
}

// -------------------------------------------------------------------------------------------
// Finalisation of one row by one warp, once all of its block records are in global memory.
// -------------------------------------------------------------------------------------------

template <int ES>
__device__ __forceinline__ float load_logit(const unsigned char* row_base, int id) {
  if (ES == 2) return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(row_base) + id) << 16);
  return __ldg(reinterpret_cast<const float*>(row_base) + id);
}

__device__ __forceinline__ void mark_row(const StepArgs& a, int row, int slot, int lane, int32_t token, unsigned dev_bit,
                                         int new_status, bool no_ticket) {
  if (lane == 0) {
    if (dev_bit) atomicOr(a.dev_status, dev_bit);
    if (new_status >= 0) a.status[slot] = (uint8_t)new_status;
    a.tokens_out[row] = token;
    a.stop_out[row] = 0;
    if (!no_ticket) a.ticket[row] = 0;   // ready for the next launch
  }
}

// What a finalizing warp reads about a row before it knows whether the row is complete: the
// trajectory slot, its state, and the critic value.  Requested early so that the loads are in
// flight while the row's ticket is being updated.
struct __align__(16) RowPre {
  int slot;         // -1: the row_ids entry was out of range
  int status, t_now;
  float z_prev, v;
  double sum_g, sum_g2;
};

__device__ __forceinline__ RowPre prefetch_row(const StepArgs& a, int row) {
  RowPre p;
  p.slot = a.row_ids ? __ldg(a.row_ids + row) : row;
  p.status = ESPO_ROW_ACTIVE; p.t_now = 0; p.z_prev = 0.f; p.sum_g = 0.0; p.sum_g2 = 0.0;
  if (p.slot < 0 || p.slot >= a.capacity) {
    p.slot = -1;
  } else {
    p.status = a.status[p.slot];
    p.t_now = a.t[p.slot];
    p.z_prev = a.z[p.slot];
    p.sum_g = a.sum_g[p.slot];
    p.sum_g2 = a.sum_g2[p.slot];
  }
  if (!a.values) p.v = 0.f;
  else if (a.values_bf16) p.v = __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(a.values) + row) << 16);
  else p.v = __ldg(reinterpret_cast<const float*>(a.values) + row);
  return p;
}

// Sum over 32 values of 2^((x - m) * k2), two per packed multiply-add.
__device__ __forceinline__ float sum_exp2_32(const float (&x)[kSubIds], float m, float k2) {
  const float c0 = -m * k2;
  const float2 k2v = make_float2(k2, k2), c0v = make_float2(c0, c0);
  float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
  for (int i = 0; i < kSubIds / 2; ++i) {
    const float2 t = __ffma2_rn(make_float2(x[2 * i], x[2 * i + 1]), k2v, c0v);
    const float2 e = make_float2(ex2_approx(t.x), ex2_approx(t.y));
    if (i & 1) acc1 = __fadd2_rn(acc1, e); else acc0 = __fadd2_rn(acc0, e);
  }
  // every exponent is off by the rounding error of m*k2 (see reduce_block): one factor takes it out
  return ((acc0.x + acc0.y) + (acc1.x + acc1.y)) * ex2_approx(-fmaf(m, k2, c0));
}

// What one thread does once a row's token is known: regret, normalisation, smoothing, stop rule and bookkeeping
// (Eq. 6, 9, 10, 11; Algorithm 1).  M: largest logit; log_S = ln sum_a exp((x_a - M)/T); l_tok: the token's logit;
// S, run_u: the sums the entropy needs (relative to M).
__device__ __forceinline__ void commit_row(const StepArgs& a, int row, const RowPre& pre, const DrawStream& ds, float M,
                                           float S, float log_S, float run_u, float l_tok, int token, bool no_ticket) {
  const int slot = pre.slot;
  const int t_now = pre.t_now;
  {
    // Eq. 6: the normaliser cancels; Eq. 9; Eq. 10; Eq. 11.
    const float g = a.greedy ? 0.f : (M - l_tok) * a.inv_temp;
    const float logp = a.greedy ? 0.f : (-g - log_S);
    float gt = (g - a.mu_g) * a.inv_sigma;
    gt = fminf(fmaxf(gt, -a.clip_c), a.clip_c);
    const float z = fmaf(a.alpha_s, pre.z_prev, a.one_minus_alpha * gt);
    const float v = pre.v;
    const bool v_nan = (v != v);
    if (v_nan) atomicOr(a.dev_status, ESPO_DEV_NAN_VALUE);
    const float thr = a.beta * fmaxf(v, a.eps);
    bool rule;
    if (a.stop_mode == ESPO_STOP_ESPO) rule = !v_nan && (z > thr);                 // Eq. 11
    else if (a.stop_mode == ESPO_STOP_VALUE_ONLY) rule = !v_nan && (v < a.tau);
    else if (a.stop_mode == ESPO_STOP_REGRET_ONLY) rule = (z > a.tau);
    else rule = (uniform_at(ds, 3u, 0u) < a.p_random);
    const bool fires = a.warmup_complete && rule;

    a.z[slot] = z;
    a.g[slot] = g;
    a.g_tilde[slot] = gt;
    a.logp[slot] = logp;
    a.sum_g[slot] = pre.sum_g + (double)g;
    a.sum_g2[slot] = pre.sum_g2 + (double)g * (double)g;
    if (a.want_entropy) {
      // H = ln S - ln2 * U / S with S, U the sums of e and of e*t relative to the row maximum
      const float h = a.greedy ? 0.f : fmaxf(log_S - 0.6931471805599453f * run_u / S, 0.f);
      a.entropy[slot] = h;
      a.sum_h[slot] += (double)h;
    }
    const int t_new = t_now + 1;
    a.t[slot] = t_new;
    uint8_t stop = 0;
    if (a.eos_token >= 0 && token == a.eos_token) {
      a.status[slot] = ESPO_ROW_EOS;
    } else if (fires && a.shadow) {
      if (a.t_stop[slot] < 0) a.t_stop[slot] = t_now;        // remembered, not acted upon
      if (t_new >= a.t_max) a.status[slot] = ESPO_ROW_TMAX;
    } else if (fires) {
      a.status[slot] = ESPO_ROW_STOPPED;
      a.t_stop[slot] = t_now;
      stop = 1;
    } else if (t_new >= a.t_max) {
      a.status[slot] = ESPO_ROW_TMAX;
    }
    a.tokens_out[row] = token;
    a.stop_out[row] = stop;
    if (!no_ticket) a.ticket[row] = 0;   // ready for the next launch
  }
}

// Where the CTA's range of the block sequence lies, in units local to the CTA: local block
// index li = b0 + q for position q of the range; local row li / nblk; block li % nblk.
struct CtaRange {
  long long r_first;   // first row the range touches
  int b0;              // block of that row at which the range starts
  int n;               // blocks in the range
  int off;             // walk order: position p of the walk is range position (p + off) mod n
  int n_local;         // rows the range touches
  int nblk;
  // blocks of local row k that belong to this CTA
  __device__ __forceinline__ int share(int k) const { return min((k + 1) * nblk, b0 + n) - max(k * nblk, b0); }
  // Rows that lie wholly inside the range need no other CTA: their records stay in shared memory.
  // Such rows are consecutive, starting at local row (b0 == 0 ? 0 : 1); returns the table index or -1.
  __device__ __forceinline__ int local_index(int k, int local_rows) const {
    const int i = k - (b0 == 0 ? 0 : 1);
    return (i >= 0 && i < local_rows && share(k) == nblk) ? i : -1;
  }
};


}  // namespace espo
