// ESPO decode-step kernel for sm_100a and the C entry points around it.
//
// One launch performs, for every logit row of the batch, the body of the rollout loop
// (Algorithm 1): log-softmax statistics, Gumbel-max sampling, the surrogate regret of
// Eq. 5, its normalisation (Eq. 8) and smoothing (Eq. 9), the value-gated stop test
// (Eq. 10) and the per-trajectory bookkeeping.
//
// Shape of the kernel
//   * The [n_rows, V] logits are cut into tiles of kConsumerWarps blocks of 1024 ids.  A
//     persistent grid (a multiple of the SM count) splits the tile sequence into equal
//     contiguous ranges, so every SM streams the same number of bytes whatever n_rows is.
//   * Inside a CTA one producer thread moves tiles from HBM into a ring of shared-memory
//     stages with bulk asynchronous copies (TMA without a tensor map) that complete on
//     mbarriers; eight consumer warps each reduce one 1024-id block of the tile to
//     (max logit, sum of exp) -- plus, for the flat sampler, the block's best perturbed
//     score -- and write that record to a small per-row table in global memory.
//   * A row may be spread over several CTAs.  Each consumer warp counts the blocks it has
//     contributed to a row and adds them to the row's ticket; whoever completes the ticket
//     hands the row to its CTA's finalizer warp, which merges the block records in a fixed
//     order (so results do not depend on the grid), draws the token, applies Eq. 5, 8, 9, 10
//     and writes the outputs and the trajectory state.  The streaming warps never wait for it.
//   * Every wait in the kernel is bounded; a wait that runs out sets ESPO_DEV_TIMEOUT.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <new>

#include "espo.h"
#include "espo_device.cuh"
#include "espo_host.h"

namespace espo {

constexpr int kConsumerWarps = 8;
constexpr int kStepThreads = (kConsumerWarps + 2) * 32;   // + producer warp + finalizer warp
constexpr int kProducerWarp = kConsumerWarps;
constexpr int kFinalizerWarp = kConsumerWarps + 1;
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
  int nblk;             // 1024-id blocks per row
  int tiles_per_row;
  long long total_tiles;
  int stages, tile_bytes, queue_cap;
  // trajectory state (indexed by slot)
  float *z, *g, *g_tilde, *logp;
  int32_t *t, *t_stop;
  uint8_t* status;
  double *sum_g, *sum_g2;
  // scratch (indexed by row of this call)
  float4* records;      // [capacity * nblk] block records (float2 view for the hierarchical sampler)
  unsigned* ticket;     // [capacity] blocks of the row reduced so far
  unsigned* dev_status; // sticky ESPO_DEV_* bits
  // frozen parameters, pre-digested on the host
  float inv_temp;       // 1/temperature (1 when greedy)
  float k2;             // inv_temp * log2(e)
  int greedy;
  float mu_g, inv_sigma, clip_c, alpha_s, one_minus_alpha, beta, eps;
  int warmup_complete, t_max, eos_token;
  uint32_t key0, key1, batch_bits;
  // outputs
  int32_t* tokens_out;
  uint8_t* stop_out;
};

struct StepCtrl {
  int fin_tail;     // rows handed to the finalizer so far
  int done_warps;   // consumer warps that have left their loop
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
        if (first < nvalid) q = sp[i * 32 + lane];
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
        if (first < nvalid) q = sp[i * 32 + lane];
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
};

// Position inside the block of the j-th value a lane holds.
template <int ES>
__device__ __forceinline__ int id_in_block(int j, int lane) {
  constexpr int P = BlockVals<ES>::kPerVec;
  return ((j / P) * 32 + lane) * P + (j % P);
}

template <int ES, int SAMPLER>
__device__ __forceinline__ void reduce_block(const StepArgs& a, const unsigned char* blk, int lane, int nvalid,
                                             int row, int block, const DrawStream& ds) {
  BlockVals<ES> bv;
  bv.load(blk, lane, nvalid);
  const float m_b = warp_max(bv.lane_max());
  const float ref = (m_b == __int_as_float(0xff800000)) ? 0.0f : m_b;   // an all -inf block sums to 0
  const float c0 = -ref * a.k2;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int j = 0; j < 32; ++j) acc[(ES == 2 ? (j >> 1) : j) & 3] += ex2_approx(fmaf(bv.val(j), a.k2, c0));
  const float s_b = warp_sum((acc[0] + acc[1]) + (acc[2] + acc[3]));

  if (SAMPLER == ESPO_SAMPLER_FLAT) {
    // one Philox block serves 4 consecutive ids; a lane's vector starts at a multiple of 4
    constexpr int P = BlockVals<ES>::kPerVec;
    float best = __int_as_float(0xff800000);
    int best_id = -1;
#pragma unroll
    for (int q = 0; q < 32 / 4; ++q) {
      const int first = block * kBlockIds + id_in_block<ES>(4 * q, lane);
      const uint4 rnd = philox4x32_10((uint32_t)first >> 2, ds.step, ds.slot, ds.batch_bits | 0u, ds.k0, ds.k1);
      const uint32_t wd[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float sc = (bv.val(4 * q + e) - ref) * a.inv_temp + gumbel_from_word(wd[e]);
        if (sc > best) { best = sc; best_id = first + e; }
      }
    }
    (void)P;
    warp_argmax(best, best_id);
    if (lane == 0)
      a.records[(size_t)row * a.nblk + block] = make_float4(m_b, s_b, best, __int_as_float(best_id));
  } else {
    if (lane == 0) reinterpret_cast<float2*>(a.records)[(size_t)row * a.nblk + block] = make_float2(m_b, s_b);
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

template <int ES, int SAMPLER>
__device__ void finalize_row(const StepArgs& a, int row, int lane) {
  const float NINF = __int_as_float(0xff800000);
  int slot = a.row_ids ? __ldg(a.row_ids + row) : row;
  if (slot < 0 || slot >= a.capacity) {
    if (lane == 0) {
      atomicOr(a.dev_status, ESPO_DEV_BAD_SLOT);
      a.tokens_out[row] = -1;
      a.stop_out[row] = 0;
      a.ticket[row] = 0;
    }
    return;
  }
  if (a.status[slot] != ESPO_ROW_ACTIVE) {   // finished trajectories are left untouched
    if (lane == 0) {
      a.tokens_out[row] = -1;
      a.stop_out[row] = 0;
      a.ticket[row] = 0;
    }
    return;
  }
  const int t_now = a.t[slot];
  const unsigned char* row_base = a.logits + (size_t)row * a.row_stride_bytes;
  const DrawStream ds{a.key0, a.key1, (uint32_t)t_now, (uint32_t)slot, a.batch_bits};

  // ---- merge the block records: M = max logit, S = sum_b s_b exp((m_b - M)/T) ----
  float M = NINF;
  bool poisoned = false;
  for (int b = lane; b < a.nblk; b += 32) {
    float m_b, s_b;
    if (SAMPLER == ESPO_SAMPLER_FLAT) {
      const float4 r = __ldcg(a.records + (size_t)row * a.nblk + b);
      m_b = r.x; s_b = r.y;
    } else {
      const float2 r = __ldcg(reinterpret_cast<const float2*>(a.records) + (size_t)row * a.nblk + b);
      m_b = r.x; s_b = r.y;
    }
    M = fmaxf(M, m_b);
    poisoned |= !(s_b >= 0.0f) || isinf(s_b);   // NaN or inf sum: the block held NaN or +inf
  }
  M = warp_max(M);
  poisoned = __any_sync(kFullMask, poisoned) || !(M > NINF) || isinf(M);
  if (poisoned) {
    if (lane == 0) {
      atomicOr(a.dev_status, ESPO_DEV_BAD_ROW);
      a.status[slot] = ESPO_ROW_BAD;
      a.tokens_out[row] = 0;
      a.stop_out[row] = 0;
      a.ticket[row] = 0;
    }
    return;
  }

  float S = 0.f;              // lane-partial, summed below
  float best = NINF;          // best perturbed score among this lane's blocks
  int best_i = -1;            // HIER: block number; FLAT: token id
  for (int b = lane; b < a.nblk; b += 32) {
    float m_b, s_b, flat_best = NINF;
    int flat_id = -1;
    if (SAMPLER == ESPO_SAMPLER_FLAT) {
      const float4 r = __ldcg(a.records + (size_t)row * a.nblk + b);
      m_b = r.x; s_b = r.y; flat_best = r.z; flat_id = __float_as_int(r.w);
    } else {
      const float2 r = __ldcg(reinterpret_cast<const float2*>(a.records) + (size_t)row * a.nblk + b);
      m_b = r.x; s_b = r.y;
    }
    if (!(s_b > 0.f)) continue;                       // all -inf block
    const float shift = (m_b - M) * a.inv_temp;
    const float rel = shift + logf(s_b);              // block log-sum-exp relative to M/T
    S += expf(rel);
    if (a.greedy) {
      if (m_b == M && best_i < 0) { best = 0.f; best_i = b; }   // lowest block holding the maximum
    } else if (SAMPLER == ESPO_SAMPLER_FLAT) {
      const float sc = flat_best + shift;
      if (flat_id >= 0 && (best_i < 0 || sc > best)) { best = sc; best_i = flat_id; }
    } else {
      const float sc = rel + gumbel_at(ds, 2u, (uint32_t)b);
      if (best_i < 0 || sc > best) { best = sc; best_i = b; }
    }
  }
  S = warp_sum(S);
  warp_argmax(best, best_i);
  if (best_i < 0) {   // no block offered a candidate: treat like an unusable row rather than index with -1
    if (lane == 0) {
      atomicOr(a.dev_status, ESPO_DEV_BAD_ROW);
      a.status[slot] = ESPO_ROW_BAD;
      a.tokens_out[row] = 0;
      a.stop_out[row] = 0;
      a.ticket[row] = 0;
    }
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
    float m_j = NINF;
#pragma unroll
    for (int i = 0; i < kSubIds; ++i) m_j = fmaxf(m_j, x[i]);

    int sub_pick;
    if (a.greedy) {
      // first id equal to the maximum
      int first = -1;
#pragma unroll
      for (int i = kSubIds - 1; i >= 0; --i) if (x[i] == M) first = sub_lo + i;
      float key = 0.f;
      warp_argmax(key, first);           // equal keys: lowest id wins
      token = first;
      l_tok = M;
      sub_pick = -1;
    } else {
      float sc = NINF;
      int j = -1;
      if (m_j > NINF) {
        float s_j = 0.f;
#pragma unroll
        for (int i = 0; i < kSubIds; ++i) s_j += expf((x[i] - m_j) * a.inv_temp);
        sc = (m_j - M) * a.inv_temp + logf(s_j) + gumbel_at(ds, 1u, (uint32_t)(sub_lo >> 5));
        j = sub_lo >> 5;
      }
      warp_argmax(sc, j);
      sub_pick = j;
      // ---- ids of the chosen sub-block: lane e owns id 32*sub_pick + e ----
      const int id = sub_pick * kSubIds + lane;
      float sc0 = NINF, l = NINF;
      int cand = -1;
      if (id < a.V) {
        l = load_logit<ES>(row_base, id);
        if (l > NINF) { sc0 = (l - M) * a.inv_temp + gumbel_at(ds, 0u, (uint32_t)id); cand = id; }
      }
      warp_argmax(sc0, cand);
      token = max(cand, sub_pick * kSubIds);   // cand < 0 cannot happen for a sub-block with a finite id
      l_tok = __shfl_sync(kFullMask, l, token & 31);
    }
    (void)sub_pick;
  } else {
    token = best_i;
    l_tok = load_logit<ES>(row_base, token);
  }

  if (lane == 0) {
    // Eq. 5: the normaliser cancels; Eq. 8; Eq. 9; Eq. 10.
    const float g = a.greedy ? 0.f : (M - l_tok) * a.inv_temp;
    const float logp = a.greedy ? 0.f : (-g - logf(S));
    float gt = (g - a.mu_g) * a.inv_sigma;
    gt = fminf(fmaxf(gt, -a.clip_c), a.clip_c);
    const float z = fmaf(a.alpha_s, a.z[slot], a.one_minus_alpha * gt);
    float v;
    if (a.values_bf16) v = __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(a.values) + row) << 16);
    else v = __ldg(reinterpret_cast<const float*>(a.values) + row);
    const bool v_nan = (v != v);
    if (v_nan) atomicOr(a.dev_status, ESPO_DEV_NAN_VALUE);
    const float thr = a.beta * fmaxf(v, a.eps);
    const bool fires = a.warmup_complete && !v_nan && (z > thr);

    a.z[slot] = z;
    a.g[slot] = g;
    a.g_tilde[slot] = gt;
    a.logp[slot] = logp;
    a.sum_g[slot] += (double)g;
    a.sum_g2[slot] += (double)g * (double)g;
    const int t_new = t_now + 1;
    a.t[slot] = t_new;
    uint8_t stop = 0;
    if (a.eos_token >= 0 && token == a.eos_token) {
      a.status[slot] = ESPO_ROW_EOS;
    } else if (fires) {
      a.status[slot] = ESPO_ROW_STOPPED;
      a.t_stop[slot] = t_now;
      stop = 1;
    } else if (t_new >= a.t_max) {
      a.status[slot] = ESPO_ROW_TMAX;
    }
    a.tokens_out[row] = token;
    a.stop_out[row] = stop;
    a.ticket[row] = 0;   // ready for the next launch
  }
}

// -------------------------------------------------------------------------------------------
// The kernel.
// -------------------------------------------------------------------------------------------

template <int ES, int SAMPLER, bool BULK>
__global__ void __launch_bounds__(kStepThreads) espo_step_kernel(const StepArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* ring = smem;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + (size_t)a.stages * a.tile_bytes);
  uint64_t* empty_bar = full_bar + a.stages;
  StepCtrl* ctrl = reinterpret_cast<StepCtrl*>(empty_bar + a.stages);
  volatile int* queue = reinterpret_cast<volatile int*>(ctrl + 1);
  volatile int* abort_flag = &ctrl->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long t_begin = (long long)blockIdx.x * a.total_tiles / gridDim.x;
  const long long t_end = (long long)(blockIdx.x + 1) * a.total_tiles / gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], kConsumerWarps);
    }
    ctrl->fin_tail = 0; ctrl->done_warps = 0; ctrl->abort_flag = 0; ctrl->pad = 0;
    mbar_init_fence();
  }
  for (int i = threadIdx.x; i < a.queue_cap; i += blockDim.x) queue[i] = -1;
  __syncthreads();

  if (warp < kConsumerWarps) {
    // ------------------------------------------------------------------ consumers
    int cur_row = -1;
    unsigned cnt = 0;
    DrawStream ds{a.key0, a.key1, 0u, 0u, a.batch_bits};
    auto flush = [&]() {
      if (lane == 0 && cnt > 0) {
        __threadfence();                                      // records before the ticket
        const unsigned old = atomicAdd(a.ticket + cur_row, cnt);
        if (old + cnt == (unsigned)a.nblk) {                   // this warp completed the row
          __threadfence();
          const int qi = atomicAdd(&ctrl->fin_tail, 1);
          if (qi < a.queue_cap) queue[qi] = cur_row;
          else atomicOr(a.dev_status, ESPO_DEV_TIMEOUT);       // cannot happen: the host sizes the queue
        }
      }
      cnt = 0;
    };
    int s = 0;
    uint32_t parity = 0;
    long long row = t_begin / a.tiles_per_row;
    int tr = (int)(t_begin - row * a.tiles_per_row);
    for (long long k = t_begin; k < t_end; ++k) {
      if ((int)row != cur_row) {
        flush();
        cur_row = (int)row;
        if (SAMPLER == ESPO_SAMPLER_FLAT) {
          // the flat sampler perturbs every id, so the streaming warps need the row's draw stream
          int slot = a.row_ids ? __ldg(a.row_ids + cur_row) : cur_row;
          slot = min(max(slot, 0), a.capacity - 1);            // a bad slot is reported by the finalizer
          ds.slot = (uint32_t)slot;
          ds.step = (uint32_t)a.t[slot];
        }
      }
      if (!mbar_wait_bounded(&full_bar[s], parity, abort_flag)) {
        if (lane == 0) { atomicOr(a.dev_status, ESPO_DEV_TIMEOUT); *abort_flag = 1; }
        break;
      }
      const int block = tr * kConsumerWarps + warp;
      if (block < a.nblk) {
        const int nvalid = min(kBlockIds, a.V - block * kBlockIds);
        reduce_block<ES, SAMPLER>(a, ring + (size_t)s * a.tile_bytes + (size_t)warp * (kBlockIds * ES), lane, nvalid,
                                  cur_row, block, ds);
        ++cnt;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[s]);
      if (++s == a.stages) { s = 0; parity ^= 1u; }
      if (++tr == a.tiles_per_row) { tr = 0; ++row; }
    }
    flush();
    if (lane == 0) { __threadfence_block(); atomicAdd(&ctrl->done_warps, 1); }
  } else if (warp == kProducerWarp) {
    // ------------------------------------------------------------------ producer
    int s = 0;
    uint32_t parity = 1;   // the first pass over the ring finds every stage free
    bool first_round = true;
    long long row = t_begin / a.tiles_per_row;
    int tr = (int)(t_begin - row * a.tiles_per_row);
    for (long long k = t_begin; k < t_end; ++k) {
      if (!first_round) {
        int ok = 1;
        if (lane == 0) ok = mbar_wait_bounded(&empty_bar[s], parity, abort_flag) ? 1 : 0;
        ok = __shfl_sync(kFullMask, ok, 0);
        if (!ok) {
          if (lane == 0) { atomicOr(a.dev_status, ESPO_DEV_TIMEOUT); *abort_flag = 1; }
          break;
        }
      }
      const int e0 = tr * kConsumerWarps * kBlockIds;
      const int n = min(kConsumerWarps * kBlockIds, a.V - e0);
      const unsigned char* src = a.logits + (size_t)row * a.row_stride_bytes + (size_t)e0 * ES;
      unsigned char* dst = ring + (size_t)s * a.tile_bytes;
      if (BULK) {
        if (lane == 0) {
          mbar_arrive_expect_tx(&full_bar[s], (uint32_t)n * ES);
          bulk_copy_g2s(dst, src, (uint32_t)n * ES, &full_bar[s]);
        }
      } else {
        if (ES == 2) {
          const unsigned short* sp = reinterpret_cast<const unsigned short*>(src);
          unsigned short* dp = reinterpret_cast<unsigned short*>(dst);
          for (int i = lane; i < n; i += 32) dp[i] = __ldg(sp + i);
        } else {
          const float* sp = reinterpret_cast<const float*>(src);
          float* dp = reinterpret_cast<float*>(dst);
          for (int i = lane; i < n; i += 32) dp[i] = __ldg(sp + i);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&full_bar[s]);
      }
      if (++s == a.stages) { s = 0; first_round = false; parity ^= 1u; }
      if (++tr == a.tiles_per_row) { tr = 0; ++row; }
    }
    // The consumers wait for every copy issued above before they leave, and the CTA's
    // shared memory outlives all of its warps, so nothing is in flight at exit.
  } else {
    // ------------------------------------------------------------------ finalizer
    int head = 0;
    for (;;) {
      int row = -1;
      bool finished = false, gave_up = true;
      if (lane == 0) {
        for (uint32_t it = 0; it < kPollSpinLimit; ++it) {
          if (head < a.queue_cap && (row = queue[head]) >= 0) { gave_up = false; break; }
          if (*(volatile int*)&ctrl->done_warps == kConsumerWarps && head >= *(volatile int*)&ctrl->fin_tail) { finished = true; gave_up = false; break; }
          if (*abort_flag) { finished = true; gave_up = false; break; }
          __nanosleep(100);
        }
        if (gave_up) { atomicOr(a.dev_status, ESPO_DEV_TIMEOUT); *abort_flag = 1; finished = true; }
      }
      row = __shfl_sync(kFullMask, row, 0);
      finished = __shfl_sync(kFullMask, finished, 0);
      if (finished && row < 0) break;
      __threadfence();
      finalize_row<ES, SAMPLER>(a, row, lane);
      ++head;
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
  int cfg_stages, cfg_ctas_per_sm;   // 0 = library default
  void* arena;
  size_t arena_bytes;
  float *z, *g, *g_tilde, *logp;
  int32_t *t, *t_stop;
  uint8_t* status;
  double *sum_g, *sum_g2;
  float4* records;
  unsigned *ticket, *dev_status;
};

namespace espo {

__global__ void espo_compact_kernel(const uint8_t* __restrict__ status, int capacity, int32_t* __restrict__ out,
                                    int32_t* __restrict__ n_out) {
  __shared__ int warp_total[32];
  __shared__ int base;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
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
  const size_t o_sg = carve(8 * cap), o_sg2 = carve(8 * cap);
  const size_t o_rec = carve(sizeof(float4) * cap * (size_t)st->nblk);
  const size_t o_tk = carve(4 * cap), o_ds = carve(4);
  st->arena_bytes = off;
  e = cudaMalloc(&st->arena, st->arena_bytes);
  if (e != cudaSuccess) { delete st; return record_cuda_error(e); }
  unsigned char* base = static_cast<unsigned char*>(st->arena);
  st->z = (float*)(base + o_z); st->g = (float*)(base + o_g); st->g_tilde = (float*)(base + o_gt);
  st->logp = (float*)(base + o_lp); st->t = (int32_t*)(base + o_t); st->t_stop = (int32_t*)(base + o_ts);
  st->status = (uint8_t*)(base + o_st); st->sum_g = (double*)(base + o_sg); st->sum_g2 = (double*)(base + o_sg2);
  st->records = (float4*)(base + o_rec); st->ticket = (unsigned*)(base + o_tk); st->dev_status = (unsigned*)(base + o_ds);

  for (int es = 2; es <= 4; es += 2)
    for (int sm = 0; sm < 2; ++sm)
      for (int b = 0; b < 2; ++b) {
        e = cudaFuncSetAttribute((const void*)pick_kernel(es, sm, b != 0), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 st->max_smem);
        if (e != cudaSuccess) { cudaFree(st->arena); delete st; return record_cuda_error(e); }
      }
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

int espo_set_launch_config(espo_state* st, int32_t stages, int32_t ctas_per_sm) {
  if (!st) return ESPO_ERR_NULL;
  if (stages < 0 || stages > 64 || ctas_per_sm < 0 || ctas_per_sm > 8) return ESPO_ERR_BAD_PARAM;
  st->cfg_stages = stages;
  st->cfg_ctas_per_sm = ctas_per_sm;
  return ESPO_OK;
}

int espo_step(const void* logits, int32_t logits_dtype, int64_t row_stride, const void* values, int32_t values_dtype,
              const int32_t* row_ids, int32_t n_rows, espo_state* st, const espo_params* p, int32_t* tokens_out,
              uint8_t* stop_out, void* stream) {
  using namespace espo;
  if (!st || !p) return ESPO_ERR_NULL;
  if (n_rows < 0) return ESPO_ERR_BAD_SHAPE;
  if (n_rows > st->capacity) return ESPO_ERR_CAPACITY;
  if ((logits_dtype != ESPO_F32 && logits_dtype != ESPO_BF16) || (values_dtype != ESPO_F32 && values_dtype != ESPO_BF16))
    return ESPO_ERR_BAD_DTYPE;
  if (!(p->temperature >= 0.f) || isinf(p->temperature)) return ESPO_ERR_BAD_PARAM;
  if (!(p->sigma2_g >= 0.f) || !(p->sigma2_g + p->delta > 0.f) || !(p->clip_c > 0.f)) return ESPO_ERR_BAD_PARAM;
  if (!(p->alpha_s >= 0.f && p->alpha_s < 1.f) || p->t_max < 1) return ESPO_ERR_BAD_PARAM;
  if (p->sampler != ESPO_SAMPLER_FLAT && p->sampler != ESPO_SAMPLER_HIER) return ESPO_ERR_BAD_PARAM;
  if (isnan(p->mu_g) || isnan(p->beta) || isnan(p->eps)) return ESPO_ERR_BAD_PARAM;
  if (n_rows == 0) return ESPO_OK;
  if (!logits || !values || !tokens_out || !stop_out) return ESPO_ERR_NULL;
  if (row_stride < st->V) return ESPO_ERR_BAD_SHAPE;
  const int es = (logits_dtype == ESPO_BF16) ? 2 : 4;
  const int ves = (values_dtype == ESPO_BF16) ? 2 : 4;
  if (((uintptr_t)logits % es) || ((uintptr_t)values % ves) || ((uintptr_t)tokens_out % 4) ||
      (row_ids && ((uintptr_t)row_ids % 4)))
    return ESPO_ERR_ALIGN;

  StepArgs a;
  memset(&a, 0, sizeof(a));
  a.logits = static_cast<const unsigned char*>(logits);
  a.row_stride_bytes = row_stride * es;
  a.values = values;
  a.values_bf16 = (values_dtype == ESPO_BF16);
  a.row_ids = row_ids;
  a.n_rows = n_rows; a.V = st->V; a.capacity = st->capacity;
  a.nblk = st->nblk;
  a.tiles_per_row = (st->nblk + kConsumerWarps - 1) / kConsumerWarps;
  a.total_tiles = (long long)n_rows * a.tiles_per_row;
  a.tile_bytes = kConsumerWarps * kBlockIds * es;
  const int ctas_per_sm = st->cfg_ctas_per_sm ? st->cfg_ctas_per_sm : 2;
  long long grid = (long long)st->sm_count * ctas_per_sm;
  if (grid > a.total_tiles) grid = a.total_tiles;
  const long long tiles_per_cta = (a.total_tiles + grid - 1) / grid;
  const long long qcap = tiles_per_cta / a.tiles_per_row + 2;
  if (qcap > kMaxQueue) return ESPO_ERR_CAPACITY;
  a.queue_cap = (int)qcap;
  const size_t fixed = sizeof(StepCtrl) + sizeof(int) * (size_t)a.queue_cap;
  const size_t budget = (size_t)st->max_smem / ctas_per_sm - (ctas_per_sm > 1 ? 1024 : 0);
  int stages = st->cfg_stages ? st->cfg_stages : (es == 2 ? 6 : 3);
  while (stages > 1 && (size_t)stages * (a.tile_bytes + 16) + fixed > budget) --stages;
  if (tiles_per_cta < stages) stages = (int)tiles_per_cta;
  a.stages = stages;
  const size_t smem = (size_t)stages * (a.tile_bytes + 16) + fixed;
  if (smem > (size_t)st->max_smem) return ESPO_ERR_CAPACITY;

  a.z = st->z; a.g = st->g; a.g_tilde = st->g_tilde; a.logp = st->logp;
  a.t = st->t; a.t_stop = st->t_stop; a.status = st->status; a.sum_g = st->sum_g; a.sum_g2 = st->sum_g2;
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
  a.key0 = (uint32_t)(st->seed & 0xffffffffull);
  a.key1 = (uint32_t)(st->seed >> 32);
  a.batch_bits = (uint32_t)(st->batch_id << 2);
  a.tokens_out = tokens_out; a.stop_out = stop_out;

  const bool bulk = ((uintptr_t)logits % 16 == 0) && (a.row_stride_bytes % 16 == 0) && (((size_t)st->V * es) % 16 == 0);
  StepKernel k = pick_kernel(es, p->sampler, bulk);
  k<<<(unsigned)grid, kStepThreads, smem, (cudaStream_t)stream>>>(a);
  ESPO_CUDA_TRY(cudaGetLastError());
  return ESPO_OK;
}

int espo_state_view(espo_state* st, const float** z, const float** g, const float** g_tilde, const float** logp,
                    const int32_t** t, const uint8_t** status, const int32_t** t_stop, const double** sum_g,
                    const double** sum_g2) {
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
  return ESPO_OK;
}

int espo_compact_active(espo_state* st, int32_t* row_ids_out, int32_t* n_active_out, void* stream) {
  if (!st || !row_ids_out || !n_active_out) return ESPO_ERR_NULL;
  espo::espo_compact_kernel<<<1, 1024, 0, (cudaStream_t)stream>>>(st->status, st->capacity, row_ids_out, n_active_out);
  ESPO_CUDA_TRY(cudaGetLastError());
  return ESPO_OK;
}

int espo_state_status(espo_state* st, uint32_t* host_out, void* stream) {
  if (!st || !host_out) return ESPO_ERR_NULL;
  ESPO_CUDA_TRY(cudaMemcpyAsync(host_out, st->dev_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  ESPO_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
  return ESPO_OK;
}

}  // extern "C"
