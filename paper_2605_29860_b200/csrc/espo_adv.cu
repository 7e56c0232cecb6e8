// TD errors and GAE over ragged, truncated trajectories (Eq. 4-5) with ESPO's absorbing
// failure transition (Eq. 13), for sm_100a.
//
// Every CTA of a persistent grid takes an equal, contiguous range of the packed token array
// (cut at multiples of four tokens, wherever trajectories begin and end), so every CTA moves the
// same number of bytes (12 per token: reward and value in, advantage out) whatever the length
// mix is, and walks it from the top down in chunks of kAdvChunk tokens.  Within a chunk the
// backward recursion A_t = delta_t + k_t A_{t+1} (k_t = gamma*lambda, or 0 on a trajectory's
// last token) is a scan over affine maps X -> b + a X: a thread folds its 12 consecutive tokens,
// the 256 threads' maps are composed by a warp-shuffle suffix scan and a small cross-warp pass,
// all in double precision (with gamma*lambda = 1 an advantage is a sum of up to 16k TD errors).
// The value that follows a chunk is carried in shared memory.  The value that follows the
// range belongs to a trajectory that continues in the next CTA's range: unrolled, Eq. 5 makes it
// a weighted sum of the rest of that one trajectory's TD errors, which the CTA takes straight from
// global memory first (read only, usually served by L2, and only as far as the weights
// (gamma*lambda)^k can still matter) -- so CTAs never wait for one another.
//
// The CTA is warp-specialised.  A producer warp keeps a ring of stages full with bulk asynchronous
// copies (TMA without a tensor map) and turns the trajectory ends that fall into a chunk into one flag
// word per scanning thread; the eight scanning warps touch global memory only to store results.  A
// thread's 12 tokens are 48 bytes: consecutive threads' rows start in different shared-memory banks
// (with 16 tokens, 64 bytes, every 128-bit read was a 4-way conflict per quarter warp).
//
// A small preparation kernel turns lengths into offsets and tells every kAdvChunk-th token which
// trajectory it belongs to; the scan is launched as its programmatic dependent, so the ring fills
// while the preparation still runs.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "espo.h"
#include "espo_device.cuh"
#include "espo_host.h"

namespace espo {

constexpr int kAdvThreads = 256;                        // scanning threads
// Tokens per scanning thread: a multiple of 4 (16-byte accesses), at most 16 (flag word), and an odd number of
// 16-byte pieces, so that the threads' shared-memory rows (48 bytes apart) fall into different banks.
constexpr int kAdvPerThread = 12;
constexpr int kAdvChunk = kAdvThreads * kAdvPerThread;   // 3072 tokens
static_assert(kAdvPerThread % 4 == 0 && kAdvPerThread <= 16, "flag word: 16 end bits and 16 stop bits");
constexpr int kAdvWarps = kAdvThreads / 32;
constexpr int kAdvCtaThreads = kAdvThreads + 32;          // the scanning threads and the producer warp
constexpr int kAdvStages = 2;
constexpr int kAdvCtasPerSm = 3;
constexpr int kMaxDevicesAdv = 64;
constexpr int kPrepThreads = 1024;

struct AdvWorkspace {
  long long* offsets;     // [B+1] exclusive prefix sum of lengths
  int* chunk_first;       // [nchunks] trajectory that owns the chunk's first token
  unsigned* status;       // sticky ESPO_DEV_* bits
  double* partials;       // [2 * grid] per-CTA sums of A and A^2 (only with stats)
  unsigned* done;         // CTAs that have written their partial sums; the last one resets it
};

struct AdvArgs {
  const float* rewards;
  const float* values;
  const int32_t* lengths;
  const uint8_t* stopped;
  float* adv;
  float* ret;             // optional: returns A_t + V_t (value targets), same layout as adv; may be null
  double* stats;          // optional: [2] sum of A_t and of A_t^2 over all tokens; may be null
  int B;
  int t_max;              // > 0: padded layout, trajectory i owns tokens [i*t_max, i*t_max + lengths[i]); 0: packed
  long long total;
  int nchunks;
  double gamma, gl;       // gamma, gamma*lambda
  long long halo_cap;     // tokens of a crossing trajectory whose weight (gamma*lambda)^k can still matter
  float r_fail;
  AdvWorkspace ws;
};

// ---------------------------------------------------------------------------------------
// Preparation: offsets = exclusive scan of lengths; chunk_first[j] = trajectory holding
// token j*kAdvChunk.  One CTA; B is a batch size, not a token count.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kPrepThreads) espo_adv_prep_kernel(const AdvArgs a) {
  __shared__ long long warp_tot[32];
  __shared__ long long carry;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // The scan kernel may be scheduled now: it starts its first copies and waits for this grid before it reads
  // anything written here.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  bool bad = false;
  for (int start = 0; start < a.B; start += kPrepThreads) {
    const int i = start + threadIdx.x;
    long long len = 0;
    if (i < a.B) {
      len = a.lengths[i];
      if (len < 0) { len = 0; bad = true; }
    }
    long long incl = len;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long up = __shfl_up_sync(kFullMask, incl, o);
      if (lane >= o) incl += up;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    long long before = carry;
    for (int w = 0; w < warp; ++w) before += warp_tot[w];
    const long long excl = before + incl - len;
    if (i < a.B) {
      a.ws.offsets[i] = excl;
      // chunks whose first token falls inside this trajectory
      const long long end = excl + len;
      for (long long j = (excl + kAdvChunk - 1) / kAdvChunk; j * kAdvChunk < end && j < a.nchunks; ++j)
        a.ws.chunk_first[j] = i;
    }
    __syncthreads();
    if (threadIdx.x == kPrepThreads - 1) carry = before + incl;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    a.ws.offsets[a.B] = carry;
    if (carry != a.total) bad = true;
  }
  if (bad) atomicOr(a.ws.status, ESPO_DEV_BAD_LENGTHS);
}

// ---------------------------------------------------------------------------------------
// The scan.
// ---------------------------------------------------------------------------------------

// Fills the discount fields.  (gamma*lambda)^k < 2^-80 from k = halo_cap on: such a term cannot move a sum of TD
// errors by more than 2^-80 times the largest of them, far below the rounding of the double-precision sum itself.
static void set_discount(AdvArgs& a, float gamma, float lambda) {
  a.gamma = (double)gamma;
  a.gl = (double)gamma * (double)lambda;
  const double g = a.gl < 0 ? -a.gl : a.gl;
  if (g >= 1.0) a.halo_cap = 0x7fffffffffffffffLL;
  else if (g <= 0.0) a.halo_cap = 1;
  else {
    const double k = -80.0 * 0.6931471805599453 / log(g);
    a.halo_cap = k < 1e15 ? (long long)k + 1 : 0x7fffffffffffffffLL;
  }
}

struct Map {   // X -> b + a * X
  double a, b;
};
// `lo` is applied after `hi` (lo belongs to the earlier tokens): lo(hi(X)).  A map that contains a trajectory end
// (a == 0) ignores its argument outright, so that a NaN or infinity in a later trajectory cannot reach an earlier one
// through 0 * NaN.
__device__ __forceinline__ Map compose(const Map& lo, const Map& hi) {
  const bool cut = (lo.a == 0.0);
  return Map{cut ? 0.0 : lo.a * hi.a, cut ? lo.b : fma(lo.a, hi.b, lo.b)};
}
// The value of `m` at X, with the same rule.
__device__ __forceinline__ double apply(const Map& m, double x) { return m.a == 0.0 ? m.b : fma(m.a, x, m.b); }

__device__ __forceinline__ double shfl_down_d(double v, int o) { return __shfl_down_sync(kFullMask, v, o); }
__device__ __forceinline__ double shfl_up_d(double v, int o) { return __shfl_up_sync(kFullMask, v, o); }
__device__ __forceinline__ double shfl_d(double v, int src) { return __shfl_sync(kFullMask, v, src); }

// Shared memory of the scan kernel: a ring of kAdvStages stages, each one chunk of rewards, one chunk of values
// followed by the value of the token after the chunk, and one flag word per scanning thread (bit e: the thread's
// token e is the last of a trajectory; bit 16 + e: that trajectory was stopped) and, for the padded layout, one word
// of padding bits (bit e: the thread's token e belongs to no trajectory).
constexpr int kAdvVStride = kAdvChunk + 4;      // floats; keeps every stage 16-byte aligned
constexpr size_t kAdvSmemBytes =
    (size_t)kAdvStages * (sizeof(float) * kAdvChunk + sizeof(float) * kAdvVStride + 2 * sizeof(uint32_t) * kAdvThreads) +
    2 * kAdvStages * sizeof(uint64_t);

// kAdvThreads threads scan; one more warp (the producer) keeps the ring full and sets the flag words, so that no
// scanning warp ever waits for a load from global memory.
// STATS: also the batch sums of A and A^2.  RET: also the returns A_t + V_t; the scanning threads then keep a stage
// until they have stored, because they read the values from it a second time.
// PADDED: the arrays are [B, t_max] with padding after every trajectory; padding reads as anything and is written as 0.
template <bool STATS, bool RET, bool PADDED>
__global__ void __launch_bounds__(kAdvCtaThreads, kAdvCtasPerSm) espo_adv_scan_kernel(const AdvArgs a) {
  extern __shared__ __align__(128) unsigned char adv_smem[];
  float* rbuf = reinterpret_cast<float*>(adv_smem);
  float* vbuf = rbuf + kAdvStages * kAdvChunk;
  uint32_t* fwbuf = reinterpret_cast<uint32_t*>(vbuf + kAdvStages * kAdvVStride);
  uint32_t* pwbuf = fwbuf + kAdvStages * kAdvThreads;
  uint64_t* full = reinterpret_cast<uint64_t*>(pwbuf + kAdvStages * kAdvThreads);   // data and flags of the stage are in place
  uint64_t* empty = full + kAdvStages;                                                // every scanning thread has read the stage
  __shared__ Map warp_agg[2][kAdvWarps];                    // double-buffered: consecutive chunks alternate
  __shared__ double pw[kAdvPerThread + 1];                   // (gamma*lambda)^i
  __shared__ double carry_buf[2];                            // value that follows the chunk, by the chunk's parity
  __shared__ int halo_traj;                                  // trajectory that crosses the range's upper end, or -1,
  __shared__ long long halo_end;                             // its end offset
  __shared__ int halo_failed;                                // and whether it was stopped
  __shared__ int all_pad[kAdvStages];                        // padded layout: the stage's chunk is padding only, nothing was copied
  __shared__ int is_last_cta;                                // statistics: this CTA adds up every CTA's partial sums

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const double r_fail_d = (double)a.r_fail;
  const int q0 = tid * kAdvPerThread;

  // This CTA's tokens: [t_lo, t_hi), cut at multiples of four tokens so that every CTA moves the same number of
  // bytes and every copy starts on a 16-byte boundary (the last range ends at the array's end rounded up).  Chunk k
  // (k = 0 is the highest) covers tokens [t_hi - (k+1)*kAdvChunk, t_hi - k*kAdvChunk) and sits in stage k mod
  // kAdvStages; the lowest chunk may begin below t_lo: those positions of its stage are never loaded, and what the
  // threads compute for them is dropped.
  const long long quads = (a.total + 3) >> 2;
  const long long t_lo = 4 * ((long long)blockIdx.x * quads / gridDim.x);
  const long long t_hi = 4 * ((long long)(blockIdx.x + 1) * quads / gridDim.x);
  const int nck = (int)((t_hi - t_lo + kAdvChunk - 1) / kAdvChunk);

  if (tid == 0) {
    halo_traj = -1;
    for (int st = 0; st < kAdvStages; ++st) {
      mbar_init(&full[st], 2);               // the producer's expect_tx arrival and its arrival after the flags
      mbar_init(&empty[st], kAdvThreads);
    }
    mbar_init_fence();
    double p = 1.0;
    for (int i = 0; i <= kAdvPerThread; ++i) { pw[i] = p; p *= a.gl; }
  }
  for (int i = tid; i < 2 * kAdvStages * kAdvThreads; i += kAdvCtaThreads) fwbuf[i] = 0u;   // flag and padding words
  __syncthreads();

  if (warp == kAdvWarps) {
    if (nck <= 0) return;
    // =============================== producer warp ===============================
    // Starts the copies of chunk `k` (lane 0).  A chunk is two bulk copies (plus 16 bytes for the value after the
    // chunk) that complete on the stage's mbarrier; of a chunk that reaches past the end of the array (only the
    // array's last, when its length is no multiple of four) the last, incomplete group of four tokens is written
    // with ordinary stores, zeros standing for the tokens that do not exist.
    auto issue_copies = [&](int k) {
      const int stage = k % kAdvStages;
      const long long p0 = t_hi - (long long)(k + 1) * kAdvChunk;
      const int skip = (int)(max(p0, t_lo) - p0);                        // unused positions at the low end, a multiple of 4
      const int n = (int)min((long long)kAdvChunk, a.total - p0);       // positions below n hold tokens
      const int n4 = n & ~3;
      float* rs = rbuf + stage * kAdvChunk;
      float* vs = vbuf + stage * kAdvVStride;
      const bool tail16 = (p0 + kAdvChunk + 4 <= a.total);               // the 16 bytes after the chunk exist
      const uint32_t bytes = n4 > skip ? (uint32_t)sizeof(float) * (uint32_t)(n4 - skip) : 0u;
      if (PADDED) {
        // A chunk that lies wholly in one row's padding is not read at all: its padding bits make the scanning
        // threads write zeros whatever the stage still holds.
        const long long p_lo = max(p0, t_lo), p_end = min(p0 + kAdvChunk, a.total);
        const long long i = p_lo / a.t_max;
        if (p_end <= (i + 1) * a.t_max) {
          const int len = a.lengths[i];
          if (p_lo >= i * a.t_max + (len < 0 ? 0 : (len > a.t_max ? a.t_max : len))) {
            all_pad[stage] = 1;                                            // published by the arrivals on full[stage]
            mbar_arrive_expect_tx(&full[stage], 0u);
            return;
          }
        }
        all_pad[stage] = 0;
      }
      fence_proxy_async();                                               // the scanning threads' reads of the stage come first
      mbar_arrive_expect_tx(&full[stage], 2u * bytes + (tail16 ? 16u : 0u));
      if (bytes) {
        bulk_copy_g2s(rs + skip, a.rewards + p0 + skip, bytes, &full[stage]);
        bulk_copy_g2s(vs + skip, a.values + p0 + skip, bytes, &full[stage]);
      }
      if (tail16) bulk_copy_g2s(vs + kAdvChunk, a.values + p0 + kAdvChunk, 16u, &full[stage]);
      else vs[kAdvChunk] = (p0 + kAdvChunk < a.total) ? __ldg(a.values + p0 + kAdvChunk) : 0.f;
      for (int q = n4; q < n4 + 4 && q < kAdvChunk; ++q) {
        rs[q] = (q < n) ? __ldg(a.rewards + p0 + q) : 0.f;
        vs[q] = (q < n) ? __ldg(a.values + p0 + q) : 0.f;
      }
    };
    // The trajectories that can end inside chunk `k` are [c_lo, c_hi]: c_lo holds a token at or below the chunk's
    // first, c_hi one at or above its last.  Values that are no trajectory (only with inconsistent lengths, which
    // the preparation flags) are pulled into range.
    auto cand_lo = [&](int k) -> int {
      const long long p0 = t_hi - (long long)(k + 1) * kAdvChunk;
      if (PADDED) return (int)min(max(p0, t_lo) / a.t_max, (long long)a.B);      // rows are t_max apart: no table needed
      const int c = __ldcg(a.ws.chunk_first + (max(p0, t_lo) / kAdvChunk));
      return c < 0 ? 0 : (c > a.B ? a.B : c);
    };
    auto cand_hi = [&](int k) -> int {
      const long long p_end = min(t_hi - (long long)k * kAdvChunk, a.total);
      if (PADDED) return (int)min((p_end - 1) / a.t_max, (long long)a.B - 1);
      const long long g = (p_end - 1) / kAdvChunk + 1;
      if (g >= a.nchunks) return a.B - 1;
      const int c = __ldcg(a.ws.chunk_first + g);
      return c < 0 ? -1 : (c >= a.B ? a.B - 1 : c);
    };
    struct Traj { long long o0, o1; unsigned st; };
    auto traj_load = [&](int i, int c_hi) -> Traj {
      Traj t{0, 0, 0u};
      if (i <= c_hi) {
        if (PADDED) {
          const int len = a.lengths[i];
          t.o0 = (long long)i * a.t_max;
          t.o1 = t.o0 + (len < 0 ? 0 : (len > a.t_max ? a.t_max : len));
        } else {
          t.o0 = __ldcg(a.ws.offsets + i);
          t.o1 = __ldcg(a.ws.offsets + i + 1);
        }
        t.st = a.stopped[i];
      }
      return t;
    };
    // Padded layout: tokens [from, to) belong to no trajectory; every lane calls this with the same arguments and
    // sets the padding bits of its share of the chunk's words.
    auto pad_mark = [&](int k, long long from, long long to) {
      const long long p0 = t_hi - (long long)(k + 1) * kAdvChunk;
      const long long lo = max(from, max(p0, t_lo)), hi = min(to, min(p0 + kAdvChunk, a.total));
      if (lo >= hi) return;
      const int q_lo = (int)(lo - p0), q_hi = (int)(hi - p0);
      uint32_t* pw = pwbuf + (k % kAdvStages) * kAdvThreads;
      for (int w = q_lo / kAdvPerThread + lane; w <= (q_hi - 1) / kAdvPerThread; w += 32) {
        const int b0 = max(q_lo - w * kAdvPerThread, 0), b1 = min(q_hi - w * kAdvPerThread, kAdvPerThread);
        atomicOr(pw + w, ((1u << (b1 - b0)) - 1u) << b0);
      }
    };
    auto traj_mark = [&](int k, const Traj& t) {
      const long long p0 = t_hi - (long long)(k + 1) * kAdvChunk;
      const long long p_lo = max(p0, t_lo);
      const long long p_end = min(p0 + kAdvChunk, a.total);
      if (t.o1 > t.o0 && t.o1 - 1 >= p_lo && t.o1 - 1 < p_end) {
        const int pos = (int)(t.o1 - 1 - p0);
        atomicOr(fwbuf + (k % kAdvStages) * kAdvThreads + (pos / kAdvPerThread), (1u | (t.st ? 0x10000u : 0u)) << (pos % kAdvPerThread));
      }
    };

    // Marks what one round of candidates (lane l holds candidate first + l) contributes to chunk k.
    auto mark_round = [&](int k, const Traj& t, int first, int c_hi) {
      traj_mark(k, t);
      if (PADDED) {
        const int n = min(32, c_hi - first + 1);
        for (int j = 0; j < n; ++j) {
          const long long o0 = __shfl_sync(kFullMask, t.o0, j), o1 = __shfl_sync(kFullMask, t.o1, j);
          pad_mark(k, o1, o0 + a.t_max);
        }
      }
    };

    const int pre = nck < kAdvStages ? nck : kAdvStages;
    if (lane == 0)
      for (int k = 0; k < pre; ++k) issue_copies(k);       // needs nothing of the preparation kernel
    if (!PADDED) asm volatile("griddepcontrol.wait;" ::: "memory");     // everything below reads what the preparation wrote
    int c_lo = cand_lo(0), c_hi = cand_hi(0);               // candidates of the chunk in hand
    int n_lo = nck > 1 ? cand_lo(1) : 0, n_hi = nck > 1 ? cand_hi(1) : -1;   // and of the next one
    Traj t0 = traj_load(c_lo + lane, c_hi);                 // the lane's first candidate, loaded one chunk ahead
    for (int k = 0; k < nck; ++k) {
      const int stage = k % kAdvStages;
      if (k >= kAdvStages) {
        if (!mbar_wait_bounded(&empty[stage], (uint32_t)((k / kAdvStages - 1) & 1), nullptr)) atomicOr(a.ws.status, ESPO_DEV_TIMEOUT);
        if (lane == 0) issue_copies(k);
      }
      mark_round(k, t0, c_lo, c_hi);
      for (int first = c_lo + 32; first <= c_hi; first += 32) mark_round(k, traj_load(first + lane, c_hi), first, c_hi);
      __syncwarp();
      if (lane == 0) mbar_arrive(&full[stage]);             // the flags (and lane 0's ordinary stores) are in place
      c_lo = n_lo; c_hi = n_hi;
      t0 = traj_load(c_lo + lane, c_hi);
      if (k + 2 < nck) { n_lo = cand_lo(k + 2); n_hi = cand_hi(k + 2); }
      else { n_lo = 0; n_hi = -1; }
    }
    return;
  }

  // =============================== scanning warps ===============================
  unsigned last_mask = 0, pad_mask = 0;
  double d[kAdvPerThread];
  Map m, after;

  // Waits for chunk `k`, folds it: leaves the thread's TD errors in d[], its end mask in last_mask, its own map in
  // m and the map of everything after the thread inside the chunk in `after`; the thread's flag word is cleared
  // and the stage handed back to the producer as soon as the thread has read its part.  Contains one rendezvous
  // of the scanning warps.
  auto fold = [&](int k) {
    const int stage = k % kAdvStages;
    const int par = k & 1;
    const float* rs = rbuf + stage * kAdvChunk;
    const float* vs = vbuf + stage * kAdvVStride;
    const long long p0 = t_hi - (long long)(k + 1) * kAdvChunk;
    if (!mbar_wait_bounded(&full[stage], (uint32_t)((k / kAdvStages) & 1), nullptr)) atomicOr(a.ws.status, ESPO_DEV_TIMEOUT);
    if (PADDED && all_pad[stage]) {
      // the whole chunk is padding (nothing was copied): every token cuts the recursion with a TD error of 0, so the
      // threads only clear their words, keep the rendezvous in step and go on to write zeros
      fwbuf[stage * kAdvThreads + tid] = 0u;
      pwbuf[stage * kAdvThreads + tid] = 0u;
      if (!RET) mbar_arrive(&empty[stage]);
      last_mask = pad_mask = (1u << kAdvPerThread) - 1u;
#pragma unroll
      for (int e = 0; e < kAdvPerThread; ++e) d[e] = 0.0;
      m = Map{0.0, 0.0};
      after = Map{0.0, 0.0};
      cta_rendezvous(kAdvThreads);
      return;
    }
    float r[kAdvPerThread], v[kAdvPerThread];
#pragma unroll
    for (int h = 0; h < kAdvPerThread / 4; ++h) {
      const float4 rr = *reinterpret_cast<const float4*>(rs + q0 + 4 * h);
      const float4 vv = *reinterpret_cast<const float4*>(vs + q0 + 4 * h);
      r[4 * h] = rr.x; r[4 * h + 1] = rr.y; r[4 * h + 2] = rr.z; r[4 * h + 3] = rr.w;
      v[4 * h] = vv.x; v[4 * h + 1] = vv.y; v[4 * h + 2] = vv.z; v[4 * h + 3] = vv.w;
    }
    const float v_after = vs[q0 + kAdvPerThread];   // the next thread's first value; for the last thread, the next chunk's
    uint32_t* fp = fwbuf + stage * kAdvThreads + tid;
    const uint32_t fw = *fp;
    *fp = 0u;
    last_mask = fw & 0xffffu;
    unsigned fail_mask = fw >> 16;
    if (PADDED) {
      uint32_t* pp = pwbuf + stage * kAdvThreads + tid;
      pad_mask = *pp;
      *pp = 0u;
      last_mask |= pad_mask;          // padding cuts the recursion like a trajectory end, with a TD error of 0
    }
    if (!RET) mbar_arrive(&empty[stage]);           // release: this thread's reads and its cleared words come first
    {
      // the array's very last token ends a trajectory even if the lengths are inconsistent
      const long long e_last = a.total - 1 - p0 - q0;
      if (e_last >= 0 && e_last < kAdvPerThread) last_mask |= 1u << (int)e_last;
    }
    fail_mask &= last_mask;
    double mb = 0.0;
    double vd_next = (double)v_after;
    if (!__any_sync(kFullMask, last_mask != 0u)) {
      // no trajectory ends among the warp's tokens (the usual case): no per-token case distinctions
#pragma unroll
      for (int e = kAdvPerThread - 1; e >= 0; --e) {
        const double vd = (double)v[e];
        const double de = fma(a.gamma, vd_next, (double)r[e]) - vd;
        d[e] = de;
        mb = fma(a.gl, mb, de);
        vd_next = vd;
      }
    } else {
#pragma unroll
      for (int e = kAdvPerThread - 1; e >= 0; --e) {
        const bool last = (last_mask >> e) & 1u;
        const double vd = (double)v[e];
        const double rd = ((fail_mask >> e) & 1u) ? r_fail_d : (double)r[e];
        double de = (last ? rd : fma(a.gamma, vd_next, rd)) - vd;
        if (PADDED) de = ((pad_mask >> e) & 1u) ? 0.0 : de;     // whatever the padding holds never enters
        d[e] = de;
        mb = last ? de : fma(a.gl, mb, de);
        vd_next = vd;
      }
    }
    // Tokens past the end of the array (at most three, in its last chunk) read as zeros; the array's last token is a
    // forced trajectory end, so nothing of them reaches a stored result.
    m = Map{last_mask ? 0.0 : pw[kAdvPerThread], mb};   // X survives the thread only if no trajectory ends in it
    Map inc = m;   // inclusive suffix inside the warp
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      Map hi{shfl_down_d(inc.a, o), shfl_down_d(inc.b, o)};
      if (lane + o < 32) inc = compose(inc, hi);
    }
    if (lane == 0) warp_agg[par][warp] = inc;
    after = Map{shfl_down_d(inc.a, 1), shfl_down_d(inc.b, 1)};   // exclusive within the warp
    if (lane == 31) after = Map{1.0, 0.0};
    cta_rendezvous(kAdvThreads);   // warp aggregates written
    for (int w = warp + 1; w < kAdvWarps; ++w) after = compose(after, warp_agg[par][w]);
  };

  if (!PADDED) asm volatile("griddepcontrol.wait;" ::: "memory");   // everything below reads what the preparation kernel wrote
  if (PADDED && blockIdx.x == 0) {   // no preparation kernel looked at the lengths
    bool bad = false;
    for (int i = tid; i < a.B; i += kAdvThreads) { const int len = a.lengths[i]; bad |= (len < 0 || len > a.t_max); }
    if (bad) atomicOr(a.ws.status, ESPO_DEV_BAD_LENGTHS);
  }

  // ---- the advantage of the token that follows the range (token t_hi).  Its trajectory continues in the next CTA's
  //      range; unrolled, Eq. 5 makes it the weighted sum of the rest of that one trajectory's TD errors,
  //      sum_k (gamma*lambda)^k delta_k, which the CTA's threads take straight from global memory (read only, usually
  //      served by L2): thread t owns tokens 4t .. 4t+3 of every 1024.  CTAs therefore never wait for one another. ----
  if (nck > 0 && t_hi < a.total) {   // find the trajectory that holds token t_hi
    int first = PADDED ? (int)min(t_hi / a.t_max, (long long)a.B) : __ldcg(a.ws.chunk_first + (t_hi / kAdvChunk));
    if ((unsigned)first >= (unsigned)a.B) first = a.B;   // only with inconsistent lengths (flagged by the preparation)
    for (int i = first + tid; i < a.B; i += kAdvThreads) {
      long long o0, o1;
      if (PADDED) {
        const int len = a.lengths[i];
        o0 = (long long)i * a.t_max;
        o1 = o0 + (len < 0 ? 0 : (len > a.t_max ? a.t_max : len));
      } else {
        o0 = __ldcg(a.ws.offsets + i);
        o1 = __ldcg(a.ws.offsets + i + 1);
      }
      const int st = a.stopped[i];
      if (o0 > t_hi) break;
      if (o1 > t_hi) { halo_traj = i; halo_end = o1; halo_failed = st; }
    }
  }
  cta_rendezvous(kAdvThreads);
  {
    double part = 0.0;
    if (halo_traj >= 0) {
      const long long t_end = min(halo_end, a.total);                              // the trajectory's end
      const long long end = (t_end - t_hi > a.halo_cap) ? t_hi + a.halo_cap : t_end; // the part whose weights matter
      const bool failed = halo_failed != 0;
      double wt = 1.0, sq = a.gl;                        // (gamma*lambda)^(4 tid) by binary powering
      for (unsigned ex = 4u * tid; ex; ex >>= 1) {
        if (ex & 1u) wt *= sq;
        sq *= sq;
      }
      double w_round = a.gl;                             // (gamma*lambda)^(4 * kAdvThreads)
#pragma unroll
      for (int h = 0; h < 10; ++h) w_round *= w_round;
      static_assert(4 * kAdvThreads == 1024, "w_round is the 1024th power");
      if (a.gamma == 1.0 && a.gl == 1.0) {
        // gamma = lambda = 1: the TD errors telescope, sum_k delta_k = sum_k r'_k - V(first token); only the rewards of
        // the rest of the trajectory are read, eight 16-byte loads per thread in flight at a time (8192 tokens per trip of
        // the CTA: a trajectory's rest takes one or two L2 round trips; sixteen at a time spill)
        constexpr int kBatch = 8;
        for (long long kb = t_hi + 4 * tid; kb < end; kb += (long long)kBatch * 4 * kAdvThreads) {
          float4 rr[kBatch];
#pragma unroll
          for (int u = 0; u < kBatch; ++u) {
            const long long k0 = kb + (long long)u * 4 * kAdvThreads;
            rr[u] = (k0 < end && k0 + 4 <= a.total) ? __ldg(reinterpret_cast<const float4*>(a.rewards + k0)) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int u = 0; u < kBatch; ++u) {
            const long long k0 = kb + (long long)u * 4 * kAdvThreads;
            if (k0 < end) {
              float r[4] = {rr[u].x, rr[u].y, rr[u].z, rr[u].w};
              if (k0 + 4 > a.total) {
#pragma unroll
                for (int e = 0; e < 4; ++e) r[e] = (k0 + e < a.total) ? __ldg(a.rewards + k0 + e) : 0.f;
              }
              if (k0 + 4 <= end && !(failed && k0 + 4 >= t_end)) {
                part += ((double)r[0] + (double)r[1]) + ((double)r[2] + (double)r[3]);
              } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const long long k = k0 + e;
                  if (k < end) part += (k == t_end - 1 && failed) ? r_fail_d : (double)r[e];
                }
              }
            }
          }
        }
        if (tid == 0) part -= (double)__ldg(a.values + t_hi);
      } else
#pragma unroll 4
      for (long long k0 = t_hi + 4 * tid; k0 < end; k0 += 4 * kAdvThreads, wt *= w_round) {
        float r[4], v[5];
        if (k0 + 4 < a.total) {                          // four tokens and the value after them exist
          const float4 rr = __ldg(reinterpret_cast<const float4*>(a.rewards + k0));
          const float4 vv = __ldg(reinterpret_cast<const float4*>(a.values + k0));
          v[4] = __ldg(a.values + k0 + 4);
          r[0] = rr.x; r[1] = rr.y; r[2] = rr.z; r[3] = rr.w;
          v[0] = vv.x; v[1] = vv.y; v[2] = vv.z; v[3] = vv.w;
        } else {
#pragma unroll
          for (int e = 0; e < 5; ++e) {
            v[e] = (k0 + e < a.total) ? __ldg(a.values + k0 + e) : 0.f;
            if (e < 4) r[e] = (k0 + e < a.total) ? __ldg(a.rewards + k0 + e) : 0.f;
          }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const long long k = k0 + e;
          if (k < end) {
            const bool last = (k == t_end - 1);
            const double rd = (last && failed) ? r_fail_d : (double)r[e];
            const double de = (last ? rd : fma(a.gamma, (double)v[e + 1], rd)) - (double)v[e];
            part = fma(wt * pw[e], de, part);
          }
        }
      }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) part += shfl_down_d(part, o);
    if (lane == 0) warp_agg[1][warp].b = part;             // chunk 0 uses warp_agg[0]
    cta_rendezvous(kAdvThreads);
    if (tid == 0) {
      double carry = 0.0;                                  // past the end of the array the value is 0
      for (int w = 0; w < kAdvWarps; ++w) carry += warp_agg[1][w].b;
      carry_buf[0] = carry;
    }
    // chunk 0's rendezvous comes between this write and its readers, and between the reads of warp_agg[1] above and
    // chunk 1's writes to it
  }

  // ---- the range, from its highest chunk down ----
  constexpr bool want_stats = STATS;
  double sum_a = 0.0, sum_a2 = 0.0;   // of the advantages this thread stores (before rounding to float)
  for (int k = 0; k < nck; ++k) {
    const int par = k & 1;
    const long long p0 = t_hi - (long long)(k + 1) * kAdvChunk;
    const int q_lo = (int)(max(p0, t_lo) - p0);                               // positions [q_lo, q_hi) hold this
    const int q_hi = (int)min((long long)kAdvChunk, a.total - p0);           // CTA's tokens
    fold(k);
    const double carry_in = carry_buf[par];
    if (tid == 0) {
      const Map whole = compose(m, after);
      carry_buf[par ^ 1] = apply(whole, carry_in);              // what follows the next (lower) chunk
    }

    // ---- replay the thread's tokens with the value that follows them ----
    double x = apply(after, carry_in);
    float out[kAdvPerThread];
    const bool whole_thread = (q0 >= q_lo && q0 + kAdvPerThread <= q_hi);
    if (!__any_sync(kFullMask, last_mask != 0u)) {
#pragma unroll
      for (int e = kAdvPerThread - 1; e >= 0; --e) {
        x = fma(a.gl, x, d[e]);
        out[e] = (float)x;
        if (want_stats && (whole_thread || (q0 + e >= q_lo && q0 + e < q_hi))) { sum_a += x; sum_a2 = fma(x, x, sum_a2); }
      }
    } else {
#pragma unroll
      for (int e = kAdvPerThread - 1; e >= 0; --e) {
        x = ((last_mask >> e) & 1u) ? d[e] : fma(a.gl, x, d[e]);
        out[e] = (float)x;
        if (want_stats && (whole_thread || (q0 + e >= q_lo && q0 + e < q_hi))) { sum_a += x; sum_a2 = fma(x, x, sum_a2); }
      }
    }
    if (whole_thread) {
#pragma unroll
      for (int h = 0; h < kAdvPerThread / 4; ++h)
        __stcs(reinterpret_cast<float4*>(a.adv + p0 + q0) + h, make_float4(out[4 * h], out[4 * h + 1], out[4 * h + 2], out[4 * h + 3]));
      if (RET) {
        const float* vs = vbuf + (k % kAdvStages) * kAdvVStride;
#pragma unroll
        for (int h = 0; h < kAdvPerThread / 4; ++h) {
          const float4 vv = *reinterpret_cast<const float4*>(vs + q0 + 4 * h);
          float4 rt = make_float4(out[4 * h] + vv.x, out[4 * h + 1] + vv.y, out[4 * h + 2] + vv.z, out[4 * h + 3] + vv.w);
          if (PADDED && pad_mask) {
            rt.x = ((pad_mask >> (4 * h)) & 1u) ? 0.f : rt.x;
            rt.y = ((pad_mask >> (4 * h + 1)) & 1u) ? 0.f : rt.y;
            rt.z = ((pad_mask >> (4 * h + 2)) & 1u) ? 0.f : rt.z;
            rt.w = ((pad_mask >> (4 * h + 3)) & 1u) ? 0.f : rt.w;
          }
          __stcs(reinterpret_cast<float4*>(a.ret + p0 + q0) + h, rt);
        }
      }
    } else {
#pragma unroll
      for (int e = 0; e < kAdvPerThread; ++e)
        if (q0 + e >= q_lo && q0 + e < q_hi) {
          a.adv[p0 + q0 + e] = out[e];
          if (RET) a.ret[p0 + q0 + e] = (PADDED && ((pad_mask >> e) & 1u)) ? 0.f : out[e] + vbuf[(k % kAdvStages) * kAdvVStride + q0 + e];
        }
    }
    if (RET) mbar_arrive(&empty[k % kAdvStages]);   // release: the second read of the values comes first
    // No rendezvous here: the next chunk's carry is read after the rendezvous inside its fold(), and the warp
    // aggregates alternate between two buffers.
  }

  // ---- optional batch sums of A and A^2: one pair per CTA, added up in a fixed order by whichever CTA finishes
  //      last, so that repeated calls give bit-identical sums ----
  if (want_stats) {
    cta_rendezvous(kAdvThreads);            // the last chunk's readers of warp_agg are done
#pragma unroll
    for (int o = 16; o; o >>= 1) { sum_a += shfl_down_d(sum_a, o); sum_a2 += shfl_down_d(sum_a2, o); }
    if (lane == 0) warp_agg[0][warp] = Map{sum_a, sum_a2};
    cta_rendezvous(kAdvThreads);
    if (tid == 0) {
      double t1 = 0.0, t2 = 0.0;
      for (int w = 0; w < kAdvWarps; ++w) { t1 += warp_agg[0][w].a; t2 += warp_agg[0][w].b; }
      a.ws.partials[2 * blockIdx.x] = t1;
      a.ws.partials[2 * blockIdx.x + 1] = t2;
      __threadfence();                      // the partial sums are visible before the count moves
      is_last_cta = (atomicAdd(a.ws.done, 1u) == gridDim.x - 1);
    }
    cta_rendezvous(kAdvThreads);
    if (is_last_cta) {
      __threadfence();
      double t1 = 0.0, t2 = 0.0;
      for (unsigned b = tid; b < gridDim.x; b += kAdvThreads) {
        t1 += __ldcg(a.ws.partials + 2 * b);
        t2 += __ldcg(a.ws.partials + 2 * b + 1);
      }
#pragma unroll
      for (int o = 16; o; o >>= 1) { t1 += shfl_down_d(t1, o); t2 += shfl_down_d(t2, o); }
      if (lane == 0) warp_agg[1][warp] = Map{t1, t2};
      cta_rendezvous(kAdvThreads);
      if (tid == 0) {
        double u1 = 0.0, u2 = 0.0;
        for (int w = 0; w < kAdvWarps; ++w) { u1 += warp_agg[1][w].a; u2 += warp_agg[1][w].b; }
        a.stats[0] = u1;
        a.stats[1] = u2;
        *a.ws.done = 0u;                    // ready for the next call
      }
    }
  }
}

// Launches both kernels; `sm_count` sizes the persistent grid of the scan.
static int launch_advantages(const AdvArgs& a, int sm_count, cudaStream_t s) {
  static bool attr_set[kMaxDevicesAdv] = {};
  int dev = 0;
  ESPO_CUDA_TRY(cudaGetDevice(&dev));
  if (dev >= 0 && dev < kMaxDevicesAdv && !attr_set[dev]) {
    const void* variants[6] = {(const void*)espo_adv_scan_kernel<false, false, false>, (const void*)espo_adv_scan_kernel<false, true, false>,
                               (const void*)espo_adv_scan_kernel<true, false, false>, (const void*)espo_adv_scan_kernel<true, true, false>,
                               (const void*)espo_adv_scan_kernel<false, false, true>, (const void*)espo_adv_scan_kernel<false, true, true>};
    for (const void* f : variants)
      ESPO_CUDA_TRY(cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAdvSmemBytes));
    attr_set[dev] = true;
  }
  // The packed layout needs offsets and chunk owners from a preparation kernel, and the scan is launched as its
  // programmatic dependent so that its ring fills meanwhile; the padded layout's offsets are arithmetic: one launch.
  if (a.t_max == 0) {
    espo_adv_prep_kernel<<<1, kPrepThreads, 0, s>>>(a);
    ESPO_CUDA_TRY(cudaGetLastError());
  }
  long long grid = (long long)sm_count * kAdvCtasPerSm;
  if (grid > a.nchunks) grid = a.nchunks;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kAdvCtaThreads);
  cfg.dynamicSmemBytes = kAdvSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start before the preparation kernel ends
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  if (a.t_max == 0) {
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  if (a.t_max > 0 && a.ret) ESPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, espo_adv_scan_kernel<false, true, true>, a));
  else if (a.t_max > 0) ESPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, espo_adv_scan_kernel<false, false, true>, a));
  else if (a.stats && a.ret) ESPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, espo_adv_scan_kernel<true, true, false>, a));
  else if (a.stats) ESPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, espo_adv_scan_kernel<true, false, false>, a));
  else if (a.ret) ESPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, espo_adv_scan_kernel<false, true, false>, a));
  else ESPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, espo_adv_scan_kernel<false, false, false>, a));
  return ESPO_OK;
}

// ---------------------------------------------------------------------------------------
// Per-device workspace, grown on demand.
// ---------------------------------------------------------------------------------------
struct AdvPool {
  int sm_count = 0;
  void* arena = nullptr;
  int cap_B = 0;
  long long cap_chunks = 0;
  AdvWorkspace ws{};
};
constexpr int kMaxDevices = 64;
static AdvPool g_pool[kMaxDevices];
static std::mutex g_pool_mu;

static int ensure_pool(int dev, int B, long long nchunks, AdvPool** out) {
  if (dev < 0 || dev >= kMaxDevices) return ESPO_ERR_CAPACITY;
  AdvPool& p = g_pool[dev];
  if (B > p.cap_B || nchunks > p.cap_chunks) {
    const int nb = B > p.cap_B ? B : p.cap_B;
    const long long nc = nchunks > p.cap_chunks ? nchunks : p.cap_chunks;
    if (p.arena) {
      ESPO_CUDA_TRY(cudaDeviceSynchronize());
      ESPO_CUDA_TRY(cudaFree(p.arena));
      p.arena = nullptr; p.cap_B = 0; p.cap_chunks = 0;
    }
    size_t off = 0;
    auto carve = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    if (!p.sm_count) ESPO_CUDA_TRY(cudaDeviceGetAttribute(&p.sm_count, cudaDevAttrMultiProcessorCount, dev));
    const size_t o_off = carve(8 * ((size_t)nb + 1)), o_cf = carve(4 * (size_t)nc), o_st = carve(4);
    const size_t o_pa = carve(16 * (size_t)p.sm_count * kAdvCtasPerSm), o_dn = carve(4);
    ESPO_CUDA_TRY(cudaMalloc(&p.arena, off));
    ESPO_CUDA_TRY(cudaMemset(p.arena, 0, off));
    unsigned char* b = static_cast<unsigned char*>(p.arena);
    p.ws.offsets = (long long*)(b + o_off); p.ws.chunk_first = (int*)(b + o_cf);
    p.ws.status = (unsigned*)(b + o_st);
    p.ws.partials = (double*)(b + o_pa); p.ws.done = (unsigned*)(b + o_dn);
    p.cap_B = nb; p.cap_chunks = nc;
  }
  *out = &p;
  return ESPO_OK;
}

// ---------------------------------------------------------------------------------------
// Fixed scratch for espo_advantages_noalloc: the same workspace layout as AdvPool's arena,
// carved out of an array that is part of the loaded module, sized for kNoAllocMaxB
// trajectories and kNoAllocMaxChunks chunks.  Zero-filled when the module is loaded.
// ---------------------------------------------------------------------------------------
constexpr int kNoAllocMaxB = ESPO_NOALLOC_MAX_B;
constexpr long long kNoAllocMaxChunks = ((ESPO_NOALLOC_MAX_TOKENS + kAdvChunk - 1) / kAdvChunk + 63) / 64 * 64;
constexpr size_t kNaOffOffsets = 0;
constexpr size_t kNaOffChunkFirst = kNaOffOffsets + ((8 * ((size_t)kNoAllocMaxB + 1) + 255) / 256) * 256;
constexpr size_t kNaOffStatus = kNaOffChunkFirst + 4 * (size_t)kNoAllocMaxChunks;
constexpr size_t kNoAllocBytes = kNaOffStatus + 256;
static_assert(kNoAllocMaxChunks % 64 == 0, "keeps every sub-array 256-byte aligned");

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

struct NoAllocSlot {
  unsigned char* base = nullptr;   // device address of g_noalloc_scratch on this device
  int sm_count = 0;
};
static NoAllocSlot g_noalloc[kMaxDevices];

}  // namespace espo

extern "C" {

int espo_advantages_noalloc(const float* rewards, const float* values, const int32_t* lengths, const uint8_t* stopped,
                            int32_t B, int64_t total_tokens, float gamma, float lambda, float r_fail, float* adv_out,
                            uint32_t* status_out, void* stream) {
  using namespace espo;
  if (B < 0 || total_tokens < 0) return ESPO_ERR_BAD_SHAPE;
  if (B > kNoAllocMaxB || total_tokens > (int64_t)ESPO_NOALLOC_MAX_TOKENS) return ESPO_ERR_CAPACITY;
  if (B == 0 || total_tokens == 0) return ESPO_OK;
  if (!rewards || !values || !lengths || !stopped || !adv_out) return ESPO_ERR_NULL;
  if (((uintptr_t)rewards % 16) || ((uintptr_t)values % 16) || ((uintptr_t)adv_out % 16) || ((uintptr_t)lengths % 4) ||
      ((uintptr_t)status_out % 4))
    return ESPO_ERR_ALIGN;
  if (gamma != gamma || lambda != lambda || r_fail != r_fail) return ESPO_ERR_BAD_PARAM;
  const long long nchunks = (total_tokens + kAdvChunk - 1) / kAdvChunk;
  int dev;
  ESPO_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return ESPO_ERR_CAPACITY;
  std::lock_guard<std::mutex> lk(g_pool_mu);
  NoAllocSlot& slot = g_noalloc[dev];
  if (!slot.base) {
    // In host code the array's name is only a handle; the kernels need its address on this device.
    void* p = nullptr;
    ESPO_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    ESPO_CUDA_TRY(cudaDeviceGetAttribute(&slot.sm_count, cudaDevAttrMultiProcessorCount, dev));
    slot.base = static_cast<unsigned char*>(p);
  }
  cudaStream_t s = (cudaStream_t)stream;
  unsigned char* b = slot.base;
  // The array keeps whatever the previous call left.  Nothing in it has to start at zero: the preparation
  // kernel rewrites every offset and chunk owner this call reads, and the built-in status word is only OR-ed into.
  AdvArgs a;
  a.rewards = rewards; a.values = values; a.lengths = lengths; a.stopped = stopped; a.adv = adv_out; a.ret = nullptr;
  a.stats = nullptr; a.ws.partials = nullptr; a.ws.done = nullptr;
  a.B = B; a.t_max = 0; a.total = total_tokens; a.nchunks = (int)nchunks;
  set_discount(a, gamma, lambda);
  a.r_fail = r_fail;
  a.ws.offsets = (long long*)(b + kNaOffOffsets);
  a.ws.chunk_first = (int*)(b + kNaOffChunkFirst);
  a.ws.status = status_out ? status_out : (unsigned*)(b + kNaOffStatus);
  return launch_advantages(a, slot.sm_count, s);
}

int espo_advantages_reserve(int32_t max_B, int64_t max_tokens) {
  using namespace espo;
  if (max_B < 1 || max_tokens < 1) return ESPO_ERR_BAD_SHAPE;
  int dev;
  ESPO_CUDA_TRY(cudaGetDevice(&dev));
  std::lock_guard<std::mutex> lk(g_pool_mu);
  AdvPool* p;
  return ensure_pool(dev, max_B, (max_tokens + kAdvChunk - 1) / kAdvChunk, &p);
}

int espo_advantages_stats(const float* rewards, const float* values, const int32_t* lengths, const uint8_t* stopped,
                          int32_t B, int64_t total_tokens, float gamma, float lambda, float r_fail, float* adv_out,
                          float* returns_out, double* stats_out, void* stream) {
  using namespace espo;
  if (B < 0 || total_tokens < 0) return ESPO_ERR_BAD_SHAPE;
  if ((uintptr_t)stats_out % 8) return ESPO_ERR_ALIGN;
  if (B == 0 || total_tokens == 0) {
    if (stats_out) ESPO_CUDA_TRY(cudaMemsetAsync(stats_out, 0, 2 * sizeof(double), (cudaStream_t)stream));
    return ESPO_OK;
  }
  if (!rewards || !values || !lengths || !stopped || !adv_out) return ESPO_ERR_NULL;
  if (((uintptr_t)rewards % 16) || ((uintptr_t)values % 16) || ((uintptr_t)adv_out % 16) || ((uintptr_t)lengths % 4) ||
      ((uintptr_t)returns_out % 16))
    return ESPO_ERR_ALIGN;
  if (gamma != gamma || lambda != lambda || r_fail != r_fail) return ESPO_ERR_BAD_PARAM;
  const long long nchunks = (total_tokens + kAdvChunk - 1) / kAdvChunk;
  if (nchunks > 0x7fffffffLL) return ESPO_ERR_CAPACITY;
  int dev;
  ESPO_CUDA_TRY(cudaGetDevice(&dev));
  std::lock_guard<std::mutex> lk(g_pool_mu);
  AdvPool* p;
  int rc = ensure_pool(dev, B, nchunks, &p);
  if (rc != ESPO_OK) return rc;
  cudaStream_t s = (cudaStream_t)stream;
  AdvArgs a;
  a.rewards = rewards; a.values = values; a.lengths = lengths; a.stopped = stopped; a.adv = adv_out; a.ret = returns_out;
  a.stats = stats_out;
  a.B = B; a.t_max = 0; a.total = total_tokens; a.nchunks = (int)nchunks;
  set_discount(a, gamma, lambda);
  a.r_fail = r_fail;
  a.ws = p->ws;
  return launch_advantages(a, p->sm_count, s);
}

int espo_advantages_padded(const float* rewards, const float* values, const int32_t* lengths, const uint8_t* stopped,
                           int32_t B, int32_t t_max, float gamma, float lambda, float r_fail, float* adv_out,
                           float* returns_out, void* stream) {
  using namespace espo;
  if (B < 0 || t_max < 0) return ESPO_ERR_BAD_SHAPE;
  if (B == 0 || t_max == 0) return ESPO_OK;
  if (!rewards || !values || !lengths || !stopped || !adv_out) return ESPO_ERR_NULL;
  if (((uintptr_t)rewards % 16) || ((uintptr_t)values % 16) || ((uintptr_t)adv_out % 16) || ((uintptr_t)lengths % 4) ||
      ((uintptr_t)returns_out % 16))
    return ESPO_ERR_ALIGN;
  if (gamma != gamma || lambda != lambda || r_fail != r_fail) return ESPO_ERR_BAD_PARAM;
  const long long total = (long long)B * t_max;
  const long long nchunks = (total + kAdvChunk - 1) / kAdvChunk;
  if (nchunks > 0x7fffffffLL) return ESPO_ERR_CAPACITY;
  int dev;
  ESPO_CUDA_TRY(cudaGetDevice(&dev));
  std::lock_guard<std::mutex> lk(g_pool_mu);
  AdvPool* p;
  int rc = ensure_pool(dev, B, nchunks, &p);
  if (rc != ESPO_OK) return rc;
  AdvArgs a;
  a.rewards = rewards; a.values = values; a.lengths = lengths; a.stopped = stopped; a.adv = adv_out; a.ret = returns_out;
  a.stats = nullptr;
  a.B = B; a.t_max = t_max; a.total = total; a.nchunks = (int)nchunks;
  set_discount(a, gamma, lambda);
  a.r_fail = r_fail;
  a.ws = p->ws;
  return launch_advantages(a, p->sm_count, (cudaStream_t)stream);
}

int espo_advantages_returns(const float* rewards, const float* values, const int32_t* lengths, const uint8_t* stopped,
                            int32_t B, int64_t total_tokens, float gamma, float lambda, float r_fail, float* adv_out,
                            float* returns_out, void* stream) {
  return espo_advantages_stats(rewards, values, lengths, stopped, B, total_tokens, gamma, lambda, r_fail, adv_out,
                               returns_out, nullptr, stream);
}

int espo_advantages(const float* rewards, const float* values, const int32_t* lengths, const uint8_t* stopped,
                    int32_t B, int64_t total_tokens, float gamma, float lambda, float r_fail, float* adv_out,
                    void* stream) {
  return espo_advantages_returns(rewards, values, lengths, stopped, B, total_tokens, gamma, lambda, r_fail, adv_out,
                                 nullptr, stream);
}

int espo_advantages_status(uint32_t* host_out, void* stream) {
  using namespace espo;
  if (!host_out) return ESPO_ERR_NULL;
  int dev;
  ESPO_CUDA_TRY(cudaGetDevice(&dev));
  std::lock_guard<std::mutex> lk(g_pool_mu);
  *host_out = 0;
  if (dev < 0 || dev >= kMaxDevices || !g_pool[dev].arena) return ESPO_OK;
  cudaStream_t s = (cudaStream_t)stream;
  ESPO_CUDA_TRY(cudaMemcpyAsync(host_out, g_pool[dev].ws.status, 4, cudaMemcpyDeviceToHost, s));
  ESPO_CUDA_TRY(cudaMemsetAsync(g_pool[dev].ws.status, 0, 4, s));
  ESPO_CUDA_TRY(cudaStreamSynchronize(s));
  return ESPO_OK;
}

}  // extern "C"
