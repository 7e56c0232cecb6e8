// TD errors and GAE over ragged, truncated trajectories (Eq. 4-5) with ESPO's absorbing
// failure transition (Eq. 13), for sm_100a.
//
// The packed token array is cut into fixed chunks of kAdvChunk tokens regardless of where
// trajectories begin and end, so every CTA moves the same number of bytes (12 per token:
// reward and value in, advantage out) whatever the length mix is.  Within a chunk the
// backward recursion A_t = delta_t + k_t A_{t+1} (k_t = gamma*lambda, or 0 on a trajectory's
// last token) is a scan over affine maps X -> b + a X: each thread composes the maps of its
// 8 tokens, a warp-shuffle suffix scan and a small cross-warp pass compose them across the
// CTA.  A chunk whose last token is not a trajectory end needs A of the next chunk's first
// token; chunks are handed out from the END of the array by an atomic counter and pass that
// value backwards through per-chunk descriptors (aggregate map first, final value when
// known), so the array is read and written exactly once.  The maps are composed in double
// precision, which costs nothing next to the memory traffic and keeps gamma*lambda = 1 sums
// over 16k tokens exact to float32 rounding of the result.
//
// A small preparation kernel turns lengths into offsets and tells every chunk which
// trajectory its first token belongs to.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "espo.h"
#include "espo_device.cuh"
#include "espo_host.h"

namespace espo {

constexpr int kAdvThreads = 256;
constexpr int kAdvPerThread = 8;
constexpr int kAdvChunk = kAdvThreads * kAdvPerThread;   // 2048 tokens
constexpr int kAdvWarps = kAdvThreads / 32;
constexpr int kPrepThreads = 1024;

struct AdvWorkspace {
  long long* offsets;     // [B+1] exclusive prefix sum of lengths
  int* chunk_first;       // [nchunks] trajectory that owns the chunk's first token
  unsigned* flag;         // [nchunks] epoch*4 + {1: aggregate published, 2: final value published}
  double2* agg;           // [nchunks] chunk map X -> agg.y + agg.x * X
  double* fin;            // [nchunks] A of the chunk's first token
  unsigned* counters;     // [0] next chunk ticket, [1] chunks finished
  unsigned* status;       // sticky ESPO_DEV_* bits
};

struct AdvArgs {
  const float* rewards;
  const float* values;
  const int32_t* lengths;
  const uint8_t* stopped;
  float* adv;
  int B;
  long long total;
  int nchunks;
  double gamma, gl;       // gamma, gamma*lambda
  float r_fail;
  unsigned epoch4;        // epoch * 4
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

struct Map {   // X -> b + a * X
  double a, b;
};
// `lo` is applied after `hi` (lo belongs to the earlier tokens): lo(hi(X)).
__device__ __forceinline__ Map compose(const Map& lo, const Map& hi) { return Map{lo.a * hi.a, fma(lo.a, hi.b, lo.b)}; }

__device__ __forceinline__ double shfl_down_d(double v, int o) { return __shfl_down_sync(kFullMask, v, o); }

__global__ void __launch_bounds__(kAdvThreads) espo_adv_scan_kernel(const AdvArgs a) {
  __shared__ __align__(16) unsigned char flags[kAdvChunk];   // bit0: last token of a trajectory, bit1: it was stopped
  __shared__ Map warp_agg[kAdvWarps];
  __shared__ float warp_first_v[kAdvWarps];
  __shared__ int chunk_s;
  __shared__ double carry_s;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) chunk_s = a.nchunks - 1 - (int)atomicAdd(a.ws.counters, 1u);   // highest positions first
  reinterpret_cast<unsigned long long*>(flags)[tid] = 0ull;
  __syncthreads();
  const int j = chunk_s;
  const long long p0 = (long long)j * kAdvChunk;
  const int n = (int)min((long long)kAdvChunk, a.total - p0);
  const int q0 = tid * kAdvPerThread;

  // ---- this thread's 8 rewards and values (issued before anything that depends on the prep data) ----
  float r[kAdvPerThread], v[kAdvPerThread + 1];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int q = q0 + 4 * h;
    if (q + 4 <= n) {
      const float4 rr = __ldcs(reinterpret_cast<const float4*>(a.rewards + p0 + q));
      const float4 vv = __ldcs(reinterpret_cast<const float4*>(a.values + p0 + q));
      r[4 * h] = rr.x; r[4 * h + 1] = rr.y; r[4 * h + 2] = rr.z; r[4 * h + 3] = rr.w;
      v[4 * h] = vv.x; v[4 * h + 1] = vv.y; v[4 * h + 2] = vv.z; v[4 * h + 3] = vv.w;
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        r[4 * h + e] = (q + e < n) ? __ldcs(a.rewards + p0 + q + e) : 0.f;
        v[4 * h + e] = (q + e < n) ? __ldcs(a.values + p0 + q + e) : 0.f;
      }
    }
  }
  // value of the token after this thread's last one: next lane, next warp, or next chunk
  float v_after = __shfl_down_sync(kFullMask, v[0], 1);
  if (lane == 0) warp_first_v[warp] = v[0];

  // ---- mark trajectory ends inside the chunk ----
  {
    const long long p_end = p0 + n;
    for (int i = a.ws.chunk_first[j] + tid; i < a.B; i += kAdvThreads) {
      const long long o0 = a.ws.offsets[i];
      if (o0 >= p_end) break;
      const long long o1 = a.ws.offsets[i + 1];
      if (o1 > o0 && o1 - 1 >= p0 && o1 - 1 < p_end) flags[o1 - 1 - p0] = (unsigned char)(1u | (a.stopped[i] ? 2u : 0u));
    }
  }
  __syncthreads();
  if (lane == 31) {
    if (warp + 1 < kAdvWarps) v_after = warp_first_v[warp + 1];
    else v_after = (p0 + kAdvChunk < a.total) ? __ldg(a.values + p0 + kAdvChunk) : 0.f;
  }
  v[kAdvPerThread] = v_after;

  // ---- per-token TD error and coefficient; compose the thread's map right to left ----
  const unsigned long long f8 = reinterpret_cast<const unsigned long long*>(flags)[tid];
  double delta[kAdvPerThread];
  unsigned last_mask = 0;
  Map m{1.0, 0.0};
#pragma unroll
  for (int e = kAdvPerThread - 1; e >= 0; --e) {
    const unsigned f = (unsigned)(f8 >> (8 * e)) & 0xffu;
    const bool in = (q0 + e < n);
    // the array's very last token ends a trajectory even if the lengths are inconsistent
    const bool last = (f & 1u) || (p0 + q0 + e == a.total - 1);
    const double rew = (last && (f & 2u)) ? (double)a.r_fail : (double)r[e];
    const double d = rew + (last ? 0.0 : a.gamma * (double)v[e + 1]) - (double)v[e];
    delta[e] = d;
    if (last) last_mask |= 1u << e;
    if (in) {
      const double k = last ? 0.0 : a.gl;
      m = Map{k * m.a, fma(k, m.b, d)};
    }
  }

  // ---- suffix scan over the CTA: what comes after each thread, as a map of the chunk's carry-in ----
  Map inc = m;   // inclusive: this thread and everything after it inside the warp
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    Map hi{shfl_down_d(inc.a, o), shfl_down_d(inc.b, o)};
    if (lane + o < 32) inc = compose(inc, hi);
  }
  if (lane == 0) warp_agg[warp] = inc;
  Map after{shfl_down_d(inc.a, 1), shfl_down_d(inc.b, 1)};   // exclusive within the warp
  if (lane == 31) after = Map{1.0, 0.0};
  __syncthreads();
  for (int w = warp + 1; w < kAdvWarps; ++w) after = compose(after, warp_agg[w]);

  // ---- chunk descriptor and carry-in ----
  if (tid == 0) {
    const Map whole = compose(m, after);     // the whole chunk
    const bool has_next = (p0 + kAdvChunk < a.total);
    // Tokens after the chunk's last trajectory end still need the value that follows the chunk,
    // even though the chunk as a whole (whole.a == 0) passes nothing through.
    const bool need_carry = has_next && !(flags[n - 1] & 1u);
    volatile unsigned* my_flag = reinterpret_cast<volatile unsigned*>(a.ws.flag + j);
    if (whole.a == 0.0) {                    // A of the first token does not depend on what follows
      a.ws.fin[j] = whole.b;
      __threadfence();
      *my_flag = a.epoch4 | 2u;
    } else {
      a.ws.agg[j] = make_double2(whole.a, whole.b);
      __threadfence();
      *my_flag = a.epoch4 | 1u;
    }
    double carry = 0.0;
    if (need_carry) {
      // walk forward through the chunks after this one until the chain closes
      Map acc{1.0, 0.0};
      int jj = j + 1;
      bool resolved = false;
      for (uint32_t it = 0; it < kPollSpinLimit && !resolved; ++it) {
        const unsigned f = *reinterpret_cast<volatile unsigned*>(a.ws.flag + jj);
        if (f == (a.epoch4 | 2u)) {
          __threadfence();
          carry = fma(acc.a, __ldcg(a.ws.fin + jj), acc.b);
          resolved = true;
        } else if (f == (a.epoch4 | 1u)) {
          __threadfence();
          const double2 g = __ldcg(a.ws.agg + jj);
          acc = compose(acc, Map{g.x, g.y});
          ++jj;
          if (acc.a == 0.0 || jj >= a.nchunks) { carry = acc.b; resolved = true; }
        } else {
          __nanosleep(40);
        }
      }
      if (!resolved) atomicOr(a.ws.status, ESPO_DEV_TIMEOUT);
    }
    if (whole.a != 0.0) {
      a.ws.fin[j] = fma(whole.a, carry, whole.b);
      __threadfence();
      *my_flag = a.epoch4 | 2u;
    }
    carry_s = carry;
  }
  __syncthreads();

  // ---- replay the thread's tokens with the now known value that follows them ----
  double x = fma(after.a, carry_s, after.b);
  float out[kAdvPerThread];
#pragma unroll
  for (int e = kAdvPerThread - 1; e >= 0; --e) {
    if (q0 + e < n) {
      const double k = ((last_mask >> e) & 1u) ? 0.0 : a.gl;
      x = fma(k, x, delta[e]);
      out[e] = (float)x;
    } else {
      out[e] = 0.f;
    }
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int q = q0 + 4 * h;
    if (q + 4 <= n) {
      __stcs(reinterpret_cast<float4*>(a.adv + p0 + q), make_float4(out[4 * h], out[4 * h + 1], out[4 * h + 2], out[4 * h + 3]));
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) if (q + e < n) a.adv[p0 + q + e] = out[4 * h + e];
    }
  }

  // ---- the last CTA to finish rewinds the counters for the next call ----
  if (tid == 0) {
    __threadfence();
    if (atomicAdd(a.ws.counters + 1, 1u) == (unsigned)a.nchunks - 1u) {
      a.ws.counters[0] = 0u;
      a.ws.counters[1] = 0u;
    }
  }
}

// ---------------------------------------------------------------------------------------
// Per-device workspace, grown on demand.
// ---------------------------------------------------------------------------------------
struct AdvPool {
  void* arena = nullptr;
  int cap_B = 0;
  long long cap_chunks = 0;
  unsigned epoch = 0;
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
    const size_t o_off = carve(8 * ((size_t)nb + 1)), o_cf = carve(4 * (size_t)nc), o_fl = carve(4 * (size_t)nc);
    const size_t o_ag = carve(16 * (size_t)nc), o_fi = carve(8 * (size_t)nc), o_ct = carve(8), o_st = carve(4);
    ESPO_CUDA_TRY(cudaMalloc(&p.arena, off));
    ESPO_CUDA_TRY(cudaMemset(p.arena, 0, off));
    unsigned char* b = static_cast<unsigned char*>(p.arena);
    p.ws.offsets = (long long*)(b + o_off); p.ws.chunk_first = (int*)(b + o_cf); p.ws.flag = (unsigned*)(b + o_fl);
    p.ws.agg = (double2*)(b + o_ag); p.ws.fin = (double*)(b + o_fi); p.ws.counters = (unsigned*)(b + o_ct);
    p.ws.status = (unsigned*)(b + o_st);
    p.cap_B = nb; p.cap_chunks = nc; p.epoch = 0;
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
constexpr long long kNoAllocMaxChunks = (ESPO_NOALLOC_MAX_TOKENS + kAdvChunk - 1) / kAdvChunk;
constexpr size_t kNaOffOffsets = 0;
constexpr size_t kNaOffChunkFirst = kNaOffOffsets + ((8 * ((size_t)kNoAllocMaxB + 1) + 255) / 256) * 256;
constexpr size_t kNaOffFlag = kNaOffChunkFirst + 4 * (size_t)kNoAllocMaxChunks;
constexpr size_t kNaOffAgg = kNaOffFlag + 4 * (size_t)kNoAllocMaxChunks;
constexpr size_t kNaOffFin = kNaOffAgg + 16 * (size_t)kNoAllocMaxChunks;
constexpr size_t kNaOffCounters = kNaOffFin + 8 * (size_t)kNoAllocMaxChunks;
constexpr size_t kNaOffStatus = kNaOffCounters + 256;
constexpr size_t kNoAllocBytes = kNaOffStatus + 256;
static_assert(kNoAllocMaxChunks % 64 == 0, "keeps every sub-array 256-byte aligned");

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

struct NoAllocSlot {
  unsigned char* base = nullptr;   // device address of g_noalloc_scratch on this device
  unsigned epoch = 0;
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
    slot.base = static_cast<unsigned char*>(p);
    slot.epoch = 0;
  }
  cudaStream_t s = (cudaStream_t)stream;
  unsigned char* b = slot.base;
  if (++slot.epoch >= (1u << 30)) {   // the descriptors' flags carry the epoch; start over before it wraps
    ESPO_CUDA_TRY(cudaMemsetAsync(b + kNaOffFlag, 0, 4 * (size_t)kNoAllocMaxChunks, s));
    slot.epoch = 1;
  }
  // The array keeps whatever the previous call left: the chunk tickets must start at zero even if
  // that call was cut short, and the built-in status word is only ever OR-ed into.
  ESPO_CUDA_TRY(cudaMemsetAsync(b + kNaOffCounters, 0, 8, s));
  AdvArgs a;
  a.rewards = rewards; a.values = values; a.lengths = lengths; a.stopped = stopped; a.adv = adv_out;
  a.B = B; a.total = total_tokens; a.nchunks = (int)nchunks;
  a.gamma = (double)gamma; a.gl = (double)gamma * (double)lambda;
  a.r_fail = r_fail;
  a.epoch4 = slot.epoch << 2;
  a.ws.offsets = (long long*)(b + kNaOffOffsets);
  a.ws.chunk_first = (int*)(b + kNaOffChunkFirst);
  a.ws.flag = (unsigned*)(b + kNaOffFlag);
  a.ws.agg = (double2*)(b + kNaOffAgg);
  a.ws.fin = (double*)(b + kNaOffFin);
  a.ws.counters = (unsigned*)(b + kNaOffCounters);
  a.ws.status = status_out ? status_out : (unsigned*)(b + kNaOffStatus);
  espo_adv_prep_kernel<<<1, kPrepThreads, 0, s>>>(a);
  ESPO_CUDA_TRY(cudaGetLastError());
  espo_adv_scan_kernel<<<(unsigned)nchunks, kAdvThreads, 0, s>>>(a);
  ESPO_CUDA_TRY(cudaGetLastError());
  return ESPO_OK;
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

int espo_advantages(const float* rewards, const float* values, const int32_t* lengths, const uint8_t* stopped,
                    int32_t B, int64_t total_tokens, float gamma, float lambda, float r_fail, float* adv_out,
                    void* stream) {
  using namespace espo;
  if (B < 0 || total_tokens < 0) return ESPO_ERR_BAD_SHAPE;
  if (B == 0 || total_tokens == 0) return ESPO_OK;
  if (!rewards || !values || !lengths || !stopped || !adv_out) return ESPO_ERR_NULL;
  if (((uintptr_t)rewards % 16) || ((uintptr_t)values % 16) || ((uintptr_t)adv_out % 16) || ((uintptr_t)lengths % 4))
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
  if (++p->epoch >= (1u << 30)) {   // flags carry the epoch; start over before it wraps
    ESPO_CUDA_TRY(cudaMemsetAsync(p->ws.flag, 0, 4 * (size_t)p->cap_chunks, s));
    p->epoch = 1;
  }
  AdvArgs a;
  a.rewards = rewards; a.values = values; a.lengths = lengths; a.stopped = stopped; a.adv = adv_out;
  a.B = B; a.total = total_tokens; a.nchunks = (int)nchunks;
  a.gamma = (double)gamma; a.gl = (double)gamma * (double)lambda;
  a.r_fail = r_fail;
  a.epoch4 = p->epoch << 2;
  a.ws = p->ws;
  espo_adv_prep_kernel<<<1, kPrepThreads, 0, s>>>(a);
  ESPO_CUDA_TRY(cudaGetLastError());
  espo_adv_scan_kernel<<<(unsigned)nchunks, kAdvThreads, 0, s>>>(a);
  ESPO_CUDA_TRY(cudaGetLastError());
  return ESPO_OK;
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
