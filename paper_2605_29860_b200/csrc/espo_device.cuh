// Device-side building blocks shared by the ESPO kernels: mbarrier / bulk-copy PTX
// wrappers with bounded waits, Philox4x32-10, warp reductions.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace espo {

constexpr int kBlockIds = 1024;  // ids per sampling block (level 2 of the hierarchical sampler)
constexpr int kSubIds = 32;      // ids per sub-block (level 1)
constexpr unsigned kFullMask = 0xffffffffu;

// Iteration caps of the in-kernel waits.  A wait that runs out records ESPO_DEV_TIMEOUT and
// the kernel winds down instead of spinning forever.
constexpr uint32_t kMbarSpinLimit = 1u << 22;   // try_wait calls (each may suspend in hardware)
constexpr uint32_t kPollSpinLimit = 1u << 22;   // polls with a short sleep in between

// ---------------------------------------------------------------- shared-memory barriers

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_init_fence() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Wait for the phase with the given parity, giving up after kMbarSpinLimit tries or as soon
// as another warp of the CTA has raised `*abort_flag` (may be null).  Returns false when it gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < kMbarSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u && abort_flag && *abort_flag) return false;
  }
  return false;
}

// Orders this thread's earlier generic-proxy accesses to shared memory before later
// asynchronous-proxy ones (a bulk copy that overwrites a stage the warp has just read).
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Bulk asynchronous copy global -> shared (TMA without a tensor map, into this CTA only).  Both addresses
// 16-byte aligned, bytes a multiple of 16.  Completion is signalled on `bar` as transaction bytes.
__device__ __forceinline__ void bulk_copy_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_addr(dst_smem)),
      "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar))
      : "memory");
}

// Barrier 1 of the CTA, for `threads` threads (a multiple of 32): warps running different code
// (streaming warps, the finalizer warp) meet here once; unlike __syncthreads() it may be reached
// from different places in the program.
__device__ __forceinline__ void cta_rendezvous(unsigned threads) {
  asm volatile("bar.sync 1, %0;" ::"r"(threads) : "memory");
}

// ---------------------------------------------------------------- ordered global accesses

// Adds to a counter in global memory; everything this thread wrote or observed before is
// visible to whoever reads the new count with acquire semantics at device scope, and the
// thread's later reads see what earlier adders published.
__device__ __forceinline__ unsigned atom_add_acq_rel_gpu(unsigned* p, unsigned v) {
  unsigned old;
  asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}

// Loads that are not served from the (incoherent) L1; the address may be shared or global.
__device__ __forceinline__ float2 ld_volatile_f2(const void* p) {
  float2 v;
  asm volatile("ld.volatile.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "l"(p) : "memory");
  return v;
}
// 16-byte accesses that are performed as one transaction and bypass L1 (global memory).
__device__ __forceinline__ uint4 ld_volatile_u4(const uint4* p) {
  uint4 v;
  asm volatile("ld.volatile.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_volatile_u4(uint4* p, uint4 v) {
  asm volatile("st.volatile.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ int2 ld_volatile_i2(const void* p) {
  int2 v;
  asm volatile("ld.volatile.v2.s32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ float4 ld_volatile_f4(const void* p) {
  float4 v;
  asm volatile("ld.volatile.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
  return v;
}

// ---------------------------------------------------------------- Philox4x32-10

// Counter-based generator of Salmon et al. (SC'11): ten rounds, each two 32x32->64 multiplies
// and a key-dependent xor; the key advances by the Weyl constants between rounds.
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                               uint32_t k1) {
  constexpr uint32_t MA = 0xD2511F53u, MB = 0xCD9E8D57u, WA = 0x9E3779B9u, WB = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t ha = __umulhi(MA, c0), la = MA * c0;
    const uint32_t hb = __umulhi(MB, c2), lb = MB * c2;
    const uint32_t n0 = hb ^ c1 ^ k0;
    const uint32_t n2 = ha ^ c3 ^ k1;
    c0 = n0; c1 = lb; c2 = n2; c3 = la;
    k0 += WA; k1 += WB;
  }
  return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint32_t pick_word(const uint4& w, uint32_t i) {
  return i == 0 ? w.x : (i == 1 ? w.y : (i == 2 ? w.z : w.w));
}

// ln E of an exponential draw E = -ln u in [6e-8, 17]: the Gumbel is -ln E.  E itself comes from the precise
// logf (u close to 1 makes E tiny, and its relative accuracy is what the large Gumbels rest on); its logarithm
// may be lg2.approx: absolute error below 2^-22 for E in (0.5, 2), relative error below 2^-22 elsewhere, i.e.
// below 6e-6 at the far ends and below 1e-6 typically -- two orders under the sampler's tie margin.
__device__ __forceinline__ float ln_expo(float e) {
  float y;
  asm("lg2.approx.f32 %0, %1;" : "=f"(y) : "f"(e));
  return y * 0.6931471805599453f;
}

// 23 random bits k -> u = (2k+1)/2^24 in (0,1), exact in float32; G = -log(-log u): the inner logarithm in full
// precision, the outer one as ln_expo.
__device__ __forceinline__ float gumbel_from_word(uint32_t word) {
  const float u = __uint2float_rn(2u * (word >> 9) + 1u) * 5.9604644775390625e-08f;
  return -ln_expo(-logf(u));
}

// The same uniform as a standard exponential draw E = -ln u > 0 (the Gumbel is -ln E).
__device__ __forceinline__ float expo_from_word(uint32_t word) {
  const float u = __uint2float_rn(2u * (word >> 9) + 1u) * 5.9604644775390625e-08f;
  return -logf(u);
}

// Which Philox stream a draw belongs to: (step, slot, batch|level) are counter words 1..3.
struct DrawStream {
  uint32_t k0, k1;     // seed halves
  uint32_t step, slot;
  uint32_t batch_bits; // batch_id << 2
};

__device__ __forceinline__ float gumbel_at(const DrawStream& ds, uint32_t level, uint32_t index) {
  const uint4 w = philox4x32_10(index >> 2, ds.step, ds.slot, ds.batch_bits | level, ds.k0, ds.k1);
  return gumbel_from_word(pick_word(w, index & 3u));
}

// The uniform itself, u = (2k+1)/2^24 in (0,1).
__device__ __forceinline__ float uniform_at(const DrawStream& ds, uint32_t level, uint32_t index) {
  const uint4 w = philox4x32_10(index >> 2, ds.step, ds.slot, ds.batch_bits | level, ds.k0, ds.k1);
  return __uint2float_rn(2u * (pick_word(w, index & 3u) >> 9) + 1u) * 5.9604644775390625e-08f;
}

__device__ __forceinline__ float expo_at(const DrawStream& ds, uint32_t level, uint32_t index) {
  const uint4 w = philox4x32_10(index >> 2, ds.step, ds.slot, ds.batch_bits | level, ds.k0, ds.k1);
  return expo_from_word(pick_word(w, index & 3u));
}

// ---------------------------------------------------------------- warp reductions

__device__ __forceinline__ float warp_max(float v) {
  float r;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
  return r;
}

// Butterfly sum: every lane ends with the same bits, independent of anything but the inputs.
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
  return v;
}

// Argmax of (score, index) over the warp; the lower index wins equal scores.  Lanes with
// nothing to offer pass index < 0.  Every lane gets the result.  Scores are never NaN here.
// Two warp-wide reductions in hardware: the largest offered score, then the smallest index
// among the lanes that offer it.
__device__ __forceinline__ void warp_argmax(float& score, int& index) {
  const float offered = index >= 0 ? score : __int_as_float(0xff800000);
  float best;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(best) : "f"(offered));
  const int cand = (index >= 0 && score == best) ? index : 0x7fffffff;
  int first;
  asm volatile("redux.sync.min.s32 %0, %1, 0xffffffff;" : "=r"(first) : "r"(cand));
  score = best;
  index = first == 0x7fffffff ? -1 : first;
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ln of a sum of exponentials that is known to lie in [1, 1024 * 32]: lg2.approx has an absolute error below
// 2^-22 on the mantissa's logarithm, i.e. below 2e-7 here -- two orders under the sampler's tie margin.
__device__ __forceinline__ float log_sum(float s) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(s));
  return y * 0.6931471805599453f;
}

__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
  uint32_t c;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(c) : "r"(a), "r"(b));
  return c;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

}  // namespace espo
