// Device-side building blocks shared by the decode and prefill kernels:
// Philox4x32-10, the uniform -> Gumbel map (Eq. 7), mbarrier / bulk-copy
// wrappers with bounded waits, warp reductions.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace kf {

// Device error word values (mirrors KF_ETIMEOUT / KF_EBOUNDS of the C header).
constexpr int ERR_TIMEOUT = -5;
constexpr int ERR_BOUNDS = -6;

constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

// ------------------------------------------------------------------ Philox
// Philox4x32-10 (Salmon et al., SC'11).  The key schedule of the ten rounds
// depends only on the seed, so it is expanded once on the host.
struct PhiloxKeys {
  uint32_t k0[10];
  uint32_t k1[10];
};

__host__ inline PhiloxKeys philox_expand_key(uint64_t seed) {
  PhiloxKeys pk;
  uint32_t a = (uint32_t)(seed & 0xffffffffu), b = (uint32_t)(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    pk.k0[r] = a;
    pk.k1[r] = b;
    a += 0x9E3779B9u;
    b += 0xBB67AE85u;
  }
  return pk;
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxKeys& pk) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi_a = __umulhi(0xD2511F53u, c0);
    const uint32_t lo_a = 0xD2511F53u * c0;
    const uint32_t hi_b = __umulhi(0xCD9E8D57u, c2);
    const uint32_t lo_b = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi_b ^ c1 ^ pk.k0[r];
    const uint32_t n2 = hi_a ^ c3 ^ pk.k1[r];
    c0 = n0; c1 = lo_b; c2 = n2; c3 = lo_a;
  }
  return make_uint4(c0, c1, c2, c3);
}

// Noise word of logit (query position i, key position j): counter
// (j / 4, i, layer * H + head, batch), output word j mod 4.
__device__ __forceinline__ uint32_t noise_word(const PhiloxKeys& pk, uint32_t b, uint32_t lh, uint32_t i, uint32_t j) {
  const uint4 r = philox4x32_10(j >> 2, i, lh, b, pk);
  const uint32_t s = j & 3u;
  return s == 0 ? r.x : (s == 1 ? r.y : (s == 2 ? r.z : r.w));
}

// u = (top 23 bits + 1/2) / 2^23, exact in binary32, inside (0, 1).
__device__ __forceinline__ float uniform_from_word(uint32_t r) {
  return ((float)(r >> 9) + 0.5f) * (1.0f / 8388608.0f);
}

// E = -ln(u) with a relative error of a few 1e-6 over the whole grid of u:
// the fast logarithm has an absolute error near 2^-22, which is not good
// enough once u approaches 1, so there the series of -ln(1 - v) takes over
// (v = 1 - u is exact).
__device__ __forceinline__ float neg_log_uniform(float u) {
  const float v = 1.0f - u;
  const float series = v * fmaf(v, fmaf(v, fmaf(v, 0.25f, 0.33333334f), 0.5f), 1.0f);
  const float direct = -LN2 * __log2f(u);
  return v < 0.03125f ? series : direct;
}

// Standard Gumbel variate zeta = -ln(-ln u) (inverse cdf of Eq. 7).
__device__ __forceinline__ float gumbel_from_word(uint32_t r) {
  return -LN2 * __log2f(neg_log_uniform(uniform_from_word(r)));
}

// Standard normal variate by the Box-Muller transform: radius from word a, angle from word b.
// cos(2 pi u) is evaluated as -cos(2 pi (u - 1/2)) so that the fast cosine sees an angle inside (-pi, pi).
__device__ __forceinline__ float gauss_from_words(uint32_t ra, uint32_t rb) {
  const float radius = sqrtf(2.0f * neg_log_uniform(uniform_from_word(ra)));
  const float angle = 6.2831853071795865f * (uniform_from_word(rb) - 0.5f);
  return -radius * __cosf(angle);
}
// The second word of the Gaussian adjustment comes from a separate counter plane: bit 31 of the batch word.
constexpr uint32_t GAUSS_PLANE = 0x80000000u;

// ------------------------------------------------------------------ warp reductions
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ------------------------------------------------------------------ mbarrier + bulk async copy
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Non-blocking form: reports at once whether the phase with this parity has completed (try_wait may suspend the thread
// for a while when it has not).
__device__ __forceinline__ bool mbar_poll(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `limit` polls and reports false.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t limit = (1u << 22)) {
  for (uint32_t it = 0; it < limit; ++it) {
    if (mbar_test(bar, parity)) return true;
    if (it > 64) __nanosleep(64);
  }
  return false;
}
// 1-D bulk copy global -> shared of `bytes` (multiple of 16, both addresses
// 16-byte aligned), completion counted on `bar`.  Each CTA fetches its own copy.
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

}  // namespace kf
