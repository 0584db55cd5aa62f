// Generation-phase kernels (Algorithm 1, t >= 1): one layer call does
//   logits -> attention output + Gumbel-softmax score -> accumulate -> evict -> replace
// in two launches.
//
// decode_kernel, grid = (splits, units); a unit is one (batch row, head).  Each CTA streams a
// contiguous range of cache slots exactly once: every warp owns 32-row tiles,
// fetched into a private shared-memory ring by 1-D bulk async copies
// (cp.async.bulk + mbarrier, one copy per CTA), computes the logits x_j = q.K_j
// once and uses them twice -- for the value-weighted output (Eq. 1) and for
// the score softmax of (x_j + zeta_j) / tau (Eq. 4, 11) -- and leaves one partial per split.
//
// decode_close_kernel, one CTA per unit, launched as the streaming kernel's programmatic dependent
// (its CTAs become resident during the streaming kernel's last wave, request what does not depend
// on it, then pass griddepcontrol.wait): merges the split partials, normalises the scores, adds
// them into f_theta, picks the entry to evict and writes the new token's row into the freed slot.
#include "kf_decode.cuh"

#include <algorithm>
#include <cstdio>
#include <mutex>

namespace kf {

namespace {

constexpr int TILE_ROWS = 32;
constexpr int MAX_SPLITS = 64;   // CTAs per unit (the closing CTA keeps one weight per split in shared memory)

// o[0..8) += p * v[0..8) for one 16-byte chunk of a value row.  `pp` holds the softmax weight p twice, as a
// binary16 pair: the products p * v are then exact in binary32 and each mixed-precision fma rounds once, with
// no conversion instructions (p <= 1 carries a relative rounding error of 2^-11, far inside the output tolerance).
__device__ __forceinline__ void axpy8(float (&o)[8], uint32_t pp, const uint4& vv) {
  const uint32_t vw[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    asm("{\n\t.reg .b16 pl, ph, vl, vh;\n\t"
        "mov.b32 {pl, ph}, %2;\n\t"
        "mov.b32 {vl, vh}, %3;\n\t"
        "fma.rn.f32.f16 %0, pl, vl, %0;\n\t"
        "fma.rn.f32.f16 %1, ph, vh, %1;\n\t}"
        : "+f"(o[2 * c]), "+f"(o[2 * c + 1]) : "r"(pp), "r"(vw[c]));
  }
}

__device__ __forceinline__ unsigned long long evict_key(float a, int pos) {
  // smallest key = smallest accumulated score; equal scores: the higher position leaves
  return ((unsigned long long)__float_as_uint(a) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)pos);
}

// The eviction decision and the replacement, common to every form of the closing stage: `best` / `best_j` are the
// thread's smallest eviction key (accumulated score, inverted position) among its non-recent entries and its slot,
// z_new the new token's own score, kn_r / vn_r the thread's columns of the new token's row.
template <int D, int NT, int CPT>
__device__ __forceinline__ void evict_and_replace(const DecodeParams& P, int u, int len, unsigned long long best, int best_j,
                                                  float z_new, const __half (&kn_r)[CPT], const __half (&vn_r)[CPT]) {
  __shared__ unsigned long long sh_key[NT / 32];
  __shared__ int sh_j[NT / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int BATCH = 8;
  float* __restrict__ acc = P.acc + (size_t)u * P.k;
  int32_t* __restrict__ pos = P.pos + (size_t)u * P.k;
  const unsigned long long key_new = evict_key(z_new, P.p);
  int slot;   // where the new token's row goes
  if (len < P.k) {  // cache not full yet: append
    slot = len;
    if (tid == 0) P.len[u] = len + 1;
  } else {
    // smallest key over the CTA: warp minimum by shuffles, the owning lane publishes it with its slot
    const unsigned long long mine = best;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
      best = other < best ? other : best;
    }
    if (best == ~0ull ? lane == 0 : mine == best) { sh_key[warp] = best; sh_j[warp] = best_j; }   // keys are unique
    __syncthreads();
    best = sh_key[0];
    slot = sh_j[0];
#pragma unroll
    for (int wi = 1; wi < NT / 32; ++wi)
      if (sh_key[wi] < best) { best = sh_key[wi]; slot = sh_j[wi]; }
    if (P.w == 0 && key_new < best) return;  // the new token itself has the lowest score: it is not stored
    if (best == ~0ull || slot < 0 || slot >= len) {  // cannot happen for 0 <= w <= k; flag it instead of guessing
      if (tid == 0) atomicExch(P.err, ERR_BOUNDS);
      return;
    }
  }
  if (P.place) {
    // the entries behind the one that leaves move up one place; the new token takes the last place
    int32_t* __restrict__ place = P.place + (size_t)u * P.k;
    if (len >= P.k) {
      const int pos_out = (int)(0xffffffffu - (uint32_t)best);   // the key's low word is 2^32 - 1 - position
      for (int j0 = tid; j0 < len; j0 += NT * BATCH) {   // loads of a batch first, so that they overlap
        int pp[BATCH], pl[BATCH];
#pragma unroll
        for (int i = 0; i < BATCH; ++i) {
          const int j = j0 + i * NT;
          pp[i] = j < len ? pos[j] : -1;
          pl[i] = j < len ? place[j] : 0;
        }
#pragma unroll
        for (int i = 0; i < BATCH; ++i) {
          const int j = j0 + i * NT;
          if (j != slot && pp[i] > pos_out) place[j] = pl[i] - 1;   // pp = -1 beyond the end never passes
        }
      }
    }
    if (tid == 0) place[slot] = len < P.k ? len : P.k - 1;
  }
  if (tid == 0) { pos[slot] = P.p; acc[slot] = z_new; }
  __half* Kr = const_cast<__half*>(P.K) + ((size_t)u * P.k + slot) * D;
  __half* Vr = const_cast<__half*>(P.V) + ((size_t)u * P.k + slot) * D;
#pragma unroll
  for (int i = 0; i < CPT; ++i) {
    const int c = tid + i * NT;
    if (c < D) { Kr[c] = kn_r[i]; Vr[c] = vn_r[i]; }
  }
}

// Closing a unit: merge splits, normalise, accumulate, evict, replace.  Everything that does not depend on the
// streaming kernel (scores and positions of the entries, the new token's own logit) is requested before
// `griddepcontrol.wait`, i.e. while the streaming kernel's last CTAs are still running.
// G query heads share the unit's cache (G = 1: the method as printed): every head has its own split partials,
// adjusted logits and output row; the score added to f_theta is the mean of the heads' softmaxes (Eq. 11).
template <int D, int NT, int G>
__device__ void combine_and_evict(const DecodeParams& P, int u, int len) {
  const int tid = threadIdx.x, lane = tid & 31;
  const int Hkv = P.H / G;
  const uint32_t b = (uint32_t)(u / Hkv), h0 = (uint32_t)(u % Hkv) * G, lh0 = (uint32_t)P.layer * P.H + h0;
  const __half* q = P.q + (size_t)u * G * D;
  const __half* kn = P.knew + (size_t)u * D;
  const __half* vn = P.vnew + (size_t)u * D;
  constexpr int PSTRIDE = 4 + D;
  constexpr int CPT = (D + NT - 1) / NT;   // output columns per thread
  constexpr float INV_G = 1.0f / (float)G;
  const float* part = P.partials + (size_t)u * P.splits * G * PSTRIDE;   // [split][head][4 + D]
  float* __restrict__ acc = P.acc + (size_t)u * P.k;
  int32_t* __restrict__ pos = P.pos + (size_t)u * P.k;
  const float* __restrict__ ys = P.y_scratch + (size_t)u * G * (P.k + 1);   // [head][k + 1]

  // ---- independent of the streaming kernel: scores and positions of the first batch of entries, the new
  //      token's row, its own logit and adjusted logit (every warp computes these for itself: no hand-over)
  constexpr int BATCH = 8;   // 64 registers per thread keep all closing CTAs of 1024 units resident at once
  float yv[BATCH], av[BATCH];
  int pv[BATCH];
#pragma unroll
  for (int i = 0; i < BATCH; ++i) {
    const int j = tid + i * NT;
    const bool in = j < len;
    av[i] = in ? acc[j] : 0.f;
    pv[i] = in ? pos[j] : 0x7fffffff;
  }
  // entries beyond the first batch: pull their scores and positions into L2 (one request per 128-byte line)
  for (int line = tid + (NT * BATCH) / 32; line * 32 < len; line += NT) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(acc + line * 32));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(pos + line * 32));
  }
  __half kn_r[CPT], vn_r[CPT];
#pragma unroll
  for (int i = 0; i < CPT; ++i) {
    const int c = tid + i * NT;
    kn_r[i] = c < D ? kn[c] : __float2half(0.f);
    vn_r[i] = c < D ? vn[c] : __float2half(0.f);
  }
  float x_new[G], y_new[G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    float s = 0.f;
    for (int c = lane; c < D; c += 32) s = fmaf(__half2float(q[g * D + c]), __half2float(kn[c]), s);
    x_new[g] = warp_sum(s) * P.scale;  // bias(p, p) = 0
    float yn = 0.f;
    if (lane == 0) yn = (x_new[g] + noise_for(P, b, lh0 + g, (uint32_t)P.p, (uint32_t)P.p)) * P.inv_tau;
    y_new[g] = __shfl_sync(0xffffffffu, yn, 0);
  }

  asm volatile("griddepcontrol.wait;" ::: "memory");   // the streaming kernel has finished; its writes are visible

  // ---- everything the streaming kernel produced is requested at once
  if (G == 1) {
#pragma unroll
    for (int i = 0; i < BATCH; ++i) {
      const int j = tid + i * NT;
      yv[i] = j < len ? __ldcg(ys + j) : 0.f;
    }
  }
  float my[G], inv_ly[G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    // (max, sum) pairs of both softmaxes: split `lane` and split `lane + 32`
    float4 ps0 = make_float4(-INFINITY, 0.f, -INFINITY, 0.f), ps1 = ps0;
    if (lane < P.splits) ps0 = __ldcg(reinterpret_cast<const float4*>(part + ((size_t)lane * G + g) * PSTRIDE));
    if (lane + 32 < P.splits) ps1 = __ldcg(reinterpret_cast<const float4*>(part + ((size_t)(lane + 32) * G + g) * PSTRIDE));
    const float mx = warp_max(fmaxf(x_new[g], fmaxf(ps0.y > 0.f ? ps0.x : -INFINITY, ps1.y > 0.f ? ps1.x : -INFINITY)));
    my[g] = warp_max(fmaxf(y_new[g], fmaxf(ps0.w > 0.f ? ps0.z : -INFINITY, ps1.w > 0.f ? ps1.z : -INFINITY)));
    const float w0 = ps0.y > 0.f ? fast_exp2((ps0.x - mx) * LOG2E) : 0.f;   // weight of split `lane` in the output
    const float w1 = ps1.y > 0.f ? fast_exp2((ps1.x - mx) * LOG2E) : 0.f;
    float lx = fmaf(ps0.y, w0, ps1.y * w1);
    float ly = (ps0.w > 0.f ? ps0.w * fast_exp2((ps0.z - my[g]) * LOG2E) : 0.f) + (ps1.w > 0.f ? ps1.w * fast_exp2((ps1.z - my[g]) * LOG2E) : 0.f);
    const float inv_lx = 1.f / (warp_sum(lx) + fast_exp2((x_new[g] - mx) * LOG2E));
    inv_ly[g] = 1.f / (warp_sum(ly) + fast_exp2((y_new[g] - my[g]) * LOG2E));

    // ---- attention output of this head (Eq. 1): merged partial sums plus the new token's own value row
    float o[CPT];
#pragma unroll
    for (int i = 0; i < CPT; ++i) o[i] = fast_exp2((x_new[g] - mx) * LOG2E) * __half2float(vn_r[i]);
#pragma unroll 4
    for (int sp = 0; sp < P.splits; ++sp) {
      const float w = __shfl_sync(0xffffffffu, sp < 32 ? w0 : w1, sp & 31);
#pragma unroll
      for (int i = 0; i < CPT; ++i) {
        const int c = tid + i * NT;
        if (c < D) o[i] = fmaf(__ldcg(part + ((size_t)sp * G + g) * PSTRIDE + 4 + c), w, o[i]);
      }
    }
#pragma unroll
    for (int i = 0; i < CPT; ++i) {
      const int c = tid + i * NT;
      if (c < D) P.out[((size_t)u * G + g) * D + c] = __float2half_rn(o[i] * inv_lx);
    }
  }

  // ---- score (Eq. 11; the mean over the group's heads), accumulation and the eviction candidate
  float* __restrict__ sc = P.score_opt ? P.score_opt + (size_t)u * (P.k + 1) : nullptr;
  unsigned long long best = ~0ull;
  int best_j = -1;
  const int cutoff = P.p - P.w;  // entries with pos <= cutoff are outside the recent window
  for (int j0 = tid; j0 < len; j0 += NT * BATCH) {
    if (j0 != tid) {   // the first batch was loaded above
#pragma unroll
      for (int i = 0; i < BATCH; ++i) {
        const int j = j0 + i * NT;
        const bool in = j < len;
        if (G == 1) yv[i] = in ? __ldcg(ys + j) : 0.f;
        av[i] = in ? acc[j] : 0.f;
        pv[i] = in ? pos[j] : 0x7fffffff;
      }
    }
    float zv[BATCH];
    if (G == 1) {
#pragma unroll
      for (int i = 0; i < BATCH; ++i) zv[i] = fast_exp2((yv[i] - my[0]) * LOG2E) * inv_ly[0];
    } else {
#pragma unroll
      for (int i = 0; i < BATCH; ++i) zv[i] = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int i = 0; i < BATCH; ++i) {
          const int j = j0 + i * NT;
          yv[i] = j < len ? __ldcg(ys + (size_t)g * (P.k + 1) + j) : 0.f;
        }
#pragma unroll
        for (int i = 0; i < BATCH; ++i) zv[i] = fmaf(fast_exp2((yv[i] - my[g]) * LOG2E), inv_ly[g], zv[i]);
      }
#pragma unroll
      for (int i = 0; i < BATCH; ++i) zv[i] *= INV_G;
    }
#pragma unroll
    for (int i = 0; i < BATCH; ++i) {
      const int j = j0 + i * NT;
      if (j < len) {
        const float z = zv[i];
        const float a = av[i] + z;
        acc[j] = a;
        if (sc) sc[j] = z;
        if (pv[i] <= cutoff) {
          const unsigned long long key = evict_key(a, pv[i]);
          if (key < best) { best = key; best_j = j; }
        }
      }
    }
  }
  float z_new = 0.f;
#pragma unroll
  for (int g = 0; g < G; ++g) z_new = fmaf(fast_exp2((y_new[g] - my[g]) * LOG2E), inv_ly[g], z_new);
  if (G > 1) z_new *= INV_G;
  if (sc && tid == 0) sc[len] = z_new;
  evict_and_replace<D, NT, CPT>(P, u, len, best, best_j, z_new, kn_r, vn_r);
}

// The closing stage with many threads per unit (NT = 128 * min(G, 4) for G > 1 query heads on one cache, so that the heads are
// worked on side by side instead of one after the other; 512 for a single head with a long cache and few units): warp n merges the split statistics of head n and leaves them in shared
// memory; then every thread owns one (head, column) of the outputs and a few entries of the score update, all of whose
// loads are issued together.
template <int D, int NT, int G>
__device__ void combine_and_evict_group(const DecodeParams& P, int u, int len) {
  static_assert(NT >= 32 * G && NT >= D, "one warp per head for the statistics, one thread per column of the new row");
  __shared__ float sh_mx[G], sh_inv_lx[G], sh_my[G], sh_inv_ly[G], sh_xnew[G], sh_ynew[G];
  __shared__ float sh_w[G][MAX_SPLITS];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Hkv = P.H / G;
  const uint32_t b = (uint32_t)(u / Hkv), h0 = (uint32_t)(u % Hkv) * G, lh0 = (uint32_t)P.layer * P.H + h0;
  const __half* q = P.q + (size_t)u * G * D;
  const __half* kn = P.knew + (size_t)u * D;
  const __half* vn = P.vnew + (size_t)u * D;
  constexpr int PSTRIDE = 4 + D;
  constexpr float INV_G = 1.0f / (float)G;
  const float* part = P.partials + (size_t)u * P.splits * G * PSTRIDE;   // [split][head][4 + D]
  float* __restrict__ acc = P.acc + (size_t)u * P.k;
  int32_t* __restrict__ pos = P.pos + (size_t)u * P.k;
  const float* __restrict__ ys = P.y_scratch + (size_t)u * G * (P.k + 1);   // [head][k + 1]

  // ---- independent of the streaming kernel
  constexpr int BATCH = 4;
  float av[BATCH];
  int pv[BATCH];
#pragma unroll
  for (int i = 0; i < BATCH; ++i) {
    const int j = tid + i * NT;
    const bool in = j < len;
    av[i] = in ? acc[j] : 0.f;
    pv[i] = in ? pos[j] : 0x7fffffff;
  }
  for (int line = tid + (NT * BATCH) / 32; line * 32 < len; line += NT) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(acc + line * 32));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(pos + line * 32));
  }
  __half kn_r[1], vn_r[1];
  kn_r[0] = tid < D ? kn[tid] : __float2half(0.f);
  vn_r[0] = tid < D ? vn[tid] : __float2half(0.f);
  float x_new = 0.f, y_new = 0.f;
  if (warp < G) {   // warp n: head n's logit of the new token against itself
    float s = 0.f;
    for (int c = lane; c < D; c += 32) s = fmaf(__half2float(q[warp * D + c]), __half2float(kn[c]), s);
    x_new = warp_sum(s) * P.scale;  // bias(p, p) = 0
    if (lane == 0) y_new = (x_new + noise_for(P, b, lh0 + warp, (uint32_t)P.p, (uint32_t)P.p)) * P.inv_tau;
    y_new = __shfl_sync(0xffffffffu, y_new, 0);
  }

  asm volatile("griddepcontrol.wait;" ::: "memory");   // the streaming kernel has finished; its writes are visible

  if (warp < G) {
    const int g = warp;
    float4 ps0 = make_float4(-INFINITY, 0.f, -INFINITY, 0.f), ps1 = ps0;
    if (lane < P.splits) ps0 = __ldcg(reinterpret_cast<const float4*>(part + ((size_t)lane * G + g) * PSTRIDE));
    if (lane + 32 < P.splits) ps1 = __ldcg(reinterpret_cast<const float4*>(part + ((size_t)(lane + 32) * G + g) * PSTRIDE));
    const float mx = warp_max(fmaxf(x_new, fmaxf(ps0.y > 0.f ? ps0.x : -INFINITY, ps1.y > 0.f ? ps1.x : -INFINITY)));
    const float my = warp_max(fmaxf(y_new, fmaxf(ps0.w > 0.f ? ps0.z : -INFINITY, ps1.w > 0.f ? ps1.z : -INFINITY)));
    const float w0 = ps0.y > 0.f ? fast_exp2((ps0.x - mx) * LOG2E) : 0.f;
    const float w1 = ps1.y > 0.f ? fast_exp2((ps1.x - mx) * LOG2E) : 0.f;
    const float lx = fmaf(ps0.y, w0, ps1.y * w1);
    const float ly = (ps0.w > 0.f ? ps0.w * fast_exp2((ps0.z - my) * LOG2E) : 0.f) + (ps1.w > 0.f ? ps1.w * fast_exp2((ps1.z - my) * LOG2E) : 0.f);
    const float inv_lx = 1.f / (warp_sum(lx) + fast_exp2((x_new - mx) * LOG2E));
    const float inv_ly = 1.f / (warp_sum(ly) + fast_exp2((y_new - my) * LOG2E));
    sh_w[g][lane] = w0;
    sh_w[g][lane + 32] = w1;
    if (lane == 0) { sh_mx[g] = mx; sh_inv_lx[g] = inv_lx; sh_my[g] = my; sh_inv_ly[g] = inv_ly; sh_xnew[g] = x_new; sh_ynew[g] = y_new; }
  }
  __syncthreads();

  // ---- attention outputs (Eq. 1): one (head, column) per thread and round
  for (int idx = tid; idx < G * D; idx += NT) {
    const int g = idx / D, c = idx % D;
    float o = fast_exp2((sh_xnew[g] - sh_mx[g]) * LOG2E) * __half2float(vn[c]);
    const float* col = part + (size_t)g * PSTRIDE + 4 + c;
#pragma unroll 8
    for (int sp = 0; sp < P.splits; ++sp) o = fmaf(__ldcg(col + (size_t)sp * G * PSTRIDE), sh_w[g][sp], o);
    P.out[((size_t)u * G + g) * D + c] = __float2half_rn(o * sh_inv_lx[g]);
  }

  // ---- score (Eq. 11; the mean over the group's heads), accumulation and the eviction candidate
  float my[G], inv_ly[G];
#pragma unroll
  for (int g = 0; g < G; ++g) { my[g] = sh_my[g]; inv_ly[g] = sh_inv_ly[g] * INV_G; }
  float* __restrict__ sc = P.score_opt ? P.score_opt + (size_t)u * (P.k + 1) : nullptr;
  unsigned long long best = ~0ull;
  int best_j = -1;
  const int cutoff = P.p - P.w;  // entries with pos <= cutoff are outside the recent window
  for (int j0 = tid; j0 < len; j0 += NT * BATCH) {
    if (j0 != tid) {
#pragma unroll
      for (int i = 0; i < BATCH; ++i) {
        const int j = j0 + i * NT;
        const bool in = j < len;
        av[i] = in ? acc[j] : 0.f;
        pv[i] = in ? pos[j] : 0x7fffffff;
      }
    }
    float yv[G][BATCH];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
      for (int i = 0; i < BATCH; ++i) {
        const int j = j0 + i * NT;
        yv[g][i] = j < len ? __ldcg(ys + (size_t)g * (P.k + 1) + j) : 0.f;
      }
#pragma unroll
    for (int i = 0; i < BATCH; ++i) {
      const int j = j0 + i * NT;
      if (j < len) {
        float z = 0.f;
#pragma unroll
        for (int g = 0; g < G; ++g) z = fmaf(fast_exp2((yv[g][i] - my[g]) * LOG2E), inv_ly[g], z);
        const float a = av[i] + z;
        acc[j] = a;
        if (sc) sc[j] = z;
        if (pv[i] <= cutoff) {
          const unsigned long long key = evict_key(a, pv[i]);
          if (key < best) { best = key; best_j = j; }
        }
      }
    }
  }
  float z_new = 0.f;
#pragma unroll
  for (int g = 0; g < G; ++g) z_new = fmaf(fast_exp2((sh_ynew[g] - my[g]) * LOG2E), inv_ly[g], z_new);
  if (sc && tid == 0) sc[len] = z_new;
  evict_and_replace<D, NT, 1>(P, u, len, best, best_j, z_new, kn_r, vn_r);
}

// Warp-wide maximum in one instruction (f32 redux is an sm_100a feature).
__device__ __forceinline__ float warp_max_redux(float v) {
  float r;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
  return r;
}

// acc += sum over the 8 binary16 pairs of a 16-byte chunk; products are exact in binary32 and
// each fma rounds once (mixed-precision fma, an sm_100 instruction: no separate conversions).
__device__ __forceinline__ void dot8_mixed(float& acc, const uint4& kv, const uint4& qv) {
  const uint32_t kw[4] = {kv.x, kv.y, kv.z, kv.w};
  const uint32_t qw[4] = {qv.x, qv.y, qv.z, qv.w};
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    asm("{\n\t.reg .b16 kl, kh, ql, qh;\n\t"
        "mov.b32 {kl, kh}, %1;\n\t"
        "mov.b32 {ql, qh}, %2;\n\t"
        "fma.rn.f32.f16 %0, kl, ql, %0;\n\t"
        "fma.rn.f32.f16 %0, kh, qh, %0;\n\t}"
        : "+f"(acc) : "r"(kw[c]), "r"(qw[c]));
  }
}

// G query heads share the unit's cache: every K and V tile is fetched once and used for all G of them
// (G logits per row, G pairs of running softmaxes, G output rows).
// ROT: the cache holds keys without rotary embedding; the logit of a row gets the rotation by the distance between
// the query and that key (in positions or in places) from a table of cos / sin.
template <int D, int NW, int NSTAGE, bool NEWPOS, int G, bool ROT>
__global__ void __launch_bounds__(NW * 32) decode_kernel(const __grid_constant__ DecodeParams P) {
  constexpr int CPR = D / 8;          // 16-byte chunks per row
  constexpr int LPR = CPR;            // lanes that share one row in the value phase
  constexpr int NLD = LPR;            // 128-bit loads per lane and 32-row value tile
  constexpr int NT = NW * 32;
  constexpr int TILE_BYTES = TILE_ROWS * D * 2;
  constexpr int PSTRIDE = 4 + D;
  constexpr int ACC = G == 1 ? 4 : (G == 2 ? 2 : 1);   // independent accumulators per logit

  extern __shared__ __align__(128) unsigned char dyn_smem[];
  __shared__ float sh_m[NW][G], sh_l[NW][G], sh_my[NW][G], sh_ly[NW][G];
  __shared__ float sh_o[NW][G][D];
  __shared__ __align__(16) __half sh_q[G][D];

  // Both kernels of a step are launched with programmatic stream serialization: this grid's CTAs may become
  // resident while the kernel before it in the stream is draining, and wait here until that kernel has
  // completed (so nothing is read or written early); the closing kernel in turn may be scheduled as soon as
  // every CTA of this grid has started, and only prefetches until this grid has completed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int s = blockIdx.x, u = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sub = lane % LPR, grp = lane / LPR;
  const int len = P.len[u];
  if (len < 0 || len > P.k) {   // a damaged entry count: touch nothing of this unit, report it
    if (tid == 0 && s == 0) atomicExch(P.err, ERR_BOUNDS);
    return;
  }
  const int row_begin = s * P.tiles_per_split * TILE_ROWS;
  const int row_end = min(len, row_begin + P.tiles_per_split * TILE_ROWS);
  const int n_tiles = row_end > row_begin ? (row_end - row_begin + TILE_ROWS - 1) / TILE_ROWS : 0;
  const int my_tiles = n_tiles > warp ? (n_tiles - warp + NW - 1) / NW : 0;
  const __half* Ku = P.K + (size_t)u * P.k * D;
  const __half* Vu = P.V + (size_t)u * P.k * D;
  const int32_t* pos_u = P.pos + (size_t)u * P.k;
  const int Hkv = P.H / G;
  const uint32_t b = (uint32_t)(u / Hkv), h0 = (uint32_t)(u % Hkv) * G, lh0 = (uint32_t)P.layer * P.H + h0;
  float slope[G];
#pragma unroll
  for (int g = 0; g < G; ++g) slope[g] = (P.bias_mode == 1 && P.slopes) ? P.slopes[h0 + g] : 0.f;

  // warp-private ring of shared-memory slots filled by bulk async copies
  unsigned char* ring = dyn_smem + (size_t)warp * NSTAGE * TILE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(dyn_smem + (size_t)NW * NSTAGE * TILE_BYTES) + warp * NSTAGE;
  const int n_items = 2 * my_tiles;  // K tile, V tile, K tile, ...
  bool failed = false;
  auto tile_base_of = [&](int ti) { return row_begin + (warp + ti * NW) * TILE_ROWS; };
  auto issue = [&](int it) {
    if (lane == 0) {
      const int tb = tile_base_of(it >> 1);
      const uint32_t bytes = (uint32_t)min(TILE_ROWS, row_end - tb) * D * 2;
      const __half* src = ((it & 1) ? Vu : Ku) + (size_t)tb * D;
      uint64_t* bar = bars + (it % NSTAGE);
      mbar_expect_tx(bar, bytes);
      bulk_load(ring + (size_t)(it % NSTAGE) * TILE_BYTES, src, bytes, bar);
    }
  };
  if (lane == 0) {
    for (int i = 0; i < NSTAGE; ++i) mbar_init(bars + i, 1);
    mbar_fence_init();
  }
  __syncwarp();
  for (int it = 0; it < NSTAGE && it < n_items; ++it) issue(it);

  if (tid < G * D / 8)
    reinterpret_cast<uint4*>(&sh_q[0][0])[tid] = reinterpret_cast<const uint4*>(P.q + (size_t)u * G * D)[tid];
  if (G * D / 8 > NT && tid + NT < G * D / 8)   // eight heads of 256 features: a second round
    reinterpret_cast<uint4*>(&sh_q[0][0])[tid + NT] = reinterpret_cast<const uint4*>(P.q + (size_t)u * G * D)[tid + NT];
  __syncthreads();

  float m_x[G], l_x[G], m_y[G], l_y[G];  // l_* are per-lane partial sums
  float o[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m_x[g] = -INFINITY; l_x[g] = 0.f; m_y[g] = -INFINITY; l_y[g] = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) o[g][c] = 0.f;
  }
  int pos_next = 0;
  // "New Pos": the bias counts places within the cache; the current token stands at place len
  const int32_t* place_u = NEWPOS ? P.place + (size_t)u * P.k : nullptr;
  int place_next = 0;
  if (my_tiles > 0) {
    const int tb = tile_base_of(0);
    pos_next = (tb + lane < row_end) ? pos_u[tb + lane] : 0;
    if (NEWPOS) place_next = (tb + lane < row_end) ? place_u[tb + lane] : 0;
  }

  int consumed = 0;  // ring items whose slot has been released
  for (int ti = 0; ti < my_tiles; ++ti) {
    const int tile_base = tile_base_of(ti);
    const int rows = min(TILE_ROWS, row_end - tile_base);
    const int pj = pos_next;
    const int dist = NEWPOS ? len - place_next : P.p - pj;   // distance between the query and this key in the bias
    if (ti + 1 < my_tiles) {
      const int tb = tile_base_of(ti + 1);
      pos_next = (tb + lane < row_end) ? pos_u[tb + lane] : 0;
      if (NEWPOS) place_next = (tb + lane < row_end) ? place_u[tb + lane] : 0;
    }

    // ---- logits: lane r computes x of row tile_base + r (for each of the G heads).  Chunks are visited in a rotated
    //      order ((c + lane) mod CPR) so that the 16-byte reads of a quarter warp hit distinct banks.
    float x_mine[G];
    {
      const int it = 2 * ti;
      const bool ok = mbar_wait_bounded(bars + (it % NSTAGE), (uint32_t)((it / NSTAGE) & 1),
                                        ti == 0 ? P.first_wait_limit : DECODE_WAIT_LIMIT);
      if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
      const unsigned char* krow = ring + (size_t)(it % NSTAGE) * TILE_BYTES + (size_t)lane * D * 2;
      float part[G][ACC];
#pragma unroll
      for (int g = 0; g < G; ++g)
#pragma unroll
        for (int a = 0; a < ACC; ++a) part[g][a] = 0.f;
#pragma unroll
      for (int c0 = 0; c0 < CPR; c0 += 4) {
        uint4 kv[4];
        int ch[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          ch[j] = (c0 + j + lane) & (CPR - 1);
          kv[j] = *reinterpret_cast<const uint4*>(krow + ch[j] * 16);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const unsigned char* qb = reinterpret_cast<const unsigned char*>(&sh_q[g][0]);
          uint4 qv[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) qv[j] = *reinterpret_cast<const uint4*>(qb + ch[j] * 16);
#pragma unroll
          for (int j = 0; j < 4; ++j) dot8_mixed(part[g][j % ACC], kv[j], qv[j]);
        }
      }
#pragma unroll
      for (int g = 0; g < G; ++g)
        x_mine[g] = ACC == 4 ? (part[g][0] + part[g][1 % ACC]) + (part[g][2 % ACC] + part[g][3 % ACC])
                             : (ACC == 2 ? part[g][0] + part[g][1 % ACC] : part[g][0]);
      if (ROT) {
        // The sum above took the rotary features as they are.  With q and k as complex pairs (x_2i + i x_2i+1) the rotated
        // product of pair i is A c - B s, A + iB = q conj(k), (c, s) = cos / sin(dist theta_i): add A (c - 1) - B s.
        const int RC = P.rot_chunks;                       // 16-byte chunks (4 pairs) that carry the rotation
        const float2* tab = P.rope_tab + (size_t)(lane < rows ? dist : 0) * (RC * 4);
        for (int c = 0; c < RC; ++c) {
          const int ch = (c + lane) & (RC - 1);            // rotated order: distinct banks within a quarter warp
          const uint4 kv = *reinterpret_cast<const uint4*>(krow + ch * 16);
          const float4 t01 = __ldg(reinterpret_cast<const float4*>(tab + ch * 4));
          const float4 t23 = __ldg(reinterpret_cast<const float4*>(tab + ch * 4 + 2));
          const float cs[8] = {t01.x, t01.y, t01.z, t01.w, t23.x, t23.y, t23.z, t23.w};
          const uint32_t kw[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const uint4 qv = *reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned char*>(&sh_q[g][0]) + ch * 16);
            const uint32_t qw[4] = {qv.x, qv.y, qv.z, qv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 kf2 = __half22float2(*reinterpret_cast<const __half2*>(&kw[e]));
              const float2 qf2 = __half22float2(*reinterpret_cast<const __half2*>(&qw[e]));
              const float A = fmaf(qf2.x, kf2.x, qf2.y * kf2.y), B = fmaf(qf2.y, kf2.x, -qf2.x * kf2.y);
              x_mine[g] = fmaf(A, cs[2 * e] - 1.0f, fmaf(-B, cs[2 * e + 1], x_mine[g]));
            }
          }
        }
      }
      __syncwarp();
      consumed = it + 1;
      if (it + NSTAGE < n_items) issue(it + NSTAGE);
    }

    // ---- per-row work: bias, noise, the two running softmaxes (warp-common maxima, per-lane sums)
    const bool valid = lane < rows;
    uint32_t pr_pair[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float x = -INFINITY, y = -INFINITY;
      if (valid) {
        x = fmaf(x_mine[g], P.scale, -slope[g] * (float)dist);
        y = (x + noise_for(P, b, lh0 + g, (uint32_t)P.p, (uint32_t)pj)) * P.inv_tau;
        P.y_scratch[((size_t)u * G + g) * (P.k + 1) + tile_base + lane] = y;
      }
      const float mx_new = fmaxf(m_x[g], warp_max_redux(x));
      const float my_new = fmaxf(m_y[g], warp_max_redux(y));
      const float corr_x = fast_exp2((m_x[g] - mx_new) * LOG2E);   // 0 on the first tile (m_x = -inf)
      const float corr_y = fast_exp2((m_y[g] - my_new) * LOG2E);
      const float pr = valid ? fast_exp2((x - mx_new) * LOG2E) : 0.f;
      const float ey = valid ? fast_exp2((y - my_new) * LOG2E) : 0.f;
      const __half2 pr_h2 = __float2half2_rn(pr);
      pr_pair[g] = *reinterpret_cast<const uint32_t*>(&pr_h2);   // (p, p) as binary16, for the value phase
      l_x[g] = fmaf(l_x[g], corr_x, pr);
      l_y[g] = fmaf(l_y[g], corr_y, ey);
      m_x[g] = mx_new; m_y[g] = my_new;
#pragma unroll
      for (int c = 0; c < 8; ++c) o[g][c] *= corr_x;
    }

    // ---- value accumulation: LPR lanes share a row, each owns 8 columns
    {
      const int it = 2 * ti + 1;
      const bool ok = mbar_wait_bounded(bars + (it % NSTAGE), (uint32_t)((it / NSTAGE) & 1));
      if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
      const unsigned char* slot = ring + (size_t)(it % NSTAGE) * TILE_BYTES + sub * 16;
      constexpr int CH = NLD < 4 ? NLD : 4;
#pragma unroll
      for (int i0 = 0; i0 < NLD; i0 += CH) {
        uint4 vv[CH];
#pragma unroll
        for (int i = 0; i < CH; ++i) {
          const int r = grp * LPR + i0 + i;
          vv[i] = r < rows ? *reinterpret_cast<const uint4*>(slot + (size_t)r * D * 2) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
          uint32_t a[CH];
#pragma unroll
          for (int i = 0; i < CH; ++i) a[i] = __shfl_sync(0xffffffffu, pr_pair[g], grp * LPR + i0 + i);
#pragma unroll
          for (int i = 0; i < CH; ++i) axpy8(o[g], a[i], vv[i]);
        }
      }
      __syncwarp();
      consumed = it + 1;
      if (it + NSTAGE < n_items) issue(it + NSTAGE);
    }
  }

  if (failed) {
    // a copy did not land in time: flag it, then give every copy still in flight a second bounded wait
    if (lane == 0) atomicExch(P.err, ERR_TIMEOUT);
    const int issued = min(n_items, consumed + NSTAGE);
    for (int it = consumed; it < issued; ++it)
      (void)mbar_wait_bounded(bars + (it % NSTAGE), (uint32_t)((it / NSTAGE) & 1));
  }

  // ---- merge the lanes, then the warps of this CTA
#pragma unroll
  for (int g = 0; g < G; ++g) {
    l_x[g] = warp_sum(l_x[g]);
    l_y[g] = warp_sum(l_y[g]);
#pragma unroll
    for (int off = LPR; off < 32; off <<= 1) {
#pragma unroll
      for (int c = 0; c < 8; ++c) o[g][c] += __shfl_xor_sync(0xffffffffu, o[g][c], off);
    }
    if (grp == 0) {
#pragma unroll
      for (int c = 0; c < 8; ++c) sh_o[warp][g][sub * 8 + c] = o[g][c];
    }
    if (lane == 0) { sh_m[warp][g] = m_x[g]; sh_l[warp][g] = l_x[g]; sh_my[warp][g] = m_y[g]; sh_ly[warp][g] = l_y[g]; }
  }
  __syncthreads();
#pragma unroll
  for (int g = 0; g < G; ++g) {
    float* part = P.partials + (((size_t)u * P.splits + s) * G + g) * PSTRIDE;
    float M = -INFINITY, MY = -INFINITY;
#pragma unroll
    for (int wi = 0; wi < NW; ++wi) { M = fmaxf(M, sh_m[wi][g]); MY = fmaxf(MY, sh_my[wi][g]); }
    float sc[NW];
#pragma unroll
    for (int wi = 0; wi < NW; ++wi) sc[wi] = sh_l[wi][g] > 0.f ? fast_exp2((sh_m[wi][g] - M) * LOG2E) : 0.f;
    for (int c = tid; c < D; c += NT) {
      float acc_o = 0.f;
#pragma unroll
      for (int wi = 0; wi < NW; ++wi) acc_o = fmaf(sh_o[wi][g][c], sc[wi], acc_o);
      part[4 + c] = acc_o;
    }
    if (tid == 0) {
      float L = 0.f, LY = 0.f;
#pragma unroll
      for (int wi = 0; wi < NW; ++wi) {
        L = fmaf(sh_l[wi][g], sc[wi], L);
        if (sh_ly[wi][g] > 0.f) LY = fmaf(sh_ly[wi][g], fast_exp2((sh_my[wi][g] - MY) * LOG2E), LY);
      }
      part[0] = M; part[1] = L; part[2] = MY; part[3] = LY;
    }
  }
}

// One CTA per unit, launched behind the streaming kernel as its programmatic dependent.
inline bool close_is_wide(int units, int k) { return units <= 148 && k >= 2048; }
__host__ __device__ constexpr int close_threads(int d, int g) { return g == 1 ? 128 : (128 * (g < 4 ? g : 4) < d ? d : 128 * (g < 4 ? g : 4)); }

// Few units with long caches (one layer of a long-context model): 128 threads would walk a unit's thousands of entries
// in several dependent rounds while most SMs idle; 512 threads take them in one.
template <int D>
__global__ void __launch_bounds__(512, 1) decode_close_wide_kernel(const __grid_constant__ DecodeParams P) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int u = blockIdx.x;
  const int len = P.len[u];
  if (len < 0 || len > P.k) return;
  combine_and_evict_group<D, 512, 1>(P, u, len);
}

template <int D, int G>
__global__ void __launch_bounds__(close_threads(D, G), G == 1 ? 8 : (G == 8 ? 1 : 2)) decode_close_kernel(const __grid_constant__ DecodeParams P) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // lets the next kernel's CTAs queue up behind this grid
  const int u = blockIdx.x;
  const int len = P.len[u];
  if (len < 0 || len > P.k) return;   // reported by the streaming kernel; nothing of the unit is written
  if constexpr (G == 1) combine_and_evict<D, 128, 1>(P, u, len);
  else combine_and_evict_group<D, close_threads(D, G), G>(P, u, len);
}

// The closing kernel behind whichever streaming kernel ran, as its programmatic dependent.
template <int D, int G>
cudaError_t launch_close(const DecodeParams& P, int units, cudaStream_t stream) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)units);
  cfg.blockDim = dim3(close_threads(D, G));
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if constexpr (G == 1) {
    if (close_is_wide(units, P.k)) {
      cfg.blockDim = dim3(512);
      return cudaLaunchKernelEx(&cfg, decode_close_wide_kernel<D>, P);
    }
  }
  return cudaLaunchKernelEx(&cfg, decode_close_kernel<D, G>, P);
}

template <int D, int NW, int NSTAGE, int G, bool ROT = false>
cudaError_t launch_one(const DecodeParams& P, int units, cudaStream_t stream) {
  constexpr size_t smem = (size_t)NW * NSTAGE * (TILE_ROWS * D * 2) + (size_t)NW * NSTAGE * 8;
  auto kern = P.place ? decode_kernel<D, NW, NSTAGE, true, G, ROT> : decode_kernel<D, NW, NSTAGE, false, G, ROT>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  // Programmatic stream serialization on both launches: a kernel's CTAs may become resident while its
  // predecessor in the stream drains; griddepcontrol.wait inside each kernel keeps the ordering.
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)P.splits, (unsigned)units);
  cfg.blockDim = dim3(NW * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kern, P);
  if (e != cudaSuccess) return e;
  return launch_close<D, G>(P, units, stream);
}

// One CTA per unit: place[j] = #{i : pos[i] < pos[j]} (positions of a unit are distinct).
__global__ void __launch_bounds__(256) rebuild_place_kernel(const int32_t* __restrict__ pos, const int32_t* __restrict__ len,
                                                            int32_t* __restrict__ place, int k) {
  const int u = blockIdx.x;
  const int n = min(len[u], k);
  const int32_t* pu = pos + (size_t)u * k;
  for (int j = threadIdx.x; j < n; j += blockDim.x) {
    const int pj = pu[j];
    int c = 0;
    for (int i = 0; i < n; ++i) c += pu[i] < pj ? 1 : 0;
    place[(size_t)u * k + j] = c;
  }
}

}  // namespace

cudaError_t launch_rebuild_place(const int32_t* pos, const int32_t* len, int32_t* place, int k, int units,
                                 cudaStream_t stream) {
  rebuild_place_kernel<<<units, 256, 0, stream>>>(pos, len, place, k);
  return cudaGetLastError();
}

int decode_tile_rows() { return TILE_ROWS; }
int decode_max_splits() { return MAX_SPLITS; }

void decode_plan(int units, int budget_k, int requested, int* splits_out, int* tiles_per_split_out) {
  const int tiles = (budget_k + TILE_ROWS - 1) / TILE_ROWS;
  int splits = requested;
  if (splits <= 0) {
    // many units (inputs larger than L2, bandwidth-bound): about ten waves of the two resident CTAs per SM;
    // few units (cache-resident, latency-bound): one wave of CTAs that each stream a long run of tiles
    const int target_ctas = units >= 148 ? 148 * 20 : 148 * 2;
    splits = (target_ctas + units - 1) / units;
  }
  splits = std::max(1, std::min(splits, std::min(MAX_SPLITS, (tiles + 3) / 4)));
  int tps = (tiles + splits - 1) / splits;
  tps = (tps + 3) / 4 * 4;  // whole rounds of the CTA's four warps
  *splits_out = (tiles + tps - 1) / tps;
  *tiles_per_split_out = tps;
}

// Template arguments <D, NW, NSTAGE> of the streaming kernel launch_decode picks for a shape (one table for the
// launcher and for kf_describe_decode).
static void decode_variant(int head_dim, int tiles_per_split, int group, bool rotary, int* nw, int* nstage) {
  *nw = (head_dim == 128 && tiles_per_split >= 16 && group == 1 && !rotary) ? 5 : 4;
  *nstage = head_dim == 64 ? 4 : 2;
}

int decode_describe(char* buf, size_t n, int head_dim, int units, int budget_k, int splits, int tiles_per_split, bool new_pos,
                    int group, bool tensor_cores, bool rotary) {
  if (tensor_cores)
    return snprintf(buf, n, "decode_tc_kernel<%d,%d> + decode_close_kernel<%d,%d>; units=%d k=%d ctas=%d pieces=%d group=%d",
                    head_dim, group, head_dim, group, units, budget_k, tiles_per_split, splits, group);
  int nw = 4, nstage = 2;
  decode_variant(head_dim, tiles_per_split, group, rotary, &nw, &nstage);
  if (group == 1)
    return snprintf(buf, n, "decode_kernel<%d,%d,%d,%d%s> + %s<%d>; units=%d k=%d splits=%d tiles_per_split=%d group=1",
                    head_dim, nw, nstage, new_pos ? 1 : 0, rotary ? ",1,rot" : "", close_is_wide(units, budget_k) ? "decode_close_wide_kernel" : "decode_close_kernel",
                    head_dim, units, budget_k, splits, tiles_per_split);
  return snprintf(buf, n, "decode_kernel<%d,%d,%d,%d,%d> + decode_close_kernel<%d,%d>; units=%d k=%d splits=%d tiles_per_split=%d group=%d",
                  head_dim, nw, nstage, new_pos ? 1 : 0, group, head_dim, group, units, budget_k, splits, tiles_per_split, group);
}

bool decode_group_supported(int group) { return group == 1 || group == 2 || group == 4 || group == 8; }

namespace {
template <int G>
cudaError_t launch_group(const DecodeParams& P, int head_dim, int units, cudaStream_t stream) {
  int nw = 4, nstage = 2;
  decode_variant(head_dim, P.tiles_per_split, G, P.rope_tab != nullptr, &nw, &nstage);
  if (P.rope_tab) {
    switch (head_dim) {
      case 64: return launch_one<64, 4, 4, G, true>(P, units, stream);
      case 128: return launch_one<128, 4, 2, G, true>(P, units, stream);
      case 256: return launch_one<256, 4, 2, G, true>(P, units, stream);
      default: return cudaErrorInvalidValue;
    }
  }
  switch (head_dim) {
    case 64: return launch_one<64, 4, 4, G>(P, units, stream);
    case 128:
      // long items (bandwidth-bound workloads): five warps and 80 KB of ring per CTA, two CTAs per SM, measured best;
      // short items (few units, latency-bound): four warps, three CTAs per SM
      if constexpr (G == 1) {
        if (nw == 5) return launch_one<128, 5, 2, 1>(P, units, stream);
      }
      return launch_one<128, 4, 2, G>(P, units, stream);
    case 256: return launch_one<256, 4, 2, G>(P, units, stream);
    default: return cudaErrorInvalidValue;
  }
}
}  // namespace

cudaError_t launch_decode_close(const DecodeParams& P, int head_dim, int units, cudaStream_t stream) {
  if (head_dim != 128) return cudaErrorInvalidValue;   // the tensor-core streaming kernel is built for head_dim 128
  switch (P.group) {
    case 1: return launch_close<128, 1>(P, units, stream);
    case 2: return launch_close<128, 2>(P, units, stream);
    case 4: return launch_close<128, 4>(P, units, stream);
    case 8: return launch_close<128, 8>(P, units, stream);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_decode(const DecodeParams& P, int head_dim, int units, cudaStream_t stream) {
  if (P.splits < 1 || P.splits > MAX_SPLITS) return cudaErrorInvalidValue;
  switch (P.group) {
    case 1: return launch_group<1>(P, head_dim, units, stream);
    case 2: return launch_group<2>(P, head_dim, units, stream);
    case 4: return launch_group<4>(P, head_dim, units, stream);
    case 8: return launch_group<8>(P, head_dim, units, stream);
    default: return cudaErrorInvalidValue;
  }
}

// ---------------------------------------------------------------------------------------------
// Scratch for kf_decode_step_static: a fixed block of device memory that exists from the moment
// the library is loaded on a GPU until the process exits, so that the entry point never has to
// ask anyone for memory.  In host code `g_static_scratch` is only a handle for the symbol; its
// device address comes from cudaGetSymbolAddress, once per device.
__device__ __align__(256) static unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

namespace {
std::mutex g_static_mutex;
void* g_static_addr[64] = {};
}  // namespace

cudaError_t launch_decode_static(DecodeParams P, int head_dim, int units, size_t y_bytes, size_t partial_bytes,
                                 cudaStream_t stream) {
  if (y_bytes + partial_bytes + 256 > STATIC_SCRATCH_BYTES) return cudaErrorMemoryAllocation;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  void* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_addr[dev]) {
      void* ptr = nullptr;
      e = cudaGetSymbolAddress(&ptr, g_static_scratch);  // the current device's copy of the array
      if (e != cudaSuccess) return e;
      g_static_addr[dev] = ptr;
    }
    base = g_static_addr[dev];
  }
  unsigned char* b = static_cast<unsigned char*>(base);
  P.y_scratch = reinterpret_cast<float*>(b);
  P.partials = reinterpret_cast<float*>(b + y_bytes);
  P.err = reinterpret_cast<int*>(b + STATIC_SCRATCH_BYTES - 256);  // error word of the kernel's self-checks
  // nothing in the block has to start at zero: every word the closing kernel reads was written by this call's
  // streaming kernel first
  return launch_decode(P, head_dim, units, stream);
}

}  // namespace kf
