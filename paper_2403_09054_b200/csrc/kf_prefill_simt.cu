// Prompt-phase kernels (Algorithm 1, t = 0; section 3.4), CUDA-core version:
//   prefill_score_simt : causal logits -> Gumbel-softmax per query row -> column sums f_theta(j)
//   prefill_select     : keep w recent + top-(k-w) by f_theta (radix select, ties -> lower position)
//   prefill_gather     : copy the kept K/V rows, positions and scores into the k-slot cache
#include "kf_prefill.cuh"

#include <algorithm>

namespace kf {

namespace {

constexpr int BM = 64;   // query rows per CTA
constexpr int BN = 64;   // key columns per inner tile
constexpr int NTH = 256; // 16 x 16 threads, 4 x 4 logits each

__device__ __forceinline__ float prefill_noise(const PrefillParams& P, uint32_t b, uint32_t lh, uint32_t i, uint32_t j) {
  if (P.noise_mode == 0) return gumbel_from_word(noise_word(P.pk, b, lh, i, j));
  if (P.noise_mode == 2) return P.noise_const;
  if (P.noise_mode == 3)
    return fmaf(P.noise_sigma, gauss_from_words(noise_word(P.pk, b, lh, i, j), noise_word(P.pk, b | GAUSS_PLANE, lh, i, j)), P.noise_mu);
  return 0.f;
}

// Two sweeps over the key tiles of one 64-row query tile: the first finds each
// row's maximum and normaliser of (x + zeta) / tau, the second recomputes the
// logits and adds the normalised scores into the column sums.
template <int D>
__global__ void __launch_bounds__(NTH) prefill_score_simt(const __grid_constant__ PrefillParams P) {
  extern __shared__ float sm[];
  float* Qs = sm;                         // [BM][D + 1]
  float* Ks = sm + BM * (D + 1);          // [BN][D + 1]
  __shared__ float colsum[BN];
  const int it = blockIdx.x, u = blockIdx.y;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int n = P.n;
  const int i0 = it * BM;
  const uint32_t b = (uint32_t)(u / P.H), h = (uint32_t)(u % P.H), lh = (uint32_t)P.layer * P.H + h;
  const float slope = (P.bias_mode == 1 && P.slopes) ? P.slopes[h] : 0.f;
  const __half* Qu = P.Q + (size_t)u * n * D;
  const __half* Ku = P.K + (size_t)(u / P.group) * n * D;   // the keys of this query head's cache
  float* acc_u = P.acc_full + (size_t)u * n;

  for (int e = tid; e < BM * D; e += NTH) {
    const int r = e / D, c = e % D;
    Qs[r * (D + 1) + c] = (i0 + r < n) ? __half2float(Qu[(size_t)(i0 + r) * D + c]) : 0.f;
  }

  float row_m[4], row_l[4];
#pragma unroll
  for (int a = 0; a < 4; ++a) { row_m[a] = -INFINITY; row_l[a] = 0.f; }
  const int last_jt = min(it, (n - 1) / BN);

  for (int sweep = 0; sweep < 2; ++sweep) {
    for (int jt = 0; jt <= last_jt; ++jt) {
      const int j0 = jt * BN;
      __syncthreads();
      for (int e = tid; e < BN * D; e += NTH) {
        const int r = e / D, c = e % D;
        Ks[r * (D + 1) + c] = (j0 + r < n) ? __half2float(Ku[(size_t)(j0 + r) * D + c]) : 0.f;
      }
      if (sweep == 1 && tid < BN) colsum[tid] = 0.f;
      __syncthreads();
      float x[4][4];
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < 4; ++c) x[a][c] = 0.f;
      for (int dd = 0; dd < D; ++dd) {
        float qv[4], kv[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) qv[a] = Qs[(ty + 16 * a) * (D + 1) + dd];
#pragma unroll
        for (int c = 0; c < 4; ++c) kv[c] = Ks[(tx + 16 * c) * (D + 1) + dd];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int c = 0; c < 4; ++c) x[a][c] = fmaf(qv[a], kv[c], x[a][c]);
      }
      float csum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const int i = i0 + ty + 16 * a;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int j = j0 + tx + 16 * c;
          if (i < n && j <= i) {
            const float xv = fmaf(x[a][c], P.scale, -slope * (float)(i - j));
            const float y = (xv + prefill_noise(P, b, lh, (uint32_t)i, (uint32_t)j)) * P.inv_tau;
            if (sweep == 0) {
              const float mn = fmaxf(row_m[a], y);
              row_l[a] = row_l[a] * fast_exp2((row_m[a] - mn) * LOG2E) + fast_exp2((y - mn) * LOG2E);
              row_m[a] = mn;
            } else {
              csum[c] += fast_exp2((y - row_m[a]) * LOG2E) * row_l[a];  // row_l holds 1 / normaliser here
            }
          }
        }
      }
      if (sweep == 1) {
#pragma unroll
        for (int c = 0; c < 4; ++c) atomicAdd(&colsum[tx + 16 * c], csum[c]);
        __syncthreads();
        if (tid < BN && j0 + tid < n && j0 + tid <= i0 + BM - 1) atomicAdd(acc_u + j0 + tid, colsum[tid]);
      }
    }
    if (sweep == 0) {
      // merge the 16 threads that share a row (they are 16 consecutive lanes)
#pragma unroll
      for (int a = 0; a < 4; ++a) {
#pragma unroll
        for (int off = 8; off > 0; off >>= 1) {
          const float om = __shfl_xor_sync(0xffffffffu, row_m[a], off);
          const float ol = __shfl_xor_sync(0xffffffffu, row_l[a], off);
          const float mn = fmaxf(row_m[a], om);
          const float sa = row_l[a] > 0.f ? row_l[a] * fast_exp2((row_m[a] - mn) * LOG2E) : 0.f;
          const float sb = ol > 0.f ? ol * fast_exp2((om - mn) * LOG2E) : 0.f;
          row_m[a] = mn;
          row_l[a] = sa + sb;
        }
        row_l[a] = row_l[a] > 0.f ? 1.f / row_l[a] : 0.f;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Selection: one CTA per unit.  Candidates are positions j < n - w; the k - w with the largest
// f_theta stay (ties: lower position).  An 8-bit-per-pass radix select over the score bits
// (non-negative binary32 values order like unsigned integers) finds the threshold score; an
// ordered block scan then emits the kept positions in ascending order.
constexpr int SEL_T = 256;

__global__ void __launch_bounds__(SEL_T) prefill_select(const __grid_constant__ SelectParams P) {
  __shared__ unsigned int hist[256];
  __shared__ unsigned int sh_prefix, sh_remaining;
  __shared__ unsigned int warp_a[SEL_T / 32], warp_b[SEL_T / 32];
  const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = P.n, k = P.k, w = P.w;
  const float* acc = P.acc_full + (size_t)u * n;
  int32_t* idx = P.idx + (size_t)u * k;

  if (n <= k) {
    for (int j = tid; j < k; j += SEL_T) idx[j] = j < n ? j : -1;
    if (tid == 0) P.len[u] = n;
    return;
  }
  const int n_cand = n - w;
  const int r = k - w;  // candidates to keep; n_cand > r because n > k
  unsigned int thresh = 0xFFFFFFFFu, need_eq = 0;
  if (r > 0) {
    if (tid == 0) { sh_prefix = 0u; sh_remaining = (unsigned)r; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      hist[tid] = 0u;
      __syncthreads();
      const unsigned int prefix = sh_prefix;
      const unsigned int mask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
      for (int j = tid; j < n_cand; j += SEL_T) {
        const unsigned int bits = __float_as_uint(acc[j]);
        if ((bits & mask) == prefix) atomicAdd(&hist[(bits >> shift) & 0xFFu], 1u);
      }
      __syncthreads();
      // the digit where the count of larger-or-equal digits first reaches `remaining`: thread d holds bin d
      // and the suffix sum above[d] = sum of the bins d' > d (warp shuffles, then the warps' totals)
      const unsigned int remaining = sh_remaining;
      const unsigned int mine = hist[tid];
      unsigned int incl = mine;   // bins tid .. end of this warp
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const unsigned int other = __shfl_down_sync(0xffffffffu, incl, off);
        if (lane + off < 32) incl += other;
      }
      if (lane == 0) warp_a[warp] = incl;
      __syncthreads();
      unsigned int above = incl - mine;
      for (int wi = warp + 1; wi < SEL_T / 32; ++wi) above += warp_a[wi];
      if (above < remaining && above + mine >= remaining) {   // exactly one thread
        sh_prefix = prefix | ((unsigned)tid << shift);
        sh_remaining = remaining - above;
      }
      __syncthreads();
    }
    thresh = sh_prefix;      // score bits of the r-th largest candidate
    need_eq = sh_remaining;  // how many candidates equal to it are kept (lowest positions first)
  }
  unsigned int base_eq = 0u, base_out = 0u;   // every thread keeps the same running totals
  __syncthreads();

  for (int j0 = 0; j0 < n; j0 += SEL_T) {
    const int j = j0 + tid;
    bool keep = false, is_eq = false;
    if (j < n) {
      if (j >= n_cand) keep = true;
      else if (r > 0) {
        const unsigned int bits = __float_as_uint(acc[j]);
        keep = bits > thresh;
        is_eq = bits == thresh;
      }
    }
    // ordered rank among the equal-score candidates
    const unsigned int eq_ballot = __ballot_sync(0xffffffffu, is_eq);
    if (lane == 0) warp_a[warp] = __popc(eq_ballot);
    __syncthreads();
    unsigned int eq_before = base_eq, eq_total = 0;
    for (int wi = 0; wi < SEL_T / 32; ++wi) {
      if (wi < warp) eq_before += warp_a[wi];
      eq_total += warp_a[wi];
    }
    eq_before += __popc(eq_ballot & ((1u << lane) - 1u));
    if (is_eq && eq_before < need_eq) keep = true;
    const unsigned int keep_ballot = __ballot_sync(0xffffffffu, keep);
    if (lane == 0) warp_b[warp] = __popc(keep_ballot);
    __syncthreads();
    unsigned int out_before = base_out, out_total = 0;
    for (int wi = 0; wi < SEL_T / 32; ++wi) {
      if (wi < warp) out_before += warp_b[wi];
      out_total += warp_b[wi];
    }
    out_before += __popc(keep_ballot & ((1u << lane) - 1u));
    if (keep) {
      if (out_before < (unsigned)k) idx[out_before] = j;
      else atomicExch(P.err, ERR_BOUNDS);
    }
    base_eq += eq_total;
    base_out += out_total;
  }
  if (tid == 0) {
    if (base_out != (unsigned)k) atomicExch(P.err, ERR_BOUNDS);
    P.len[u] = k;
  }
}

// ---------------------------------------------------------------------------------------------
// Gather: slot s of unit u receives prompt row idx[u][s] (K, V, position, score); unused slots
// are cleared.  One warp per slot.
template <int D>
__global__ void __launch_bounds__(128) prefill_gather(const __grid_constant__ GatherParams P) {
  const int u = blockIdx.y;
  const int slot = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (slot >= P.k) return;
  const int j = P.idx[(size_t)u * P.k + slot];
  if (P.place && lane == 0) P.place[(size_t)u * P.k + slot] = slot;
  uint4* Kd = reinterpret_cast<uint4*>(P.Kc + ((size_t)u * P.k + slot) * D);
  uint4* Vd = reinterpret_cast<uint4*>(P.Vc + ((size_t)u * P.k + slot) * D);
  if (j < 0 || j >= P.n) {
    for (int c = lane; c < D / 8; c += 32) { Kd[c] = make_uint4(0, 0, 0, 0); Vd[c] = make_uint4(0, 0, 0, 0); }
    if (lane == 0) { P.pos[(size_t)u * P.k + slot] = -1; P.acc[(size_t)u * P.k + slot] = 0.f; }
    return;
  }
  const uint4* Ks = reinterpret_cast<const uint4*>(P.K + ((size_t)u * P.n + j) * D);
  const uint4* Vs = reinterpret_cast<const uint4*>(P.V + ((size_t)u * P.n + j) * D);
  for (int c = lane; c < D / 8; c += 32) { Kd[c] = Ks[c]; Vd[c] = Vs[c]; }
  if (lane == 0) {
    P.pos[(size_t)u * P.k + slot] = j;
    P.acc[(size_t)u * P.k + slot] = P.acc_full[(size_t)u * P.n + j];
  }
}

}  // namespace

cudaError_t launch_prefill_score_simt(const PrefillParams& P, int head_dim, int units, cudaStream_t stream) {
  dim3 grid((unsigned)((P.n + BM - 1) / BM), (unsigned)units);
  const size_t smem = (size_t)(BM + BN) * (head_dim + 1) * sizeof(float);
  cudaError_t e = cudaSuccess;
  switch (head_dim) {
    case 64:
      e = cudaFuncSetAttribute(prefill_score_simt<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      prefill_score_simt<64><<<grid, NTH, smem, stream>>>(P);
      break;
    case 128:
      e = cudaFuncSetAttribute(prefill_score_simt<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      prefill_score_simt<128><<<grid, NTH, smem, stream>>>(P);
      break;
    case 256:
      e = cudaFuncSetAttribute(prefill_score_simt<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      prefill_score_simt<256><<<grid, NTH, smem, stream>>>(P);
      break;
    default:
      return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

namespace {
__global__ void __launch_bounds__(256) group_mean_kernel(const float* __restrict__ src, float* __restrict__ dst, int group, int n) {
  const int c = blockIdx.y;
  const float inv = 1.0f / (float)group;
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < n; j += gridDim.x * blockDim.x) {
    float s = 0.f;
    for (int r = 0; r < group; ++r) s += src[((size_t)c * group + r) * n + j];
    dst[(size_t)c * n + j] = s * inv;
  }
}
}  // namespace

cudaError_t launch_group_mean(const float* src, float* dst, int caches, int group, int n, cudaStream_t stream) {
  dim3 grid((unsigned)std::min((n + 255) / 256, 64), (unsigned)caches);
  group_mean_kernel<<<grid, 256, 0, stream>>>(src, dst, group, n);
  return cudaGetLastError();
}

cudaError_t launch_prefill_select(const SelectParams& P, int units, cudaStream_t stream) {
  prefill_select<<<units, SEL_T, 0, stream>>>(P);
  return cudaGetLastError();
}

cudaError_t launch_prefill_gather(const GatherParams& P, int head_dim, int units, cudaStream_t stream) {
  dim3 grid((unsigned)((P.k + 3) / 4), (unsigned)units);
  switch (head_dim) {
    case 64: prefill_gather<64><<<grid, 128, 0, stream>>>(P); break;
    case 128: prefill_gather<128><<<grid, 128, 0, stream>>>(P); break;
    case 256: prefill_gather<256><<<grid, 128, 0, stream>>>(P); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace kf
