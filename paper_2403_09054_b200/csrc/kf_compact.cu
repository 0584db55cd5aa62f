// In-place compaction of a layer's cache into position order.
//
// Algorithm 1 describes the reduced cache as a subsequence of the token sequence (S_key and the recent
// window S_w, section 3.4).  The generation kernels keep it as an unordered set instead: the token that
// leaves is overwritten by the one that arrives, so after some steps the slots of a unit are a permutation
// of that subsequence.  This kernel applies the inverse permutation in place -- K rows, V rows, positions,
// scores -- so that slot s holds the entry with the s-th smallest position again, the layout the prompt
// phase produces.  Nothing later depends on the order (entries are identified by their positions); the
// compaction exists for callers that want the canonical layout: comparable state images, contiguous recent
// window, slot = place.
//
// Two launches.  compact_rank_kernel, one CTA per unit: the rank of every entry among the positions of its unit
// (counted in shared memory) is its destination slot.  compact_move_kernel, one warp per unit: the permutation is
// applied cycle by cycle, a row travelling through the registers of the warp (each lane holds 1/32 of a K row and
// of a V row), so no staging buffer is needed; the rows of the next destinations are requested in batches before
// any of them is overwritten, so the walk pays one memory latency per batch rather than per row, and a warp
// per unit keeps enough units resident to fill the memory system.
#include "kf_decode.cuh"

namespace kf {

namespace {

constexpr int CP_THREADS = 256;
constexpr int CP_MAX_K = 16384;   // one int32 per slot and warp in shared memory
__host__ __device__ constexpr int cp_ahead(int d) { return d == 256 ? 8 : 16; }   // rows in flight per warp

template <int D> struct RowPart;   // what one lane holds of a row of D binary16 values
template <> struct RowPart<64> { using type = uint32_t; };
template <> struct RowPart<128> { using type = uint2; };
template <> struct RowPart<256> { using type = uint4; };

__global__ void __launch_bounds__(CP_THREADS) compact_rank_kernel(const int32_t* __restrict__ pos, const int32_t* __restrict__ len,
                                                                  int32_t* __restrict__ dst, int k) {
  extern __shared__ __align__(16) int32_t cp_smem[];
  int32_t* spos = cp_smem;
  const int u = blockIdx.x, tid = threadIdx.x;
  const int n = min(len[u], k);
  const int32_t* pos_u = pos + (size_t)u * k;
  const int n4 = (n + 3) & ~3;   // padded with the largest value, which counts for nobody
  for (int j = tid; j < n4; j += CP_THREADS) spos[j] = j < n ? pos_u[j] : 0x7fffffff;
  __syncthreads();
  for (int j = tid; j < n; j += CP_THREADS) {
    const int pj = spos[j];
    int c = 0;
    for (int i = 0; i < n4; i += 4) {   // positions of a unit are distinct
      const int4 q = *reinterpret_cast<const int4*>(spos + i);
      c += (q.x < pj ? 1 : 0) + (q.y < pj ? 1 : 0) + (q.z < pj ? 1 : 0) + (q.w < pj ? 1 : 0);
    }
    dst[(size_t)u * k + j] = c;
  }
}

template <int D>
__global__ void compact_move_kernel(__half* __restrict__ K, __half* __restrict__ V, float* __restrict__ acc,
                                    int32_t* __restrict__ pos, const int32_t* __restrict__ len,
                                    const int32_t* __restrict__ dst, int32_t* __restrict__ place, int k, int units) {
  using Part = typename RowPart<D>::type;
  constexpr int CP_AHEAD = cp_ahead(D);
  extern __shared__ __align__(16) int32_t cp_smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int u = blockIdx.x * (blockDim.x >> 5) + warp;
  if (u >= units) return;
  int32_t* sdst = cp_smem + (size_t)warp * k;   // where the entry in each slot still has to go; s itself once it is home
  const int n = min(len[u], k);
  int32_t* pos_u = pos + (size_t)u * k;
  float* acc_u = acc + (size_t)u * k;
  Part* Ku = reinterpret_cast<Part*>(K + (size_t)u * k * D);
  Part* Vu = reinterpret_cast<Part*>(V + (size_t)u * k * D);
  for (int j = lane; j < n; j += 32) sdst[j] = dst[(size_t)u * k + j];
  __syncwarp();

  // The entry in slot j goes to slot sdst[j].  Every lane walks the same way, so there is no divergence.
  for (int s = 0; s < n; ++s) {
    if (sdst[s] == s) continue;
    Part ck = Ku[(size_t)s * 32 + lane], cv = Vu[(size_t)s * 32 + lane];
    float ca = acc_u[s];
    int cp = pos_u[s];
    int t = sdst[s];        // destination of the travelling entry
    bool done = false;
    while (!done) {
      int tt[CP_AHEAD];
      Part rk[CP_AHEAD], rv[CP_AHEAD];
      float ra[CP_AHEAD];
      int rp[CP_AHEAD];
      int cnt = 0;
#pragma unroll
      for (int i = 0; i < CP_AHEAD; ++i) {
        if (!done) {
          tt[i] = t;
          cnt = i + 1;
          if (t == s) done = true;        // the cycle closes at its first slot, whose entry already travels
          else t = sdst[t];
        }
      }
#pragma unroll
      for (int i = 0; i < CP_AHEAD; ++i) {
        if (i < cnt && tt[i] != s) {
          rk[i] = Ku[(size_t)tt[i] * 32 + lane];
          rv[i] = Vu[(size_t)tt[i] * 32 + lane];
          ra[i] = acc_u[tt[i]];
          rp[i] = pos_u[tt[i]];
        }
      }
      __syncwarp();   // every lane has read the scores and positions before lane 0 overwrites them
#pragma unroll
      for (int i = 0; i < CP_AHEAD; ++i) {
        if (i < cnt) {
          Ku[(size_t)tt[i] * 32 + lane] = ck;
          Vu[(size_t)tt[i] * 32 + lane] = cv;
          if (lane == 0) { pos_u[tt[i]] = cp; acc_u[tt[i]] = ca; sdst[tt[i]] = tt[i]; }
          if (tt[i] != s) { ck = rk[i]; cv = rv[i]; ca = ra[i]; cp = rp[i]; }
        }
      }
      __syncwarp();
    }
  }
  if (place) {
    int32_t* place_u = place + (size_t)u * k;
    for (int j = lane; j < n; j += 32) place_u[j] = j;
  }
}

}  // namespace

int compact_max_k() { return CP_MAX_K; }

cudaError_t launch_compact(__half* K, __half* V, float* acc, int32_t* pos, const int32_t* len, int32_t* place,
                           int32_t* dst_scratch, int k, int head_dim, int units, cudaStream_t stream) {
  if (k < 1 || k > CP_MAX_K || units < 1 || !dst_scratch) return cudaErrorInvalidValue;
  const size_t smem_rank = (size_t)((k + 3) & ~3) * 4;
  cudaError_t e = cudaSuccess;
  if (smem_rank > 48 * 1024) e = cudaFuncSetAttribute(compact_rank_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_rank);
  if (e != cudaSuccess) return e;
  compact_rank_kernel<<<units, CP_THREADS, smem_rank, stream>>>(pos, len, dst_scratch, k);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int wpc = k <= 4096 ? 4 : 1;                // warps (units) per CTA: at most 64 KB of destinations per CTA
  const size_t smem = (size_t)wpc * k * 4;
  auto go = [&](auto kern) -> cudaError_t {
    if (smem > 48 * 1024) {
      cudaError_t e2 = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e2 != cudaSuccess) return e2;
    }
    kern<<<(units + wpc - 1) / wpc, wpc * 32, smem, stream>>>(K, V, acc, pos, len, dst_scratch, place, k, units);
    return cudaGetLastError();
  };
  switch (head_dim) {
    case 64: return go(compact_move_kernel<64>);
    case 128: return go(compact_move_kernel<128>);
    case 256: return go(compact_move_kernel<256>);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace kf
