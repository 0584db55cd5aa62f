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
// One CTA per unit.  The rank of every entry (its destination) comes from counting smaller positions in shared
// memory; the permutation is then applied cycle by cycle, one warp per cycle, a row travelling through the
// registers of the warp (each lane holds 1/32 of a K row and of a V row), so no staging buffer is needed.
#include "kf_decode.cuh"

namespace kf {

namespace {

constexpr int CP_THREADS = 256;
constexpr int CP_MAX_K = 16384;   // two int32 per slot in shared memory: 128 KB

template <int D> struct RowPart;   // what one lane holds of a row of D binary16 values
template <> struct RowPart<64> { using type = uint32_t; };
template <> struct RowPart<128> { using type = uint2; };
template <> struct RowPart<256> { using type = uint4; };

template <int D>
__global__ void __launch_bounds__(CP_THREADS) compact_kernel(__half* __restrict__ K, __half* __restrict__ V,
                                                            float* __restrict__ acc, int32_t* __restrict__ pos,
                                                            const int32_t* __restrict__ len, int32_t* __restrict__ place,
                                                            int k) {
  using Part = typename RowPart<D>::type;
  extern __shared__ int32_t cp_smem[];
  int32_t* spos = cp_smem;        // positions as they are before the compaction
  int32_t* sdst = cp_smem + k;    // destination slot of every entry
  const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = min(len[u], k);
  int32_t* pos_u = pos + (size_t)u * k;
  float* acc_u = acc + (size_t)u * k;
  Part* Ku = reinterpret_cast<Part*>(K + (size_t)u * k * D);
  Part* Vu = reinterpret_cast<Part*>(V + (size_t)u * k * D);

  for (int j = tid; j < n; j += CP_THREADS) spos[j] = pos_u[j];
  __syncthreads();
  for (int j = tid; j < n; j += CP_THREADS) {
    const int pj = spos[j];
    int c = 0;
    for (int i = 0; i < n; ++i) c += spos[i] < pj ? 1 : 0;   // positions of a unit are distinct
    sdst[j] = c;
  }
  __syncthreads();

  // The entry in slot j goes to slot sdst[j].  A cycle of that permutation is rotated by the warp that finds
  // its smallest slot among the slots it visits; every lane walks the same way, so there is no divergence.
  for (int s = warp; s < n; s += CP_THREADS / 32) {
    if (sdst[s] == s) continue;
    bool leader = true;
    for (int j = sdst[s]; j != s; j = sdst[j])
      if (j < s) { leader = false; break; }
    if (!leader) continue;
    Part ck = Ku[(size_t)s * 32 + lane], cv = Vu[(size_t)s * 32 + lane];
    float ca = acc_u[s];
    int j = s;
    do {
      const int t = sdst[j];
      Part tk = ck, tv = cv;
      float ta = ca;
      if (t != s) {   // the entry that sits in the destination travels next
        tk = Ku[(size_t)t * 32 + lane];
        tv = Vu[(size_t)t * 32 + lane];
        ta = acc_u[t];
      }
      Ku[(size_t)t * 32 + lane] = ck;
      Vu[(size_t)t * 32 + lane] = cv;
      if (lane == 0) { pos_u[t] = spos[j]; acc_u[t] = ca; }
      ck = tk; cv = tv; ca = ta;
      j = t;
    } while (j != s);
  }
  if (place) {
    int32_t* place_u = place + (size_t)u * k;
    for (int j = tid; j < n; j += CP_THREADS) place_u[j] = j;
  }
}

}  // namespace

int compact_max_k() { return CP_MAX_K; }

cudaError_t launch_compact(__half* K, __half* V, float* acc, int32_t* pos, const int32_t* len, int32_t* place, int k,
                           int head_dim, int units, cudaStream_t stream) {
  if (k < 1 || k > CP_MAX_K || units < 1) return cudaErrorInvalidValue;
  const size_t smem = (size_t)k * 8;
  auto go = [&](auto kern) -> cudaError_t {
    if (smem > 48 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    kern<<<units, CP_THREADS, smem, stream>>>(K, V, acc, pos, len, place, k);
    return cudaGetLastError();
  };
  switch (head_dim) {
    case 64: return go(compact_kernel<64>);
    case 128: return go(compact_kernel<128>);
    case 256: return go(compact_kernel<256>);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace kf
