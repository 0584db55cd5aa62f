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
// (a sort in shared memory, then a bisection per entry) is its destination slot.  compact_move_kernel, one CTA of eight warps per unit:
// what the generation steps leave behind -- old entries that only have to move down, a few new ones that belong at the
// end -- is carried over in ascending chunks by the whole CTA (see "the ordered shift" in the kernel); any other
// permutation is applied cycle by cycle, a row travelling through the registers of a warp (each lane holds 1/32 of a
// K row and of a V row), so no staging buffer is needed.  Long cycles are cut into segments that the warps walk at
// the same time (see the kernel), and within a segment the rows of the next destinations are requested in batches
// before any of them is overwritten, so a walk pays one memory latency per batch rather than per row.
#include "kf_decode.cuh"

namespace kf {

namespace {

constexpr int CP_THREADS = 256;
constexpr int CP_MAX_K = 16384;   // one int32 per slot in shared memory
__host__ __device__ constexpr int cp_ahead(int d) { return d == 256 ? 8 : 16; }   // rows in flight per warp

template <int D> struct RowPart;   // what one lane holds of a row of D binary16 values
template <> struct RowPart<64> { using type = uint32_t; };
template <> struct RowPart<128> { using type = uint2; };
template <> struct RowPart<256> { using type = uint4; };

constexpr int CP_FAST_N = 4096;    // entries up to which the nearly-sorted shortcut of the rank kernel has its shared memory
constexpr int CP_FAST_OUT = 128;   // out-of-order entries it handles

// dst[j] = number of the unit's positions smaller than pos[j] (positions of a unit are distinct).
// Shortcut for what generation steps leave behind: call an entry "in order" if every later slot holds a larger
// position (a suffix minimum tells).  The in-order entries form an ascending run; if the others are few (the tokens
// that arrived since the last compaction) every rank is a prefix count within the run plus a handful of comparisons
// with the others, and the others find their place in the run by bisection.  Otherwise: the positions are sorted in
// shared memory (bitonic network, padded to a power of two with the largest value) and every entry finds its own
// position in the sorted array by bisection.
__global__ void __launch_bounds__(CP_THREADS) compact_rank_kernel(const int32_t* __restrict__ pos, const int32_t* __restrict__ len,
                                                                  int32_t* __restrict__ dst, int k, int n_pow2) {
  extern __shared__ __align__(16) int32_t cp_smem[];
  int32_t* key = cp_smem;
  const int u = blockIdx.x, tid = threadIdx.x;
  const int n = min(len[u], k);
  const int32_t* pos_u = pos + (size_t)u * k;
  if (n <= CP_FAST_N && n > 0) {
    __shared__ int32_t red[CP_THREADS];
    __shared__ int32_t opos[CP_FAST_OUT], oidx[CP_FAST_OUT];
    __shared__ int s_out;
    int32_t* run = key + n;          // positions of the in-order entries, ascending
    int32_t* code = run + n;         // per slot: index within the run, or -1
    const int per = (n + CP_THREADS - 1) / CP_THREADS;
    const int lo = min(n, tid * per), hi = min(n, lo + per);
    for (int j = tid; j < n; j += CP_THREADS) key[j] = pos_u[j];
    if (tid == 0) s_out = 0;
    __syncthreads();
    int mn = 0x7fffffff;
    for (int j = lo; j < hi; ++j) mn = min(mn, key[j]);
    red[tid] = mn;
    __syncthreads();
    // smallest position in the slots behind this thread's range; how many in-order entries this range holds
    int behind = 0x7fffffff;
    for (int t = tid + 1; t < CP_THREADS; ++t) behind = min(behind, red[t]);
    int running = behind, mine = 0;
    for (int j = hi - 1; j >= lo; --j) {
      const int pj = key[j];
      const bool in_order = pj < running;
      code[j] = in_order ? 0 : -1;
      mine += in_order ? 1 : 0;
      running = min(running, pj);
    }
    __syncthreads();                 // everybody has read red[]
    red[tid] = mine;
    __syncthreads();
    int base = 0;
    for (int t = 0; t < tid; ++t) base += red[t];
    for (int j = lo; j < hi; ++j) {
      if (code[j] == 0) {
        code[j] = base;
        run[base++] = key[j];
      } else {
        const int at = atomicAdd(&s_out, 1);
        if (at < CP_FAST_OUT) { opos[at] = key[j]; oidx[at] = j; }
      }
    }
    __syncthreads();
    const int m = s_out, n_run = n - m;
    if (m <= CP_FAST_OUT) {          // (every thread reads the same count)
      for (int j = tid; j < n; j += CP_THREADS) {
        const int cj = code[j];
        if (cj >= 0) {
          const int pj = key[j];
          int below = 0;
          for (int o = 0; o < m; ++o) below += opos[o] < pj ? 1 : 0;
          dst[(size_t)u * k + j] = cj + below;
        }
      }
      for (int o = tid; o < m; o += CP_THREADS) {
        const int p = opos[o];
        int a = 0, b = n_run;        // first index of the run whose position is not below p
        while (a < b) {
          const int mid = (a + b) >> 1;
          if (run[mid] < p) a = mid + 1; else b = mid;
        }
        int below = 0;
        for (int o2 = 0; o2 < m; ++o2) below += opos[o2] < p ? 1 : 0;
        dst[(size_t)u * k + oidx[o]] = a + below;
      }
      return;
    }
    __syncthreads();                 // too many entries out of order: the general way, from the start
  }
  int np = 1;
  while (np < n) np <<= 1;          // the network only has to cover this unit's entries (np <= n_pow2)
  for (int j = tid; j < np; j += CP_THREADS) key[j] = j < n ? pos_u[j] : 0x7fffffff;
  for (int size = 2; size <= np; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      __syncthreads();
      for (int p = tid; p < (np >> 1); p += CP_THREADS) {
        const int i = ((p & ~(stride - 1)) << 1) | (p & (stride - 1));   // lower index of the pair
        const int j = i | stride;
        const bool up = (i & size) == 0;
        const int a = key[i], b = key[j];
        if ((a > b) == up) { key[i] = b; key[j] = a; }
      }
    }
  }
  __syncthreads();
  for (int j = tid; j < n; j += CP_THREADS) {
    const int pj = pos_u[j];
    int lo = 0, hi = n;             // first index whose key is not below pj
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (key[mid] < pj) lo = mid + 1; else hi = mid;
    }
    dst[(size_t)u * k + j] = lo;
  }
  (void)n_pow2;
}

// One CTA of CP_WARPS (8 or 16) warps per unit.  A cycle of the permutation is cut at "boundary" slots: a segment starts at a
// boundary slot and follows the cycle up to, and including the write into, the next boundary slot.  In every round
// the CTA picks up to cp_heads(D) boundary slots among the entries that are not home yet and copies their entries
// (rows, score, position) into shared memory; after one barrier the segments are independent -- a slot inside a
// segment is read and written by that segment's warp only, and the boundary slot a segment ends in has been saved --
// so the warps take segments from a common counter and walk them at the same time, each with the rows of its next
// destinations requested in batches.  Every cycle that contains a boundary slot is finished in that round.  The first
// rounds pick boundary slots by a hash of the slot number, so that a long cycle is cut into many segments (a regular
// choice such as every 64th slot can miss whole cycles of a regular permutation, e.g. the shift by two that two
// evictions leave behind); the later rounds take whatever is left, until every entry is home.
constexpr int CP_FLAG = 1 << 30;   // marks a boundary slot in the shared-memory copy of the permutation
__host__ __device__ constexpr int cp_heads(int d) { return d == 256 ? 32 : 64; }   // boundary slots per round (32 KB of rows)

// CP_WARPS = 8 with two CTAs per SM when there are units enough to fill the SMs twice over, 16 otherwise.
template <int D, int CP_WARPS>
__global__ void __launch_bounds__(CP_WARPS * 32, CP_WARPS == 8 ? 2 : 1) compact_move_kernel(__half* __restrict__ K, __half* __restrict__ V, float* __restrict__ acc,
                                                                        int32_t* __restrict__ pos, const int32_t* __restrict__ len,
                                                                        const int32_t* __restrict__ dst, int32_t* __restrict__ place, int k) {
  using Part = typename RowPart<D>::type;
  constexpr int CP_AHEAD = cp_ahead(D);
  constexpr int NH = cp_heads(D);
  extern __shared__ __align__(16) int32_t cp_smem[];
  Part* head_k = reinterpret_cast<Part*>(cp_smem);          // [NH][32] the boundary entries' K rows, one part per lane
  Part* head_v = head_k + NH * 32;
  float* head_a = reinterpret_cast<float*>(head_v + NH * 32);
  int32_t* head_p = reinterpret_cast<int32_t*>(head_a + NH);
  int32_t* head_t = head_p + NH;                            // where the boundary entry has to go
  int32_t* head_b = head_t + NH;                            // the boundary slot itself
  int32_t* sdst = head_b + NH;   // [k] where the entry in each slot still has to go; s itself once it is home
  __shared__ int sb_count, sb_next;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int u = blockIdx.x;
  const int n = min(len[u], k);
  int32_t* pos_u = pos + (size_t)u * k;
  float* acc_u = acc + (size_t)u * k;
  Part* Ku = reinterpret_cast<Part*>(K + (size_t)u * k * D);
  Part* Vu = reinterpret_cast<Part*>(V + (size_t)u * k * D);
  for (int j = threadIdx.x; j < n; j += CP_WARPS * 32) sdst[j] = dst[(size_t)u * k + j];
  const uint32_t n_buckets = (uint32_t)max(1, n / (NH * 3 / 4));   // a hashed round expects 3/4 of the head buffer
  const int hashed_rounds = max(1, min(8, n / (NH * 12)));          // in all about one slot in sixteen, spread by the hash

  // Walks from the entry (ck, cv, ca, cp) that has to go to slot t: writes it there, picks up what was there, and so on,
  // until the walk has written into a boundary slot (whose entry is in the head buffer).
  auto walk = [&](int t, Part ck, Part cv, float ca, int cp) {
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
          const int v = sdst[t];
          if (v & CP_FLAG) done = true;
          else t = v;
        }
      }
      const int last = done ? cnt - 1 : cnt;   // the slot the walk ends in is written but not picked up
#pragma unroll
      for (int i = 0; i < CP_AHEAD; ++i) {
        if (i < last) {
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
          if (i < last) { ck = rk[i]; cv = rv[i]; ca = ra[i]; cp = rp[i]; }
        }
      }
      __syncwarp();
    }
  };

  // ---- The ordered shift: the case the generation steps leave behind.  Entries that were in the cache at the last
  // compaction have not moved, so they are still in position order and only have to move DOWN past the slots of the
  // entries that left; the tokens that arrived since sit in those slots and belong at the end.  Whenever the entries
  // that have to move UP fit the head buffer, they are set aside there, every entry that moves down is carried over in
  // ascending chunks by the whole CTA (rows of a chunk read, one barrier, rows written: a destination lies below its
  // source, so what it holds was read in this chunk or an earlier one, or has been set aside), and the entries set
  // aside are written last.  No cycle is followed and no load waits for another.  Any other permutation (an imported
  // state, say) goes through the rounds below.
  bool shifted = false;
  {
    constexpr int R = D == 256 ? 4 : 8;   // rows a warp carries per chunk
    if (threadIdx.x == 0) sb_count = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < n; j += CP_WARPS * 32) {
      const int t = sdst[j];
      if (t > j) {
        const int at = atomicAdd(&sb_count, 1);
        if (at < NH) { head_b[at] = j; head_t[at] = t; }
      }
    }
    __syncthreads();
    const int nup = sb_count;             // (every thread reads the same count)
    if (nup <= NH) {
      shifted = true;
      for (int i = warp; i < nup; i += CP_WARPS) {
        const int b = head_b[i];
        head_k[i * 32 + lane] = Ku[(size_t)b * 32 + lane];
        head_v[i * 32 + lane] = Vu[(size_t)b * 32 + lane];
        if (lane == 0) { head_a[i] = acc_u[b]; head_p[i] = pos_u[b]; }
      }
      __syncthreads();
      for (int c0 = 0; c0 < n; c0 += CP_WARPS * R) {
        int tt[R];
        Part rk[R], rv[R];
        float ra[R];
        int rp[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
          const int sl = c0 + warp * R + i;
          const int t = sl < n ? sdst[sl] : sl;
          tt[i] = t < sl ? t : -1;
          if (tt[i] >= 0) {
            rk[i] = Ku[(size_t)sl * 32 + lane];
            rv[i] = Vu[(size_t)sl * 32 + lane];
            ra[i] = acc_u[sl];
            rp[i] = pos_u[sl];
          }
        }
        __syncthreads();   // every row of the chunk is in registers before any slot of it is overwritten
#pragma unroll
        for (int i = 0; i < R; ++i) {
          if (tt[i] >= 0) {
            Ku[(size_t)tt[i] * 32 + lane] = rk[i];
            Vu[(size_t)tt[i] * 32 + lane] = rv[i];
            if (lane == 0) { pos_u[tt[i]] = rp[i]; acc_u[tt[i]] = ra[i]; }
          }
        }
      }
      __syncthreads();
      for (int i = warp; i < nup; i += CP_WARPS) {
        const int t = head_t[i];
        Ku[(size_t)t * 32 + lane] = head_k[i * 32 + lane];
        Vu[(size_t)t * 32 + lane] = head_v[i * 32 + lane];
        if (lane == 0) { pos_u[t] = head_p[i]; acc_u[t] = head_a[i]; }
      }
    }
  }

  if (!shifted) {
    for (int r = 0;; ++r) {
      // ---- this round's boundary slots among the entries that are not home yet
      if (threadIdx.x == 0) { sb_count = 0; sb_next = 0; }
      __syncthreads();
      const bool hashed = r < hashed_rounds;
      for (int j = threadIdx.x; j < n; j += CP_WARPS * 32) {
        if (sdst[j] != j && (!hashed || ((uint32_t)j * 0x9E3779B1u >> 8) % n_buckets == (uint32_t)r)) {
          const int at = atomicAdd(&sb_count, 1);
          if (at < NH) { head_b[at] = j; head_t[at] = sdst[j]; sdst[j] |= CP_FLAG; }
        }
      }
      __syncthreads();
      const int nb = min(sb_count, NH);   // (every thread reads the same count)
      if (nb == 0) {
        if (hashed) continue;
        break;       // an unrestricted round found nothing: every entry is home
      }
      // ---- their entries into shared memory, before anything is overwritten
      for (int i = warp; i < nb; i += CP_WARPS) {
        const int b = head_b[i];
        head_k[i * 32 + lane] = Ku[(size_t)b * 32 + lane];
        head_v[i * 32 + lane] = Vu[(size_t)b * 32 + lane];
        if (lane == 0) { head_a[i] = acc_u[b]; head_p[i] = pos_u[b]; }
      }
      __syncthreads();
      // ---- the segments, first come first served
      for (;;) {
        int i = 0;
        if (lane == 0) i = atomicAdd(&sb_next, 1);
        i = __shfl_sync(0xffffffffu, i, 0);
        if (i >= nb) break;
        walk(head_t[i], head_k[i * 32 + lane], head_v[i * 32 + lane], head_a[i], head_p[i]);
      }
      __syncthreads();
    }
  }
  if (place) {
    int32_t* place_u = place + (size_t)u * k;
    for (int j = threadIdx.x; j < n; j += CP_WARPS * 32) place_u[j] = j;
  }
}

}  // namespace

int compact_max_k() { return CP_MAX_K; }

cudaError_t launch_compact(__half* K, __half* V, float* acc, int32_t* pos, const int32_t* len, int32_t* place,
                           int32_t* dst_scratch, int k, int head_dim, int units, cudaStream_t stream) {
  if (k < 1 || k > CP_MAX_K || units < 1 || !dst_scratch) return cudaErrorInvalidValue;
  int n_pow2 = 1;
  while (n_pow2 < k) n_pow2 <<= 1;
  const size_t smem_rank = std::max((size_t)n_pow2 * 4, (size_t)3 * std::min(k, CP_FAST_N) * 4);   // the sort, or the shortcut's three arrays
  cudaError_t e = cudaSuccess;
  // (the kernel also has 2 KB of static shared memory: ask as soon as the sum could pass the 48 KB every kernel may have)
  if (smem_rank > 40 * 1024) e = cudaFuncSetAttribute(compact_rank_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_rank);
  if (e != cudaSuccess) return e;
  compact_rank_kernel<<<units, CP_THREADS, smem_rank, stream>>>(pos, len, dst_scratch, k, n_pow2);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  // the head buffer (rows, scores, positions, destinations, slots of a round's boundary entries), then one destination per slot
  const size_t smem = (size_t)cp_heads(head_dim) * ((size_t)head_dim * 4 + 16) + (size_t)k * 4;
  const bool many = units >= 2 * 148;
  auto go = [&](auto kern) -> cudaError_t {
    if (smem > 48 * 1024) {
      cudaError_t e2 = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e2 != cudaSuccess) return e2;
    }
    kern<<<units, many ? 256 : 512, smem, stream>>>(K, V, acc, pos, len, dst_scratch, place, k);
    return cudaGetLastError();
  };
  switch (head_dim) {
    case 64: return many ? go(compact_move_kernel<64, 8>) : go(compact_move_kernel<64, 16>);
    case 128: return many ? go(compact_move_kernel<128, 8>) : go(compact_move_kernel<128, 16>);
    case 256: return many ? go(compact_move_kernel<256, 8>) : go(compact_move_kernel<256, 16>);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace kf
