// Generation-phase streaming kernel for query heads that share a key/value head (section 6 of the paper:
// multi-query / grouped-query attention), on the 5th-generation tensor cores.
//
// With g query heads on one cache every K and V row is used g times, so the logits and the value-weighted
// sums are small dense contractions: per tile of 128 cache slots
//     S[128 slots][16] = K_tile[128][d] * Q^T[d][16]           (tcgen05.mma, K-major operands; heads zero-padded to 16)
//     O[d][16]        += V_tile^T[d][128] * P^T[128][16]       (A = the V tile as TMA wrote it, MN-major; B = P from shared memory)
// with both accumulators in tensor memory.  Everything the method adds -- bias, the logit adjustment zeta of
// Eq. 4, the temperature, the two softmaxes (Eq. 1 for the output, Eq. 11 for the score) -- is per-logit
// CUDA-core arithmetic on S as it is read back: an accumulator lane is a cache slot, a column a query head.
//
// Persistent grid, one CTA per SM.  Warp 0 issues the TMA loads (a ring of K+V tile stages, the query block of
// each item), warp 1 owns tensor memory and issues the logit MMAs, warp 2 the value MMAs (one thread each: two
// warps, so that neither instruction stream waits for the other), the other warps are groups of four compute warps
// (128 threads = the 128 accumulator lanes); each group owns some of the heads' columns, so that every scheduler
// has several warps to hide the latency of the per-logit chains (Philox, two logarithms, three exponentials).  A work item is one split of one cache (the same split plan, partial format and closing
// kernel as the CUDA-core streaming kernel); the pipeline keeps running across items.  The output accumulator
// needs a reference exponent common to the whole CTA: it is the first tile's maximum and moves only when a later
// tile exceeds it by more than 2^8, in which case the accumulator is rescaled in tensor memory.
// Every wait is bounded; a wait that runs out raises the error word, and the CTA drains its copies and frees
// tensor memory before it leaves.
#include "kf_decode.cuh"
#include "kf_tc.cuh"

#include <algorithm>

namespace kf {

namespace {

constexpr int DT_ROWS = 128;          // cache slots per tile = accumulator lanes of the logit MMA
constexpr int DT_NH = 16;             // head columns of both MMAs (the group's heads, zero padded)
constexpr int DT_STAGES = 3;          // K+V tile stages in flight
__host__ __device__ constexpr int dt_threads(int hg) { return (3 + 4 * hg) * 32; }   // TMA warp, two MMA warps, hg groups of four compute warps
constexpr uint32_t DT_TMEM_COLS = 64; // S: 2 x 16 columns, O: 2 x 16 columns
constexpr uint32_t DT_O_COL = 32;
constexpr float DT_REF_SLACK = 5.545177f;   // 8 ln 2: a probability may reach 2^8 before the reference moves

struct DecodeTcParams {
  DecodeParams P;
  CUtensorMap tmK, tmV;   // fp16 [units][k][d] of the layer, boxes of 64 columns x 128 rows, 128-byte swizzle
  CUtensorMap tmQ;        // fp16 [units][group][d], boxes of 64 columns x 16 rows (rows past the group read as zeros)
  int32_t units;          // caches of the layer
  int32_t tiles_unit;     // tiles of 128 slots per cache, by capacity
};

__device__ __forceinline__ uint64_t desc_mn(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}

// 32 lanes x N consecutive binary32 columns (N = 1, 2, 4 or 8): thread t of the warp receives lane (base + t).
template <int N>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, float (&v)[N]) {
  static_assert(N == 1 || N == 2 || N == 4 || N == 8, "shapes of tcgen05.ld used here");
  uint32_t r[8];
  if constexpr (N == 1) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r[0]) : "r"(taddr) : "memory");
  } else if constexpr (N == 2) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(taddr) : "memory");
  } else if constexpr (N == 4) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
  } else {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "r"(taddr) : "memory");
  }
  tmem_wait_ld();
#pragma unroll
  for (int e = 0; e < N; ++e) v[e] = __uint_as_float(r[e]);
}
template <int N>
__device__ __forceinline__ void tmem_st_cols(uint32_t taddr, const float (&v)[N]) {
  static_assert(N == 1 || N == 2 || N == 4 || N == 8, "shapes of tcgen05.st used here");
  uint32_t r[8];
#pragma unroll
  for (int e = 0; e < N; ++e) r[e] = __float_as_uint(v[e]);
  if constexpr (N == 1) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x1.b32 [%0], {%1};" ::"r"(taddr), "r"(r[0]) : "memory");
  } else if constexpr (N == 2) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1, %2};" ::"r"(taddr), "r"(r[0]), "r"(r[1]) : "memory");
  } else if constexpr (N == 4) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};" ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
  } else {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
  }
  tmem_wait_st();
}

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// A cursor over the tiles of one CTA, in order.  The CTA owns the global tiles [lo, hi) of the sequence
// (cache 0 tile 0, cache 0 tile 1, ..., cache 1 tile 0, ...) counted by capacity (tiles_unit per cache), so every
// CTA streams the same number of tiles whatever the number of caches; a cache cut by a CTA boundary is shared by
// the CTAs on either side, each producing one partial ("piece") of it.  An item is the part of one cache inside
// [lo, hi); tiles beyond the cache's entry count do not exist (nt counts the ones that do).
struct TileCursor {
  long long lo, hi;
  int tiles_unit, units, k;
  const int32_t* len_ptr;
  int u, rb, nt, len, t, ni, gt;   // cache, first row, tiles, entry count of the item; tile in it; items with tiles and tiles so far
  int len_ahead;                   // entry count of cache u + 1, requested one item early
  bool last_piece;                 // this item reaches the end of its cache
  bool live;
  __device__ __forceinline__ void load_item(bool have_ahead) {   // the item of cache u (which overlaps [lo, hi))
    const long long base = (long long)u * tiles_unit;
    const int t0 = (int)((lo > base ? lo : base) - base);
    const int t1 = (int)((hi < base + tiles_unit ? hi : base + tiles_unit) - base);
    len = have_ahead ? len_ahead : len_ptr[u];
    len_ahead = len_ptr[u + 1 < units ? u + 1 : u];
    const bool bad = len < 0 || len > k;
    rb = t0 * 128;
    const int row_end = bad ? rb : min(len, t1 * 128);
    nt = row_end > rb ? (row_end - rb + 127) / 128 : 0;
    if (bad) len = -1;
    last_piece = t1 == tiles_unit;
    t = 0;
  }
  __device__ __forceinline__ bool first(bool skip_empty) {
    u = (int)(lo / tiles_unit);
    ni = 0; gt = 0;
    live = lo < hi && u < units;
    if (live) load_item(false);
    if (skip_empty) while (live && nt == 0) next_item_raw();
    return live;
  }
  __device__ __forceinline__ void next_item_raw() {
    ++u;
    live = (long long)u * tiles_unit < hi && u < units;
    if (live) load_item(true);
  }
  // to the next tile; crosses into the next item that has tiles (skip_empty) when this one is exhausted
  __device__ __forceinline__ void next_tile() {
    ++gt;
    if (++t < nt) return;
    ++ni;
    do { next_item_raw(); } while (live && nt == 0);
  }
};

// G query heads per cache, handled by HG groups of compute warps (HPT = G / HG heads per thread).
template <int D, int G, int HG, bool GUMBEL>
__global__ void __launch_bounds__(dt_threads(HG), 1) decode_tc_kernel(const __grid_constant__ DecodeTcParams A) {
  static_assert(D == 128, "one accumulator lane per output feature");
  static_assert(G >= 1 && G <= DT_NH && G % HG == 0, "heads of a group fit the MMA's columns and split evenly over the compute groups");
  constexpr int HPT = G / HG;
  constexpr int NCW = 4 * HG;
  constexpr int DT_THREADS = dt_threads(HG);
  const DecodeParams& P = A.P;
  constexpr int KCH = D / 64;                    // 64-column boxes per row
  constexpr int KBOX = DT_ROWS * 128;            // one box of a K or V tile: 128 rows x 128 bytes
  constexpr int TILE_BYTES = KCH * KBOX;         // 32 KB
  constexpr int QBOX = DT_NH * 128;              // one box of the query block / of P: 16 rows x 128 bytes
  constexpr int QBYTES = KCH * QBOX;
  constexpr int PBYTES = (DT_ROWS / 64) * QBOX;  // P^T [16 heads][128 slots] binary16: two 64-slot boxes
  constexpr int PSTRIDE = 4 + D;
  constexpr uint32_t IDESC_QK = umma_idesc_kk(DT_NH);
  constexpr uint32_t IDESC_PV = (1u << 4) | (1u << 15) | ((uint32_t)(DT_NH >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);   // A MN-major

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* sK = smem;                                    // ring of K tiles
  unsigned char* sV = sK + (size_t)DT_STAGES * TILE_BYTES;     // ring of V tiles (released later than the K tiles: after the value MMA)
  unsigned char* sQ = sV + (size_t)DT_STAGES * TILE_BYTES;     // two query blocks
  unsigned char* sP = sQ + 2 * QBYTES;
  float* red_max = reinterpret_cast<float*>(sP + PBYTES);      // [2][4 warps][G] tile maxima of x
  float* red_end = red_max + 2 * 4 * G;                         // [4 warps][G][3] (l_x, m_y, l_y) at the end of an item
  uint64_t* bars = reinterpret_cast<uint64_t*>(red_end + 4 * G * 3 + 2);   // 8-byte aligned: (20 G + 2) floats
  uint64_t* k_full = bars;
  uint64_t* k_empty = k_full + DT_STAGES;
  uint64_t* v_full = k_empty + DT_STAGES;
  uint64_t* v_empty = v_full + DT_STAGES;
  uint64_t* q_full = v_empty + DT_STAGES;
  uint64_t* q_empty = q_full + 2;
  uint64_t* s_full = q_empty + 2;
  uint64_t* s_empty = s_full + 2;
  uint64_t* o_full = s_empty + 2;
  uint64_t* o_empty = o_full + 2;
  uint64_t* p_full = o_empty + 2;
  uint64_t* pv_done = p_full + 1;
  uint64_t* x_bar = pv_done + 1;      // [HG] the four warps of a compute group exchange their tile maxima
  uint64_t* e_bar = x_bar + HG;       // [HG] ... and their end-of-item sums
  uint64_t* drain = e_bar + HG;       // [2] one per MMA-issuing thread
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* issued = const_cast<int*>(abort_flag) + 1;   // [0] K tiles, [1] V tiles, [2] query blocks the producer has issued

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long total_tiles = (long long)A.units * A.tiles_unit;
  auto make_cursor = [&]() {
    TileCursor c;
    c.lo = (long long)blockIdx.x * total_tiles / gridDim.x;
    c.hi = (long long)(blockIdx.x + 1) * total_tiles / gridDim.x;
    c.tiles_unit = A.tiles_unit; c.units = A.units; c.k = P.k; c.len_ptr = P.len;
    return c;
  };

  if (tid == 0) {
    for (int s = 0; s < DT_STAGES; ++s) {
      mbar_init(k_full + s, 1); mbar_init(k_empty + s, 1);
      mbar_init(v_full + s, 1); mbar_init(v_empty + s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(q_full + b, 1); mbar_init(q_empty + b, 1);
      mbar_init(s_full + b, 1); mbar_init(s_empty + b, NCW);
      mbar_init(o_full + b, 1); mbar_init(o_empty + b, NCW);
    }
    mbar_init(p_full, NCW);
    mbar_init(pv_done, 1);
    for (int g = 0; g < HG; ++g) { mbar_init(x_bar + g, 4); mbar_init(e_bar + g, 4); }
    mbar_init(drain, 1);
    mbar_init(drain + 1, 1);
    *abort_flag = 0;
    issued[0] = 0;
    issued[1] = 0;
    issued[2] = 0;
    mbar_fence_init();
  }
  if (tid == 32) {   // the TMA descriptors are kernel parameters: fetch them while the set-up runs
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&A.tmK)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&A.tmV)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&A.tmQ)) : "memory");
  }
  // rows of P beyond the group's heads stay zero for the whole kernel
  for (int i = tid; i < PBYTES / 16; i += DT_THREADS) reinterpret_cast<uint4*>(sP)[i] = make_uint4(0, 0, 0, 0);
  fence_async_smem();
  if (warp == 1) {
    tmem_alloc(tmem_slot, DT_TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Everything above touches this CTA's shared and tensor memory only, so it may run while the kernel before this one
  // in the stream is still finishing (programmatic stream serialization); nothing global is read or written before this.
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer: two streams (K tiles with the query
    //      blocks, V tiles), each issued as soon as its ring has room, whichever that is
    if (lane == 0) {
      bool ok = true;
      TileCursor kc = make_cursor(), vc = make_cursor();
      kc.first(true);
      vc.first(true);
      uint32_t idle = 0;
      while (ok && (kc.live || vc.live)) {
        bool progress = false;
        if (kc.live) {
          const int s = kc.gt % DT_STAGES, qb = kc.ni & 1;
          const bool room = (kc.gt < DT_STAGES || mbar_poll(k_empty + s, (uint32_t)((kc.gt / DT_STAGES - 1) & 1))) &&
                            (kc.t != 0 || kc.ni < 2 || mbar_poll(q_empty + qb, (uint32_t)(((kc.ni >> 1) - 1) & 1)));
          if (room) {
            if (kc.t == 0) {
              mbar_expect_tx(q_full + qb, QBYTES);
              for (int c = 0; c < KCH; ++c) tma_load_3d(sQ + qb * QBYTES + c * QBOX, &A.tmQ, c * 64, 0, kc.u, q_full + qb);
              issued[2] = kc.ni + 1;
            }
            mbar_expect_tx(k_full + s, TILE_BYTES);
            for (int c = 0; c < KCH; ++c)
              tma_load_3d(sK + (size_t)s * TILE_BYTES + c * KBOX, &A.tmK, c * 64, kc.rb + kc.t * DT_ROWS, kc.u, k_full + s);
            issued[0] = kc.gt + 1;
            kc.next_tile();
            progress = true;
          }
        }
        if (vc.live && (!kc.live || vc.gt < kc.gt)) {
          const int s = vc.gt % DT_STAGES;
          if (vc.gt < DT_STAGES || mbar_poll(v_empty + s, (uint32_t)((vc.gt / DT_STAGES - 1) & 1))) {
            mbar_expect_tx(v_full + s, TILE_BYTES);
            for (int c = 0; c < KCH; ++c)
              tma_load_3d(sV + (size_t)s * TILE_BYTES + c * KBOX, &A.tmV, c * 64, vc.rb + vc.t * DT_ROWS, vc.u, v_full + s);
            issued[1] = vc.gt + 1;
            vc.next_tile();
            progress = true;
          }
        }
        if (progress) {
          idle = 0;
        } else if (++idle > TC_WAIT_LIMIT) {
          ok = false;
        } else if (idle > 4096) {
          __nanosleep(40);
          if ((idle & 127u) == 0u && *abort_flag) ok = false;
        }
      }
      if (!ok) { *abort_flag = 1; atomicExch(P.err, ERR_TIMEOUT); }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ logit MMAs: S[tile & 1] = K_tile Q^T, as soon as the tile
    //      has landed and the accumulator buffer has been read (up to two tiles ahead of the compute warps)
    if (lane == 0) {
      bool ok = true;
      TileCursor qk = make_cursor();
      qk.first(true);
      const uint64_t kd0 = umma_smem_desc(smem_u32(sK)), qd0 = umma_smem_desc(smem_u32(sQ));
      while (ok && qk.live) {
        const int qb = qk.ni & 1, s = qk.gt % DT_STAGES, sb = qk.gt & 1;
        if (qk.t == 0) ok = wait_bar_eager(q_full + qb, (uint32_t)((qk.ni >> 1) & 1), abort_flag);
        if (ok) ok = wait_bar_eager(k_full + s, (uint32_t)((qk.gt / DT_STAGES) & 1), abort_flag);
        if (ok && qk.gt >= 2) ok = wait_bar_eager(s_empty + sb, (uint32_t)(((qk.gt >> 1) - 1) & 1), abort_flag);
        if (!ok) break;
        tc_fence_after();
        // descriptors differ from those of the rings' first buffers by the byte offset / 16 in their address field
        const uint64_t kd = kd0 + (uint64_t)((s * TILE_BYTES) >> 4), qd = qd0 + (uint64_t)((qb * QBYTES) >> 4);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {   // 64-column box, then 16 columns = 32 bytes inside it
          const uint32_t koff = (uint32_t)((kk >> 2) * KBOX + (kk & 3) * 32), qoff = (uint32_t)((kk >> 2) * QBOX + (kk & 3) * 32);
          umma_f16(tmem_base + (uint32_t)(sb * DT_NH), kd + (koff >> 4), qd + (qoff >> 4), IDESC_QK, kk > 0 ? 1u : 0u);
        }
        umma_commit(k_empty + s);     // the K tile may be replaced as soon as the logits are there
        umma_commit(s_full + sb);
        if (qk.t == qk.nt - 1) umma_commit(q_empty + qb);   // the item's last use of its query block
        qk.next_tile();
      }
      if (!ok) { *abort_flag = 1; atomicExch(P.err, ERR_TIMEOUT); }
      umma_commit(drain);
      (void)wait_bar(drain, 0, abort_flag);
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ value MMAs: O[item & 1] += V_tile^T P^T once the compute
    //      warps have written the tile's probabilities
    if (lane == 0) {
      bool ok = true;
      TileCursor pv = make_cursor();
      pv.first(true);
      const uint64_t vd0 = desc_mn(smem_u32(sV), KBOX, 1024), pd0 = umma_smem_desc(smem_u32(sP));
      while (ok && pv.live) {
        const int s = pv.gt % DT_STAGES, ob = pv.ni & 1;
        ok = wait_bar_eager(p_full, (uint32_t)(pv.gt & 1), abort_flag);
        if (ok) ok = wait_bar_eager(v_full + s, (uint32_t)((pv.gt / DT_STAGES) & 1), abort_flag);
        if (ok && pv.t == 0 && pv.ni >= 2) ok = wait_bar_eager(o_empty + ob, (uint32_t)(((pv.ni >> 1) - 1) & 1), abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint64_t vd = vd0 + (uint64_t)((s * TILE_BYTES) >> 4);
#pragma unroll
        for (int kk = 0; kk < DT_ROWS / 16; ++kk) {   // 16 slots per MMA: 16 rows of the V tile, 32 bytes of a row of P
          umma_f16(tmem_base + DT_O_COL + (uint32_t)(ob * DT_NH), vd + (uint64_t)((kk * 16 * 128) >> 4),
                   pd0 + (uint64_t)(((kk >> 2) * QBOX + (kk & 3) * 32) >> 4), IDESC_PV, (pv.t > 0 || kk > 0) ? 1u : 0u);
        }
        umma_commit(v_empty + s);
        umma_commit(pv_done);
        if (pv.t == pv.nt - 1) umma_commit(o_full + ob);
        pv.next_tile();
      }
      if (!ok) { *abort_flag = 1; atomicExch(P.err, ERR_TIMEOUT); }
      umma_commit(drain + 1);
      (void)wait_bar(drain + 1, 0, abort_flag);
    }
  } else {
    // ------------------------------------------------------------ compute warps
    const int quarter = warp & 3;                 // accumulator lanes this warp may read
    const int grp = (warp - 3) >> 2;              // heads grp * HPT .. grp * HPT + HPT - 1 are this thread's
    const int hb = grp * HPT;
    const int row = quarter * 32 + lane;          // cache slot within a tile; output feature at the end of an item
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const int Hkv = P.H / G;
    bool ok = true;
    int gt = 0, ni = 0, xn = 0, en = 0;           // tiles, items with tiles, exchanges done so far
    TileCursor it = make_cursor();
    const int c_self = (int)blockIdx.x;

    // The end of an item -- its accumulator and softmax sums become the piece's partial -- is postponed until the first
    // tile of the next item has been handled: by then the last value MMA has long finished, so nobody waits for it,
    // and the pipeline of the next item is already running.
    struct Pending { bool any; int ob, ni; float* part; float m_ref[HPT], l_x[HPT], m_y[HPT], l_y[HPT]; } pend;
    pend.any = false;
    auto finish_item = [&]() {
      if (!pend.any || !ok) return;
      pend.any = false;
      ok = __all_sync(0xffffffffu, wait_bar(o_full + pend.ob, (uint32_t)((pend.ni >> 1) & 1), abort_flag));
      if (!ok) return;
      tc_fence_after();
      float ov[HPT];
      tmem_ld_cols<HPT>(lane_addr + DT_O_COL + (uint32_t)(pend.ob * DT_NH + hb), ov);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(o_empty + pend.ob);
#pragma unroll
      for (int n = 0; n < HPT; ++n) {
        pend.part[n * PSTRIDE + 4 + row] = ov[n];
        const float lx = warp_sum(pend.l_x[n]);
        const float my = warp_max(pend.m_y[n]);
        const float ly = warp_sum(pend.l_y[n] > 0.f ? pend.l_y[n] * fast_exp2((pend.m_y[n] - my) * LOG2E) : 0.f);
        if (lane == 0) {
          float* re = red_end + (quarter * G + hb + n) * 3;
          re[0] = lx; re[1] = my; re[2] = ly;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(e_bar + grp);
      ok = __all_sync(0xffffffffu, wait_bar(e_bar + grp, (uint32_t)(en & 1), abort_flag));
      ++en;
      if (!ok) return;
#pragma unroll
      for (int n = 0; n < HPT; ++n) {
        if (row == n) {
          float L = 0.f, MY = -INFINITY, LY = 0.f;
#pragma unroll
          for (int w = 0; w < 4; ++w) MY = fmaxf(MY, red_end[(w * G + hb + n) * 3 + 1]);
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            const float* re = red_end + (w * G + hb + n) * 3;
            L += re[0];
            if (re[2] > 0.f) LY = fmaf(re[2], fast_exp2((re[1] - MY) * LOG2E), LY);
          }
          *reinterpret_cast<float4*>(pend.part + n * PSTRIDE) = make_float4(pend.m_ref[n], L, MY, LY);
        }
      }
      // red_end is written again only at the next call, which comes after another pass through x_bar: every reader is done
    };

    // positions (and places) of the first tile of the next item are requested during the last tile of this one
    int pos_ahead = 0, place_ahead = 0;
    bool have_ahead = false;
    for (it.first(false); it.live; it.next_item_raw()) {
      const int u = it.u, rb = it.rb, nt = it.nt, len = it.len;
      // which piece of its cache this item is: CTAs c_first .. share the cache, in tile order
      const int c_first = (int)((((long long)u * A.tiles_unit + 1) * gridDim.x - 1) / total_tiles);
      const int piece = c_self - c_first;
      float* part = P.partials + (((size_t)u * P.splits + piece) * G + hb) * PSTRIDE;   // this group's heads
      if (it.last_piece) {
        // the CTA that reaches the end of a cache marks the pieces nobody produces as empty (sum 0)
        for (int e = piece + 1; e < P.splits; ++e) {
          float* pe = P.partials + (((size_t)u * P.splits + e) * G + hb) * PSTRIDE;
#pragma unroll
          for (int n = 0; n < HPT; ++n) {
            pe[n * PSTRIDE + 4 + row] = 0.f;
            if (row == n) *reinterpret_cast<float4*>(pe + n * PSTRIDE) = make_float4(-INFINITY, 0.f, -INFINITY, 0.f);
          }
        }
      }
      if (nt == 0) {
        // nothing cached in this piece: an empty partial for the closing kernel
        if (len < 0 && rb == 0 && tid == 96) atomicExch(P.err, ERR_BOUNDS);
#pragma unroll
        for (int n = 0; n < HPT; ++n) {
          part[n * PSTRIDE + 4 + row] = 0.f;
          if (row == n) *reinterpret_cast<float4*>(part + n * PSTRIDE) = make_float4(-INFINITY, 0.f, -INFINITY, 0.f);
        }
        have_ahead = false;
        continue;
      }
      if (!ok) break;
      const uint32_t b = (uint32_t)(u / Hkv), h0 = (uint32_t)(u % Hkv) * G + hb, lh0 = (uint32_t)P.layer * P.H + h0;
      float slope[HPT], m_ref[HPT], l_x[HPT], m_y[HPT], l_y[HPT];
#pragma unroll
      for (int n = 0; n < HPT; ++n) {
        slope[n] = (P.bias_mode == 1 && P.slopes) ? P.slopes[h0 + n] : 0.f;
        m_ref[n] = -INFINITY; l_x[n] = 0.f; m_y[n] = -INFINITY; l_y[n] = 0.f;
      }
      const int32_t* pos_u = P.pos + (size_t)u * P.k;
      const int32_t* place_u = P.place ? P.place + (size_t)u * P.k : nullptr;
      float* ys = P.y_scratch + ((size_t)u * G + hb) * (P.k + 1);
      int pos_next, place_next = 0;
      if (have_ahead && rb == 0) {
        pos_next = pos_ahead;
        place_next = place_ahead;
      } else {
        pos_next = (rb + row < len) ? pos_u[rb + row] : 0;
        if (place_u) place_next = (rb + row < len) ? place_u[rb + row] : 0;
      }
      have_ahead = false;
      const int ob = ni & 1;
      const uint32_t o_addr = lane_addr + DT_O_COL + (uint32_t)(ob * DT_NH + hb);

      for (int t = 0; t < nt; ++t, ++gt) {
        const int slot = rb + t * DT_ROWS + row;
        const bool valid = slot < len;
        const int pj = pos_next;
        const int dist = place_u ? len - place_next : P.p - pj;   // distance between the query and this key in the bias
        if (t + 1 < nt) {
          const int sn = slot + DT_ROWS;
          pos_next = sn < len ? pos_u[sn] : 0;
          if (place_u) place_next = sn < len ? place_u[sn] : 0;
        } else if (u + 1 < A.units) {
          // the next item, if this CTA has one, starts at row 0 of the next cache (an index inside the cache whatever its
          // entry count: the value is used only for a valid slot)
          const size_t ia = (size_t)(u + 1) * P.k + (row < P.k ? row : P.k - 1);
          pos_ahead = P.pos[ia];
          if (P.place) place_ahead = P.place[ia];
          have_ahead = true;
        }
        const int sb = gt & 1;
        ok = __all_sync(0xffffffffu, wait_bar(s_full + sb, (uint32_t)((gt >> 1) & 1), abort_flag));
        if (!ok) break;
        tc_fence_after();
        float sv[HPT];
        tmem_ld_cols<HPT>(lane_addr + (uint32_t)(sb * DT_NH + hb), sv);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(s_empty + sb);

        // ---- per logit: bias, adjustment, the score softmax's running pair (private to the thread), tile maximum of x
        float x[HPT];
#pragma unroll
        for (int n = 0; n < HPT; ++n) {
          x[n] = -INFINITY;
          if (valid) {
            x[n] = fmaf(sv[n], P.scale, -slope[n] * (float)dist);
            const float zeta = GUMBEL ? gumbel_from_word(noise_word(P.pk, b, lh0 + n, (uint32_t)P.p, (uint32_t)pj))
                                      : noise_for(P, b, lh0 + n, (uint32_t)P.p, (uint32_t)pj);
            const float y = (x[n] + zeta) * P.inv_tau;
            ys[(size_t)n * (P.k + 1) + slot] = y;
            const float mn = fmaxf(m_y[n], y);
            l_y[n] = fmaf(l_y[n], fast_exp2((m_y[n] - mn) * LOG2E), fast_exp2((y - mn) * LOG2E));
            m_y[n] = mn;
          }
          float wm;
          asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(wm) : "f"(x[n]));
          if (lane == 0) red_max[((gt & 1) * 4 + quarter) * G + hb + n] = wm;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(x_bar + grp);
        ok = __all_sync(0xffffffffu, wait_bar(x_bar + grp, (uint32_t)(xn & 1), abort_flag));
        ++xn;
        if (!ok) break;
        // ---- the reference exponent of the output accumulator: the same decision in every thread of the group
        float fac[HPT];
        bool moved = false;
#pragma unroll
        for (int n = 0; n < HPT; ++n) {
          const float* rm = red_max + (gt & 1) * 4 * G + hb + n;
          const float tm = fmaxf(fmaxf(rm[0], rm[G]), fmaxf(rm[2 * G], rm[3 * G]));
          float nr = m_ref[n];
          if (tm > nr + DT_REF_SLACK) nr = tm;
          fac[n] = fast_exp2((m_ref[n] - nr) * LOG2E);   // 1 when unchanged, 0 on the item's first tile
          moved = moved || (nr != m_ref[n]);
          m_ref[n] = nr;
        }
        // the value MMA of the previous tile has read P (and, for a rescale, finished with the accumulator)
        if (gt > 0) ok = __all_sync(0xffffffffu, wait_bar(pv_done, (uint32_t)((gt - 1) & 1), abort_flag));
        if (!ok) break;
        if (moved && t > 0) {
          // rare: a later tile carries a much larger logit; lane = output feature, column = head
          tc_fence_after();
          float ov[HPT];
          tmem_ld_cols<HPT>(o_addr, ov);
#pragma unroll
          for (int n = 0; n < HPT; ++n) ov[n] *= fac[n];
          tmem_st_cols<HPT>(o_addr, ov);
          tc_fence_before();
        }
        unsigned char* prow = sP + (row >> 6) * QBOX + (row & 7) * 2;
        const int chunk = (row & 63) >> 3;
#pragma unroll
        for (int n = 0; n < HPT; ++n) {
          const float p = valid ? fast_exp2((x[n] - m_ref[n]) * LOG2E) : 0.f;
          l_x[n] = fmaf(l_x[n], fac[n], p);
          const int hn = hb + n;
          *reinterpret_cast<__half*>(prow + hn * 128 + ((chunk ^ (hn & 7)) << 4)) = __float2half_rn(p);
        }
        if (grp == 0 && rb + (t + 1) * DT_ROWS > len) {
          // slots past the entry count inside the cache hold whatever was there: clear this slot's V row (its weight
          // is 0, but 0 x NaN would poison the sum), once the tile has landed.
          ok = __all_sync(0xffffffffu, wait_bar(v_full + (gt % DT_STAGES), (uint32_t)((gt / DT_STAGES) & 1), abort_flag));
          if (!ok) break;
          if (!valid) {
            unsigned char* vrow = sV + (size_t)(gt % DT_STAGES) * TILE_BYTES + row * 128;
#pragma unroll
            for (int kc = 0; kc < KCH; ++kc)
#pragma unroll
              for (int c = 0; c < 8; ++c) reinterpret_cast<uint4*>(vrow + kc * KBOX)[c] = make_uint4(0, 0, 0, 0);
          }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_full);
        if (t == 0) finish_item();   // the previous item's partial, now that this item's pipeline is running
        if (!ok) break;
      }
      if (!ok) break;
      pend.any = true; pend.ob = ob; pend.ni = ni; pend.part = part;
#pragma unroll
      for (int n = 0; n < HPT; ++n) { pend.m_ref[n] = m_ref[n]; pend.l_x[n] = l_x[n]; pend.m_y[n] = m_y[n]; pend.l_y[n] = l_y[n]; }
      ++ni;
    }
    finish_item();
    if (!ok && lane == 0) { *abort_flag = 1; atomicExch(P.err, ERR_TIMEOUT); }
  }

  // ---- teardown: on the failure path give the copies still in flight a bounded wait, then free tensor memory
  __syncthreads();
  if (tid == 0 && *abort_flag) {
    const int nk = issued[0], nv = issued[1], nq = issued[2];
    for (int i = nk > DT_STAGES ? nk - DT_STAGES : 0; i < nk; ++i)
      (void)mbar_wait_bounded(k_full + (i % DT_STAGES), (uint32_t)((i / DT_STAGES) & 1), TC_WAIT_LIMIT);
    for (int i = nv > DT_STAGES ? nv - DT_STAGES : 0; i < nv; ++i)
      (void)mbar_wait_bounded(v_full + (i % DT_STAGES), (uint32_t)((i / DT_STAGES) & 1), TC_WAIT_LIMIT);
    for (int i = nq > 2 ? nq - 2 : 0; i < nq; ++i) (void)mbar_wait_bounded(q_full + (i & 1), (uint32_t)((i >> 1) & 1), TC_WAIT_LIMIT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, DT_TMEM_COLS);
  }
}

constexpr size_t dt_smem_bytes(int d) {
  return 1024 + (size_t)DT_STAGES * 2 * DT_ROWS * d * 2 + 2 * (size_t)(d / 64) * DT_NH * 128 + (DT_ROWS / 64) * DT_NH * 128 +
         (2 * 4 * DT_NH + 4 * DT_NH * 3 + 2) * 4 + 48 * 8 + 64;
}

template <int G, int HG>
cudaError_t launch_tc(const DecodeTcParams& A, int ctas, cudaStream_t stream) {
  constexpr size_t smem = dt_smem_bytes(128);
  static_assert(smem <= 227 * 1024, "shared memory budget of one CTA");
  auto kern = A.P.noise_mode == 0 ? decode_tc_kernel<128, G, HG, true> : decode_tc_kernel<128, G, HG, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)ctas);   // persistent: at most one CTA per SM
  cfg.blockDim = dim3(dt_threads(HG));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, A);
}

}  // namespace

bool decode_tc_supported(int head_dim, int group) { return head_dim == 128 && (group == 1 || group == 2 || group == 4 || group == 8); }

bool decode_tc_cache_maps(CUtensorMap* tmK, CUtensorMap* tmV, const __half* K, const __half* V, int units, int budget_k, int head_dim) {
  return make_operand_map(tmK, K, units, budget_k, head_dim, DT_ROWS) && make_operand_map(tmV, V, units, budget_k, head_dim, DT_ROWS);
}

// The CTAs of a launch and the largest number of CTAs that share one cache (= partials per cache).  CTA c streams the
// global tiles [c T / ctas, (c + 1) T / ctas); fewer CTAs are used when a cache would otherwise be cut into more pieces
// than the closing kernel merges.
cudaError_t decode_tc_plan(int units, int budget_k, int* ctas_out, int* pieces_out) {
  static int sms = 0;
  if (sms == 0) {
    int dev = 0, n = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    sms = n;
  }
  const long long tu = (budget_k + DT_ROWS - 1) / DT_ROWS, total = tu * units;
  long long ctas = total < sms ? total : sms;
  for (;; --ctas) {
    int worst = 1;
    for (int u = 0; u < units; ++u) {   // first and last CTA that touch cache u
      const long long first = ((u * tu + 1) * ctas - 1) / total, last = (((u + 1) * tu) * ctas - 1) / total;
      worst = std::max(worst, (int)(last - first + 1));
    }
    if (worst <= decode_max_splits() || ctas == 1) {
      *ctas_out = (int)ctas;
      *pieces_out = worst;
      return cudaSuccess;
    }
  }
}

cudaError_t launch_decode_tc(DecodeParams P, const CUtensorMap& tmK, const CUtensorMap& tmV, int head_dim, int units,
                             cudaStream_t stream) {
  if (!decode_tc_supported(head_dim, P.group)) return cudaErrorInvalidValue;
  int ctas = 1, pieces = 1;
  cudaError_t e = decode_tc_plan(units, P.k, &ctas, &pieces);
  if (e != cudaSuccess) return e;
  P.splits = pieces;          // partials per cache, for this kernel and for the closing kernel
  P.tiles_per_split = 0;
  DecodeTcParams A{};
  A.P = P;
  A.tmK = tmK;
  A.tmV = tmV;
  if (!make_operand_map(&A.tmQ, P.q, units, P.group, head_dim, DT_NH)) return cudaErrorNotSupported;
  A.units = units;
  A.tiles_unit = (P.k + DT_ROWS - 1) / DT_ROWS;
  switch (P.group) {
    case 1: e = launch_tc<1, 1>(A, ctas, stream); break;
    case 2: e = launch_tc<2, 2>(A, ctas, stream); break;
    case 4: e = launch_tc<4, 4>(A, ctas, stream); break;
    case 8: e = launch_tc<8, 4>(A, ctas, stream); break;
    default: return cudaErrorInvalidValue;
  }
  if (e != cudaSuccess) return e;
  return launch_decode_close(P, head_dim, units, stream);
}

}  // namespace kf
