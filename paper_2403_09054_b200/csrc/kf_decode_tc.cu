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
// each item), warp 1 owns tensor memory and issues the MMAs, warps 2..5 are the compute warps (128 threads = 128
// accumulator lanes).  A work item is one split of one cache (the same split plan, partial format and closing
// kernel as the CUDA-core streaming kernel); the pipeline keeps running across items.  The output accumulator
// needs a reference exponent common to the whole CTA: it is the first tile's maximum and moves only when a later
// tile exceeds it by more than 2^8, in which case the accumulator is rescaled in tensor memory.
// Every wait is bounded; a wait that runs out raises the error word, and the CTA drains its copies and frees
// tensor memory before it leaves.
#include "kf_decode.cuh"
#include "kf_tc.cuh"

namespace kf {

namespace {

constexpr int DT_ROWS = 128;          // cache slots per tile = accumulator lanes of the logit MMA
constexpr int DT_NH = 16;             // head columns of both MMAs (the group's heads, zero padded)
constexpr int DT_STAGES = 3;          // K+V tile stages in flight
constexpr int DT_THREADS = 6 * 32;    // TMA warp, MMA warp, four compute warps
constexpr uint32_t DT_TMEM_COLS = 64; // S: 2 x 16 columns, O: 2 x 16 columns
constexpr uint32_t DT_O_COL = 32;
constexpr float DT_REF_SLACK = 5.545177f;   // 8 ln 2: a probability may reach 2^8 before the reference moves

struct DecodeTcParams {
  DecodeParams P;
  CUtensorMap tmK, tmV;   // fp16 [units][k][d] of the layer, boxes of 64 columns x 128 rows, 128-byte swizzle
  CUtensorMap tmQ;        // fp16 [units][group][d], boxes of 64 columns x 16 rows (rows past the group read as zeros)
  int32_t n_items;        // units x splits
};

__device__ __forceinline__ uint64_t desc_mn(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}

// 32 lanes x 16 consecutive binary32 columns: thread t of the warp receives lane (base + t).
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
  tmem_wait_ld();
#pragma unroll
  for (int e = 0; e < 16; ++e) v[e] = __uint_as_float(r[e]);
}

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

template <int D, int G>
__global__ void __launch_bounds__(DT_THREADS, 1) decode_tc_kernel(const __grid_constant__ DecodeTcParams A) {
  static_assert(D == 128, "one accumulator lane per output feature");
  static_assert(G >= 1 && G <= DT_NH, "heads of a group fit the MMA's columns");
  const DecodeParams& P = A.P;
  constexpr int KCH = D / 64;                    // 64-column boxes per row
  constexpr int KBOX = DT_ROWS * 128;            // one box of a K or V tile: 128 rows x 128 bytes
  constexpr int TILE_BYTES = KCH * KBOX;         // 32 KB
  constexpr int STAGE_BYTES = 2 * TILE_BYTES;    // K tile, then V tile
  constexpr int QBOX = DT_NH * 128;              // one box of the query block / of P: 16 rows x 128 bytes
  constexpr int QBYTES = KCH * QBOX;
  constexpr int PBYTES = (DT_ROWS / 64) * QBOX;  // P^T [16 heads][128 slots] binary16: two 64-slot boxes
  constexpr int PSTRIDE = 4 + D;
  constexpr uint32_t IDESC_QK = umma_idesc_kk(DT_NH);
  constexpr uint32_t IDESC_PV = (1u << 4) | (1u << 15) | ((uint32_t)(DT_NH >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);   // A MN-major

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* sKV = smem;
  unsigned char* sQ = sKV + (size_t)DT_STAGES * STAGE_BYTES;   // two query blocks
  unsigned char* sP = sQ + 2 * QBYTES;
  float* red_max = reinterpret_cast<float*>(sP + PBYTES);      // [2][4 warps][G] tile maxima of x
  float* red_end = red_max + 2 * 4 * G;                         // [4 warps][G][3] (l_x, m_y, l_y) at the end of an item
  uint64_t* bars = reinterpret_cast<uint64_t*>(red_end + 4 * G * 3 + 2);
  uint64_t* kv_full = bars;
  uint64_t* kv_empty = kv_full + DT_STAGES;
  uint64_t* q_full = kv_empty + DT_STAGES;
  uint64_t* q_empty = q_full + 2;
  uint64_t* s_full = q_empty + 2;
  uint64_t* s_empty = s_full + 2;
  uint64_t* o_full = s_empty + 2;
  uint64_t* o_empty = o_full + 2;
  uint64_t* p_full = o_empty + 2;
  uint64_t* pv_done = p_full + 1;
  uint64_t* x_bar = pv_done + 1;      // the compute warps exchange their tile maxima
  uint64_t* e_bar = x_bar + 1;        // ... and their end-of-item sums
  uint64_t* drain = e_bar + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* issued = const_cast<int*>(abort_flag) + 1;   // [0] tiles, [1] query blocks the producer has issued

  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // item j of this CTA: a split of a cache; nt = its tiles of 128 slots (0: nothing to stream)
  auto item_at = [&](int j, int& u, int& sp, int& row_begin, int& nt, int& len) -> bool {
    const long long e = (long long)blockIdx.x + (long long)j * gridDim.x;
    if (e >= A.n_items) return false;
    u = (int)(e / P.splits);
    sp = (int)(e % P.splits);
    len = P.len[u];
    row_begin = sp * P.tiles_per_split * 32;
    const bool bad = len < 0 || len > P.k;
    const int row_end = bad ? row_begin : min(len, row_begin + P.tiles_per_split * 32);
    nt = row_end > row_begin ? (row_end - row_begin + DT_ROWS - 1) / DT_ROWS : 0;
    if (bad) len = -1;
    return true;
  };

  if (tid == 0) {
    for (int s = 0; s < DT_STAGES; ++s) { mbar_init(kv_full + s, 1); mbar_init(kv_empty + s, 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(q_full + b, 1); mbar_init(q_empty + b, 1);
      mbar_init(s_full + b, 1); mbar_init(s_empty + b, 4);
      mbar_init(o_full + b, 1); mbar_init(o_empty + b, 4);
    }
    mbar_init(p_full, 4);
    mbar_init(pv_done, 1);
    mbar_init(x_bar, 4);
    mbar_init(e_bar, 4);
    mbar_init(drain, 1);
    *abort_flag = 0;
    issued[0] = 0;
    issued[1] = 0;
    mbar_fence_init();
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

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      int gt = 0, ni = 0;
      for (int j = 0, u, sp, rb, nt, len; ok && item_at(j, u, sp, rb, nt, len); ++j) {
        if (nt == 0) continue;
        const int qb = ni & 1;
        if (ni >= 2) ok = wait_bar(q_empty + qb, (uint32_t)(((ni >> 1) - 1) & 1), abort_flag);
        if (!ok) break;
        mbar_expect_tx(q_full + qb, QBYTES);
        for (int kc = 0; kc < KCH; ++kc) tma_load_3d(sQ + qb * QBYTES + kc * QBOX, &A.tmQ, kc * 64, 0, u, q_full + qb);
        ++ni;
        issued[1] = ni;
        for (int t = 0; t < nt; ++t, ++gt) {
          const int s = gt % DT_STAGES;
          if (gt >= DT_STAGES) ok = wait_bar(kv_empty + s, (uint32_t)((gt / DT_STAGES - 1) & 1), abort_flag);
          if (!ok) break;
          mbar_expect_tx(kv_full + s, STAGE_BYTES);
          unsigned char* dst = sKV + (size_t)s * STAGE_BYTES;
          const int row = rb + t * DT_ROWS;
          for (int kc = 0; kc < KCH; ++kc) tma_load_3d(dst + kc * KBOX, &A.tmK, kc * 64, row, u, kv_full + s);
          for (int kc = 0; kc < KCH; ++kc) tma_load_3d(dst + TILE_BYTES + kc * KBOX, &A.tmV, kc * 64, row, u, kv_full + s);
          issued[0] = gt + 1;
        }
      }
      if (!ok) { *abort_flag = 1; atomicExch(P.err, ERR_TIMEOUT); }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true;
      // a cursor over the CTA's tiles in order; the logit MMA runs one tile ahead of the value MMA
      struct Cur { int j, t, nt, ni, gt; bool live; };
      auto next_item = [&](Cur& c) {   // moves to the first tile of the next item that has tiles
        int u, sp, rb, len;
        c.live = false;
        while (item_at(c.j, u, sp, rb, c.nt, len)) {
          if (c.nt > 0) { c.live = true; c.t = 0; return; }
          ++c.j;
        }
      };
      auto advance = [&](Cur& c) {
        ++c.gt;
        if (++c.t < c.nt) return;
        ++c.j; ++c.ni;
        next_item(c);
      };
      Cur qk{0, 0, 0, 0, 0, false}, pv{0, 0, 0, 0, 0, false};
      next_item(qk);
      next_item(pv);
      auto issue_qk = [&]() {
        const int qb = qk.ni & 1, s = qk.gt % DT_STAGES, sb = qk.gt & 1;
        if (qk.t == 0) ok = wait_bar(q_full + qb, (uint32_t)((qk.ni >> 1) & 1), abort_flag);
        if (ok) ok = wait_bar(kv_full + s, (uint32_t)((qk.gt / DT_STAGES) & 1), abort_flag);
        if (ok && qk.gt >= 2) ok = wait_bar(s_empty + sb, (uint32_t)(((qk.gt >> 1) - 1) & 1), abort_flag);
        if (!ok) return;
        tc_fence_after();
        const uint32_t k_addr = smem_u32(sKV + (size_t)s * STAGE_BYTES), q_addr = smem_u32(sQ + qb * QBYTES);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {   // 64-column box, then 16 columns = 32 bytes inside it
          const uint32_t koff = (uint32_t)((kk >> 2) * KBOX + (kk & 3) * 32), qoff = (uint32_t)((kk >> 2) * QBOX + (kk & 3) * 32);
          umma_f16(tmem_base + (uint32_t)(sb * DT_NH), umma_smem_desc(k_addr + koff), umma_smem_desc(q_addr + qoff), IDESC_QK,
                   kk > 0 ? 1u : 0u);
        }
        umma_commit(s_full + sb);
        if (qk.t == qk.nt - 1) umma_commit(q_empty + qb);   // the item's last use of its query block
        advance(qk);
      };
      if (qk.live) issue_qk();
      while (ok && pv.live) {
        if (qk.live) issue_qk();   // logits of the next tile while the probabilities of this one are being written
        if (!ok) break;
        const int s = pv.gt % DT_STAGES, ob = pv.ni & 1;
        ok = wait_bar(p_full, (uint32_t)(pv.gt & 1), abort_flag);
        if (ok && pv.t == 0 && pv.ni >= 2) ok = wait_bar(o_empty + ob, (uint32_t)(((pv.ni >> 1) - 1) & 1), abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t v_addr = smem_u32(sKV + (size_t)s * STAGE_BYTES + TILE_BYTES), p_addr = smem_u32(sP);
#pragma unroll
        for (int kk = 0; kk < DT_ROWS / 16; ++kk) {   // 16 slots per MMA
          const uint64_t da = desc_mn(v_addr + (uint32_t)(kk * 16 * 128), KBOX, 1024);
          const uint64_t db = umma_smem_desc(p_addr + (uint32_t)((kk >> 2) * QBOX + (kk & 3) * 32));
          umma_f16(tmem_base + DT_O_COL + (uint32_t)(ob * DT_NH), da, db, IDESC_PV, (pv.t > 0 || kk > 0) ? 1u : 0u);
        }
        umma_commit(kv_empty + s);
        umma_commit(pv_done);
        if (pv.t == pv.nt - 1) umma_commit(o_full + ob);
        advance(pv);
      }
      if (!ok) { *abort_flag = 1; atomicExch(P.err, ERR_TIMEOUT); }
      umma_commit(drain);
      (void)wait_bar(drain, 0, abort_flag);
    }
  } else {
    // ------------------------------------------------------------ compute warps
    const int quarter = warp & 3;                 // accumulator lanes this warp may read
    const int row = quarter * 32 + lane;          // cache slot within a tile; output feature at the end of an item
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const int Hkv = P.H / G;
    bool ok = true;
    int gt = 0, ni = 0, xn = 0, en = 0;           // tiles, items with tiles, exchanges done so far
    for (int j = 0, u, sp, rb, nt, len; item_at(j, u, sp, rb, nt, len); ++j) {
      float* part = P.partials + (((size_t)u * P.splits + sp) * G) * PSTRIDE;
      if (nt == 0) {
        // nothing cached in this split: an empty partial (sum 0) for the closing kernel
        if (len < 0 && sp == 0 && tid == 64) atomicExch(P.err, ERR_BOUNDS);
#pragma unroll
        for (int n = 0; n < G; ++n) {
          part[n * PSTRIDE + 4 + row] = 0.f;
          if (row == n) *reinterpret_cast<float4*>(part + n * PSTRIDE) = make_float4(-INFINITY, 0.f, -INFINITY, 0.f);
        }
        continue;
      }
      if (!ok) break;
      const uint32_t b = (uint32_t)(u / Hkv), h0 = (uint32_t)(u % Hkv) * G, lh0 = (uint32_t)P.layer * P.H + h0;
      float slope[G], m_ref[G], l_x[G], m_y[G], l_y[G];
#pragma unroll
      for (int n = 0; n < G; ++n) {
        slope[n] = (P.bias_mode == 1 && P.slopes) ? P.slopes[h0 + n] : 0.f;
        m_ref[n] = -INFINITY; l_x[n] = 0.f; m_y[n] = -INFINITY; l_y[n] = 0.f;
      }
      const int32_t* pos_u = P.pos + (size_t)u * P.k;
      const int32_t* place_u = P.place ? P.place + (size_t)u * P.k : nullptr;
      int pos_next = (rb + row < len) ? pos_u[rb + row] : 0;
      int place_next = (place_u && rb + row < len) ? place_u[rb + row] : 0;
      const int ob = ni & 1;

      for (int t = 0; t < nt; ++t, ++gt) {
        const int slot = rb + t * DT_ROWS + row;
        const bool valid = slot < len;
        const int pj = pos_next;
        const int dist = place_u ? len - place_next : P.p - pj;   // distance between the query and this key in the bias
        if (t + 1 < nt) {
          const int sn = slot + DT_ROWS;
          pos_next = sn < len ? pos_u[sn] : 0;
          if (place_u) place_next = sn < len ? place_u[sn] : 0;
        }
        const int sb = gt & 1;
        ok = __all_sync(0xffffffffu, wait_bar(s_full + sb, (uint32_t)((gt >> 1) & 1), abort_flag));
        if (!ok) break;
        tc_fence_after();
        float sv[16];
        tmem_ld_32x16(lane_addr + (uint32_t)(sb * DT_NH), sv);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(s_empty + sb);

        // ---- per logit: bias, adjustment, the score softmax's running pair (private to the thread), tile maximum of x
        float x[G];
#pragma unroll
        for (int n = 0; n < G; ++n) {
          x[n] = -INFINITY;
          if (valid) {
            x[n] = fmaf(sv[n], P.scale, -slope[n] * (float)dist);
            const float y = (x[n] + noise_for(P, b, lh0 + n, (uint32_t)P.p, (uint32_t)pj)) * P.inv_tau;
            P.y_scratch[((size_t)u * G + n) * (P.k + 1) + slot] = y;
            const float mn = fmaxf(m_y[n], y);
            l_y[n] = fmaf(l_y[n], fast_exp2((m_y[n] - mn) * LOG2E), fast_exp2((y - mn) * LOG2E));
            m_y[n] = mn;
          }
          float wm;
          asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(wm) : "f"(x[n]));
          if (lane == 0) red_max[((gt & 1) * 4 + quarter) * G + n] = wm;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(x_bar);
        ok = __all_sync(0xffffffffu, wait_bar(x_bar, (uint32_t)(xn & 1), abort_flag));
        ++xn;
        if (!ok) break;
        // ---- the reference exponent of the output accumulator: the same decision in every thread
        float fac[G];
        bool moved = false;
#pragma unroll
        for (int n = 0; n < G; ++n) {
          const float* rm = red_max + (gt & 1) * 4 * G + n;
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
          float ov[16];
          tmem_ld_32x16(lane_addr + DT_O_COL + (uint32_t)(ob * DT_NH), ov);
          uint32_t w[16];
#pragma unroll
          for (int n = 0; n < 16; ++n) w[n] = __float_as_uint(n < G ? ov[n] * fac[n < G ? n : 0] : 0.f);
          tmem_st_32x16(lane_addr + DT_O_COL + (uint32_t)(ob * DT_NH), w);
          tmem_wait_st();
          tc_fence_before();
        }
        unsigned char* prow = sP + (row >> 6) * QBOX + (row & 7) * 2;
        const int chunk = (row & 63) >> 3;
#pragma unroll
        for (int n = 0; n < G; ++n) {
          const float p = valid ? fast_exp2((x[n] - m_ref[n]) * LOG2E) : 0.f;
          l_x[n] = fmaf(l_x[n], fac[n], p);
          *reinterpret_cast<__half*>(prow + n * 128 + ((chunk ^ (n & 7)) << 4)) = __float2half_rn(p);
        }
        if (rb + (t + 1) * DT_ROWS > len && !valid) {
          // slots past the entry count inside the cache hold whatever was there: clear this slot's V row (its weight
          // is 0, but 0 x NaN would poison the sum).  The tile has landed: the logit MMA was issued after it.
          unsigned char* vrow = sKV + (size_t)(gt % DT_STAGES) * STAGE_BYTES + TILE_BYTES + row * 128;
#pragma unroll
          for (int kc = 0; kc < KCH; ++kc)
#pragma unroll
            for (int c = 0; c < 8; ++c) reinterpret_cast<uint4*>(vrow + kc * KBOX)[c] = make_uint4(0, 0, 0, 0);
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_full);
      }
      if (!ok) break;

      // ---- end of the item: the accumulator and the softmax sums become this split's partial
      ok = __all_sync(0xffffffffu, wait_bar(o_full + ob, (uint32_t)((ni >> 1) & 1), abort_flag));
      if (!ok) break;
      tc_fence_after();
      float ov[16];
      tmem_ld_32x16(lane_addr + DT_O_COL + (uint32_t)(ob * DT_NH), ov);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(o_empty + ob);
#pragma unroll
      for (int n = 0; n < G; ++n) {
        part[n * PSTRIDE + 4 + row] = ov[n];
        const float lx = warp_sum(l_x[n]);
        const float my = warp_max(m_y[n]);
        const float ly = warp_sum(l_y[n] > 0.f ? l_y[n] * fast_exp2((m_y[n] - my) * LOG2E) : 0.f);
        if (lane == 0) {
          float* re = red_end + (quarter * G + n) * 3;
          re[0] = lx; re[1] = my; re[2] = ly;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(e_bar);
      ok = __all_sync(0xffffffffu, wait_bar(e_bar, (uint32_t)(en & 1), abort_flag));
      ++en;
      if (!ok) break;
#pragma unroll
      for (int n = 0; n < G; ++n) {
        if (row == n) {
          float L = 0.f, MY = -INFINITY, LY = 0.f;
#pragma unroll
          for (int w = 0; w < 4; ++w) MY = fmaxf(MY, red_end[(w * G + n) * 3 + 1]);
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            const float* re = red_end + (w * G + n) * 3;
            L += re[0];
            if (re[2] > 0.f) LY = fmaf(re[2], fast_exp2((re[1] - MY) * LOG2E), LY);
          }
          *reinterpret_cast<float4*>(part + n * PSTRIDE) = make_float4(m_ref[n], L, MY, LY);
        }
      }
      ++ni;
    }
    if (!ok && lane == 0) { *abort_flag = 1; atomicExch(P.err, ERR_TIMEOUT); }
  }

  // ---- teardown: on the failure path give the copies still in flight a bounded wait, then free tensor memory
  __syncthreads();
  if (tid == 0 && *abort_flag) {
    const int nt = issued[0], nq = issued[1];
    for (int it = nt > DT_STAGES ? nt - DT_STAGES : 0; it < nt; ++it)
      (void)mbar_wait_bounded(kv_full + (it % DT_STAGES), (uint32_t)((it / DT_STAGES) & 1), TC_WAIT_LIMIT);
    for (int it = nq > 2 ? nq - 2 : 0; it < nq; ++it) (void)mbar_wait_bounded(q_full + (it & 1), (uint32_t)((it >> 1) & 1), TC_WAIT_LIMIT);
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
         (2 * 4 * DT_NH + 4 * DT_NH * 3 + 2) * 4 + 32 * 8 + 64;
}

template <int G>
cudaError_t launch_tc(const DecodeTcParams& A, cudaStream_t stream) {
  constexpr size_t smem = dt_smem_bytes(128);
  static_assert(smem <= 227 * 1024, "shared memory budget of one CTA");
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_tc_kernel<128, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(A.n_items < sms ? A.n_items : sms));   // persistent: one CTA per SM
  cfg.blockDim = dim3(DT_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_tc_kernel<128, G>, A);
}

}  // namespace

bool decode_tc_supported(int head_dim, int group) { return head_dim == 128 && (group == 1 || group == 2 || group == 4 || group == 8); }

bool decode_tc_cache_maps(CUtensorMap* tmK, CUtensorMap* tmV, const __half* K, const __half* V, int units, int budget_k, int head_dim) {
  return make_operand_map(tmK, K, units, budget_k, head_dim, DT_ROWS) && make_operand_map(tmV, V, units, budget_k, head_dim, DT_ROWS);
}

cudaError_t launch_decode_tc(const DecodeParams& P, const CUtensorMap& tmK, const CUtensorMap& tmV, int head_dim, int units,
                             cudaStream_t stream) {
  if (!decode_tc_supported(head_dim, P.group) || P.splits < 1 || P.splits > decode_max_splits() || (P.tiles_per_split & 3))
    return cudaErrorInvalidValue;
  DecodeTcParams A{};
  A.P = P;
  A.tmK = tmK;
  A.tmV = tmV;
  if (!make_operand_map(&A.tmQ, P.q, units, P.group, head_dim, DT_NH)) return cudaErrorNotSupported;
  A.n_items = units * P.splits;
  cudaError_t e;
  switch (P.group) {
    case 1: e = launch_tc<1>(A, stream); break;
    case 2: e = launch_tc<2>(A, stream); break;
    case 4: e = launch_tc<4>(A, stream); break;
    case 8: e = launch_tc<8>(A, stream); break;
    default: return cudaErrorInvalidValue;
  }
  if (e != cudaSuccess) return e;
  return launch_decode_close(P, head_dim, units, stream);
}

}  // namespace kf
