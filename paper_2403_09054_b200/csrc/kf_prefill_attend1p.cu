// Causal attention output of the prompt (Eq. 1: out_i = sum_{j <= i} softmax_j(x_ij) V_j, plain softmax, no logit
// adjustment) in ONE pass over the keys, for head_dim 64 and 128.
//
// A CTA owns two adjacent blocks of 128 query rows of one (batch row, head) and walks the key tiles once.  Each block
// has its own accumulators in tensor memory (S: 128 columns, O: head_dim columns; 2 x (128 + 128) = all 512 columns at
// head_dim 128) and its own group of four compute warps in which a thread IS a query row: the row's running maximum
// and sum live in that thread's registers, and so does the decision to rescale the row of O (the same accumulator
// lane), so no reduction or exchange between threads is ever needed.  Per key tile and block:
//   S = Q_blk K_tile^T                         tcgen05.mma, K-major operands from shared memory
//   P = 2^(x2 - ref) as binary16 pairs, from ONE read of S, against the reference exponent the row already has;
//           the row's maximum over the tile falls out of the same pass, and only if it exceeds the reference by more
//           than 2^8 (or on the first and the diagonal tile) is the reference moved, the row of O rescaled in tensor
//           memory, and P taken again.  P is written over the first half of S itself once the row has been read.
//   O += P V_tile                              tcgen05.mma with A = P from tensor memory, B = the V tile as TMA wrote it
// The two blocks alternate on the tensor pipe: while one block's warps work on their tile, the other block's
// MMAs run.  Warp 0 issues the TMA loads (the K and V tiles are shared by the two blocks; they pass through ONE ring of
// five slots in the order the MMAs use them: K0, K1, V0, K2, V1, ... so that the loads run two and a half key tiles
// ahead), warp 1 owns tensor memory and issues every MMA.  Every wait is bounded; a wait that runs out raises the error word and the CTA drains its
// copies and frees tensor memory before it leaves.
#include "kf_prefill.cuh"
#include "kf_tc.cuh"

namespace kf {

namespace {

constexpr int A1_THREADS = 10 * 32;     // TMA warp, MMA warp, two groups of four compute warps
constexpr int A1_RING = 5;              // shared-memory slots of one ring that K and V tiles go through in the order of use
constexpr uint32_t A1_TMEM_COLS = 512;
constexpr float A1_SLACK = 8.0f;        // log2 units a row's maximum may exceed its reference before the reference moves

struct Attend1pParams {
  CUtensorMap tmQ, tmK, tmV;   // fp16 [units][n][d] (K, V: [units / group][n][d]), boxes of 64 columns x 128 rows, 128-byte swizzle
  __half* out;                 // [units][n][d]
  const float* slopes;         // [H] or null
  int* err;
  int32_t n, nblk, H, group;
  float a_scale;               // logit scale * log2(e)
};

__device__ __forceinline__ uint64_t a1_desc_mn(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}

__device__ __forceinline__ float a1_max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// (a0, a1) * b + c and (a0, a1) + (b0, b1) as packed binary32 pairs: one instruction for two elements.
__device__ __forceinline__ void a1_fma2(float& d0, float& d1, float a0, float a1, float b, float c) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\tmov.b64 rc, {%5, %5};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b), "f"(c));
}
__device__ __forceinline__ void a1_add2(float& d0, float& d1, float b0, float b1) {
  asm("{\n\t.reg .b64 ra, rb;\n\t"
      "mov.b64 ra, {%0, %1};\n\tmov.b64 rb, {%2, %3};\n\t"
      "add.rn.f32x2 ra, ra, rb;\n\tmov.b64 {%0, %1}, ra;\n\t}"
      : "+f"(d0), "+f"(d1) : "f"(b0), "f"(b1));
}

// A thread's row of one key tile: the largest adjusted logit x2 = a_scale x (+ slope (j - i) log2 e), in log2 units,
// over the columns the causal mask leaves (`diag`: the tile on the diagonal; quarter = the warp's 32-row group, so
// chunk `quarter` of 32 columns is cut by the diagonal and later chunks are masked altogether).
template <bool ALIBI>
__device__ __forceinline__ float a1_tile_max(uint32_t s_addr, float A, float sb, float bias_t, int lane, int quarter, bool diag) {
  const int nch = diag ? quarter + 1 : 4;
  float tmax = -INFINITY;
#pragma unroll 1
  for (int c = 0; c < nch; ++c) {
    float v[32];
    tmem_ld_32x32(s_addr + (uint32_t)(c * 32), v);
    const bool edge = diag && c == quarter;
    float bias0 = 0.f;
    if (ALIBI) bias0 = fmaf(sb, (float)(c * 32), bias_t);
    float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
      float a4[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        a4[q] = v[e + q];
        if (ALIBI) a4[q] = fmaf(sb, (float)(e + q), fmaf(a4[q], A, bias0));
        if (edge && e + q > lane) a4[q] = -INFINITY;
      }
      m0 = a1_max3(m0, a4[0], a4[1]);
      m1 = a1_max3(m1, a4[2], a4[3]);
    }
    const float cm = fmaxf(m0, m1);
    tmax = fmaxf(tmax, ALIBI ? cm : cm * A);   // the scale is positive: maximum of the raw logits first, scale after
  }
  return tmax;
}

// The row's probabilities 2^(x2 - m_ref) of one key tile as 64 binary16 pairs in registers, their sum (binary32, of the
// unrounded values) in `lsum`.  MASK = false is the common case (a tile wholly below the diagonal): it also returns
// the row's largest x2, so that the caller can tell afterwards whether m_ref was still a valid reference.  MASK =
// true applies the causal mask of the diagonal tile when `diag` is set (and returns nothing of use).
#define A1_R32(r) "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),        \
                  "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),        \
                  "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),      \
                  "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
// 32 lanes x 32 columns of tensor memory into r[0..32) WITHOUT waiting: the registers hold the values only after
// a1_ld_wait(r), which also ties their later uses to the wait for the compiler.
__device__ __forceinline__ void a1_ld_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void a1_ld_wait(uint32_t (&r)[32]) { asm volatile("tcgen05.wait::ld.sync.aligned;" : A1_R32(r)::"memory"); }

template <bool ALIBI, bool MASK>
__device__ __forceinline__ float a1_tile_probs(uint32_t s_addr, float A, float m_ref, float sb, float bias_t, int lane, int quarter,
                                               bool diag, uint32_t (&packed)[64], float& lsum) {
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  auto chunk = [&](const uint32_t (&r)[32], int c) {
    const bool edge = MASK && diag && c == quarter;
    float bias0 = 0.f;
    if (ALIBI) bias0 = fmaf(sb, (float)(c * 32), bias_t);
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
      const float v0 = __uint_as_float(r[e]), v1 = __uint_as_float(r[e + 1]);
      float y0, y1;
      if (ALIBI) {
        const float x0 = fmaf(sb, (float)e, fmaf(v0, A, bias0)), x1 = fmaf(sb, (float)(e + 1), fmaf(v1, A, bias0));
        if (!MASK) { if (e & 2) m1 = a1_max3(m1, x0, x1); else m0 = a1_max3(m0, x0, x1); }
        y0 = x0 - m_ref;
        y1 = x1 - m_ref;
      } else {
        if (!MASK) { if (e & 2) m1 = a1_max3(m1, v0, v1); else m0 = a1_max3(m0, v0, v1); }
        a1_fma2(y0, y1, v0, v1, A, -m_ref);
      }
      float p0 = fast_exp2(y0), p1 = fast_exp2(y1);
      if (edge) { p0 = e <= lane ? p0 : 0.f; p1 = e + 1 <= lane ? p1 : 0.f; }
      a1_add2(l0, l1, p0, p1);
      const __half2 h = __floats2half2_rn(p0, p1);
      packed[c * 16 + (e >> 1)] = *reinterpret_cast<const uint32_t*>(&h);
    }
  };
  if (MASK) {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      if (diag && c > quarter) {
#pragma unroll
        for (int e = 0; e < 16; ++e) packed[c * 16 + e] = 0u;
        continue;
      }
      uint32_t r[32];
      a1_ld_issue(s_addr + (uint32_t)(c * 32), r);
      a1_ld_wait(r);
      chunk(r, c);
    }
  } else {
    // the logits of the next 32 columns are on their way while the current ones are worked on
    uint32_t ra[32], rb[32];
    a1_ld_issue(s_addr, ra);
    a1_ld_wait(ra);
    a1_ld_issue(s_addr + 32u, rb);
    chunk(ra, 0);
    a1_ld_wait(rb);
    a1_ld_issue(s_addr + 64u, ra);
    chunk(rb, 1);
    a1_ld_wait(ra);
    a1_ld_issue(s_addr + 96u, rb);
    chunk(ra, 2);
    a1_ld_wait(rb);
    chunk(rb, 3);
  }
  lsum = l0 + l1;
  const float m = fmaxf(m0, m1);
  return ALIBI ? m : m * A;
}

template <int D, bool ALIBI>
__global__ void __launch_bounds__(A1_THREADS, 1) prefill_attend1p(const __grid_constant__ Attend1pParams P) {
  constexpr int OP_BYTES = 128 * D * 2;    // a block of 128 rows (queries, keys or values)
  constexpr int KCH = D / 64;              // 64-column boxes per row
  constexpr int KBOX = 128 * 128;          // one box: 128 rows x 64 binary16
  constexpr uint32_t O_COL = 256;          // S0 at 0, S1 at 128, O0 at 256, O1 at 256 + D
  constexpr uint32_t IDESC_QK = umma_idesc_kk(128);
  constexpr uint32_t IDESC_PV = (1u << 4) | (1u << 16) | ((uint32_t)(D >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* sQ = smem;                               // two query blocks
  unsigned char* sR = sQ + 2 * OP_BYTES;                  // the ring of K and V tiles
  uint64_t* bars = reinterpret_cast<uint64_t*>(sR + (size_t)A1_RING * OP_BYTES);
  uint64_t* q_full = bars;
  uint64_t* r_full = q_full + 1;
  uint64_t* r_empty = r_full + A1_RING;
  uint64_t* s_full = r_empty + A1_RING;   // [2] per block
  uint64_t* p_full = s_full + 2;          // [2]
  uint64_t* o_full = p_full + 2;          // [2]
  uint64_t* drain = o_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* issued = const_cast<int*>(abort_flag) + 1;   // ring positions whose loads have been issued

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = blockIdx.y;
  const int npairs = (P.nblk + 1) >> 1;
  const int pair = npairs - 1 - (int)blockIdx.x;   // the longest CTAs of a unit start first
  const int blk0 = 2 * pair, blk1 = 2 * pair + 1;
  const bool has1 = blk1 < P.nblk;
  const int T0 = blk0 + 1;                         // key tiles of block 0 (up to its diagonal tile)
  const int T = has1 ? blk1 + 1 : T0;              // key tiles the CTA walks

  if (tid == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < A1_RING; ++s) { mbar_init(r_full + s, 1); mbar_init(r_empty + s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(s_full + b, 1); mbar_init(p_full + b, 4); mbar_init(o_full + b, 1); }
    mbar_init(drain, 1);
    *abort_flag = 0;
    issued[0] = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, A1_TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(q_full, has1 ? 2 * OP_BYTES : OP_BYTES);
      for (int kc = 0; kc < KCH; ++kc) tma_load_3d(sQ + kc * KBOX, &P.tmQ, kc * 64, blk0 * 128, u, q_full);
      if (has1)
        for (int kc = 0; kc < KCH; ++kc) tma_load_3d(sQ + OP_BYTES + kc * KBOX, &P.tmQ, kc * 64, blk1 * 128, u, q_full);
      bool ok = true;
      const int ukv = u / P.group;
      // Ring position 0 is K tile 0; position 2t + 1 is K tile t + 1 and position 2t + 2 is V tile t: the order in which
      // the MMA warp first needs them.  (Position 2T - 1 would be K tile T, which does not exist: skipped.)
      for (int j = 0; ok && j <= 2 * T; ++j) {
        const bool is_v = j >= 2 && (j & 1) == 0;
        const int t = j == 0 ? 0 : (is_v ? (j - 2) >> 1 : (j + 1) >> 1);
        if (!is_v && t >= T) continue;
        const int s = j % A1_RING;
        if (j >= A1_RING) ok = wait_bar(r_empty + s, (uint32_t)((j / A1_RING - 1) & 1), abort_flag);
        if (!ok) break;
        mbar_expect_tx(r_full + s, OP_BYTES);
        const CUtensorMap* tm = is_v ? &P.tmV : &P.tmK;
        for (int kc = 0; kc < KCH; ++kc) tma_load_3d(sR + (size_t)s * OP_BYTES + kc * KBOX, tm, kc * 64, t * 128, ukv, r_full + s);
        issued[0] = j + 1;
      }
      if (!ok) { *abort_flag = 1; atomicExch(P.err, ERR_TIMEOUT); }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = wait_bar_eager(q_full, 0, abort_flag);
      const uint64_t qd0 = umma_smem_desc(smem_u32(sQ)), kd0 = umma_smem_desc(smem_u32(sR));
      const uint64_t vd0 = a1_desc_mn(smem_u32(sR), KBOX, 1024);   // descriptors of other slots / offsets: + bytes / 16
      auto kpos = [](int t) { return t == 0 ? 0 : 2 * t - 1; };    // ring positions of K tile t and V tile t
      auto vpos = [](int t) { return 2 * t + 2; };
      // S_b = Q_b K_t^T for tile t (K-major operands, eight MMAs of K = 16 at head_dim 128)
      auto qk = [&](int b, int t) {
        const uint64_t kd = kd0 + (uint64_t)(((kpos(t) % A1_RING) * OP_BYTES) >> 4), qd = qd0 + (uint64_t)((b * OP_BYTES) >> 4);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (uint32_t)(((kk >> 2) * KBOX + (kk & 3) * 32) >> 4);
          umma_f16(tmem_base + (uint32_t)(b * 128), qd + off, kd + off, IDESC_QK, kk > 0 ? 1u : 0u);
        }
        umma_commit(s_full + b);
      };
      // O_b += P_b V_t (A = P from tensor memory, 16 keys = 8 columns per MMA; B = V, MN-major)
      auto pv = [&](int b, int t) {
        const uint64_t vd = vd0 + (uint64_t)(((vpos(t) % A1_RING) * OP_BYTES) >> 4);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          umma_f16_ts(tmem_base + O_COL + (uint32_t)(b * D), tmem_base + (uint32_t)(b * 128 + kk * 8), vd + (uint64_t)((kk * 16 * 128) >> 4),
                      IDESC_PV, (t > 0 || kk > 0) ? 1u : 0u);
      };
      // Tile 0 of both blocks, then per tile: block 0's value MMA and its next logits, block 1's value MMA and its next
      // logits.  A slot is handed back by a commit placed right after the last MMA that reads it.
      if (ok) ok = wait_bar_eager(r_full, 0, abort_flag);
      if (ok) {
        tc_fence_after();
        qk(0, 0);
        if (has1) qk(1, 0);
        umma_commit(r_empty);
      }
      for (int t = 0; ok && t < T; ++t) {
        const bool more = t + 1 < T;
        const int jk = kpos(t + 1), jv = vpos(t);
        if (more) ok = wait_bar_eager(r_full + (jk % A1_RING), (uint32_t)((jk / A1_RING) & 1), abort_flag);
        if (ok) ok = wait_bar_eager(r_full + (jv % A1_RING), (uint32_t)((jv / A1_RING) & 1), abort_flag);
        if (!ok) break;
        const bool do0 = t < T0;
        if (do0) {
          ok = wait_bar_eager(p_full, (uint32_t)(t & 1), abort_flag);
          if (!ok) break;
          tc_fence_after();
          pv(0, t);
          if (!has1) umma_commit(r_empty + (jv % A1_RING));
          if (t == T0 - 1) umma_commit(o_full);
          else qk(0, t + 1);
        }
        if (has1) {
          ok = wait_bar_eager(p_full + 1, (uint32_t)(t & 1), abort_flag);
          if (!ok) break;
          tc_fence_after();
          pv(1, t);
          umma_commit(r_empty + (jv % A1_RING));                 // both blocks' value MMAs of tile t have been issued
          if (t == T - 1) umma_commit(o_full + 1);
          else qk(1, t + 1);
        }
        if (more) umma_commit(r_empty + (jk % A1_RING));         // every logit MMA that reads K tile t + 1 has been issued
      }
      if (!ok) { *abort_flag = 1; atomicExch(P.err, ERR_TIMEOUT); }
      umma_commit(drain);
      (void)wait_bar(drain, 0, abort_flag);
    }
  } else {
    // ------------------------------------------------------------ compute warps: a thread is a query row
    const int b = (warp - 2) >> 2;          // which of the CTA's two blocks
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const int blk = b ? blk1 : blk0;
    const int g_row = blk * 128 + row;      // query position i
    const int Tb = b ? T : T0;
    const bool active = b == 0 || has1;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t s_addr = lane_addr + (uint32_t)(b * 128), o_addr = lane_addr + O_COL + (uint32_t)(b * D);
    const float A = P.a_scale;
    float sb = 0.f;
    if (ALIBI) sb = P.slopes[u % P.H] * LOG2E;
    bool ok = true;
    float m_ref = 0.f, l = 0.f;
    for (int t = 0; active && ok && t < Tb; ++t) {
      const bool diag = t == blk;
      ok = __all_sync(0xffffffffu, wait_bar(s_full + b, (uint32_t)(t & 1), abort_flag));
      if (!ok) break;
      tc_fence_after();
      const float bias_t = ALIBI ? sb * (float)(t * 128 - g_row) : 0.f;
      uint32_t packed[64];
      float lt = 0.f, tmax;
      // The common tile (below the diagonal, not the first): ONE read of S, probabilities taken against the reference the
      // row already has; the row's maximum comes out of the same pass and tells whether that was good enough.
      bool exact = t == 0 || diag;
      if (!exact) {
        tmax = a1_tile_probs<ALIBI, false>(s_addr, A, m_ref, sb, bias_t, lane, quarter, false, packed, lt);
        exact = __any_sync(0xffffffffu, tmax > m_ref + A1_SLACK);
      } else {
        tmax = a1_tile_max<ALIBI>(s_addr, A, sb, bias_t, lane, quarter, diag);
      }
      if (exact) {
        // The first tile, the diagonal tile, or a row whose maximum outgrew its reference by more than the slack: set
        // or move the reference (rescaling the row of O and its sum), then take the probabilities again from S, which
        // is still whole.
        float fac = 1.f;
        bool move = false;
        if (t == 0) { m_ref = tmax; }
        else if (tmax > m_ref + A1_SLACK) { fac = fast_exp2(m_ref - tmax); m_ref = tmax; move = true; }
        if (__any_sync(0xffffffffu, move)) {
          // rows of O are accumulator lanes of these same threads; the value MMAs of the tiles before have completed
          // (their commit precedes the one that published S)
          l *= fac;
#pragma unroll 1
          for (int oc = 0; oc < D / 32; ++oc) {
            float v[32];
            tmem_ld_32x32(o_addr + (uint32_t)(oc * 32), v);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              uint32_t w[16];
#pragma unroll
              for (int e = 0; e < 16; ++e) w[e] = __float_as_uint(v[h * 16 + e] * fac);
              tmem_st_32x16(o_addr + (uint32_t)(oc * 32 + h * 16), w);
            }
          }
          tmem_wait_st();
        }
        if (diag) (void)a1_tile_probs<ALIBI, true>(s_addr, A, m_ref, sb, bias_t, lane, quarter, true, packed, lt);
        else (void)a1_tile_probs<ALIBI, false>(s_addr, A, m_ref, sb, bias_t, lane, quarter, false, packed, lt);
      }
      l += lt;
      // P over the first half of S (every logit of the tile has been read by now)
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_st_32x16(s_addr + (uint32_t)(c * 16), reinterpret_cast<const uint32_t(&)[16]>(packed[c * 16]));
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full + b);
    }
    // ---- output: O / l
    if (active && ok) ok = __all_sync(0xffffffffu, wait_bar(o_full + b, 0, abort_flag));
    if (active && ok) {
      tc_fence_after();
      const float inv_l = 1.f / l;
#pragma unroll 1
      for (int oc = 0; oc < D / 32; ++oc) {
        float v[32];
        tmem_ld_32x32(o_addr + (uint32_t)(oc * 32), v);
        if (g_row < P.n) {
          uint4* dst = reinterpret_cast<uint4*>(P.out + ((size_t)u * P.n + g_row) * D + oc * 32);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const __half2 h = __floats2half2_rn(v[8 * q4 + 2 * e] * inv_l, v[8 * q4 + 2 * e + 1] * inv_l);
              w[e] = *reinterpret_cast<const uint32_t*>(&h);
            }
            dst[q4] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      tc_fence_before();
    }
    if (!ok && lane == 0) { *abort_flag = 1; atomicExch(P.err, ERR_TIMEOUT); }
  }

  // ---- teardown: on the failure path give the copies still in flight a bounded wait, then free tensor memory
  __syncthreads();
  if (tid == 0 && *abort_flag) {
    const int nj = issued[0];
    for (int j = nj > A1_RING ? nj - A1_RING : 0; j < nj; ++j) {
      if (j == 2 * T - 1) continue;                       // the position that is never loaded
      (void)mbar_wait_bounded(r_full + (j % A1_RING), (uint32_t)((j / A1_RING) & 1), TC_WAIT_LIMIT);
    }
    (void)mbar_wait_bounded(q_full, 0, TC_WAIT_LIMIT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, A1_TMEM_COLS);
  }
}

}  // namespace

namespace {

template <int D>
cudaError_t launch_attend1p(const Attend1pParams& P, int units, bool alibi, cudaStream_t st) {
  constexpr size_t smem = 1024 + (size_t)(2 + A1_RING) * 128 * D * 2 + 32 * 8 + 64;
  static_assert(smem <= 227 * 1024, "shared memory budget of one CTA");
  constexpr size_t smem_req = smem < 120 * 1024 ? 120 * 1024 : smem;   // one CTA per SM: it takes all of tensor memory
  dim3 grid((unsigned)((P.nblk + 1) / 2), (unsigned)units);
  auto go = [&](auto kern) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_req);
    if (e != cudaSuccess) return e;
    kern<<<grid, A1_THREADS, smem_req, st>>>(P);
    return cudaGetLastError();
  };
  return alibi ? go(prefill_attend1p<D, true>) : go(prefill_attend1p<D, false>);
}

}  // namespace

bool prefill_attend_one_pass_supported(int head_dim) { return head_dim == 64 || head_dim == 128; }

cudaError_t launch_prefill_attend_one_pass(const PrefillAttendArgs& a, int head_dim, int units, cudaStream_t stream) {
  if (a.n < 1 || units < 1 || units > 65535 || a.group < 1 || units % a.group != 0) return cudaErrorInvalidValue;
  Attend1pParams P{};
  if (!make_operand_map(&P.tmQ, a.Q, units, a.n, head_dim, 128)) return cudaErrorNotSupported;
  if (!make_operand_map(&P.tmK, a.K, units / a.group, a.n, head_dim, 128)) return cudaErrorNotSupported;
  if (!make_operand_map(&P.tmV, a.V, units / a.group, a.n, head_dim, 128)) return cudaErrorNotSupported;
  P.out = a.out;
  P.slopes = a.slopes;
  P.err = a.err;
  P.n = a.n;
  P.nblk = (a.n + 127) / 128;
  P.H = a.H;
  P.group = a.group;
  P.a_scale = a.scale * LOG2E;
  const bool alibi = a.bias_mode == 1 && a.slopes != nullptr;
  switch (head_dim) {
    case 64: return launch_attend1p<64>(P, units, alibi, stream);
    case 128: return launch_attend1p<128>(P, units, alibi, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace kf
