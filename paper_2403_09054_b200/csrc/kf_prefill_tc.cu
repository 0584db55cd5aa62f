// Prompt-phase scoring on the 5th-generation tensor cores (Algorithm 1, t = 0; section 3.4).
//
// The causal logits X = Q K^T are a dense contraction, so they run as tcgen05.mma tiles with
// the accumulators in tensor memory; everything the method adds on top of them -- the logit
// adjustment zeta of Eq. 4, the temperature, the row softmax of Eq. 11 and the accumulation of
// the scores over query rows -- is per-element arithmetic done by the CUDA cores on the
// accumulator tiles as they are read back.  Two launches of one kernel template:
//
//   sweep 1  D = Q_blk K_tile^T : an accumulator lane is a QUERY row, so a thread keeps that
//            row's running maximum and normaliser in registers; output lse2[i] =
//            log2 sum_j 2^(y2_ij) with y2 = (x + zeta) log2(e) / tau.
//   sweep 2  D = K_blk Q_tile^T : the operands swap places, an accumulator lane is a KEY, so a
//            thread sums z_ij = 2^(y2_ij - lse2[i]) over the queries i >= j in a register and
//            stores f_theta(j) directly: no atomics, a reproducible summation order.
//
// A work item is a block of 128 rows of the resident operand together with the 128-row tiles of the
// other operand it meets under the causal mask, streamed through a ring of shared-memory stages.
// The grid is persistent (one CTA per SM): every CTA walks a fixed list of items, long and short
// ones paired so that all lists weigh the same, and its pipeline keeps running across the items --
// the loads and MMAs of the next item are issued while the compute warps still work on the
// accumulator tiles of the current one, so no SM idles through a prologue per item.
// Warp 0 issues the TMA loads (128-byte swizzled boxes, one copy per CTA), warp 1 owns tensor
// memory and issues the MMAs, the other warps are groups of four compute warps that take
// accumulator tiles in turn (a warp can read the 32 accumulator lanes selected by warp id mod 4).
// Every wait is bounded; a wait that runs out raises the error word and the CTA drains and frees
// tensor memory before it leaves.
#include "kf_prefill.cuh"
#include "kf_tc.cuh"

#include <cuda.h>

#include <mutex>
#include <type_traits>

namespace kf {

namespace {

constexpr int TC_BM = 128;                    // rows of the resident operand (accumulator lanes)
constexpr int TC_BN = 128;                    // rows of a streamed tile (accumulator columns)
constexpr int tc_threads(int ng) { return (2 + 4 * ng) * 32; }   // TMA warp + MMA warp + NG groups of 4 compute warps
#ifndef KF_TC_NG
#define KF_TC_NG 3
#endif
constexpr int TC_NG = KF_TC_NG;               // compute groups for head_dim 64 / 128 (256 leaves room for 2)
constexpr int TC_NACC = 4;                    // accumulator buffers: 4 x 128 columns = all of tensor memory
constexpr uint32_t TC_TMEM_COLS = 512;
constexpr int TC_XBUF_FLOATS = 4 * 32 * 4;    // per warp and buffer: 4 noise calls x 32 lanes x 4 words
__host__ __device__ constexpr int tc_xbufs(int d) { return d == 256 ? 1 : 2; }   // buffers per warp (two where shared memory allows)
__host__ __device__ constexpr int tc_comb_buffers(int d) { return d == 256 ? 2 : 4; }   // what the shared memory left over allows
constexpr float LG2_LN2 = -0.5287663729448977f;  // log2(ln 2)

// Instruction descriptor: binary16 A and B, both K-major, binary32 accumulator, M = 128, N = 128.
constexpr uint32_t UMMA_IDESC = (1u << 4) | ((uint32_t)(TC_BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);

// ------------------------------------------------------------------ the logit adjustment
__device__ __forceinline__ float fast_lg2(float x) {   // arguments here are normal numbers: no subnormal handling
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Same u as uniform_from_word(): ((r >> 9) + 1/2) / 2^23, built without an int->float conversion:
// the funnel shift places the 23 random bits under the exponent of 1.0, giving a value of [1, 2).
__device__ __forceinline__ float uniform_from_word_bits(uint32_t r) {
  return __uint_as_float(__funnelshift_r(r, 0x7Fu, 9)) - 0.99999994f;   // minus (1 - 2^-24): exact
}
// -log2(u).  The fast logarithm has an absolute error near 2^-22, too coarse once u approaches 1;
// there (v = 1 - u < 2^-8, v exact) two terms of the series of -ln(1 - v) take over.  Relative
// error below 5e-5 everywhere.
__device__ __forceinline__ float neg_lg2_uniform(float u) {
  const float v = 1.0f - u;
  const float series = v * fmaf(v, 0.5f * LOG2E, LOG2E);
  const float direct = -fast_lg2(u);
  return v < 0.00390625f ? series : direct;
}
// The four noise terms of one Philox call in the scaled log2 domain:
//   zeta * log2(e) / tau = -(log2(-log2 u) + log2 ln 2) / tau     with zeta = -ln(-ln u)   (Eq. 7)
// `offset` carries -log2(ln 2) / tau plus whatever the caller wants added to all four logits.
// MODE 1 (Gumbel): `mult` = -1 / tau.  MODE 2 (Gaussian alternative of section 4.4.3): the four terms are
// sigma * N(0,1) * log2(e) / tau with `mult` = sigma * log2(e) / tau and the mean inside `offset`; the angle words
// come from the counter plane with bit 31 of the batch word set.
constexpr int NOISE_OFF = 0, NOISE_GUMBEL_T = 1, NOISE_GAUSS_T = 2;
template <int MODE>
__device__ __forceinline__ float4 noise_terms(const PhiloxKeys& pk, uint32_t jgroup, uint32_t i, uint32_t lh, uint32_t b,
                                              float mult, float offset) {
  const uint4 r = philox4x32_10(jgroup, i, lh, b, pk);
  float4 t;
  if (MODE == NOISE_GAUSS_T) {
    const uint4 a = philox4x32_10(jgroup, i, lh, b | GAUSS_PLANE, pk);
    t.x = fmaf(gauss_from_words(r.x, a.x), mult, offset);
    t.y = fmaf(gauss_from_words(r.y, a.y), mult, offset);
    t.z = fmaf(gauss_from_words(r.z, a.z), mult, offset);
    t.w = fmaf(gauss_from_words(r.w, a.w), mult, offset);
  } else {
    t.x = fmaf(fast_lg2(neg_lg2_uniform(uniform_from_word_bits(r.x))), mult, offset);
    t.y = fmaf(fast_lg2(neg_lg2_uniform(uniform_from_word_bits(r.y))), mult, offset);
    t.z = fmaf(fast_lg2(neg_lg2_uniform(uniform_from_word_bits(r.z))), mult, offset);
    t.w = fmaf(fast_lg2(neg_lg2_uniform(uniform_from_word_bits(r.w))), mult, offset);
  }
  return t;
}

// ------------------------------------------------------------------ the kernel
template <int D, int NST, int NG, bool SWEEP2, int NOISE, bool ALIBI, bool WANT_X>
__global__ void __launch_bounds__(tc_threads(NG), 1) prefill_tc(const __grid_constant__ PrefillTcParams P) {
  constexpr int OP_BYTES = TC_BM * D * 2;  // one operand block: D / 64 boxes
  constexpr int KCH = D / 64;              // 64-column boxes per operand row
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* sR = smem;                                  // resident operand
  unsigned char* sS = smem + OP_BYTES;                       // NST stages of the streamed operand
  constexpr int NCW = 4 * NG;                                // compute warps
  float* xbuf = reinterpret_cast<float*>(sS + (size_t)NST * OP_BYTES);  // [NCW][TC_XBUF_FLOATS] noise exchange
  constexpr int XB = tc_xbufs(D);
  float* lse_s = xbuf + NCW * XB * TC_XBUF_FLOATS;           // [NCW][128] lse2 of the current query tile
  constexpr int COMB_FLOATS = NG * 4 * 128;
  constexpr int NCB = tc_comb_buffers(D);                    // items whose hand-over may be pending at one time
  float* comb = lse_s + NCW * 128;                           // [NCB][NG][4][128] hand-over between the compute groups
  uint64_t* bars = reinterpret_cast<uint64_t*>(comb + NCB * COMB_FLOATS);
  uint64_t* r_full = bars;
  uint64_t* r_empty = bars + 1;
  uint64_t* s_full = bars + 2;
  uint64_t* s_empty = s_full + NST;
  uint64_t* t_full = s_empty + NST;
  uint64_t* t_empty = t_full + TC_NACC;
  uint64_t* drain = t_empty + TC_NACC;
  uint64_t* c_full = drain + 1;
  uint64_t* c_empty = c_full + NCB;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(c_empty + NCB);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* issued_slot = const_cast<int*>(abort_flag) + 1;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nblk = P.nblk;
  const CUtensorMap* mapR = SWEEP2 ? &P.tmK : &P.tmQ;
  const CUtensorMap* mapS = SWEEP2 ? &P.tmQ : &P.tmK;

  // The items of this CTA.  All (unit, block) pairs are listed unit by unit, the blocks of a unit in the
  // order longest, shortest, second longest, second shortest, ...; the list is cut into chunks of two
  // (together nblk + 1 tiles, whatever the pair) and chunk q belongs to CTA q mod gridDim.x.  Consecutive
  // chunks belong to the same few units, so the CTAs running at one time share their operands in L2.
  const long long n_items = (long long)P.units * nblk;
  auto item_at = [&](int k, int& u, int& Rb) -> bool {
    const long long e = 2 * ((long long)blockIdx.x + (long long)(k >> 1) * gridDim.x) + (k & 1);
    if (e >= n_items) return false;
    u = (int)(e / nblk);
    const int z = (int)(e % nblk);
    const int r = (z & 1) ? nblk - 1 - (z >> 1) : (z >> 1);   // rank by length, 0 = longest
    Rb = SWEEP2 ? r : nblk - 1 - r;
    return true;
  };
  auto tiles_of = [&](int Rb) { return SWEEP2 ? nblk - Rb : Rb + 1; };

  if (tid == 0) {
    mbar_init(r_full, 1);
    mbar_init(r_empty, 1);
    for (int s = 0; s < NST; ++s) { mbar_init(s_full + s, 1); mbar_init(s_empty + s, 1); }
    for (int a = 0; a < TC_NACC; ++a) { mbar_init(t_full + a, 1); mbar_init(t_empty + a, 4); }
    mbar_init(drain, 1);
    for (int cb = 0; cb < NCB; ++cb) { mbar_init(c_full + cb, (NG - 1) * 4); mbar_init(c_empty + cb, 4); }
    *abort_flag = 0;
    issued_slot[0] = 0;
    issued_slot[1] = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, TC_TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // per-thread results of the compute warps
  float row_m = 0.f, row_l = 0.f;         // sweep 1: reference exponent and sum_j 2^(y2_j - row_m) of this query row
  bool started = false;
  // sweep 1, when the caller also wants the attention layer's own statistics: the same for the plain logits
  float rowx_m = 0.f, rowx_l = 0.f;
  bool started_x = false;
  float col_sum = 0.f;                    // sweep 2: f_theta partial of this key

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int gt = 0, k = 0;     // streamed tiles and items issued so far
      bool ok = true;
      for (int u, Rb; ok && item_at(k, u, Rb); ++k) {
        // the resident block may be replaced once the MMAs of the previous item have read it
        if (k > 0 && !wait_bar(r_empty, (uint32_t)((k - 1) & 1), abort_flag)) { ok = false; break; }
        mbar_expect_tx(r_full, OP_BYTES);
        // unit u is a (batch row, query head); its keys are those of cache u / group
        const int uR = SWEEP2 ? u / P.group : u, uS = SWEEP2 ? u : u / P.group;
        for (int kc = 0; kc < KCH; ++kc) tma_load_3d(sR + kc * TC_BOX_BYTES, mapR, kc * 64, Rb * TC_BM, uR, r_full);
        issued_slot[1] = k + 1;
        const int t_begin = SWEEP2 ? Rb : 0, n_tiles = tiles_of(Rb);
        for (int it = 0; it < n_tiles; ++it, ++gt) {
          const int s = gt % NST;
          if (gt >= NST && !wait_bar(s_empty + s, (uint32_t)((gt / NST - 1) & 1), abort_flag)) { ok = false; break; }
          mbar_expect_tx(s_full + s, OP_BYTES);
          unsigned char* dst = sS + (size_t)s * OP_BYTES;
          for (int kc = 0; kc < KCH; ++kc) tma_load_3d(dst + kc * TC_BOX_BYTES, mapS, kc * 64, (t_begin + it) * TC_BN, uS, s_full + s);
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicExch(P.err, ERR_TIMEOUT);
      }
      issued_slot[0] = gt;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true;
      const uint32_t r_addr = smem_u32(sR);
      int gt = 0;
      for (int k = 0, u, Rb; ok && item_at(k, u, Rb); ++k) {
        ok = wait_bar(r_full, (uint32_t)(k & 1), abort_flag);
        const int n_tiles = tiles_of(Rb);
        for (int it = 0; ok && it < n_tiles; ++it, ++gt) {
          const int s = gt % NST, a = gt % TC_NACC;
          ok = wait_bar(s_full + s, (uint32_t)((gt / NST) & 1), abort_flag);
          if (ok && gt >= TC_NACC) ok = wait_bar(t_empty + a, (uint32_t)((gt / TC_NACC - 1) & 1), abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t s_addr = smem_u32(sS + (size_t)s * OP_BYTES);
          const uint32_t d_addr = tmem_base + (uint32_t)(a * TC_BN);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = (uint32_t)((kk >> 2) * TC_BOX_BYTES + (kk & 3) * 32);  // box, then 16 columns = 32 bytes
            umma_f16(d_addr, umma_smem_desc(r_addr + off), umma_smem_desc(s_addr + off), UMMA_IDESC, kk > 0 ? 1u : 0u);
          }
          umma_commit(s_empty + s);   // the stage may be refilled once these MMAs have read it
          umma_commit(t_full + a);    // the accumulator tile is complete
        }
        if (ok) umma_commit(r_empty); // the resident block may be replaced once this item's MMAs have read it
      }
      if (!ok) {
        *abort_flag = 1;
        atomicExch(P.err, ERR_TIMEOUT);
      }
      umma_commit(drain);           // nothing of this thread's MMAs is in flight once this lands
      (void)wait_bar(drain, 0, abort_flag);
    }
  } else {
    // ------------------------------------------------------------ compute warps
    const int cw = warp - 2;            // 0..7
    const int grp = cw >> 2;            // takes the accumulator tiles whose running index is grp mod NG
    const int quarter = warp & 3;       // accumulator lanes this warp may read
    const int row = quarter * 32 + lane;               // row of the resident block owned by this thread
    const float A = P.a_scale;
    const float n_mult = NOISE == NOISE_GAUSS_T ? P.gauss_scale : -P.inv_tau;
    const float n_off = NOISE == NOISE_GUMBEL_T ? -P.inv_tau * LG2_LN2 : P.const_term;   // additive term common to all logits
    float* my_x0 = xbuf + cw * XB * TC_XBUF_FLOATS;
    float* my_lse = lse_s + cw * 128;
    bool ok = true;

    // sweep 2: the lse2 values of the next tile this group will take (of this item or the next one) are requested
    // one tile ahead; (lse_u_next, lse_t_next) say which tile they belong to
    float4 lse_next = make_float4(0.f, 0.f, 0.f, 0.f);
    int lse_u_next = -1, lse_t_next = -1;
    auto fetch_lse = [&](int uu, int tt) {
      lse_next = reinterpret_cast<const float4*>(P.lse2 + ((size_t)uu * nblk + tt) * TC_BN)[lane];
      lse_u_next = uu; lse_t_next = tt;
    };

    int gt_base = 0;   // streamed tiles of the items before this one: tile `it` of the item is the CTA's tile gt_base + it
    for (int k = 0, u, Rb; item_at(k, u, Rb); ++k) {
    const int t_begin = SWEEP2 ? Rb : 0, n_tiles = tiles_of(Rb);
    const int g_row = Rb * TC_BM + row;                // query i (sweep 1) or key j (sweep 2)
    const uint32_t b = (uint32_t)(u / P.H), h = (uint32_t)(u % P.H), lh = (uint32_t)P.layer * P.H + h;
    float sb = 0.f;
    if (ALIBI) sb = P.slopes[h] * P.c1;
    row_m = 0.f; row_l = 0.f; started = false;
    rowx_m = 0.f; rowx_l = 0.f; started_x = false;
    col_sum = 0.f;

    // the groups take the CTA's accumulator tiles in turn, across item boundaries
    for (int it = (grp + NG - gt_base % NG) % NG; ok && it < n_tiles; it += NG) {
      const int gt = gt_base + it;
      const int a = gt % TC_NACC;
      const int t = t_begin + it;
      const bool diag = (t == Rb);
      if (SWEEP2) {
        if (lse_u_next != u || lse_t_next != t) fetch_lse(u, t);
        __syncwarp();
        reinterpret_cast<float4*>(my_lse)[lane] = lse_next;
        if (it + NG < n_tiles) {
          fetch_lse(u, t + NG);
        } else {
          int u2, Rb2;
          if (item_at(k + 1, u2, Rb2)) {
            const int it2 = (grp + NG - (gt_base + n_tiles) % NG) % NG;
            if (it2 < tiles_of(Rb2)) fetch_lse(u2, Rb2 + it2);   // sweep 2: an item's first tile is its diagonal one
          }
        }
        __syncwarp();
      }
      ok = wait_bar(t_full + a, (uint32_t)((gt / TC_NACC) & 1), abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * TC_BN);

#pragma unroll 1
      for (int c = 0; c < TC_BN / 32; ++c) {
        // on the diagonal tile whole 32-column chunks are causally masked for this warp
        if (diag && (SWEEP2 ? c < quarter : c > quarter)) continue;
        const bool edge = diag && c == quarter;
        float v[32];
        tmem_ld_32x32(t_addr + (uint32_t)(c * 32), v);
        const int col0 = t * TC_BN + c * 32;   // first key j (sweep 1) / first query i (sweep 2) of the chunk

        // causally masked logits of the diagonal chunk: -inf in, 0 out of every exponential below
        if (edge) {
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = (SWEEP2 ? e >= lane : e <= lane) ? v[e] : -INFINITY;
        }

        if (!SWEEP2) {
          // ---- thread = query row i: add sum_j 2^(y2_j - row_m) over 32 keys to row_l.  The reference
          //      row_m is not the exact running maximum: any value within 2^+-100 of it serves, so it moves
          //      only when the sum leaves that range, which saves a max and a subtract per logit.
          float bias0 = 0.f;
          if (ALIBI) bias0 = sb * (float)(col0 - g_row);   // -slope (i - j) log2(e) / tau at e = 0
          if (!started) {
            row_m = fmaf(v[0], A, n_off + bias0);          // element 0 of a row's first chunk is never masked
            started = true;
          }
          // mode 0: sum of 2^(y2 - ref); mode 1: max of y2 - ref (exact fallback, see below)
          auto sweep_chunk = [&](float ref, auto mode) -> float {
            constexpr bool WANT_MAX = decltype(mode)::value;
            const float off = n_off + bias0 - ref;
            float r0 = WANT_MAX ? -INFINITY : 0.f, r1 = r0, r2 = r0, r3 = r0;
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              float4 nz = make_float4(off, off, off, off);
              if (NOISE) nz = noise_terms<NOISE>(P.pk, (uint32_t)(col0 >> 2) + g, (uint32_t)g_row, lh, b, n_mult, off);
              const float nn[4] = {nz.x, nz.y, nz.z, nz.w};
              float a4[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const int e = 4 * g + q;
                a4[q] = fmaf(v[e], A, nn[q]);
                if (ALIBI) a4[q] = fmaf(sb, (float)e, a4[q]);
              }
              if (WANT_MAX) {
                r0 = fmaxf(r0, a4[0]); r1 = fmaxf(r1, a4[1]); r2 = fmaxf(r2, a4[2]); r3 = fmaxf(r3, a4[3]);
              } else {
                r0 += fast_exp2(a4[0]); r1 += fast_exp2(a4[1]); r2 += fast_exp2(a4[2]); r3 += fast_exp2(a4[3]);
              }
            }
            return WANT_MAX ? fmaxf(fmaxf(r0, r1), fmaxf(r2, r3)) : (r0 + r1) + (r2 + r3);
          };
          float ref = row_m;
          float sum = sweep_chunk(ref, std::false_type{});
          if (!(sum < 1e30f)) {
            // some logit lies about 2^100 or more above the reference: take the chunk's exact maximum instead
            const float cm = sweep_chunk(ref, std::true_type{});
            if (cm < INFINITY) {
              ref += cm;
              sum = sweep_chunk(ref, std::false_type{});
            }
          }
          if (ref != row_m) {
            row_l *= fast_exp2(row_m - ref);
            row_m = ref;
          }
          row_l += sum;
          if (row_l > 1.8446744e19f) {   // 2^64: keep the sum far from overflow
            row_l *= 5.4210109e-20f;     // 2^-64
            row_m += 64.f;
          }
          if (WANT_X) {
            // plain softmax of x (no adjustment, temperature 1): log-sum-exp for the attention output kernel
            const float Ax = P.ax;
            float bias0x = 0.f, sbx = 0.f;
            if (ALIBI) { sbx = P.slopes[h] * LOG2E; bias0x = sbx * (float)(col0 - g_row); }
            if (!started_x) { rowx_m = fmaf(v[0], Ax, bias0x); started_x = true; }
            auto fold_x = [&](float rx, auto mode) -> float {
              constexpr bool WANT_MAX = decltype(mode)::value;
              float r0 = WANT_MAX ? -INFINITY : 0.f, r1 = r0, r2 = r0, r3 = r0;
#pragma unroll
              for (int e = 0; e < 32; e += 4) {
                float a4[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  a4[q] = fmaf(v[e + q], Ax, bias0x - rx);
                  if (ALIBI) a4[q] = fmaf(sbx, (float)(e + q), a4[q]);
                }
                if (WANT_MAX) { r0 = fmaxf(r0, a4[0]); r1 = fmaxf(r1, a4[1]); r2 = fmaxf(r2, a4[2]); r3 = fmaxf(r3, a4[3]); }
                else { r0 += fast_exp2(a4[0]); r1 += fast_exp2(a4[1]); r2 += fast_exp2(a4[2]); r3 += fast_exp2(a4[3]); }
              }
              return WANT_MAX ? fmaxf(fmaxf(r0, r1), fmaxf(r2, r3)) : (r0 + r1) + (r2 + r3);
            };
            float rx = rowx_m;
            float sx = fold_x(rx, std::false_type{});
            if (!(sx < 1e30f)) {
              const float cm = fold_x(rx, std::true_type{});
              if (cm < INFINITY) { rx += cm; sx = fold_x(rx, std::false_type{}); }
            }
            if (rx != rowx_m) { rowx_l *= fast_exp2(rowx_m - rx); rowx_m = rx; }
            rowx_l += sx;
            if (rowx_l > 1.8446744e19f) { rowx_l *= 5.4210109e-20f; rowx_m += 64.f; }
          }
        } else {
          // ---- thread = key j: add z_ij = 2^(y2_ij - lse2_i) over 32 queries to col_sum
          float bias0 = 0.f;
          if (ALIBI) bias0 = sb * (float)(g_row - col0);   // -slope (i - j) log2(e) / tau at e = 0
          const float* lse_t = my_lse + c * 32;
          float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
          if (NOISE) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              // Lane L draws the Philox call of key group (L & 7) of this warp and query 4 g + (L >> 3) and
              // folds that query's -lse2 into the four terms; afterwards lane L reads word (L & 3) of its
              // own key group (L >> 2) for each query.  Both access patterns are bank-conflict free.  With two
              // buffers the halves alternate, and the barrier after a half's writes is also what tells that the
              // buffer written next (read one half earlier) is free.
              float* my_x = my_x0 + (XB == 2 ? half * TC_XBUF_FLOATS : 0);
              if (XB == 1) __syncwarp();
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                const int ql = half * 16 + 4 * g + (lane >> 3);
                const uint32_t jg = (uint32_t)((Rb * TC_BM + quarter * 32) >> 2) + (uint32_t)(lane & 7);
                reinterpret_cast<float4*>(my_x)[g * 32 + lane] =
                    noise_terms<NOISE>(P.pk, jg, (uint32_t)(col0 + ql), lh, b, n_mult, n_off - lse_t[ql]);
              }
              __syncwarp();
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                float pp[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  const int e = half * 16 + 4 * g + q;
                  float arg = fmaf(v[e], A, my_x[(g * 32 + 8 * q + (lane >> 2)) * 4 + (lane & 3)]);
                  if (ALIBI) arg += fmaf(-sb, (float)e, bias0);
                  pp[q] = fast_exp2(arg);
                }
                s0 += pp[0]; s1 += pp[1]; s2 += pp[2]; s3 += pp[3];
              }
            }
          } else {
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              const float4 l4 = reinterpret_cast<const float4*>(lse_t)[g];
              const float ll[4] = {l4.x, l4.y, l4.z, l4.w};
              float pp[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const int e = 4 * g + q;
                float arg = fmaf(v[e], A, n_off - ll[q]);
                if (ALIBI) arg += fmaf(-sb, (float)e, bias0);
                pp[q] = fast_exp2(arg);
              }
              s0 += pp[0]; s1 += pp[1]; s2 += pp[2]; s3 += pp[3];
            }
          }
          col_sum += (s0 + s1) + (s2 + s3);
        }
      }
      // hand the accumulator buffer back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(t_empty + a);
    }
    gt_base += n_tiles;
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicExch(P.err, ERR_TIMEOUT);
    }

    // ---- the item is complete: the group that took its last tile (most likely the last to finish) collects
    //      the partial results of the others from a ring of hand-over buffers and stores the rows' results.
    //      Nobody else waits for it: a group only has to find a free buffer, NCB items later.
    const int merger = (gt_base - 1) % NG;
    const int cb = k % NCB;
    float* cmb = comb + cb * COMB_FLOATS;
    if (grp != merger) {
      if (ok && k >= NCB) ok = __all_sync(0xffffffffu, wait_bar(c_empty + cb, (uint32_t)((k / NCB - 1) & 1), abort_flag));
      float* mine = cmb + grp * 512;
      mine[row] = SWEEP2 ? col_sum : row_m;
      mine[128 + row] = row_l;
      mine[256 + row] = rowx_m;
      mine[384 + row] = rowx_l;
      __syncwarp();
      if (lane == 0) mbar_arrive(c_full + cb);
    } else {
      if (ok) ok = __all_sync(0xffffffffu, wait_bar(c_full + cb, (uint32_t)((k / NCB) & 1), abort_flag));
      if (!SWEEP2) {
        // merge the groups' (reference, sum) pairs; a sum of 0 marks a group that had no tile
        auto merged = [&](float m, float l, int off) -> float {
#pragma unroll
          for (int g = 0; g < NG; ++g) {
            if (g == merger) continue;
            const float m1 = cmb[g * 512 + off + row], l1 = cmb[g * 512 + off + 128 + row];
            if (l1 > 0.f) {
              if (l > 0.f) {
                const float mm = fmaxf(m, m1);
                l = l * fast_exp2(m - mm) + l1 * fast_exp2(m1 - mm);
                m = mm;
              } else {
                m = m1; l = l1;
              }
            }
          }
          return m + log2f(l);
        };
        // rows past the prompt get +inf: their scores vanish in sweep 2 (and their attention weights likewise)
        P.lse2[(size_t)u * nblk * TC_BN + g_row] = g_row < P.n ? merged(row_m, row_l, 0) : INFINITY;
        if (WANT_X) P.lse_x[(size_t)u * nblk * TC_BN + g_row] = g_row < P.n ? merged(rowx_m, rowx_l, 256) : INFINITY;
      } else {
        // a fixed order of summation (group 0, 1, ...), whichever group collects
        float total = 0.f;
#pragma unroll
        for (int g = 0; g < NG; ++g) total += g == merger ? col_sum : cmb[g * 512 + row];
        if (g_row < P.n) P.acc_full[(size_t)u * P.n + g_row] = total;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(c_empty + cb);
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicExch(P.err, ERR_TIMEOUT);
    }
    }   // items
  }

  // ---- teardown: on the failure path give the copies still in flight a bounded wait, then free tensor memory
  __syncthreads();
  if (tid == 0 && *abort_flag) {
    const int issued = issued_slot[0], items = issued_slot[1];
    for (int it = issued > NST ? issued - NST : 0; it < issued; ++it)
      (void)mbar_wait_bounded(s_full + (it % NST), (uint32_t)((it / NST) & 1), TC_WAIT_LIMIT);
    if (items > 0) (void)mbar_wait_bounded(r_full, (uint32_t)((items - 1) & 1), TC_WAIT_LIMIT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TC_TMEM_COLS);
  }
}

// ------------------------------------------------------------------ host side
}  // namespace

namespace {
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static std::once_flag once;
  static EncodeTiledFn fn = nullptr;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

}  // namespace

bool make_operand_map(CUtensorMap* map, const __half* base, int units, int n, int d, int box_rows) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)n, (cuuint64_t)units};
  const cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)n * d * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<__half*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

template <int D, int NST, int NG>
constexpr size_t tc_smem_bytes() {
  size_t b = 1024 + (size_t)(1 + NST) * TC_BM * D * 2 + (size_t)4 * NG * tc_xbufs(D) * TC_XBUF_FLOATS * 4 + (size_t)4 * NG * 128 * 4 +
             (size_t)tc_comb_buffers(D) * NG * 4 * 128 * 4 + 40 * 8 + 64;
  return b < 120 * 1024 ? 120 * 1024 : b;   // one CTA per SM: each takes all of tensor memory
}

template <int D, int NST, int NG, bool SWEEP2>
cudaError_t launch_variant(const PrefillTcParams& P, int units, int noise, bool alibi, cudaStream_t st) {
  constexpr size_t smem = tc_smem_bytes<D, NST, NG>();
  static_assert(smem <= 227 * 1024, "shared memory budget of one CTA");
  // persistent grid: one CTA per SM (each takes all of tensor memory), fewer when there are fewer item pairs
  int dev = 0, sms = 0;
  cudaError_t e0 = cudaGetDevice(&dev);
  if (e0 == cudaSuccess) e0 = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e0 != cudaSuccess) return e0;
  const long long pairs = ((long long)P.nblk * units + 1) / 2;
  dim3 grid((unsigned)(pairs < sms ? pairs : sms));
  auto go = [&](auto kern) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, tc_threads(NG), smem, st>>>(P);
    return cudaGetLastError();
  };
  // the plain-softmax statistics are an extra of sweep 1 only
  const bool want_x = !SWEEP2 && P.lse_x != nullptr;
  auto pick = [&](auto noise_c, auto alibi_c) -> cudaError_t {
    constexpr int NZ = decltype(noise_c)::value;
    constexpr bool AL = decltype(alibi_c)::value;
    if constexpr (!SWEEP2) {
      if (want_x) return go(prefill_tc<D, NST, NG, false, NZ, AL, true>);
    }
    return go(prefill_tc<D, NST, NG, SWEEP2, NZ, AL, false>);
  };
  using std::integral_constant;
  if (noise == NOISE_GUMBEL_T)
    return alibi ? pick(integral_constant<int, NOISE_GUMBEL_T>{}, std::true_type{}) : pick(integral_constant<int, NOISE_GUMBEL_T>{}, std::false_type{});
  if (noise == NOISE_GAUSS_T)
    return alibi ? pick(integral_constant<int, NOISE_GAUSS_T>{}, std::true_type{}) : pick(integral_constant<int, NOISE_GAUSS_T>{}, std::false_type{});
  return alibi ? pick(integral_constant<int, NOISE_OFF>{}, std::true_type{}) : pick(integral_constant<int, NOISE_OFF>{}, std::false_type{});
}

}  // namespace

cudaError_t launch_prefill_score_tc(const PrefillTcArgs& a, int head_dim, int units, cudaStream_t stream) {
  if (a.n < 1 || units < 1 || units > 65535) return cudaErrorInvalidValue;
  PrefillTcParams P{};
  if (!make_operand_map(&P.tmQ, a.Q, units, a.n, head_dim)) return cudaErrorNotSupported;
  if (a.group < 1 || units % a.group != 0) return cudaErrorInvalidValue;
  if (!make_operand_map(&P.tmK, a.K, units / a.group, a.n, head_dim)) return cudaErrorNotSupported;
  P.lse2 = a.lse2;
  P.lse_x = a.lse_x;
  P.ax = a.scale * LOG2E;
  P.acc_full = a.acc_full;
  P.slopes = a.slopes;
  P.err = a.err;
  P.n = a.n;
  P.nblk = (a.n + TC_BM - 1) / TC_BM;
  P.units = units;
  P.group = a.group;
  P.H = a.H;
  P.layer = a.layer;
  P.inv_tau = a.inv_tau;
  P.c1 = LOG2E * a.inv_tau;
  P.a_scale = a.scale * P.c1;
  P.const_term = a.noise_mode == 2 ? a.noise_const * P.c1 : (a.noise_mode == 3 ? a.noise_mu * P.c1 : 0.f);
  P.gauss_scale = a.noise_sigma * P.c1;
  P.pk = a.pk;
  const int noise = a.noise_mode == 0 ? NOISE_GUMBEL_T : (a.noise_mode == 3 ? NOISE_GAUSS_T : NOISE_OFF);
  const bool alibi = a.bias_mode == 1 && a.slopes != nullptr;
  cudaError_t e;
  switch (head_dim) {
    case 64:
      e = launch_variant<64, 4, TC_NG, false>(P, units, noise, alibi, stream);
      if (e == cudaSuccess) e = launch_variant<64, 4, TC_NG, true>(P, units, noise, alibi, stream);
      return e;
    case 128:
      e = launch_variant<128, 3, TC_NG, false>(P, units, noise, alibi, stream);
      if (e == cudaSuccess) e = launch_variant<128, 3, TC_NG, true>(P, units, noise, alibi, stream);
      return e;
    case 256:
      e = launch_variant<256, 2, 2, false>(P, units, noise, alibi, stream);
      if (e == cudaSuccess) e = launch_variant<256, 2, 2, true>(P, units, noise, alibi, stream);
      return e;
    default:
      return cudaErrorInvalidValue;
  }
}

size_t prefill_tc_lse_floats(int units, int n_max) {
  return (size_t)units * (size_t)((n_max + TC_BM - 1) / TC_BM) * TC_BM;
}

}  // namespace kf
