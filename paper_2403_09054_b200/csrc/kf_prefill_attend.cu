// Causal attention output of the prompt (Eq. 1: out_i = sum_{j <= i} softmax_j(x_ij) V_j, plain softmax,
// no logit adjustment) on the tensor cores, for callers that want the prompt phase to return what the
// model's attention layer needs together with the Keyformer scores.
//
// One CTA owns 128 query rows and walks the key tiles j <= i twice:
//   phase A  S = Q_blk K_tile^T (tcgen05.mma, accumulator in tensor memory); the compute warps fold each
//            tile into the row's softmax reference and sum, giving lse2_i = log2 sum_j 2^(x2_ij).
//   phase B  S again; the compute warps turn it into the normalised probabilities P = 2^(x2 - lse2) (exact
//            softmax weights, so no running rescale of the output is ever needed), round them to binary16
//            and store them back into tensor memory (two buffers); a second MMA takes P from there as its A
//            operand and accumulates O += P V_tile (V is the MN-major B operand, read as TMA wrote it).
// Warp 0 issues the TMA loads (one copy per CTA), warp 1 owns tensor memory and issues both MMAs, the other warps are
// groups of four compute warps (four groups at head_dim 128), each taking an equal share of a tile's 128 key columns.  Every wait is bounded;
// a wait that runs out raises the error word and the CTA drains and frees tensor memory before it leaves.
#include "kf_prefill.cuh"
#include "kf_tc.cuh"

#include <type_traits>

namespace kf {

namespace {

constexpr int at_threads(int ng) { return (2 + 4 * ng) * 32; }   // TMA warp, MMA warp, NG groups of four compute warps
constexpr uint32_t AT_TMEM_COLS = 512;   // two S tiles (BN columns each), then O (D columns), then two P buffers (BN / 2 columns of binary16 pairs each)

struct AttendParams {
  CUtensorMap tmQ, tmK, tmV;   // fp16 [units][n][d], boxes of 64 columns x 128 rows (Q) or BN rows (K, V), 128-byte swizzle
  __half* out;                 // [units][n][d]
  const float* lse_in;         // null, or [units][nblk * 128] log2-domain log-sum-exp of the rows: phase A is skipped
  const float* slopes;         // [H] or null
  int* err;
  int32_t n, nblk, H;
  int32_t group;               // query heads per key/value head: unit u reads the keys and values of cache u / group
  float a_scale;               // logit scale * log2(e)
};

// MN-major operand (rows = K index, 128-byte swizzled runs along N): `lbo` bytes between 64-element chunks
// along N, `sbo` bytes between groups of eight K rows.
__device__ __forceinline__ uint64_t umma_smem_desc_mn(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}

template <int D, int BN, int KST, int VST, int NG, bool ALIBI>
__global__ void __launch_bounds__(at_threads(NG), 1) prefill_attend(const __grid_constant__ AttendParams P) {
  constexpr int OP_BYTES = 128 * D * 2;   // the query block
  constexpr int KOP_BYTES = BN * D * 2;   // one key / value tile of BN rows
  constexpr int KBOX = BN * 128;          // one TMA box of a key / value tile: BN rows x 64 binary16
  constexpr uint32_t AT_O_COL = 2 * BN, AT_P_COL = 2 * BN + D;
  static_assert(2 * BN + D + BN <= 512, "tensor memory plan");
  constexpr int KCH = D / 64;
  constexpr int NCW = 4 * NG;          // compute warps
  constexpr int CPG = BN / 32 / NG;    // 32-column chunks of a tile per group
  constexpr int OCH = D / NG / 32;     // 32-column chunks of the output per group
  static_assert(CPG >= 1 && CPG * NG * 32 == BN && OCH >= 1 && OCH * NG * 32 == D, "column split over the compute groups");
  constexpr uint32_t IDESC_QK = umma_idesc_kk(BN);
  constexpr uint32_t IDESC_PV = (1u << 4) | (1u << 16) | ((uint32_t)(D >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* sQ = smem;
  unsigned char* sK = sQ + OP_BYTES;
  unsigned char* sV = sK + (size_t)KST * KOP_BYTES;
  float* stats = reinterpret_cast<float*>(sV + (size_t)VST * KOP_BYTES);   // [NG groups][ref, sum][128 rows]
  uint64_t* bars = reinterpret_cast<uint64_t*>(stats + NG * 2 * 128);
  uint64_t* q_full = bars;
  uint64_t* k_full = q_full + 1;
  uint64_t* k_empty = k_full + KST;
  uint64_t* v_full = k_empty + KST;
  uint64_t* v_empty = v_full + VST;
  uint64_t* s_full = v_empty + VST;
  uint64_t* s_empty = s_full + 2;
  uint64_t* p_full = s_empty + 2;
  uint64_t* p_empty = p_full + 2;
  uint64_t* o_full = p_empty + 2;
  uint64_t* stats_bar = o_full + 1;
  uint64_t* drain = stats_bar + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* issued_k = const_cast<int*>(abort_flag) + 1;
  int* issued_v = issued_k + 1;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = blockIdx.y;
  const int Rb = P.nblk - 1 - (int)blockIdx.x;   // the longest CTAs of a unit start first
  const int T = (Rb + 1) * (128 / BN);           // key tiles of BN rows up to the end of this query block
  const int TA = P.lse_in ? 0 : T;               // tiles of the statistics phase

  if (tid == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < KST; ++s) { mbar_init(k_full + s, 1); mbar_init(k_empty + s, 1); }
    for (int s = 0; s < VST; ++s) { mbar_init(v_full + s, 1); mbar_init(v_empty + s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(s_full + b, 1); mbar_init(s_empty + b, NCW); }
    for (int b = 0; b < 2; ++b) { mbar_init(p_full + b, NCW); mbar_init(p_empty + b, 1); }
    mbar_init(o_full, 1);
    mbar_init(stats_bar, NCW);
    mbar_init(drain, 1);
    *abort_flag = 0;
    *issued_k = 0;
    *issued_v = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, AT_TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(q_full, OP_BYTES);
      for (int kc = 0; kc < KCH; ++kc) tma_load_3d(sQ + kc * TC_BOX_BYTES, &P.tmQ, kc * 64, Rb * 128, u, q_full);
      bool ok = true;
      int kit = 0, vit = 0;
      for (int pass = (TA == 0 ? 1 : 0); ok && pass < 2; ++pass) {
        for (int t = 0; ok && t < T; ++t) {
          const int s = kit % KST;
          if (kit >= KST) ok = wait_bar(k_empty + s, (uint32_t)((kit / KST - 1) & 1), abort_flag);
          if (!ok) break;
          mbar_expect_tx(k_full + s, KOP_BYTES);
          for (int kc = 0; kc < KCH; ++kc) tma_load_3d(sK + (size_t)s * KOP_BYTES + kc * KBOX, &P.tmK, kc * 64, t * BN, u / P.group, k_full + s);
          ++kit;
          if (pass == 1) {
            const int sv = vit % VST;
            if (vit >= VST) ok = wait_bar(v_empty + sv, (uint32_t)((vit / VST - 1) & 1), abort_flag);
            if (!ok) break;
            mbar_expect_tx(v_full + sv, KOP_BYTES);
            for (int kc = 0; kc < KCH; ++kc) tma_load_3d(sV + (size_t)sv * KOP_BYTES + kc * KBOX, &P.tmV, kc * 64, t * BN, u / P.group, v_full + sv);
            ++vit;
          }
        }
      }
      if (!ok) { *abort_flag = 1; atomicExch(P.err, ERR_TIMEOUT); }
      *issued_k = kit;
      *issued_v = vit;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = wait_bar(q_full, 0, abort_flag);
      const uint32_t q_addr = smem_u32(sQ);
      int kit = 0, sit = 0;
      auto mma_qk = [&]() {   // S[sit % 2] = Q_blk K_tile^T for the next K stage
        const int s = kit % KST, b = sit % 2;
        ok = wait_bar(k_full + s, (uint32_t)((kit / KST) & 1), abort_flag);
        if (ok && sit >= 2) ok = wait_bar(s_empty + b, (uint32_t)((sit / 2 - 1) & 1), abort_flag);
        if (!ok) return;
        tc_fence_after();
        const uint32_t k_addr = smem_u32(sK + (size_t)s * KOP_BYTES);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {   // 64-column box, then 16 columns = 32 bytes inside it
          const uint32_t qoff = (uint32_t)((kk >> 2) * TC_BOX_BYTES + (kk & 3) * 32);
          const uint32_t koff = (uint32_t)((kk >> 2) * KBOX + (kk & 3) * 32);
          umma_f16(tmem_base + (uint32_t)(b * BN), umma_smem_desc(q_addr + qoff), umma_smem_desc(k_addr + koff), IDESC_QK,
                   kk > 0 ? 1u : 0u);
        }
        umma_commit(k_empty + s);
        umma_commit(s_full + b);
        ++kit;
        ++sit;
      };
      for (int t = 0; ok && t < TA; ++t) mma_qk();         // phase A
      if (ok) mma_qk();                                     // phase B, tile 0
      for (int t = 0; ok && t < T; ++t) {
        if (t + 1 < T) mma_qk();                            // S of the next tile while P of this one is being written
        if (!ok) break;
        const int sv = t % VST;
        ok = wait_bar(p_full + (t & 1), (uint32_t)((t >> 1) & 1), abort_flag);
        if (ok) ok = wait_bar(v_full + sv, (uint32_t)((t / VST) & 1), abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t p_tmem = tmem_base + AT_P_COL + (uint32_t)((t & 1) * (BN / 2));
        const uint32_t v_addr = smem_u32(sV + (size_t)sv * KOP_BYTES);
#pragma unroll
        for (int kk = 0; kk < BN / 16; ++kk) {              // 16 keys per MMA; 16 binary16 = 8 columns of P
          const uint64_t db = umma_smem_desc_mn(v_addr + (uint32_t)(kk * 16 * 128), KBOX, 1024);
          umma_f16_ts(tmem_base + AT_O_COL, p_tmem + (uint32_t)(kk * 8), db, IDESC_PV, (t > 0 || kk > 0) ? 1u : 0u);
        }
        umma_commit(p_empty + (t & 1));
        umma_commit(v_empty + sv);
      }
      if (ok) umma_commit(o_full);
      if (!ok) { *abort_flag = 1; atomicExch(P.err, ERR_TIMEOUT); }
      umma_commit(drain);
      (void)wait_bar(drain, 0, abort_flag);
    }
  } else {
    // ------------------------------------------------------------ compute warps
    const int cw = warp - 2;
    const int grp = cw >> 2;                 // key columns [128 / NG * grp, 128 / NG * (grp + 1)) of every tile
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const int g_row = Rb * 128 + row;        // query position i
    const float A = P.a_scale;
    float sb = 0.f;
    if (ALIBI) sb = P.slopes[u % P.H] * LOG2E;
    bool ok = true;
    float row_m = 0.f, row_l = 0.f;
    bool started = false;

    // ---- phase A: softmax statistics of this row over this group's columns
    for (int it = 0; it < TA; ++it) {
      const int b = it % 2;
      const int dj = it * BN - Rb * 128;   // first key of the tile relative to the first query of the block
      ok = __all_sync(0xffffffffu, wait_bar(s_full + b, (uint32_t)((it / 2) & 1), abort_flag));
      if (!ok) break;
      tc_fence_after();
#pragma unroll 1
      for (int cc = 0; cc < CPG; ++cc) {
        const int c = grp * CPG + cc;
        if (dj + c * 32 > quarter * 32) continue;   // causally masked for the whole warp
        float v[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(b * BN + c * 32), v);
        if (dj + c * 32 == quarter * 32) {          // the chunk that holds the diagonal of these 32 rows
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = e <= lane ? v[e] : -INFINITY;
        }
        float bias0 = 0.f;
        if (ALIBI) bias0 = sb * (float)(it * BN + c * 32 - g_row);
        if (!started) { row_m = fmaf(v[0], A, bias0); started = true; }
        auto fold = [&](float ref, auto mode) -> float {
          constexpr bool WANT_MAX = decltype(mode)::value;
          float r0 = WANT_MAX ? -INFINITY : 0.f, r1 = r0, r2 = r0, r3 = r0;
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            float a4[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              a4[q] = fmaf(v[e + q], A, bias0 - ref);
              if (ALIBI) a4[q] = fmaf(sb, (float)(e + q), a4[q]);
            }
            if (WANT_MAX) { r0 = fmaxf(r0, a4[0]); r1 = fmaxf(r1, a4[1]); r2 = fmaxf(r2, a4[2]); r3 = fmaxf(r3, a4[3]); }
            else { r0 += fast_exp2(a4[0]); r1 += fast_exp2(a4[1]); r2 += fast_exp2(a4[2]); r3 += fast_exp2(a4[3]); }
          }
          return WANT_MAX ? fmaxf(fmaxf(r0, r1), fmaxf(r2, r3)) : (r0 + r1) + (r2 + r3);
        };
        float ref = row_m;
        float sum = fold(ref, std::false_type{});
        if (!(sum < 1e30f)) {   // a logit far above the reference: fall back to the chunk's exact maximum
          const float cm = fold(ref, std::true_type{});
          if (cm < INFINITY) { ref += cm; sum = fold(ref, std::false_type{}); }
        }
        if (ref != row_m) { row_l *= fast_exp2(row_m - ref); row_m = ref; }
        row_l += sum;
        if (row_l > 1.8446744e19f) { row_l *= 5.4210109e-20f; row_m += 64.f; }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s_empty + b);
    }
    // exchange with the thread of the other group that owns the same row
    stats[grp * 256 + row] = row_m;
    stats[grp * 256 + 128 + row] = row_l;
    __syncwarp();
    if (lane == 0) mbar_arrive(stats_bar);
    float lse = 0.f;
    if (TA == 0) lse = P.lse_in[(size_t)u * P.nblk * 128 + g_row];   // +inf past the prompt: those rows get P = 0
    if (ok && TA > 0) ok = __all_sync(0xffffffffu, wait_bar(stats_bar, 0, abort_flag));
    if (ok && TA > 0) {
      float m = row_m, l = row_l;
#pragma unroll
      for (int g = 1; g < NG; ++g) {   // the other groups' threads of this row (a sum of 0: no valid column)
        const int og = (grp + g) % NG;
        const float m1 = stats[og * 256 + row], l1 = stats[og * 256 + 128 + row];
        if (l1 > 0.f) {
          if (l > 0.f) { const float mm = fmaxf(m, m1); l = l * fast_exp2(m - mm) + l1 * fast_exp2(m1 - mm); m = mm; }
          else { m = m1; l = l1; }
        }
      }
      lse = m + log2f(l);
    }

    // ---- phase B: normalised probabilities of this group's 64 columns into the P operand
    for (int t = 0; ok && t < T; ++t) {
      const int sit = TA + t, b = sit % 2;
      const int dj = t * BN - Rb * 128;
      ok = wait_bar(s_full + b, (uint32_t)((sit / 2) & 1), abort_flag);
      if (ok && t >= 2) ok = wait_bar(p_empty + (t & 1), (uint32_t)(((t >> 1) - 1) & 1), abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
#pragma unroll 1
      for (int cc = 0; cc < CPG; ++cc) {
        const int c = grp * CPG + cc;
        uint32_t packed[16];
        if (dj + c * 32 > quarter * 32) {
#pragma unroll
          for (int e = 0; e < 16; ++e) packed[e] = 0u;
        } else {
          float v[32];
          tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(b * BN + c * 32), v);
          if (dj + c * 32 == quarter * 32) {
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] = e <= lane ? v[e] : -INFINITY;
          }
          float off = -lse;
          if (ALIBI) off += sb * (float)(t * BN + c * 32 - g_row);
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            float a0 = fmaf(v[e], A, off), a1 = fmaf(v[e + 1], A, off);
            if (ALIBI) { a0 = fmaf(sb, (float)e, a0); a1 = fmaf(sb, (float)(e + 1), a1); }
            const __half2 h = __floats2half2_rn(fast_exp2(a0), fast_exp2(a1));
            packed[e >> 1] = *reinterpret_cast<const uint32_t*>(&h);
          }
        }
        // keys 32 c .. 32 c + 31 of this row: 16 columns of binary16 pairs
        tmem_st_32x16(tmem_base + ((uint32_t)(quarter * 32) << 16) + AT_P_COL + (uint32_t)((t & 1) * (BN / 2) + c * 16), packed);
      }
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) { mbar_arrive(p_full + (t & 1)); mbar_arrive(s_empty + b); }
    }

    // ---- output: this group's half of the row
    if (ok) ok = __all_sync(0xffffffffu, wait_bar(o_full, 0, abort_flag));
    if (ok) {
      tc_fence_after();
#pragma unroll 1
      for (int oc = 0; oc < OCH; ++oc) {
        const int col = (grp * OCH + oc) * 32;
        float v[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + AT_O_COL + (uint32_t)col, v);
        if (g_row < P.n) {
          uint4* dst = reinterpret_cast<uint4*>(P.out + ((size_t)u * P.n + g_row) * D + col);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const __half2 h = __floats2half2_rn(v[8 * q4 + 2 * e], v[8 * q4 + 2 * e + 1]);
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
    const int nk = *issued_k, nv = *issued_v;
    for (int it = nk > KST ? nk - KST : 0; it < nk; ++it) (void)mbar_wait_bounded(k_full + (it % KST), (uint32_t)((it / KST) & 1), TC_WAIT_LIMIT);
    for (int it = nv > VST ? nv - VST : 0; it < nv; ++it) (void)mbar_wait_bounded(v_full + (it % VST), (uint32_t)((it / VST) & 1), TC_WAIT_LIMIT);
    (void)mbar_wait_bounded(q_full, 0, TC_WAIT_LIMIT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, AT_TMEM_COLS);
  }
}

template <int D, int BN, int KST, int VST, int NG>
cudaError_t launch_attend(const AttendParams& P, int units, bool alibi, cudaStream_t st) {
  constexpr size_t need = 1024 + (size_t)128 * D * 2 + (size_t)(KST + VST) * BN * D * 2 + NG * 2 * 128 * 4 + 32 * 8 + 64;
  constexpr size_t smem = need < 120 * 1024 ? 120 * 1024 : need;   // one CTA per SM: it takes all of tensor memory
  static_assert(smem <= 227 * 1024, "shared memory budget of one CTA");
  dim3 grid((unsigned)P.nblk, (unsigned)units);
  auto go = [&](auto kern) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, at_threads(NG), smem, st>>>(P);
    return cudaGetLastError();
  };
  return alibi ? go(prefill_attend<D, BN, KST, VST, NG, true>) : go(prefill_attend<D, BN, KST, VST, NG, false>);
}

}  // namespace

cudaError_t launch_prefill_attend(const PrefillAttendArgs& a, int head_dim, int units, cudaStream_t stream) {
  if (a.n < 1 || units < 1 || units > 65535) return cudaErrorInvalidValue;
  AttendParams P{};
  const int bn = head_dim == 256 ? 64 : 128;   // key / value rows per tile
  if (!make_operand_map(&P.tmQ, a.Q, units, a.n, head_dim, 128)) return cudaErrorNotSupported;
  if (a.group < 1 || units % a.group != 0) return cudaErrorInvalidValue;
  if (!make_operand_map(&P.tmK, a.K, units / a.group, a.n, head_dim, bn)) return cudaErrorNotSupported;
  if (!make_operand_map(&P.tmV, a.V, units / a.group, a.n, head_dim, bn)) return cudaErrorNotSupported;
  P.out = a.out;
  P.lse_in = a.lse_x;
  P.slopes = a.slopes;
  P.err = a.err;
  P.n = a.n;
  P.nblk = (a.n + 127) / 128;
  P.H = a.H;
  P.group = a.group;
  P.a_scale = a.scale * LOG2E;
  const bool alibi = a.bias_mode == 1 && a.slopes != nullptr;
  switch (head_dim) {
    case 64: return launch_attend<64, 128, 3, 2, 2>(P, units, alibi, stream);
    case 128: return launch_attend<128, 128, 3, 2, 4>(P, units, alibi, stream);
    case 256: return launch_attend<256, 64, 2, 2, 2>(P, units, alibi, stream);   // 64-row key tiles: the 64 KB query block leaves room for no more
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace kf
