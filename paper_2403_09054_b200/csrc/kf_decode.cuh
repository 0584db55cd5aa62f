// Launch interface of the generation-phase kernel (see kf_decode.cu).
#pragma once

#include <cuda.h>

#include "kf_common.cuh"

namespace kf {

struct DecodeParams {
  const __half* K;        // [units][k][d] cache of this layer
  const __half* V;
  float* acc;             // [units][k]  accumulated score f_theta
  int32_t* pos;           // [units][k]  original token positions
  int32_t* len;           // [units]     entries in use
  int32_t* place;         // [units][k]  place of each entry within the cache in position order, or null when the
                          //             bias uses the original positions (section 4.4.2)
  const __half* q;        // [units][group][d]   (a unit is a cache: one (batch row, key/value head))
  const __half* knew;     // [units][d]
  const __half* vnew;     // [units][d]
  __half* out;            // [units][group][d]
  float* score_opt;       // [units][k+1] or null
  float* y_scratch;       // [units][group][k+1] adjusted logits (x + zeta) / tau
  float* partials;        // [units][splits][group][4 + d]
  int* err;               // device error word
  const float* slopes;    // [H] ALiBi slopes or null
  const float2* rope_tab; // [distance][rot_chunks * 4] (cos, sin) of distance * theta_i, or null: the rotary embedding is applied
                          //   to the first rot_chunks * 8 features when a logit is formed (the cache holds unrotated keys)
  int32_t rot_chunks;     // rotary features / 8 (a power of two), 0 without
  int32_t k, w, p;        // budget, recent window, position of the query token
  int32_t splits, tiles_per_split;
  int32_t H, layer, noise_mode, bias_mode;   // H = query heads
  int32_t group;          // query heads per key/value head (H / group caches per batch row)
  float scale, inv_tau, noise_const, noise_mu, noise_sigma;
  uint32_t first_wait_limit;   // polls the streaming kernel grants its first tile (DECODE_WAIT_LIMIT; 0 in the self-test
                               // that makes a wait run out: the warp gives up at once, then drains with the full limit)
  PhiloxKeys pk;
};

constexpr uint32_t DECODE_WAIT_LIMIT = 1u << 22;   // polls of a bounded wait in the generation kernels

#ifdef __CUDACC__
// zeta of Eq. 4 for logit (query position i, key position j) of (batch b, layer * H + head lh), by adjustment mode.
__device__ __forceinline__ float noise_for(const DecodeParams& P, uint32_t b, uint32_t lh, uint32_t i, uint32_t j) {
  if (P.noise_mode == 0) return gumbel_from_word(noise_word(P.pk, b, lh, i, j));
  if (P.noise_mode == 2) return P.noise_const;
  if (P.noise_mode == 3)
    return fmaf(P.noise_sigma, gauss_from_words(noise_word(P.pk, b, lh, i, j), noise_word(P.pk, b | GAUSS_PLANE, lh, i, j)), P.noise_mu);
  return 0.f;
}
#endif

// Size of the built-in scratch block used by kf_decode_step_static (16 MiB per GPU).
constexpr size_t STATIC_SCRATCH_BYTES = (size_t)16 << 20;

int decode_tile_rows();
int decode_max_splits();
// How a layer call is cut into CTAs: `splits` CTAs per unit, each streaming `tiles_per_split` 32-row tiles.
// `requested` = 0 lets the grid fill the 148 SMs several times over.  The scratch layout follows from it.
void decode_plan(int units, int budget_k, int requested, int* splits, int* tiles_per_split);
cudaError_t launch_decode(const DecodeParams& P, int head_dim, int units, cudaStream_t stream);
// Names the kernels (with their template arguments) and the split plan of a layer call of this shape; snprintf semantics.
// For the tensor-core kernel `splits` = partials per cache and `tiles_per_split` = CTAs of the launch.
int decode_describe(char* buf, size_t n, int head_dim, int units, int budget_k, int splits, int tiles_per_split, bool new_pos,
                    int group, bool tensor_cores, bool rotary);
// Tensor-core streaming kernel for query heads sharing a cache (see kf_decode_tc.cu), followed by the same closing kernel.
// `tmK`, `tmV`: TMA maps of the layer's cache built by decode_tc_cache_maps (they depend on the cache addresses only).
bool decode_tc_supported(int head_dim, int group);
bool decode_tc_cache_maps(CUtensorMap* tmK, CUtensorMap* tmV, const __half* K, const __half* V, int units, int budget_k, int head_dim);
cudaError_t launch_decode_tc(DecodeParams P, const CUtensorMap& tmK, const CUtensorMap& tmV, int head_dim, int units,
                             cudaStream_t stream);
// CTAs of a tensor-core launch and the partials it leaves per cache (needs the current device's SM count).
cudaError_t decode_tc_plan(int units, int budget_k, int* ctas, int* pieces);

// Closing kernel alone (merge, normalise, accumulate, evict, replace), behind a streaming kernel launched elsewhere.
cudaError_t launch_decode_close(const DecodeParams& P, int head_dim, int units, cudaStream_t stream);
bool decode_group_supported(int group);   // query heads per key/value head the generation kernels are built for

// Reorders every unit's entries of one layer into ascending position, in place (see kf_compact.cu).  `place` may be
// null; `dst_scratch` is [units][k] int32 of scratch.  Budgets above compact_max_k() are refused (cudaErrorInvalidValue).
int compact_max_k();
cudaError_t launch_compact(__half* K, __half* V, float* acc, int32_t* pos, const int32_t* len, int32_t* place,
                           int32_t* dst_scratch, int k, int head_dim, int units, cudaStream_t stream);

// place[j] = number of entries of the unit with a smaller position, for every unit of a layer (after a state import).
cudaError_t launch_rebuild_place(const int32_t* pos, const int32_t* len, int32_t* place, int k, int units,
                                 cudaStream_t stream);

// Same launch with y_scratch / partials carved out of the built-in scratch block
// (the sizes are in bytes, each a multiple of 256).  Allocates nothing.
cudaError_t launch_decode_static(DecodeParams P, int head_dim, int units, size_t y_bytes, size_t partial_bytes,
                                 cudaStream_t stream);

}  // namespace kf
