// Launch interface of the prompt-phase kernels (see kf_prefill_tc.cu and kf_prefill_simt.cu).
#pragma once

#include <cuda.h>

#include "kf_common.cuh"

namespace kf {

struct PrefillParams {
  const __half* Q;     // [units][n][d]            a unit here is a (batch row, query head)
  const __half* K;     // [units / group][n][d]    query heads of a group read the same keys
  float* acc_full;     // [units][n] f_theta of each query head before pruning (zeroed by the caller)
  const float* slopes; // [H] or null
  int* err;
  int32_t group;       // query heads per key/value head
  int32_t n, H, layer, noise_mode, bias_mode;
  float scale, inv_tau, noise_const, noise_mu, noise_sigma;
  PhiloxKeys pk;
};

struct SelectParams {
  const float* acc_full; // [units][n]
  int32_t* idx;          // [units][k] kept positions, ascending, -1 padded
  int32_t* len;          // [units]
  int* err;
  int32_t n, k, w;
};

struct GatherParams {
  const __half* K;       // prompt [units][n][d]
  const __half* V;
  const float* acc_full; // [units][n]
  const int32_t* idx;    // [units][k]
  __half* Kc;            // cache [units][k][d]
  __half* Vc;
  int32_t* pos;          // [units][k]
  float* acc;            // [units][k]
  int32_t* place;        // [units][k] or null: place within the cache (= slot, the rows are stored in position order)
  int32_t n, k;
};

// Kernel parameters of the tensor-core scoring kernel (both sweeps).
struct PrefillTcParams {
  CUtensorMap tmQ;     // fp16 [units][n][d], 64 x 128 boxes, 128-byte swizzle
  CUtensorMap tmK;
  float* lse2;         // [units][nblk * 128] log2-domain log-sum-exp of every query row (+inf past n)
  float* lse_x;        // same for the plain logits x (sweep 1 fills it when non-null), or null
  float* acc_full;     // [units][n] f_theta before pruning
  const float* slopes; // [H] or null
  int* err;
  int32_t n, nblk, H, layer;
  int32_t units;       // (batch row, query head) pairs of the call
  int32_t group;       // query heads per key/value head: unit u reads the keys of cache u / group
  float a_scale;       // logit scale * log2(e) / tau
  float ax;            // logit scale * log2(e)
  float c1;            // log2(e) / tau
  float inv_tau;
  float const_term;    // constant logit adjustment in the scaled log2 domain (0 without one)
  float gauss_scale;   // noise_sigma * log2(e) / tau (Gaussian adjustment)
  PhiloxKeys pk;
};

// What the caller of the tensor-core scoring provides.
struct PrefillTcArgs {
  const __half* Q;     // [units][n][d]           units = (batch row, query head) pairs
  const __half* K;     // [units / group][n][d]
  int32_t group;       // query heads per key/value head
  float* lse2;         // scratch, prefill_tc_lse_floats(units, n) floats
  float* lse_x;        // null, or a second such array: receives the plain softmax statistics of the prompt rows
  float* acc_full;     // [units][n], fully overwritten
  const float* slopes;
  int* err;
  int32_t n, H, layer, noise_mode, bias_mode;
  float scale, inv_tau, noise_const, noise_mu, noise_sigma;
  PhiloxKeys pk;
};

// Causal attention output of the prompt (see kf_prefill_attend.cu).
struct PrefillAttendArgs {
  const __half* Q;     // [units][n][d]           units = (batch row, query head) pairs
  const __half* K;     // [units / group][n][d]
  const __half* V;     // [units / group][n][d]
  int32_t group;       // query heads per key/value head
  __half* out;         // [units][n][d]
  const float* lse_x;  // null, or the rows' log2-domain log-sum-exp from the scoring sweep (skips the statistics phase)
  const float* slopes; // [H] or null
  int* err;
  int32_t n, H, bias_mode;
  float scale;
};
cudaError_t launch_prefill_attend(const PrefillAttendArgs& a, int head_dim, int units, cudaStream_t stream);
// The same output in one pass over the keys (running maximum, head_dim 64 and 128; see kf_prefill_attend1p.cu); `lse_x` is not used.
bool prefill_attend_one_pass_supported(int head_dim);
cudaError_t launch_prefill_attend_one_pass(const PrefillAttendArgs& a, int head_dim, int units, cudaStream_t stream);

// Rotary embedding applied by the library (see kf_rope.cu).  `table`: [n_dist][rotary_dims / 2] (cos, sin) of dist * theta_i.
cudaError_t launch_rope_table(float2* table, int n_dist, int rotary_dims, double base, cudaStream_t stream);
// dst = src with the first rotary_dims features of row j of every unit ([units][n][head_dim]) rotated at position j.
cudaError_t launch_rope_rotate(const __half* src, __half* dst, const float2* table, int units, int n, int head_dim, int rotary_dims,
                               cudaStream_t stream);

size_t prefill_tc_lse_floats(int units, int n_max);
cudaError_t launch_prefill_score_tc(const PrefillTcArgs& a, int head_dim, int units, cudaStream_t stream);
cudaError_t launch_prefill_score_simt(const PrefillParams& P, int head_dim, int units, cudaStream_t stream);
cudaError_t launch_prefill_select(const SelectParams& P, int units, cudaStream_t stream);
// dst[c][j] = mean over r < group of src[c * group + r][j]: the prompt scores of a cache from those of its query heads
// (a fixed summation order, r ascending).
cudaError_t launch_group_mean(const float* src, float* dst, int caches, int group, int n, cudaStream_t stream);
cudaError_t launch_prefill_gather(const GatherParams& P, int head_dim, int units, cudaStream_t stream);

}  // namespace kf
