// Launch interface of the prompt-phase kernels (see kf_prefill_simt.cu).
#pragma once

#include "kf_common.cuh"

namespace kf {

struct PrefillParams {
  const __half* Q;     // [units][n][d]
  const __half* K;     // [units][n][d]
  float* acc_full;     // [units][n] f_theta before pruning (zeroed by the caller)
  const float* slopes; // [H] or null
  int* err;
  int32_t n, H, layer, noise_mode, bias_mode;
  float scale, inv_tau, noise_const;
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
  int32_t n, k;
};

cudaError_t launch_prefill_score_simt(const PrefillParams& P, int head_dim, int units, cudaStream_t stream);
cudaError_t launch_prefill_select(const SelectParams& P, int units, cudaStream_t stream);
cudaError_t launch_prefill_gather(const GatherParams& P, int head_dim, int units, cudaStream_t stream);

}  // namespace kf
