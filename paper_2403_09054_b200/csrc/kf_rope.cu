// Rotary position embedding applied by the library (section 4.4.2 of the paper compares original with new positional
// information on rotary models too; for that the cache keeps keys without rotation).  Interleaved pairs: features
// (2i, 2i+1), i < R/2, are rotated by pos * base^(-2i/R).
//   rope_table_kernel   cos / sin of dist * theta_i for every distance the context can meet, computed in double
//                       precision (a binary32 product dist * theta is off by 1e-3 rad at positions in the thousands)
//   rope_rotate_kernel  prompt phase: rows rotated at their own positions into a scratch copy, which the scoring and
//                       attention kernels then read (the cache itself is filled from the caller's unrotated rows)
#include "kf_prefill.cuh"

namespace kf {

namespace {

__global__ void __launch_bounds__(256) rope_table_kernel(float2* __restrict__ table, int n_dist, int half, double base) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)n_dist * half) return;
  const int dist = (int)(idx / half), i = (int)(idx % half);
  const double theta = pow(base, -(double)i / (double)half);   // base^(-2i/R), R = 2 half
  double s, c;
  sincos((double)dist * theta, &s, &c);
  table[idx] = make_float2((float)c, (float)s);
}

// One thread per pair of features of one row; rows of a unit are positions 0 .. n-1.
__global__ void __launch_bounds__(256) rope_rotate_kernel(const __half* __restrict__ src, __half* __restrict__ dst,
                                                          const float2* __restrict__ table, long long rows, int n, int d, int half) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;   // (row, pair) with d / 2 pairs per row
  const int pairs = d >> 1;
  if (idx >= rows * pairs) return;
  const long long row = idx / pairs;
  const int i = (int)(idx % pairs);
  const __half2 v = reinterpret_cast<const __half2*>(src)[idx];
  __half2 out = v;
  if (i < half) {
    const int pos = (int)(row % n);
    const float2 cs = table[(size_t)pos * half + i];
    const float x0 = __low2float(v), x1 = __high2float(v);
    out = __floats2half2_rn(x0 * cs.x - x1 * cs.y, x0 * cs.y + x1 * cs.x);
  }
  reinterpret_cast<__half2*>(dst)[idx] = out;
}

}  // namespace

cudaError_t launch_rope_table(float2* table, int n_dist, int rotary_dims, double base, cudaStream_t stream) {
  const int half = rotary_dims / 2;
  const long long total = (long long)n_dist * half;
  rope_table_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(table, n_dist, half, base);
  return cudaGetLastError();
}

cudaError_t launch_rope_rotate(const __half* src, __half* dst, const float2* table, int units, int n, int head_dim, int rotary_dims,
                               cudaStream_t stream) {
  const long long rows = (long long)units * n, total = rows * (head_dim / 2);
  rope_rotate_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(src, dst, table, rows, n, head_dim, rotary_dims / 2);
  return cudaGetLastError();
}

}  // namespace kf
