// C ABI of the library (see include/keyformer.h): configuration checks,
// workspace carving, temperature schedule (Eq. 12) and kernel launches.
#include "keyformer.h"

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "kf_decode.cuh"
#include "kf_prefill.cuh"

namespace {

constexpr size_t ALIGN = 256;
inline size_t align_up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }
inline bool misaligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

constexpr size_t GUARD_BYTES = 256;
constexpr int GUARD_BYTE = 0xA5;

struct Layout {
  size_t K, V, acc, pos, len;          // per-layer strides are kv_layer / sc_layer / len_layer
  size_t place;                        // KF_POS_NEW only (sc_layer per layer)
  size_t y_scratch, partials, err, slopes;
  size_t acc_full, idx, staging, lse2, lse_x;
  size_t total;
  size_t kv_layer, sc_layer, len_layer; // bytes per layer
  int units, max_splits;               // units = caches of a layer = batch x key/value heads
  int units_q, group;                  // batch x query heads; query heads per key/value head
  size_t acc_q;                        // group > 1 only: prompt scores per query head, before the group mean
  size_t rope_tab, q_rot, k_rot;       // rotary_dims > 0 only: cos / sin table, rotated copies of the prompt's Q and K
  int rope_dists;                      // distances the table covers: 0 .. max_prompt_len + max(T, 1) - 1
  // debug_canaries: a guard of GUARD_BYTES follows every sub-buffer; `guards` holds their offsets in layout order
  // (K, V, acc, pos, len, y_scratch, partials, err, slopes, acc_full, idx, staging, lse2, lse_x, [place], [acc_q],
  //  [rotary table, rotated Q, rotated K])
  std::vector<size_t> guards;
};

bool config_ok(const kf_config* c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->batch < 1 || c->n_heads < 1) return false;
  if (c->head_dim != 64 && c->head_dim != 128 && c->head_dim != 256) return false;
  if (c->budget_k < 1 || c->recent_w < 0 || c->recent_w > c->budget_k) return false;
  if (c->max_prompt_len < 1 || c->gen_len_T < 0) return false;
  if (!(c->tau_init > 0.f) || !(c->tau_end > 0.f)) return false;
  if (c->noise_mode < KF_NOISE_GUMBEL || c->noise_mode > KF_NOISE_GAUSS) return false;
  if (c->noise_mode == KF_NOISE_GAUSS && !(c->noise_sigma >= 0.f)) return false;
  if (c->bias_mode != KF_BIAS_NONE && c->bias_mode != KF_BIAS_ALIBI) return false;
  if (c->bias_mode == KF_BIAS_ALIBI && !c->h_alibi_slopes) return false;
  if (c->logit_scale < 0.f || c->decode_splits < 0 || c->decode_splits > kf::decode_max_splits()) return false;
  if (c->prefill_impl != KF_PREFILL_TENSOR && c->prefill_impl != KF_PREFILL_SIMT) return false;
  if (c->pos_mode != KF_POS_ORIGINAL && c->pos_mode != KF_POS_NEW) return false;
  if ((int64_t)c->batch * c->n_heads > 65535) return false;  // grid.y limit
  if (c->n_kv_heads < 0 || c->n_kv_heads > c->n_heads) return false;
  if (c->n_kv_heads > 0 && (c->n_heads % c->n_kv_heads != 0 || !kf::decode_group_supported(c->n_heads / c->n_kv_heads))) return false;
  if (c->rotary_dims < 0 || c->rotary_dims > c->head_dim || (c->rotary_dims & (c->rotary_dims - 1)) != 0 ||
      (c->rotary_dims > 0 && c->rotary_dims < 8))
    return false;   // 0, or a power of two from 8 to head_dim
  if (c->rotary_dims > 0 && !(c->rotary_base > 1.0f)) return false;
  if (c->rotary_dims > 0 && c->decode_impl == KF_DECODE_TENSOR) return false;   // the tensor-core kernel reads keys as stored
  if (c->decode_impl < KF_DECODE_AUTO || c->decode_impl > KF_DECODE_TENSOR) return false;
  if (c->decode_impl == KF_DECODE_TENSOR &&
      !kf::decode_tc_supported(c->head_dim, c->n_kv_heads > 0 ? c->n_heads / c->n_kv_heads : 1)) return false;
  if (c->debug_canaries < 0 || c->debug_canaries > 1 || c->debug_fail_first_wait < 0 || c->debug_fail_first_wait > 1) return false;
  return true;
}

// Which streaming kernel the generation step uses: the tensor-core one where it is built (head_dim 128) and pays
// (several query heads per cache), unless the configuration asks for one of them.
bool decode_uses_tensor_cores(const kf_config* c) {
  const int hkv = c->n_kv_heads > 0 ? c->n_kv_heads : c->n_heads;
  const int group = c->n_heads / hkv;
  if (c->decode_impl == KF_DECODE_CUDA_CORES || c->rotary_dims > 0) return false;
  if (c->decode_impl == KF_DECODE_TENSOR) return true;
  return group >= 2 && kf::decode_tc_supported(c->head_dim, group);
}

Layout make_layout(const kf_config* c) {
  Layout L{};
  const int hkv = c->n_kv_heads > 0 ? c->n_kv_heads : c->n_heads;
  const size_t units = (size_t)c->batch * hkv, units_q = (size_t)c->batch * c->n_heads;
  const size_t k = (size_t)c->budget_k, d = (size_t)c->head_dim, nl = (size_t)c->n_layers;
  L.units = (int)units;
  L.units_q = (int)units_q;
  L.group = c->n_heads / hkv;
  L.max_splits = kf::decode_max_splits();
  L.kv_layer = align_up(units * k * d * 2);
  L.sc_layer = align_up(units * k * 4);
  L.len_layer = align_up(units * 4);
  size_t off = 0;
  auto carve = [&](size_t bytes) {   // appends a sub-buffer (and, in the debug layout, the guard behind it)
    const size_t at = off;
    off += bytes;
    if (c->debug_canaries) { L.guards.push_back(off); off += GUARD_BYTES; }
    return at;
  };
  L.K = carve(nl * L.kv_layer);
  L.V = carve(nl * L.kv_layer);
  L.acc = carve(nl * L.sc_layer);
  L.pos = carve(nl * L.sc_layer);
  L.len = carve(nl * L.len_layer);
  L.y_scratch = carve(align_up(units_q * (k + 1) * 4));
  L.partials = carve(align_up(units_q * (size_t)L.max_splits * (4 + d) * 4));
  L.err = carve(ALIGN);
  L.slopes = carve(align_up((size_t)c->n_heads * 4));
  L.acc_full = carve(align_up(units * (size_t)c->max_prompt_len * 4));
  L.idx = carve(align_up(units * k * 4));
  L.staging = carve(8 * align_up(units_q * d * 2));   // two sets of (q, k_new, v_new, out)
  L.lse2 = carve(align_up(kf::prefill_tc_lse_floats((int)units_q, c->max_prompt_len) * 4));
  L.lse_x = carve(align_up(kf::prefill_tc_lse_floats((int)units_q, c->max_prompt_len) * 4));
  L.place = off;
  if (c->pos_mode == KF_POS_NEW) L.place = carve(nl * L.sc_layer);
  L.acc_q = off;
  if (L.group > 1) L.acc_q = carve(align_up(units_q * (size_t)c->max_prompt_len * 4));
  L.rope_tab = L.q_rot = L.k_rot = off;
  L.rope_dists = c->max_prompt_len + (c->gen_len_T > 1 ? c->gen_len_T : 1);
  if (c->rotary_dims > 0) {
    L.rope_tab = carve(align_up((size_t)L.rope_dists * (c->rotary_dims / 2) * 8));
    L.q_rot = carve(align_up(units_q * (size_t)c->max_prompt_len * d * 2));
    L.k_rot = carve(align_up(units * (size_t)c->max_prompt_len * d * 2));
  }
  L.total = off;
  return L;
}

}  // namespace

struct kf_ctx {
  kf_config cfg;
  Layout lay;
  unsigned char* ws;
  kf::PhiloxKeys pk;
  float scale;
  std::vector<int32_t> n_prompt;   // per layer, -1 before prefill
  std::vector<int32_t> last_step;  // per layer
  int64_t launches;
  // tensor-core generation kernel: TMA maps of every layer's cache (built on first use; they depend on addresses only)
  bool decode_tc = false;
  std::vector<CUtensorMap> tmK, tmV;
  std::vector<char> tm_ready;
  // kf_decode_step_host: copy streams and events (created on first use), two staging sets used alternately
  cudaStream_t copy_in = nullptr, copy_out = nullptr;
  cudaEvent_t in_done[2] = {nullptr, nullptr}, kernel_done[2] = {nullptr, nullptr}, out_done[2] = {nullptr, nullptr};
  int64_t host_calls = 0;
};

extern "C" {

size_t kf_workspace_bytes(const kf_config* cfg) {
  if (!config_ok(cfg)) return 0;
  return make_layout(cfg).total;
}

int kf_create(const kf_config* cfg, void* d_workspace, size_t workspace_bytes, void* stream, kf_ctx** out) {
  if (!out) return KF_EINVAL;
  *out = nullptr;
  if (!config_ok(cfg) || !d_workspace) return KF_EINVAL;
  if (((uintptr_t)d_workspace) % ALIGN != 0) return KF_EINVAL;
  const Layout lay = make_layout(cfg);
  if (workspace_bytes < lay.total) return KF_ENOSPC;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return KF_ECUDA;
  kf_ctx* ctx = new (std::nothrow) kf_ctx();
  if (!ctx) return KF_EINVAL;
  ctx->cfg = *cfg;
  ctx->cfg.h_alibi_slopes = nullptr;  // copied below; the caller's array is not referenced later
  ctx->lay = lay;
  ctx->ws = static_cast<unsigned char*>(d_workspace);
  ctx->pk = kf::philox_expand_key(cfg->noise_seed);
  ctx->scale = cfg->logit_scale > 0.f ? cfg->logit_scale : (float)(1.0 / std::sqrt((double)cfg->head_dim));
  ctx->n_prompt.assign(cfg->n_layers, -1);
  ctx->last_step.assign(cfg->n_layers, 0);
  ctx->launches = 0;
  ctx->decode_tc = decode_uses_tensor_cores(cfg);
  ctx->tmK.resize(cfg->n_layers);
  ctx->tmV.resize(cfg->n_layers);
  ctx->tm_ready.assign(cfg->n_layers, 0);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemsetAsync(ctx->ws + lay.acc, 0, lay.y_scratch - lay.acc, st);  // acc, pos, len
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->ws + lay.err, 0, lay.slopes - lay.err, st);  // error word
  if (e == cudaSuccess && cfg->bias_mode == KF_BIAS_ALIBI)
    e = cudaMemcpyAsync(ctx->ws + lay.slopes, cfg->h_alibi_slopes, (size_t)cfg->n_heads * 4, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess && cfg->bias_mode == KF_BIAS_ALIBI) e = cudaStreamSynchronize(st);  // host array may go away
  if (e == cudaSuccess && cfg->rotary_dims > 0)
    e = kf::launch_rope_table(reinterpret_cast<float2*>(ctx->ws + lay.rope_tab), lay.rope_dists, cfg->rotary_dims,
                              (double)cfg->rotary_base, st);
  for (size_t g = 0; e == cudaSuccess && g < lay.guards.size(); ++g)   // after the clears above, which span some guards
    e = cudaMemsetAsync(ctx->ws + lay.guards[g], GUARD_BYTE, GUARD_BYTES, st);
  if (e != cudaSuccess) { delete ctx; return KF_ECUDA; }
  *out = ctx;
  return KF_OK;
}

// `want_x`: the scoring sweep also leaves the plain softmax statistics of the prompt rows in the workspace
// (tensor-core scoring only), for the attention output kernel.
static int prefill_score_prune_impl(kf_ctx* ctx, int32_t layer, int32_t n_prompt,
                                    const void* d_q, const void* d_k, const void* d_v,
                                    float* d_score_opt, bool want_x, void* stream) {
  if (!ctx || !d_q || !d_k || !d_v) return KF_EINVAL;
  const kf_config& c = ctx->cfg;
  if (layer < 0 || layer >= c.n_layers) return KF_EINVAL;
  if (n_prompt < 1 || n_prompt > c.max_prompt_len) return KF_EINVAL;
  // rows are read 16 bytes at a time (TMA boxes, 128-bit loads in the gather)
  if (misaligned16(d_q) || misaligned16(d_k) || misaligned16(d_v)) return KF_EINVAL;
  const Layout& L = ctx->lay;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  float* acc_full = d_score_opt ? d_score_opt : reinterpret_cast<float*>(ctx->ws + L.acc_full);
  // with shared key/value heads the scoring kernels leave one f_theta per query head; their mean over a group is the cache's
  float* acc_scored = L.group > 1 ? reinterpret_cast<float*>(ctx->ws + L.acc_q) : acc_full;
  int* err = reinterpret_cast<int*>(ctx->ws + L.err);
  const float* slopes = c.bias_mode == KF_BIAS_ALIBI ? reinterpret_cast<const float*>(ctx->ws + L.slopes) : nullptr;
  const float inv_tau = (float)(1.0 / (double)c.tau_init);  // the prompt phase is iteration t = 0 of Eq. 12
  const void* d_k_rows = d_k;   // the cache is filled from the caller's rows (unrotated when the library applies the embedding)
  if (c.rotary_dims > 0) {
    // nothing has been dropped yet: every token is rotated at its own position; the scoring kernels read the copies
    const float2* tab = reinterpret_cast<const float2*>(ctx->ws + L.rope_tab);
    __half* qr = reinterpret_cast<__half*>(ctx->ws + L.q_rot);
    __half* kr = reinterpret_cast<__half*>(ctx->ws + L.k_rot);
    if (kf::launch_rope_rotate(static_cast<const __half*>(d_q), qr, tab, L.units_q, n_prompt, c.head_dim, c.rotary_dims, st) != cudaSuccess ||
        kf::launch_rope_rotate(static_cast<const __half*>(d_k), kr, tab, L.units, n_prompt, c.head_dim, c.rotary_dims, st) != cudaSuccess)
      return KF_ECUDA;
    ctx->launches += 2;
    d_q = qr;
    d_k = kr;
  }
  if (c.prefill_impl == KF_PREFILL_TENSOR) {
    kf::PrefillTcArgs A{};
    A.Q = static_cast<const __half*>(d_q);
    A.K = static_cast<const __half*>(d_k);
    A.lse2 = reinterpret_cast<float*>(ctx->ws + L.lse2);
    A.lse_x = want_x ? reinterpret_cast<float*>(ctx->ws + L.lse_x) : nullptr;
    A.acc_full = acc_scored;
    A.slopes = slopes;
    A.err = err;
    A.group = L.group;
    A.n = n_prompt; A.H = c.n_heads; A.layer = layer; A.noise_mode = c.noise_mode; A.bias_mode = c.bias_mode;
    A.scale = ctx->scale; A.inv_tau = inv_tau; A.noise_const = c.noise_const;
    A.noise_mu = c.noise_mu; A.noise_sigma = c.noise_sigma;
    A.pk = ctx->pk;
    if (kf::launch_prefill_score_tc(A, c.head_dim, L.units_q, st) != cudaSuccess) return KF_ECUDA;
    ctx->launches += 2;
  } else {
    if (cudaMemsetAsync(acc_scored, 0, (size_t)L.units_q * n_prompt * 4, st) != cudaSuccess) return KF_ECUDA;
    kf::PrefillParams P{};
    P.Q = static_cast<const __half*>(d_q);
    P.K = static_cast<const __half*>(d_k);
    P.acc_full = acc_scored;
    P.slopes = slopes;
    P.err = err;
    P.group = L.group;
    P.n = n_prompt; P.H = c.n_heads; P.layer = layer; P.noise_mode = c.noise_mode; P.bias_mode = c.bias_mode;
    P.scale = ctx->scale;
    P.inv_tau = inv_tau;
    P.noise_const = c.noise_const;
    P.noise_mu = c.noise_mu; P.noise_sigma = c.noise_sigma;
    P.pk = ctx->pk;
    if (kf::launch_prefill_score_simt(P, c.head_dim, L.units_q, st) != cudaSuccess) return KF_ECUDA;
    ctx->launches += 1;
  }
  if (L.group > 1) {
    if (kf::launch_group_mean(acc_scored, acc_full, L.units, L.group, n_prompt, st) != cudaSuccess) return KF_ECUDA;
    ctx->launches += 1;
  }

  kf::SelectParams S{};
  S.acc_full = acc_full;
  S.idx = reinterpret_cast<int32_t*>(ctx->ws + L.idx);
  S.len = reinterpret_cast<int32_t*>(ctx->ws + L.len + (size_t)layer * L.len_layer);
  S.err = err;
  S.n = n_prompt; S.k = c.budget_k; S.w = c.recent_w;
  if (kf::launch_prefill_select(S, L.units, st) != cudaSuccess) return KF_ECUDA;

  kf::GatherParams G{};
  G.K = static_cast<const __half*>(d_k_rows);
  G.V = static_cast<const __half*>(d_v);
  G.acc_full = acc_full;
  G.idx = S.idx;
  G.Kc = reinterpret_cast<__half*>(ctx->ws + L.K + (size_t)layer * L.kv_layer);
  G.Vc = reinterpret_cast<__half*>(ctx->ws + L.V + (size_t)layer * L.kv_layer);
  G.pos = reinterpret_cast<int32_t*>(ctx->ws + L.pos + (size_t)layer * L.sc_layer);
  G.acc = reinterpret_cast<float*>(ctx->ws + L.acc + (size_t)layer * L.sc_layer);
  G.place = c.pos_mode == KF_POS_NEW ? reinterpret_cast<int32_t*>(ctx->ws + L.place + (size_t)layer * L.sc_layer) : nullptr;
  G.n = n_prompt; G.k = c.budget_k;
  if (kf::launch_prefill_gather(G, c.head_dim, L.units, st) != cudaSuccess) return KF_ECUDA;

  ctx->launches += 2;
  ctx->n_prompt[layer] = n_prompt;
  ctx->last_step[layer] = 0;
  return KF_OK;
}

int kf_prefill_score_prune(kf_ctx* ctx, int32_t layer, int32_t n_prompt,
                           const void* d_q, const void* d_k, const void* d_v,
                           float* d_score_opt, void* stream) {
  return prefill_score_prune_impl(ctx, layer, n_prompt, d_q, d_k, d_v, d_score_opt, false, stream);
}

static int prefill_attend_impl(kf_ctx* ctx, int32_t n_prompt, const void* d_q, const void* d_k, const void* d_v,
                               void* d_out, bool have_lse_x, void* stream) {
  if (!ctx || !d_q || !d_k || !d_v || !d_out) return KF_EINVAL;
  const kf_config& c = ctx->cfg;
  if (n_prompt < 1 || n_prompt > c.max_prompt_len) return KF_EINVAL;
  if ((reinterpret_cast<uintptr_t>(d_q) | reinterpret_cast<uintptr_t>(d_k) | reinterpret_cast<uintptr_t>(d_v) |
       reinterpret_cast<uintptr_t>(d_out)) & 15u)
    return KF_EINVAL;
  const Layout& L = ctx->lay;
  if (c.rotary_dims > 0) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float2* tab = reinterpret_cast<const float2*>(ctx->ws + L.rope_tab);
    __half* qr = reinterpret_cast<__half*>(ctx->ws + L.q_rot);
    __half* kr = reinterpret_cast<__half*>(ctx->ws + L.k_rot);
    if (kf::launch_rope_rotate(static_cast<const __half*>(d_q), qr, tab, L.units_q, n_prompt, c.head_dim, c.rotary_dims, st) != cudaSuccess ||
        kf::launch_rope_rotate(static_cast<const __half*>(d_k), kr, tab, L.units, n_prompt, c.head_dim, c.rotary_dims, st) != cudaSuccess)
      return KF_ECUDA;
    ctx->launches += 2;
    d_q = qr;
    d_k = kr;
  }
  kf::PrefillAttendArgs A{};
  A.Q = static_cast<const __half*>(d_q);
  A.K = static_cast<const __half*>(d_k);
  A.V = static_cast<const __half*>(d_v);
  A.out = static_cast<__half*>(d_out);
  A.lse_x = have_lse_x ? reinterpret_cast<const float*>(ctx->ws + L.lse_x) : nullptr;
  A.slopes = c.bias_mode == KF_BIAS_ALIBI ? reinterpret_cast<const float*>(ctx->ws + L.slopes) : nullptr;
  A.err = reinterpret_cast<int*>(ctx->ws + L.err);
  A.n = n_prompt; A.H = c.n_heads; A.bias_mode = c.bias_mode;
  A.group = L.group;
  A.scale = ctx->scale;
  // one pass over the keys where that kernel is built (head_dim 64, 128); the two-phase kernel otherwise, which can take
  // the rows' softmax statistics from the scoring sweep
  const cudaError_t e = (!have_lse_x && kf::prefill_attend_one_pass_supported(c.head_dim))
                            ? kf::launch_prefill_attend_one_pass(A, c.head_dim, L.units_q, static_cast<cudaStream_t>(stream))
                            : kf::launch_prefill_attend(A, c.head_dim, L.units_q, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return KF_ECUDA;
  ctx->launches += 1;
  return KF_OK;
}

int kf_prefill_attend_score_prune(kf_ctx* ctx, int32_t layer, int32_t n_prompt,
                                  const void* d_q, const void* d_k, const void* d_v,
                                  void* d_out, float* d_score_opt, void* stream) {
  if (!ctx || layer < 0 || layer >= ctx->cfg.n_layers || n_prompt < 1 || n_prompt > ctx->cfg.max_prompt_len) return KF_EINVAL;
  // everything the second half would reject is rejected here, before anything is enqueued
  if (!d_q || !d_k || !d_v || !d_out) return KF_EINVAL;
  if ((reinterpret_cast<uintptr_t>(d_q) | reinterpret_cast<uintptr_t>(d_k) | reinterpret_cast<uintptr_t>(d_v) |
       reinterpret_cast<uintptr_t>(d_out)) & 15u)
    return KF_EINVAL;
  // with tensor-core scoring the first sweep also produces the rows' plain softmax statistics, so the attention
  // kernel skips its own statistics pass (one Q K^T pass fewer)
  const bool share = ctx->cfg.prefill_impl == KF_PREFILL_TENSOR && !kf::prefill_attend_one_pass_supported(ctx->cfg.head_dim);
  const int rc = prefill_score_prune_impl(ctx, layer, n_prompt, d_q, d_k, d_v, d_score_opt, share, stream);
  if (rc != KF_OK) return rc;
  return prefill_attend_impl(ctx, n_prompt, d_q, d_k, d_v, d_out, share, stream);
}

int kf_prefill_attend(kf_ctx* ctx, int32_t n_prompt, const void* d_q, const void* d_k, const void* d_v,
                      void* d_out, void* stream) {
  return prefill_attend_impl(ctx, n_prompt, d_q, d_k, d_v, d_out, false, stream);
}

static int decode_impl(kf_ctx* ctx, int32_t layer, int32_t step, const void* d_q, const void* d_knew,
                       const void* d_vnew, void* d_out, float* d_score_opt, cudaStream_t st) {
  const kf_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  kf::DecodeParams P{};
  P.K = reinterpret_cast<const __half*>(ctx->ws + L.K + (size_t)layer * L.kv_layer);
  P.V = reinterpret_cast<const __half*>(ctx->ws + L.V + (size_t)layer * L.kv_layer);
  P.acc = reinterpret_cast<float*>(ctx->ws + L.acc + (size_t)layer * L.sc_layer);
  P.pos = reinterpret_cast<int32_t*>(ctx->ws + L.pos + (size_t)layer * L.sc_layer);
  P.len = reinterpret_cast<int32_t*>(ctx->ws + L.len + (size_t)layer * L.len_layer);
  P.place = c.pos_mode == KF_POS_NEW ? reinterpret_cast<int32_t*>(ctx->ws + L.place + (size_t)layer * L.sc_layer) : nullptr;
  P.q = static_cast<const __half*>(d_q);
  P.knew = static_cast<const __half*>(d_knew);
  P.vnew = static_cast<const __half*>(d_vnew);
  P.out = static_cast<__half*>(d_out);
  P.score_opt = d_score_opt;
  P.y_scratch = reinterpret_cast<float*>(ctx->ws + L.y_scratch);
  P.partials = reinterpret_cast<float*>(ctx->ws + L.partials);
  P.err = reinterpret_cast<int*>(ctx->ws + L.err);
  P.slopes = c.bias_mode == KF_BIAS_ALIBI ? reinterpret_cast<const float*>(ctx->ws + L.slopes) : nullptr;
  P.k = c.budget_k; P.w = c.recent_w;
  P.p = ctx->n_prompt[layer] + step - 1;
  P.rope_tab = c.rotary_dims > 0 ? reinterpret_cast<const float2*>(ctx->ws + L.rope_tab) : nullptr;
  P.rot_chunks = c.rotary_dims / 8;

  int splits = 1, tps = 4;
  kf::decode_plan(L.units, c.budget_k, c.decode_splits, &splits, &tps);
  P.splits = splits; P.tiles_per_split = tps;
  P.H = c.n_heads; P.layer = layer; P.noise_mode = c.noise_mode; P.bias_mode = c.bias_mode;
  P.group = L.group;
  P.scale = ctx->scale;
  // Eq. 12 with t = step, clamped at T; T = 0 keeps tau_init
  double tau = c.tau_init;
  if (c.gen_len_T > 0) {
    const int t = std::min(step, c.gen_len_T);
    tau = (double)c.tau_init + (double)t * (((double)c.tau_end - (double)c.tau_init) / (double)c.gen_len_T);
  }
  P.inv_tau = (float)(1.0 / tau);
  P.noise_const = c.noise_const;
  P.noise_mu = c.noise_mu; P.noise_sigma = c.noise_sigma;
  P.first_wait_limit = c.debug_fail_first_wait ? 0u : kf::DECODE_WAIT_LIMIT;
  P.pk = ctx->pk;
  if (ctx->decode_tc) {
    if (!ctx->tm_ready[layer]) {
      if (!kf::decode_tc_cache_maps(&ctx->tmK[layer], &ctx->tmV[layer], P.K, P.V, L.units, c.budget_k, c.head_dim)) return KF_ECUDA;
      ctx->tm_ready[layer] = 1;
    }
    if (kf::launch_decode_tc(P, ctx->tmK[layer], ctx->tmV[layer], c.head_dim, L.units, st) != cudaSuccess) return KF_ECUDA;
  } else if (kf::launch_decode(P, c.head_dim, L.units, st) != cudaSuccess) {
    return KF_ECUDA;
  }
  ctx->launches += 2;   // streaming kernel + closing kernel
  ctx->last_step[layer] = step;
  return KF_OK;
}

static int decode_check(kf_ctx* ctx, int32_t layer, int32_t step) {
  if (!ctx) return KF_EINVAL;
  if (layer < 0 || layer >= ctx->cfg.n_layers || step < 1) return KF_EINVAL;
  if (ctx->n_prompt[layer] < 0) return KF_ESTATE;
  if (step != ctx->last_step[layer] + 1) return KF_ESTATE;
  // with the rotary embedding applied here the table of angles ends at position max_prompt_len + max(T, 1) - 1
  if (ctx->cfg.rotary_dims > 0 && ctx->n_prompt[layer] + step - 1 >= ctx->lay.rope_dists) return KF_EINVAL;
  return KF_OK;
}

int kf_decode_step(kf_ctx* ctx, int32_t layer, int32_t step,
                   const void* d_q, const void* d_knew, const void* d_vnew,
                   void* d_out, float* d_score_opt, void* stream) {
  const int rc = decode_check(ctx, layer, step);
  if (rc != KF_OK) return rc;
  if (!d_q || !d_knew || !d_vnew || !d_out) return KF_EINVAL;
  if (misaligned16(d_q) || misaligned16(d_knew) || misaligned16(d_vnew) || misaligned16(d_out)) return KF_EINVAL;
  return decode_impl(ctx, layer, step, d_q, d_knew, d_vnew, d_out, d_score_opt, static_cast<cudaStream_t>(stream));
}

int kf_decode_step_host(kf_ctx* ctx, int32_t layer, int32_t step,
                        const void* h_q, const void* h_knew, const void* h_vnew,
                        void* h_out, int32_t wait, void* stream) {
  const int rc = decode_check(ctx, layer, step);
  if (rc != KF_OK) return rc;
  if (!h_q || !h_knew || !h_vnew || !h_out) return KF_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!ctx->copy_in) {   // host-side resources only: two streams and six events
    bool ok = cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; ok && i < 2; ++i)
      ok = cudaEventCreateWithFlags(&ctx->in_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&ctx->kernel_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&ctx->out_done[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return KF_ECUDA;
  }
  const Layout& L = ctx->lay;
  const size_t bytes = (size_t)L.units_q * ctx->cfg.head_dim * 2;      // q and out: one row per query head
  const size_t bytes_kv = (size_t)L.units * ctx->cfg.head_dim * 2;     // k_new, v_new: one row per cache
  const size_t stride = align_up(bytes);
  const int set = (int)(ctx->host_calls & 1);
  unsigned char* sq = ctx->ws + L.staging + (size_t)set * 4 * stride;
  unsigned char* sk = sq + stride;
  unsigned char* sv = sk + stride;
  unsigned char* so = sv + stride;
  // Inputs travel on a copy stream so that they overlap the previous call's kernel; this staging set was last
  // read by the kernel of two calls ago.  (Waiting on an event that was never recorded is a no-op.)
  bool ok = cudaStreamWaitEvent(ctx->copy_in, ctx->kernel_done[set], 0) == cudaSuccess &&
            cudaMemcpyAsync(sq, h_q, bytes, cudaMemcpyHostToDevice, ctx->copy_in) == cudaSuccess &&
            cudaMemcpyAsync(sk, h_knew, bytes_kv, cudaMemcpyHostToDevice, ctx->copy_in) == cudaSuccess &&
            cudaMemcpyAsync(sv, h_vnew, bytes_kv, cudaMemcpyHostToDevice, ctx->copy_in) == cudaSuccess &&
            cudaEventRecord(ctx->in_done[set], ctx->copy_in) == cudaSuccess &&
            cudaStreamWaitEvent(st, ctx->in_done[set], 0) == cudaSuccess &&
            cudaStreamWaitEvent(st, ctx->out_done[set], 0) == cudaSuccess;   // `out` of two calls ago has left
  if (!ok) return KF_ECUDA;
  const int rc2 = decode_impl(ctx, layer, step, sq, sk, sv, so, nullptr, st);
  if (rc2 != KF_OK) return rc2;
  ctx->host_calls += 1;
  // The result leaves on the other copy stream, overlapping the next call's kernel.
  ok = cudaEventRecord(ctx->kernel_done[set], st) == cudaSuccess &&
       cudaStreamWaitEvent(ctx->copy_out, ctx->kernel_done[set], 0) == cudaSuccess &&
       cudaMemcpyAsync(h_out, so, bytes, cudaMemcpyDeviceToHost, ctx->copy_out) == cudaSuccess &&
       cudaEventRecord(ctx->out_done[set], ctx->copy_out) == cudaSuccess;
  if (!ok) return KF_ECUDA;
  if (wait) {
    if (cudaStreamSynchronize(ctx->copy_out) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) return KF_ECUDA;
  }
  return KF_OK;
}

int kf_decode_step_static(const kf_static_step* a, void* d_K, void* d_V, int32_t* d_pos, float* d_acc,
                          int32_t* d_len, const void* d_q, const void* d_knew, const void* d_vnew,
                          void* d_out, float* d_score_opt, void* stream) {
  if (!a || !d_K || !d_V || !d_pos || !d_acc || !d_len || !d_q || !d_knew || !d_vnew || !d_out) return KF_EINVAL;
  if (a->batch < 1 || a->n_heads < 1 || (int64_t)a->batch * a->n_heads > 65535) return KF_EINVAL;
  if (a->head_dim != 64 && a->head_dim != 128 && a->head_dim != 256) return KF_EINVAL;
  if (a->budget_k < 1 || a->recent_w < 0 || a->recent_w > a->budget_k) return KF_EINVAL;
  if (a->layer < 0 || a->position < 0 || !(a->tau > 0.0) || a->logit_scale < 0.f) return KF_EINVAL;
  if (a->reserved != 0) return KF_EINVAL;
  if (a->noise_mode < KF_NOISE_GUMBEL || a->noise_mode > KF_NOISE_CONST) return KF_EINVAL;   // no Gaussian here (no mu, sigma)
  // rows of the cache are sources of 16-byte bulk copies; the step's vectors are read 16 bytes at a time
  if (misaligned16(d_K) || misaligned16(d_V) || misaligned16(d_q) || misaligned16(d_knew) || misaligned16(d_vnew) ||
      misaligned16(d_out))
    return KF_EINVAL;
  if ((reinterpret_cast<uintptr_t>(d_pos) | reinterpret_cast<uintptr_t>(d_acc) | reinterpret_cast<uintptr_t>(d_len)) & 3u)
    return KF_EINVAL;
  if (a->bias_mode != KF_BIAS_NONE && a->bias_mode != KF_BIAS_ALIBI) return KF_EINVAL;
  if (a->bias_mode == KF_BIAS_ALIBI && !a->d_alibi_slopes) return KF_EINVAL;
  const int units = a->batch * a->n_heads;
  int splits = 1, tps = 4;
  kf::decode_plan(units, a->budget_k, 0, &splits, &tps);
  const size_t y_bytes = align_up((size_t)units * ((size_t)a->budget_k + 1) * 4);
  const size_t partial_bytes = align_up((size_t)units * splits * (4 + (size_t)a->head_dim) * 4);
  if (y_bytes + partial_bytes + 256 > kf::STATIC_SCRATCH_BYTES) return KF_ENOSPC;  // before any CUDA call

  kf::DecodeParams P{};
  P.K = static_cast<const __half*>(d_K);
  P.V = static_cast<const __half*>(d_V);
  P.acc = d_acc; P.pos = d_pos; P.len = d_len;
  P.q = static_cast<const __half*>(d_q);
  P.knew = static_cast<const __half*>(d_knew);
  P.vnew = static_cast<const __half*>(d_vnew);
  P.out = static_cast<__half*>(d_out);
  P.score_opt = d_score_opt;
  P.err = nullptr;
  P.slopes = a->bias_mode == KF_BIAS_ALIBI ? a->d_alibi_slopes : nullptr;
  P.k = a->budget_k; P.w = a->recent_w; P.p = a->position;
  P.splits = splits; P.tiles_per_split = tps;
  P.H = a->n_heads; P.layer = a->layer; P.noise_mode = a->noise_mode; P.bias_mode = a->bias_mode;
  P.group = 1;
  P.scale = a->logit_scale > 0.f ? a->logit_scale : (float)(1.0 / std::sqrt((double)a->head_dim));
  P.inv_tau = (float)(1.0 / a->tau);
  P.noise_const = a->noise_const;
  P.first_wait_limit = kf::DECODE_WAIT_LIMIT;
  P.rope_tab = nullptr; P.rot_chunks = 0;
  P.pk = kf::philox_expand_key(a->noise_seed);
  const cudaError_t e = kf::launch_decode_static(P, a->head_dim, units, y_bytes, partial_bytes,
                                                 static_cast<cudaStream_t>(stream));
  if (e == cudaErrorMemoryAllocation) return KF_ENOSPC;
  return e == cudaSuccess ? KF_OK : KF_ECUDA;
}

int kf_view_state(kf_ctx* ctx, int32_t layer, const void** d_K, const void** d_V,
                  const int32_t** d_pos, const float** d_acc, const int32_t** d_len) {
  if (!ctx || layer < 0 || layer >= ctx->cfg.n_layers) return KF_EINVAL;
  const Layout& L = ctx->lay;
  if (d_K) *d_K = ctx->ws + L.K + (size_t)layer * L.kv_layer;
  if (d_V) *d_V = ctx->ws + L.V + (size_t)layer * L.kv_layer;
  if (d_pos) *d_pos = reinterpret_cast<const int32_t*>(ctx->ws + L.pos + (size_t)layer * L.sc_layer);
  if (d_acc) *d_acc = reinterpret_cast<const float*>(ctx->ws + L.acc + (size_t)layer * L.sc_layer);
  if (d_len) *d_len = reinterpret_cast<const int32_t*>(ctx->ws + L.len + (size_t)layer * L.len_layer);
  return KF_OK;
}

int kf_compact_layer(kf_ctx* ctx, int32_t layer, void* stream) {
  if (!ctx || layer < 0 || layer >= ctx->cfg.n_layers) return KF_EINVAL;
  if (ctx->n_prompt[layer] < 0) return KF_ESTATE;
  const kf_config& c = ctx->cfg;
  if (c.budget_k > kf::compact_max_k()) return KF_EINVAL;
  const Layout& L = ctx->lay;
  if (kf::launch_compact(reinterpret_cast<__half*>(ctx->ws + L.K + (size_t)layer * L.kv_layer),
                         reinterpret_cast<__half*>(ctx->ws + L.V + (size_t)layer * L.kv_layer),
                         reinterpret_cast<float*>(ctx->ws + L.acc + (size_t)layer * L.sc_layer),
                         reinterpret_cast<int32_t*>(ctx->ws + L.pos + (size_t)layer * L.sc_layer),
                         reinterpret_cast<const int32_t*>(ctx->ws + L.len + (size_t)layer * L.len_layer),
                         c.pos_mode == KF_POS_NEW ? reinterpret_cast<int32_t*>(ctx->ws + L.place + (size_t)layer * L.sc_layer) : nullptr,
                         reinterpret_cast<int32_t*>(ctx->ws + L.idx),   // the prompt phase's index scratch is free here
                         c.budget_k, c.head_dim, L.units, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return KF_ECUDA;
  ctx->launches += 2;
  return KF_OK;
}

int kf_view_place(kf_ctx* ctx, int32_t layer, const int32_t** d_place) {
  if (!ctx || !d_place || layer < 0 || layer >= ctx->cfg.n_layers || ctx->cfg.pos_mode != KF_POS_NEW) return KF_EINVAL;
  *d_place = reinterpret_cast<const int32_t*>(ctx->ws + ctx->lay.place + (size_t)layer * ctx->lay.sc_layer);
  return KF_OK;
}

size_t kf_state_bytes(const kf_ctx* ctx) {
  if (!ctx) return 0;
  const Layout& L = ctx->lay;
  return 2 * L.kv_layer + 2 * L.sc_layer + L.len_layer;
}

// One layer's image: K | V | acc | pos | len, the workspace's own per-layer blocks back to back.
static int copy_state(kf_ctx* ctx, int32_t layer, unsigned char* image, bool to_image, cudaStream_t st) {
  const Layout& L = ctx->lay;
  struct Block { size_t ws_off, bytes; };
  const Block blocks[5] = {{L.K + (size_t)layer * L.kv_layer, L.kv_layer},   {L.V + (size_t)layer * L.kv_layer, L.kv_layer},
                           {L.acc + (size_t)layer * L.sc_layer, L.sc_layer}, {L.pos + (size_t)layer * L.sc_layer, L.sc_layer},
                           {L.len + (size_t)layer * L.len_layer, L.len_layer}};
  size_t off = 0;
  for (const Block& b : blocks) {
    void* dst = to_image ? (void*)(image + off) : (void*)(ctx->ws + b.ws_off);
    const void* src = to_image ? (const void*)(ctx->ws + b.ws_off) : (const void*)(image + off);
    if (cudaMemcpyAsync(dst, src, b.bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return KF_ECUDA;
    off += b.bytes;
  }
  return KF_OK;
}

int kf_export_state(kf_ctx* ctx, int32_t layer, void* d_dst, size_t bytes, int32_t* n_prompt, int32_t* last_step,
                    void* stream) {
  if (!ctx || !d_dst || layer < 0 || layer >= ctx->cfg.n_layers) return KF_EINVAL;
  if (ctx->n_prompt[layer] < 0) return KF_ESTATE;
  if (bytes < kf_state_bytes(ctx)) return KF_ENOSPC;
  const int rc = copy_state(ctx, layer, static_cast<unsigned char*>(d_dst), true, static_cast<cudaStream_t>(stream));
  if (rc != KF_OK) return rc;
  if (n_prompt) *n_prompt = ctx->n_prompt[layer];
  if (last_step) *last_step = ctx->last_step[layer];
  return KF_OK;
}

int kf_import_state(kf_ctx* ctx, int32_t layer, const void* d_src, size_t bytes, int32_t n_prompt, int32_t last_step,
                    void* stream) {
  if (!ctx || !d_src || layer < 0 || layer >= ctx->cfg.n_layers) return KF_EINVAL;
  if (n_prompt < 1 || last_step < 0) return KF_EINVAL;
  if (bytes < kf_state_bytes(ctx)) return KF_ENOSPC;
  const int rc = copy_state(ctx, layer, const_cast<unsigned char*>(static_cast<const unsigned char*>(d_src)), false,
                            static_cast<cudaStream_t>(stream));
  if (rc != KF_OK) return rc;
  if (ctx->cfg.pos_mode == KF_POS_NEW) {
    // the image carries positions only: the places follow from them
    const Layout& L = ctx->lay;
    if (kf::launch_rebuild_place(reinterpret_cast<const int32_t*>(ctx->ws + L.pos + (size_t)layer * L.sc_layer),
                                 reinterpret_cast<const int32_t*>(ctx->ws + L.len + (size_t)layer * L.len_layer),
                                 reinterpret_cast<int32_t*>(ctx->ws + L.place + (size_t)layer * L.sc_layer),
                                 ctx->cfg.budget_k, L.units, static_cast<cudaStream_t>(stream)) != cudaSuccess)
      return KF_ECUDA;
    ctx->launches += 1;
  }
  ctx->n_prompt[layer] = n_prompt;
  ctx->last_step[layer] = last_step;
  return KF_OK;
}

int kf_poll_error(kf_ctx* ctx, void* stream) {
  if (!ctx) return KF_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int word = 0;
  if (cudaMemcpyAsync(&word, ctx->ws + ctx->lay.err, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return KF_ECUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return KF_ECUDA;
  if (ctx->copy_out && cudaStreamSynchronize(ctx->copy_out) != cudaSuccess) return KF_ECUDA;
  if (word != 0) {
    if (cudaMemsetAsync(ctx->ws + ctx->lay.err, 0, sizeof(int), st) != cudaSuccess) return KF_ECUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return KF_ECUDA;
  }
  return word;
}

int kf_check_canaries(kf_ctx* ctx, void* stream, int32_t* first_bad) {
  if (first_bad) *first_bad = -1;
  if (!ctx || !ctx->cfg.debug_canaries) return KF_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const std::vector<size_t>& guards = ctx->lay.guards;
  std::vector<unsigned char> host(guards.size() * GUARD_BYTES);
  for (size_t g = 0; g < guards.size(); ++g)
    if (cudaMemcpyAsync(host.data() + g * GUARD_BYTES, ctx->ws + guards[g], GUARD_BYTES, cudaMemcpyDeviceToHost, st) != cudaSuccess)
      return KF_ECUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return KF_ECUDA;
  for (size_t i = 0; i < host.size(); ++i)
    if (host[i] != (unsigned char)GUARD_BYTE) {
      if (first_bad) *first_bad = (int32_t)(i / GUARD_BYTES);
      return KF_EBOUNDS;
    }
  return KF_OK;
}

int kf_describe_decode(const kf_ctx* ctx, char* buf, size_t n) {
  if (!ctx || !buf || n == 0) return KF_EINVAL;
  int splits = 1, tps = 4;
  if (ctx->decode_tc) {
    if (kf::decode_tc_plan(ctx->lay.units, ctx->cfg.budget_k, &tps, &splits) != cudaSuccess) return KF_ECUDA;
  } else {
    kf::decode_plan(ctx->lay.units, ctx->cfg.budget_k, ctx->cfg.decode_splits, &splits, &tps);
  }
  const int len = kf::decode_describe(buf, n, ctx->cfg.head_dim, ctx->lay.units, ctx->cfg.budget_k, splits, tps,
                                      ctx->cfg.pos_mode == KF_POS_NEW, ctx->lay.group, ctx->decode_tc, ctx->cfg.rotary_dims > 0);
  return len < 0 ? KF_EINVAL : len;
}

int64_t kf_launch_count(const kf_ctx* ctx) { return ctx ? ctx->launches : 0; }

int kf_destroy(kf_ctx* ctx) {
  if (!ctx) return KF_EINVAL;
  if (ctx->copy_in) {   // drain and release the host-variant's streams and events
    cudaStreamSynchronize(ctx->copy_in);
    cudaStreamSynchronize(ctx->copy_out);
    for (int i = 0; i < 2; ++i) {
      if (ctx->in_done[i]) cudaEventDestroy(ctx->in_done[i]);
      if (ctx->kernel_done[i]) cudaEventDestroy(ctx->kernel_done[i]);
      if (ctx->out_done[i]) cudaEventDestroy(ctx->out_done[i]);
    }
    cudaStreamDestroy(ctx->copy_in);
    if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
  }
  delete ctx;
  return KF_OK;
}

const char* kf_strerror(int code) {
  switch (code) {
    case KF_OK: return "ok";
    case KF_EINVAL: return "invalid argument or configuration";
    case KF_ENOSPC: return "workspace too small";
    case KF_ESTATE: return "call out of order";
    case KF_ECUDA: return "CUDA runtime error or no device";
    case KF_ETIMEOUT: return "a bounded device-side wait ran out";
    case KF_EBOUNDS: return "a device-side bounds check failed";
    default: return "unknown error";
  }
}

}  // extern "C"
