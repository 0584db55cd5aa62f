/*
 * keyformer.h -- C ABI of the B200 (sm_100a) Keyformer score-and-evict library.
 *
 * The library keeps, per (layer, batch row, head), a KV cache of at most k
 * entries together with each entry's original token position and accumulated
 * Keyformer score f_theta, and implements the two phases of Algorithm 1 of the
 * Keyformer paper:
 *
 *   prompt phase      kf_prefill_score_prune   (Algorithm 1 with m <- n; section 3.4)
 *   generation phase  kf_decode_step           (Algorithm 1 with m <- k; section 3.4)
 *
 * Conventions
 *   - Every pointer whose name starts with d_ is a DEVICE pointer, h_ a HOST pointer.
 *   - All device buffers, the workspace included, are owned by the caller; the
 *     context owns host metadata only and kf_destroy frees no device memory.
 *   - Q/K/V tensors are IEEE binary16 ("fp16"), contiguous, row-major in the
 *     shapes stated per call.  Scores are binary32.
 *   - Work is enqueued on the CUDA stream passed as `stream` (a cudaStream_t cast
 *     to void*; NULL = the default stream).  No call synchronises except
 *     kf_poll_error and the *_host variants' final wait when asked to.
 *   - Return value 0 = success, negative = one of the KF_E* codes; on an error
 *     detected on the host nothing has been enqueued.
 *   - There is no CPU fallback: without a CUDA device every compute call
 *     returns KF_ECUDA.
 */
#ifndef KEYFORMER_B200_H
#define KEYFORMER_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KF_OK        0
#define KF_EINVAL   -1   /* bad argument or configuration                         */
#define KF_ENOSPC   -2   /* workspace too small                                   */
#define KF_ESTATE   -3   /* call out of order (decode before prefill, ...)        */
#define KF_ECUDA    -4   /* a CUDA runtime call failed / no device                */
#define KF_ETIMEOUT -5   /* a bounded device-side wait ran out (error word)       */
#define KF_EBOUNDS  -6   /* a device-side bounds check failed (error word)        */

/* Logit adjustment zeta of Eq. 4 (section 4.4.3 lists the alternatives). */
#define KF_NOISE_GUMBEL 0   /* zeta = -ln(-ln u), standard Gumbel, Eq. 7 (the method) */
#define KF_NOISE_NONE   1   /* zeta = 0 (accumulated-attention score, H2O-like)      */
#define KF_NOISE_CONST  2   /* zeta = noise_const                                     */
#define KF_NOISE_GAUSS  3   /* zeta = noise_mu + noise_sigma * N(0,1) (the Gaussian alternative of section 4.4.3;
                               Box-Muller on two Philox words)                        */

/* How kf_prefill_score_prune computes the prompt logits Q K^T. */
#define KF_PREFILL_TENSOR 0 /* tcgen05 tensor cores, accumulators in tensor memory (default) */
#define KF_PREFILL_SIMT   1 /* CUDA cores; scores are summed with floating-point atomics     */

/* Which streaming kernel kf_decode_step uses. */
#define KF_DECODE_AUTO       0 /* tensor cores where several query heads share a cache and head_dim is 128, else CUDA cores */
#define KF_DECODE_CUDA_CORES 1 /* lane-per-row mixed-precision fma (every shape)                                          */
#define KF_DECODE_TENSOR     2 /* tcgen05 logits and value sums, accumulators in tensor memory (head_dim 128 only)        */

#define KF_BIAS_NONE  0
#define KF_BIAS_ALIBI 1     /* x_ij += -slope_h * (i - j); which i and j is chosen by pos_mode */

/* Positional information seen by the bias once the cache has been reduced (section 4.4.2). */
#define KF_POS_ORIGINAL 0   /* i, j = positions of the tokens in the text ("Org Pos", the method's default) */
#define KF_POS_NEW      1   /* i, j = places within the reduced cache, counted in position order ("New Pos"):
                               the oldest kept entry is 0, the current token is the last.  Only the generation
                               phase differs (nothing has been dropped while the prompt is scored); the noise
                               is keyed by the original positions in both modes.                              */

typedef struct kf_ctx kf_ctx;

/* Inputs of Algorithm 1 (cache size k, recent window w, generation length T,
 * tau_init, tau_end) plus the tensor geometry. */
typedef struct kf_config {
  int32_t n_layers;        /* L >= 1                                              */
  int32_t batch;           /* B >= 1 (beams are batch rows)                       */
  int32_t n_heads;         /* H >= 1                                              */
  int32_t head_dim;        /* d in {64, 128, 256}                                 */
  int32_t budget_k;        /* k >= 1 : KV cache entries kept per (layer, b, head) */
  int32_t recent_w;        /* 0 <= w <= k : most recent tokens always kept        */
  int32_t max_prompt_len;  /* largest n accepted by kf_prefill_score_prune        */
  int32_t gen_len_T;       /* T >= 0 : delta_tau = (tau_end - tau_init) / T (Eq. 12); 0 = constant tau_init */
  float   tau_init;        /* > 0, paper default 1                                */
  float   tau_end;         /* > 0, paper default 2                                */
  uint64_t noise_seed;     /* Philox key                                          */
  int32_t noise_mode;      /* KF_NOISE_*                                          */
  int32_t bias_mode;       /* KF_BIAS_*                                           */
  const float* h_alibi_slopes; /* HOST [H], read during kf_create when bias_mode == KF_BIAS_ALIBI */
  float   logit_scale;     /* 0 => 1/sqrt(d) (Eq. 1 / Eq. 4)                      */
  float   noise_const;     /* c of KF_NOISE_CONST                                 */
  int32_t decode_splits;   /* 0 = choose automatically; else CTAs per unit in the decode kernel (at most 64) */
  int32_t prefill_impl;    /* KF_PREFILL_*                                        */
  float   noise_mu;        /* mean of KF_NOISE_GAUSS (the paper matches Gumbel's 0.5772)          */
  float   noise_sigma;     /* standard deviation of KF_NOISE_GAUSS (1.2825 in the paper)         */
  int32_t pos_mode;        /* KF_POS_*; KF_POS_NEW keeps one more int32 per cache slot            */
  int32_t n_kv_heads;      /* key/value heads Hkv (section 6: multi-query / grouped-query attention).  0 or H: every head
                              has its own cache, the method as printed.  Otherwise H / Hkv must be 2, 4 or 8: that many
                              consecutive query heads share one cache and one f_theta; each of them has its own logits,
                              noise (drawn with its own head index), bias slope and softmax of Eq. 11, and f_theta
                              accumulates the mean of their scores.  Caches are then per (layer, batch row, key/value
                              head): wherever a shape below says [B][H] for K, V, k_new, v_new, scores, positions or entry
                              counts read [B][Hkv]; q and out stay [B][H].                                         */
  int32_t rotary_dims;     /* R.  0: Q and K carry whatever positional rotation the model applies (the library never looks).
                              R > 0 (a power of two, 8 <= R <= d): Q and K are passed WITHOUT rotary embedding and the cache
                              keeps keys unrotated; the library applies the embedding to the first R features (interleaved
                              pairs (2i, 2i+1), angle position * rotary_base^(-2i/R)) when a logit is formed -- in the prompt
                              phase at each token's own position, in the generation phase according to pos_mode: KF_POS_ORIGINAL
                              rotates at the positions in the text, KF_POS_NEW at the places within the reduced cache (section
                              4.4.2 on rotary models).  Generation then accepts positions below max_prompt_len + max(T, 1)
                              (KF_EINVAL beyond: the table of angles ends there); not available with KF_DECODE_TENSOR.   */
  float   rotary_base;     /* > 1 when rotary_dims > 0; 10000 in the published embedding                               */
  int32_t decode_impl;     /* KF_DECODE_*                                                                              */
  int32_t debug_canaries;  /* 1: a 256-byte guard of a known pattern follows every sub-buffer of the workspace
                              (kf_workspace_bytes grows accordingly); kf_check_canaries verifies them.  0: none */
  int32_t debug_fail_first_wait; /* self-test of the error path: 1 makes every warp of the generation kernel give up
                              its first wait for a cache tile at once, as if the bounded wait had run out: the step
                              reports KF_ETIMEOUT through kf_poll_error (after waiting, with the full limit, for the
                              copies in flight) and leaves the layer's state undefined.  0 in normal use.          */
} kf_config;

/* Bytes of device workspace kf_create needs for this configuration
 * (KV cache, positions, scores, kernel scratch).  Returns 0 if the
 * configuration is invalid. */
size_t kf_workspace_bytes(const kf_config* cfg);

/* Build a context over a caller-owned device workspace of at least
 * kf_workspace_bytes(cfg) bytes, 256-byte aligned.  Clears the cache state
 * (asynchronously, on `stream`).  *out receives the context. */
int kf_create(const kf_config* cfg, void* d_workspace, size_t workspace_bytes, void* stream, kf_ctx** out);

/* Prompt phase of Algorithm 1 (t = 0, temperature tau_init; section 3.4).
 * For every (batch row, head) of `layer`: causal logits x_ij = scale * Q_i.K_j
 * (+ bias), y_ij = (x_ij + zeta_ij) / tau_init, row-wise softmax (Eq. 11), sum
 * over query rows into f_theta(j); keep the w most recent positions plus the
 * top-(k-w) of the others by f_theta (ties: lower position), and store the
 * kept K/V rows, positions and scores in ascending position order.  If
 * n_prompt <= k everything is kept.
 *   d_q, d_k, d_v : DEVICE fp16 [B][H][n_prompt][d], read only, each 16-byte aligned (KF_EINVAL otherwise,
 *                   with either scoring implementation).
 *   d_score_opt   : DEVICE fp32 [B][H][n_prompt] or NULL; receives f_theta
 *                   before pruning.
 * Must be called once per layer before that layer's first kf_decode_step. */
int kf_prefill_score_prune(kf_ctx* ctx, int32_t layer, int32_t n_prompt,
                           const void* d_q, const void* d_k, const void* d_v,
                           float* d_score_opt, void* stream);

/* Attention output of the prompt phase (Eq. 1 under the causal mask): for every (batch row, head) and query
 * position i, out_i = sum_{j <= i} softmax_j(x_ij) V_j with the plain softmax of x_ij = scale * Q_i.K_j
 * (+ bias) -- no logit adjustment and temperature 1, i.e. what the model's attention layer produces, which
 * section 3.4 leaves untouched.  Runs on the tensor cores; does not read or change the cache state.
 *   d_q, d_k, d_v : DEVICE fp16 [B][H][n_prompt][d], read only, 16-byte aligned.
 *   d_out         : DEVICE fp16 [B][H][n_prompt][d], 16-byte aligned.
 * kf_prefill_attend_score_prune is the two calls in one: attention output, then kf_prefill_score_prune. */
int kf_prefill_attend(kf_ctx* ctx, int32_t n_prompt, const void* d_q, const void* d_k, const void* d_v,
                      void* d_out, void* stream);
int kf_prefill_attend_score_prune(kf_ctx* ctx, int32_t layer, int32_t n_prompt,
                                  const void* d_q, const void* d_k, const void* d_v,
                                  void* d_out, float* d_score_opt, void* stream);

/* One generation step of Algorithm 1 (t = step >= 1; section 3.4) for every
 * (batch row, head) of `layer`.  The new token (original position
 * p = n_prompt + step - 1) joins the cached entries, so m = len + 1 logits:
 *   out   = sum_j softmax(x)_j V_j                       (Eq. 1; no noise, temperature 1)
 *   z_j   = softmax_j((x_j + zeta_j) / tau_step)          (Eq. 4, 11; tau of Eq. 12, clamped at T)
 *   f_theta(j) += z_j                                     (the new token starts from 0)
 *   if m > k: evict the entry with the smallest f_theta among those not in
 *   the w most recent (ties: the higher position leaves); the new token's
 *   row takes the freed slot.  Slot order is therefore arbitrary; the
 *   position array identifies the entries.
 *   d_q, d_knew, d_vnew : DEVICE fp16 [B][H][d], each 16-byte aligned (KF_EINVAL otherwise).
 *   d_out               : DEVICE fp16 [B][H][d], 16-byte aligned.
 *   d_score_opt         : DEVICE fp32 [B][H][k+1] or NULL; receives z for the
 *                         slots [0, len) followed by the new token at index len.
 * The steps of a layer must be consecutive: the first call after the prompt phase (or after kf_import_state with
 * last_step = s) has step 1 (s + 1), every later call the previous step plus one; anything else is KF_ESTATE and
 * enqueues nothing.  (The position of the token, hence its noise and temperature, follows from the step.)
 * A unit whose entry count in the workspace is outside 0..k (a damaged or foreign state image) is left untouched
 * and reported as KF_EBOUNDS by kf_poll_error. */
int kf_decode_step(kf_ctx* ctx, int32_t layer, int32_t step,
                   const void* d_q, const void* d_knew, const void* d_vnew,
                   void* d_out, float* d_score_opt, void* stream);

/* Same step with HOST buffers (pinned memory recommended).  The three inputs are copied to the device on an
 * internal copy stream, so that they overlap the kernel of the previous call; the step runs on `stream`; `out`
 * is copied back on a second internal stream, overlapping the next call's kernel.
 *   - h_q, h_knew, h_vnew must hold their values when the call is made (they are read without waiting for
 *     work queued earlier on `stream`) and stay unchanged until the step has run.
 *   - h_out is valid after a call with `wait` != 0 has returned (that call drains `stream` and the result
 *     copies of all earlier calls), or after kf_poll_error.  With `wait` == 0 nothing is waited for.
 * The first call creates two streams and six events (host resources; no device memory). */
int kf_decode_step_host(kf_ctx* ctx, int32_t layer, int32_t step,
                        const void* h_q, const void* h_knew, const void* h_vnew,
                        void* h_out, int32_t wait, void* stream);

/* Size in bytes of the scratch block built into the library (see kf_decode_step_static). */
#define KF_STATIC_SCRATCH_BYTES (16u << 20)

/* Arguments of kf_decode_step_static: the quantities kf_decode_step takes from its context. */
typedef struct kf_static_step {
  int32_t batch, n_heads, head_dim;   /* B, H, d in {64, 128, 256}                          */
  int32_t budget_k, recent_w;         /* k, w                                               */
  int32_t layer;                      /* layer index (part of the noise coordinates)        */
  int32_t position;                   /* p: original position of the token being generated  */
  int32_t noise_mode, bias_mode;      /* KF_NOISE_GUMBEL, KF_NOISE_NONE or KF_NOISE_CONST (the Gaussian alternative needs
                                         its mean and deviation: use a context); KF_BIAS_*  */
  int32_t reserved;                   /* must be 0 (KF_EINVAL otherwise)                    */
  double  tau;                        /* temperature of this step (Eq. 12, computed by the caller) */
  uint64_t noise_seed;
  float   logit_scale;                /* 0 => 1/sqrt(d)                                     */
  float   noise_const;
  const float* d_alibi_slopes;        /* DEVICE [H] when bias_mode == KF_BIAS_ALIBI, else NULL */
} kf_static_step;

/* (The paper has no counterpart for this call: it is a packaging variant of kf_decode_step.)
 *
 * The same generation step, for callers that have no way to obtain device memory for the
 * library's scratch: code that runs where cudaMalloc is off limits -- inside a region that is
 * being captured or replayed and must not allocate, under a framework that owns every byte of
 * the GPU through its own pool, or in a process whose memory budget is fixed up front.  Such a
 * caller keeps the cache tensors itself and passes them in; the per-launch scratch (adjusted
 * logits, split partials) lives in a block of KF_STATIC_SCRATCH_BYTES of device
 * memory that is part of the library image.  Every GPU that loads the library holds that block
 * until the process exits.  The call itself calls no cudaMalloc, cudaFree or other allocating
 * routine.
 *
 *   d_K, d_V  : DEVICE fp16 [B][H][k][d]   cache rows, updated in place (one row replaced or appended)
 *   d_pos     : DEVICE int32 [B][H][k]     original positions, updated in place
 *   d_acc     : DEVICE fp32 [B][H][k]      accumulated scores f_theta, updated in place
 *   d_len     : DEVICE int32 [B][H]        entries in use, updated in place
 *   d_q, d_knew, d_vnew, d_out, d_score_opt : as in kf_decode_step
 *   d_K, d_V, d_q, d_knew, d_vnew, d_out must be 16-byte aligned, d_pos, d_acc, d_len 4-byte aligned (KF_EINVAL
 *   otherwise).  A unit whose d_len entry is outside 0..k is skipped: nothing of it is read or written.
 *
 * Limits and rules
 *   - The step needs about 4*B*H*(k+1) + 4*B*H*splits*(d+4) bytes of scratch; if that exceeds the
 *     block the call returns KF_ENOSPC and enqueues nothing.
 *   - The first call on a device looks up the block's device address (with that device current);
 *     make that first call outside any stream capture.
 *   - All calls on a device share the one block, which keeps the previous call's contents; no
 *     part of it has to start at zero (the step's first kernel writes every word its second
 *     kernel reads), so nothing is cleared.  Two calls whose kernels overlap on the GPU (different
 *     streams, no ordering between them) would race on it: keep them on one stream or order them.
 *   - Device-side self-checks have nowhere to report to in this variant (there is no context to
 *     poll); arguments are validated on the host as far as possible. */
int kf_decode_step_static(const kf_static_step* args,
                          void* d_K, void* d_V, int32_t* d_pos, float* d_acc, int32_t* d_len,
                          const void* d_q, const void* d_knew, const void* d_vnew,
                          void* d_out, float* d_score_opt, void* stream);

/* Borrowed DEVICE pointers into the workspace for one layer:
 *   K, V fp16 [B][H][k][d]; pos int32 [B][H][k] (original positions; -1 marks a slot left empty by the prompt phase);
 *   acc fp32 [B][H][k] (f_theta); len int32 [B][H] (entries in use).  Any may be NULL. */
int kf_view_state(kf_ctx* ctx, int32_t layer, const void** d_K, const void** d_V,
                  const int32_t** d_pos, const float** d_acc, const int32_t** d_len);

/* In-place compaction of one layer's cache into position order (Algorithm 1 describes the reduced cache as a
 * subsequence of the token sequence, S_key and the recent window S_w; section 3.4).  kf_decode_step keeps each
 * unit's entries as an unordered set -- the token that leaves is overwritten by the one that arrives -- and
 * identifies them by their positions, so no call needs this one.  It exists for callers that want the layout the
 * prompt phase produces back: slot s of every (batch row, head) holds the entry with the s-th smallest position
 * (K row, V row, position, f_theta), e.g. to compare or store state images independent of the eviction history.
 * The permutation is applied in place, cycle by cycle, with no staging buffer; asynchronous on `stream`.
 * KF_ESTATE before the layer's prompt phase; KF_EINVAL when budget_k exceeds 16384 (the ranks of a unit's
 * entries are computed in shared memory). */
int kf_compact_layer(kf_ctx* ctx, int32_t layer, void* stream);

/* KF_POS_NEW only: borrowed DEVICE pointer to the places, int32 [B][H][k]; entry j of a unit holds the
 * number of entries of that unit with a smaller position.  KF_EINVAL in the other mode. */
int kf_view_place(kf_ctx* ctx, int32_t layer, const int32_t** d_place);

/* Checkpoint of one layer's cache (section 3.3: the reduced KV cache and f_theta are the whole state the
 * method carries from step to step).  kf_state_bytes gives the size of one layer's image: K, V, f_theta,
 * positions and entry counts, each block padded to 256 bytes, in that order.  kf_export_state copies the
 * image to a caller-owned DEVICE buffer and reports how far the layer has come (prompt length, last decode
 * step); kf_import_state loads an image into a context created with the same configuration and sets that
 * progress, after which kf_decode_step continues with step last_step + 1 and reproduces the original run
 * bit for bit (noise and temperature are functions of the coordinates, not of hidden state).  Both are
 * enqueued on `stream`.  KF_ESTATE if the layer has no prompt yet; KF_ENOSPC if `bytes` is too small. */
size_t kf_state_bytes(const kf_ctx* ctx);
int kf_export_state(kf_ctx* ctx, int32_t layer, void* d_dst, size_t bytes,
                    int32_t* n_prompt, int32_t* last_step, void* stream);
int kf_import_state(kf_ctx* ctx, int32_t layer, const void* d_src, size_t bytes,
                    int32_t n_prompt, int32_t last_step, void* stream);

/* Waits for `stream`, then returns and clears the device error word:
 * 0, KF_ETIMEOUT or KF_EBOUNDS. */
int kf_poll_error(kf_ctx* ctx, void* stream);

/* Debug layout only (kf_config.debug_canaries = 1): waits for `stream`, then compares the guard behind every
 * sub-buffer of the workspace with its pattern.  KF_OK if all are intact; KF_EBOUNDS if one was overwritten, with
 * *first_bad (may be NULL) = index of the sub-buffer in front of it, in layout order: K, V, scores, positions,
 * entry counts, adjusted-logit scratch, split partials, error word, slopes, prompt scores, kept indices, host
 * staging, the two row-statistics arrays, places.  KF_EINVAL for a context without guards. */
int kf_check_canaries(kf_ctx* ctx, void* stream, int32_t* first_bad);

/* Writes into buf (n bytes, always terminated) which kernels a kf_decode_step of this context launches, with their
 * template arguments, and how a layer call is cut into CTAs, e.g.
 * "decode_kernel<128,5,2,0> + decode_close_kernel<128>; units=1024 k=2048 splits=3 tiles_per_split=24 group=1".
 * Profiles are keyed by this string.  Returns the length the full text needs (as snprintf does) or KF_EINVAL. */
int kf_describe_decode(const kf_ctx* ctx, char* buf, size_t n);

/* Number of kernel launches this context has enqueued so far. */
int64_t kf_launch_count(const kf_ctx* ctx);

/* Frees host metadata.  The workspace stays with the caller. */
int kf_destroy(kf_ctx* ctx);

const char* kf_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* KEYFORMER_B200_H */
