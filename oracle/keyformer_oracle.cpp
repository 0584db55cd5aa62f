// Keyformer CPU oracle -- TEST INFRASTRUCTURE, not a product path.
//
// A plain, slow, double-precision restatement of the Keyformer method
// (Algorithm 1 with Eq. 1, 4, 7, 11, 12 of the paper), one (batch, layer, key/value head)
// unit at a time.  It shares no code with the CUDA library.  Only the test
// suite, the smoke check and the benchmark's cpu_baseline leg may call it.
//
// Every function below cites the passage of the paper it follows.  Where the
// paper is silent the reading taken is stated next to the code.
//
// Pins (see the CPU test-suite): Philox known-answer vectors, Gumbel moments
// (0.5772 / 1.2825, section 4.4.3), the Gumbel-max frequency law, softmax
// invariants, library attention in the zero-noise special case, brute-force
// sort for the selection, conservation of accumulated mass.
// Parity unpinned: the specific kept sets on random data (the paper prints no
// worked numeric example); they are pinned only through the properties above.
//
// Build: g++ -O2 -fopenmp -shared -fPIC keyformer_oracle.cpp -o libkeyformer_oracle.so

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

// ---------------------------------------------------------------------------
// Parameters of one run (Algorithm 1 inputs: k, w, T, tau_init, tau_end).
// ---------------------------------------------------------------------------
struct ko_params {
  int32_t head_dim;      // d
  int32_t n_heads;       // H (enters the noise counter as layer*H + head)
  int32_t budget_k;      // k
  int32_t recent_w;      // w
  int32_t gen_len_T;     // T
  int32_t noise_mode;    // 0 Gumbel (Eq. 7), 1 none, 2 constant c, 3 Gaussian(mu, sigma)
  int32_t bias_mode;     // 0 none, 1 ALiBi: bias(i,j) = -slope_h * (i - j)
  int32_t pos_mode;      // 0 original token positions in the bias, 1 positions within the reduced cache (section 4.4.2)
  double tau_init;       // Eq. 12
  double tau_end;        // Eq. 12
  double logit_scale;    // 1/sqrt(d_k) of Eq. 1 / Eq. 4
  double noise_const;    // c of the constant adjustment (section 4.4.3)
  double noise_mu;       // Gaussian mean
  double noise_sigma;    // Gaussian std
  uint64_t noise_seed;
  const double* alibi_slopes;  // [H] or null
  int32_t n_kv_heads;    // key/value heads; H / n_kv_heads query heads share each of them (0 = H: none shared)
  int32_t rotary_dims;   // R: 0 = the caller's Q/K carry whatever positional rotation the model uses; R > 0 (even, <= d) = they
                         //    come without it and the rotary embedding of their first R features is applied here
  double rotary_base;    // 10000 in the published embedding
};

// Query heads per key/value head (section 6 names multi-query / grouped-query attention as compatible with the
// method without giving the rule).  Reading: a cache and its f_theta belong to a key/value head; every query head
// h = kv_head * g + r of the group has its own logits, its own noise (drawn with its own head index) and its own
// softmax of Eq. 11; f_theta accumulates the mean of the group's scores, so a step still adds a total of 1 to a
// cache and g = 1 is the method as printed.
static int group_size(const ko_params* P) {
  return (P->n_kv_heads > 0 && P->n_kv_heads < P->n_heads) ? P->n_heads / P->n_kv_heads : 1;
}

// ---------------------------------------------------------------------------
// IEEE binary16 -> double, by decoding the bit fields.
// ---------------------------------------------------------------------------
static double half_bits_to_double(uint16_t h) {
  const int sign = (h >> 15) & 1;
  const int expo = (h >> 10) & 0x1f;
  const int frac = h & 0x3ff;
  double v;
  if (expo == 0) {
    v = std::ldexp((double)frac, -24);                 // subnormal
  } else if (expo == 31) {
    v = frac ? std::numeric_limits<double>::quiet_NaN()
             : std::numeric_limits<double>::infinity();
  } else {
    v = std::ldexp((double)(1024 + frac), expo - 25);  // (1 + f/1024) 2^(e-15)
  }
  return sign ? -v : v;
}

double ko_half_to_double(uint16_t h) { return half_bits_to_double(h); }

// All 65536 decoded values, filled once from the routine above, so that the
// inner loops do a table look-up instead of an ldexp per element.
struct HalfTable {
  std::vector<double> v;
  HalfTable() : v(65536) { for (uint32_t h = 0; h < 65536; ++h) v[h] = half_bits_to_double((uint16_t)h); }
};
static const HalfTable g_half;
static inline double h2d(uint16_t h) { return g_half.v[h]; }

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
// as 1, 2, 3", SC'11).  The paper leaves the random generator open; a
// counter-based generator makes zeta a pure function of its coordinates.
// ---------------------------------------------------------------------------
void ko_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  const uint64_t mult_a = 0xD2511F53ull;  // multiplier for word 0
  const uint64_t mult_b = 0xCD9E8D57ull;  // multiplier for word 2
  const uint32_t weyl_a = 0x9E3779B9u;    // key schedule increments
  const uint32_t weyl_b = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    const uint64_t prod_a = mult_a * (uint64_t)c0;
    const uint64_t prod_b = mult_b * (uint64_t)c2;
    const uint32_t n0 = (uint32_t)(prod_b >> 32) ^ c1 ^ k0;
    const uint32_t n1 = (uint32_t)prod_b;
    const uint32_t n2 = (uint32_t)(prod_a >> 32) ^ c3 ^ k1;
    const uint32_t n3 = (uint32_t)prod_a;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += weyl_a;
    k1 += weyl_b;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Random word for logit (query position i, key position j) of unit
// (batch b, layer l, head h).  Reading (the paper is silent): key = the two
// halves of the seed; counter = (j / 4, i, l*H + h, b); word j mod 4.
static uint32_t noise_word(uint64_t seed, uint32_t b, uint32_t lh, uint32_t i, uint32_t j) {
  const uint32_t ctr[4] = {j >> 2, i, lh, b};
  const uint32_t key[2] = {(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)};
  uint32_t out[4];
  ko_philox4x32_10(ctr, key, out);
  return out[j & 3];
}

// Uniform in the open interval (0,1) from the top 23 bits of a word:
// u = (floor(r / 2^9) + 1/2) / 2^23.  (Reading; exact in binary32 too.)
double ko_uniform_from_word(uint32_t r) {
  return ((double)(r >> 9) + 0.5) * (1.0 / 8388608.0);
}

// Standard Gumbel variate by inversion of the cdf exp(-exp(-zeta)), whose
// derivative is the pdf of Eq. 7:  zeta = -ln(-ln u).
double ko_gumbel_from_word(uint32_t r) {
  const double u = ko_uniform_from_word(r);
  return -std::log(-std::log(u));
}

// Standard normal variate for the Gaussian ablation (Eq. 5) by the Box-Muller
// transform: radius from word a, angle from word b.
static double gaussian_from_words(uint32_t ra, uint32_t rb) {
  const double u1 = ko_uniform_from_word(ra);
  const double u2 = ko_uniform_from_word(rb);
  const double two_pi = 6.283185307179586476925286766559;
  return std::sqrt(-2.0 * std::log(u1)) * std::cos(two_pi * u2);
}

// zeta_{ij} of Eq. 4 for the chosen adjustment (section 4.4.3 lists the four).
double ko_noise(const ko_params* P, int32_t b, int32_t l, int32_t h, int32_t i, int32_t j) {
  const uint32_t lh = (uint32_t)l * (uint32_t)P->n_heads + (uint32_t)h;
  switch (P->noise_mode) {
    case 0:
      return ko_gumbel_from_word(noise_word(P->noise_seed, (uint32_t)b, lh, (uint32_t)i, (uint32_t)j));
    case 1:
      return 0.0;
    case 2:
      return P->noise_const;
    case 3: {
      // Gaussian: a separate counter plane (bit 31 of the batch word set) gives
      // the second word, so both draws are independent of the Gumbel stream.
      const uint32_t ra = noise_word(P->noise_seed, (uint32_t)b, lh, (uint32_t)i, (uint32_t)j);
      const uint32_t rb = noise_word(P->noise_seed, (uint32_t)b | 0x80000000u, lh, (uint32_t)i, (uint32_t)j);
      return P->noise_mu + P->noise_sigma * gaussian_from_words(ra, rb);
    }
    default:
      return 0.0;
  }
}

// Eq. 12: tau = tau_init + t * dtau, dtau = (tau_end - tau_init) / T.
// Reading: the prompt phase is t = 0; decode step s is t = s; t is clamped at
// T so generation past T stays at tau_end; T = 0 means a constant tau_init.
double ko_tau(const ko_params* P, int32_t t) {
  if (P->gen_len_T <= 0) return P->tau_init;
  const int32_t tc = std::min(std::max(t, 0), P->gen_len_T);
  const double dtau = (P->tau_end - P->tau_init) / (double)P->gen_len_T;
  return P->tau_init + (double)tc * dtau;
}

static double position_bias(const ko_params* P, int32_t h, int32_t i, int32_t j) {
  if (P->bias_mode == 1 && P->alibi_slopes) return -P->alibi_slopes[h] * (double)(i - j);
  return 0.0;
}

// Rotary position embedding (Su et al., RoFormer) in the interleaved-pair form GPT-J uses: features (2i, 2i+1), i < R/2,
// are rotated by the angle pos * base^(-2i/R).  The paper's section 4.4.2 compares feeding a model the original
// positions of the kept tokens ("Org Pos") with their positions inside the reduced cache ("New Pos") and runs the
// comparison on rotary models too; for that the cache has to hold keys without rotation and the rotation is applied
// when a logit is formed.  Reading: in the prompt phase nothing has been dropped, so every token is rotated at its own
// position in both modes; in the generation phase Org Pos rotates the query at p and key j at its original position,
// New Pos rotates the query at place m - 1 and the key in place j at j (this list is kept in position order).
static void rope_row(const ko_params* P, const uint16_t* x, int pos, double* out) {
  const int d = P->head_dim, R = P->rotary_dims;
  for (int c = 0; c < d; ++c) out[c] = h2d(x[c]);
  for (int i = 0; i < R / 2; ++i) {
    const double theta = std::pow(P->rotary_base, -2.0 * (double)i / (double)R);
    const double a = (double)pos * theta;
    const double x0 = out[2 * i], x1 = out[2 * i + 1];
    out[2 * i] = x0 * std::cos(a) - x1 * std::sin(a);
    out[2 * i + 1] = x0 * std::sin(a) + x1 * std::cos(a);
  }
}
static double dot_double(const double* a, const double* b, int d) {
  double s = 0.0;
  for (int c = 0; c < d; ++c) s += a[c] * b[c];
  return s;
}

static double dot_half(const uint16_t* a, const uint16_t* b, int d) {
  double s = 0.0;
  for (int c = 0; c < d; ++c) s += h2d(a[c]) * h2d(b[c]);
  return s;
}

// softmax of v[0..m) into p[0..m) (Eq. 1 / Eq. 11 share this normalisation).
static void softmax_inplace(const double* v, double* p, int m) {
  double mx = -std::numeric_limits<double>::infinity();
  for (int j = 0; j < m; ++j) mx = std::max(mx, v[j]);
  double sum = 0.0;
  for (int j = 0; j < m; ++j) { p[j] = std::exp(v[j] - mx); sum += p[j]; }
  for (int j = 0; j < m; ++j) p[j] /= sum;
}

// ---------------------------------------------------------------------------
// Selection (Algorithm 1: S_w = recent w tokens, S_key = argmax_(k-w) of
// f_theta[:-w], S_k = S_key U S_w).
//   pos[0..m), acc[0..m): the entries; p = position of the current query.
//   keep[j] = 1 if entry j stays.  If m <= k everything stays.
// Recent = entries with pos > p - w.  Among the others the k - #recent with
// the largest accumulated score stay; equal scores: the lower position stays
// (reading; the paper does not say).
// ---------------------------------------------------------------------------
void ko_select(const int32_t* pos, const double* acc, int32_t m, int32_t k, int32_t w,
               int32_t p, uint8_t* keep) {
  if (m <= k) { for (int j = 0; j < m; ++j) keep[j] = 1; return; }
  std::vector<int> cand;
  int n_recent = 0;
  for (int j = 0; j < m; ++j) {
    if (pos[j] > p - w) { keep[j] = 1; ++n_recent; }
    else { keep[j] = 0; cand.push_back(j); }
  }
  const int n_key = std::max(0, k - n_recent);
  std::stable_sort(cand.begin(), cand.end(), [&](int a, int b) {
    if (acc[a] != acc[b]) return acc[a] > acc[b];
    return pos[a] < pos[b];
  });
  for (int r = 0; r < n_key && r < (int)cand.size(); ++r) keep[cand[r]] = 1;
}

// ---------------------------------------------------------------------------
// Prompt phase, scoring half (Algorithm 1, t = 0, m <- n; section 3.4).
// For each query row i the causal logits x_ij (j <= i) get noise, are divided
// by tau_init and normalised (Eq. 11); the result is added into f_theta(j).
//   Q, K: [n][d] binary16 bit patterns of this unit.   acc_out: [n].
// ---------------------------------------------------------------------------
static void prefill_score_unit(const ko_params* P, int32_t b, int32_t l, int32_t hk, int32_t n,
                               const uint16_t* Q /* [g][n][d] */, const uint16_t* K, double* acc_out) {
  const int d = P->head_dim;
  const int g = group_size(P);
  const double tau = ko_tau(P, 0);
  std::vector<double> y(n), z(n);
  std::vector<double> Kr, Qr;                                             // rows rotated at their positions (rotary_dims > 0)
  const bool rot = P->rotary_dims > 0;
  if (rot) {
    Kr.resize((size_t)n * d); Qr.resize((size_t)n * d);
    for (int j = 0; j < n; ++j) rope_row(P, K + (size_t)j * d, j, Kr.data() + (size_t)j * d);
  }
  for (int j = 0; j < n; ++j) acc_out[j] = 0.0;
  for (int r = 0; r < g; ++r) {
    const int h = hk * g + r;                                             // query head r of this key/value head
    const uint16_t* Qh = Q + (size_t)r * n * d;
    if (rot) for (int i = 0; i < n; ++i) rope_row(P, Qh + (size_t)i * d, i, Qr.data() + (size_t)i * d);
    for (int i = 0; i < n; ++i) {
      const int m = i + 1;
      for (int j = 0; j < m; ++j) {
        const double qk = rot ? dot_double(Qr.data() + (size_t)i * d, Kr.data() + (size_t)j * d, d)
                              : dot_half(Qh + (size_t)i * d, K + (size_t)j * d, d);
        const double x = P->logit_scale * qk
                       + position_bias(P, h, i, j);                       // Eq. 4: x
        y[j] = (x + ko_noise(P, b, l, h, i, j)) / tau;                    // Eq. 4 then Eq. 11
      }
      softmax_inplace(y.data(), z.data(), m);
      for (int j = 0; j < m; ++j) acc_out[j] += z[j] / (double)g;         // accumulate f_theta (group mean)
    }
  }
}

// Attention output of the prompt phase (Eq. 1 with the causal mask): row i attends to keys j <= i with the
// plain softmax of x (no adjustment, temperature 1), exactly what the model's attention layer produces.
static void prefill_attend_unit(const ko_params* P, int32_t hk, int32_t n,
                                const uint16_t* Q /* [g][n][d] */, const uint16_t* K, const uint16_t* V,
                                double* out /* [g][n][d] */) {
  const int d = P->head_dim;
  const int g = group_size(P);
  std::vector<double> x(n), p(n);
  std::vector<double> Kr, qr(d);
  const bool rot = P->rotary_dims > 0;
  if (rot) {
    Kr.resize((size_t)n * d);
    for (int j = 0; j < n; ++j) rope_row(P, K + (size_t)j * d, j, Kr.data() + (size_t)j * d);
  }
  for (int r = 0; r < g; ++r) {
    const int h = hk * g + r;
    const uint16_t* Qh = Q + (size_t)r * n * d;
    double* outh = out + (size_t)r * n * d;
    for (int i = 0; i < n; ++i) {
      const int m = i + 1;
      if (rot) rope_row(P, Qh + (size_t)i * d, i, qr.data());
      for (int j = 0; j < m; ++j)
        x[j] = P->logit_scale * (rot ? dot_double(qr.data(), Kr.data() + (size_t)j * d, d)
                                     : dot_half(Qh + (size_t)i * d, K + (size_t)j * d, d)) + position_bias(P, h, i, j);
      softmax_inplace(x.data(), p.data(), m);
      for (int c = 0; c < d; ++c) {
        double s = 0.0;
        for (int j = 0; j < m; ++j) s += p[j] * h2d(V[(size_t)j * d + c]);
        outh[(size_t)i * d + c] = s;
      }
    }
  }
}

// Prompt phase, pruning half: keep w recent + top-(k-w) of the rest, store the
// kept rows in ascending position order.  keep_override (nullable, [n]) lets a
// lock-step harness impose a kept set chosen inside the tolerance band.
static void prefill_prune_unit(const ko_params* P, int32_t n, const uint16_t* K, const uint16_t* V,
                               const double* acc_full, const uint8_t* keep_override,
                               int32_t* st_len, int32_t* st_pos, double* st_acc,
                               uint16_t* st_K, uint16_t* st_V) {
  const int d = P->head_dim;
  std::vector<int32_t> pos(n);
  std::vector<uint8_t> keep(n);
  for (int j = 0; j < n; ++j) pos[j] = j;
  if (keep_override) std::memcpy(keep.data(), keep_override, n);
  else ko_select(pos.data(), acc_full, n, P->budget_k, P->recent_w, n - 1, keep.data());
  int len = 0;
  for (int j = 0; j < n; ++j) {
    if (!keep[j]) continue;
    st_pos[len] = j;
    st_acc[len] = acc_full[j];
    std::memcpy(st_K + (size_t)len * d, K + (size_t)j * d, sizeof(uint16_t) * d);
    std::memcpy(st_V + (size_t)len * d, V + (size_t)j * d, sizeof(uint16_t) * d);
    ++len;
  }
  *st_len = len;
}

// ---------------------------------------------------------------------------
// Generation phase, scoring half (Algorithm 1, t = s >= 1; section 3.4).
// The new token (position p = n_prompt + s - 1) is appended with f_theta = 0
// and attends to itself like any causal decode step, so m = len + 1 entries.
//   out  = sum_j softmax(x)_j V_j            (Eq. 1; noise-free, temperature 1)
//   z    = softmax((x + zeta) / tau_s)        (Eq. 11, Eq. 12)
//   acc += z                                  (Algorithm 1 accumulation)
// ---------------------------------------------------------------------------
static void decode_score_unit(const ko_params* P, int32_t b, int32_t l, int32_t hk,
                              int32_t step, int32_t n_prompt,
                              const uint16_t* q /* [g][d] */, const uint16_t* knew, const uint16_t* vnew,
                              int32_t* st_len, int32_t* st_pos, double* st_acc,
                              uint16_t* st_K, uint16_t* st_V,
                              double* out /* [g][d] */, double* z_out /* [cap]: the group's mean score */) {
  const int d = P->head_dim;
  const int g = group_size(P);
  const int p = n_prompt + step - 1;
  int len = *st_len;
  st_pos[len] = p;
  st_acc[len] = 0.0;
  std::memcpy(st_K + (size_t)len * d, knew, sizeof(uint16_t) * d);
  std::memcpy(st_V + (size_t)len * d, vnew, sizeof(uint16_t) * d);
  ++len;
  *st_len = len;
  const int m = len;
  const double tau = ko_tau(P, step);
  std::vector<double> x(m), y(m), a(m), z(m);
  std::vector<double> Kr, qr(d);
  const bool rot = P->rotary_dims > 0;
  if (rot) {   // keys rotated at their original positions (Org Pos) or at their places in the reduced cache (New Pos)
    Kr.resize((size_t)m * d);
    for (int j = 0; j < m; ++j) rope_row(P, st_K + (size_t)j * d, P->pos_mode == 1 ? j : st_pos[j], Kr.data() + (size_t)j * d);
  }
  for (int j = 0; j < m; ++j) z_out[j] = 0.0;
  for (int r = 0; r < g; ++r) {
    const int h = hk * g + r;                                             // query head r of this key/value head
    if (rot) rope_row(P, q + (size_t)r * d, P->pos_mode == 1 ? m - 1 : p, qr.data());
    for (int j = 0; j < m; ++j) {
      // "New Pos" (section 4.4.2): the bias sees the entries' places in the reduced cache, which this list
      // keeps in position order, so entry j sits at place j and the current token at place m - 1.
      const double bias = P->pos_mode == 1 ? position_bias(P, h, m - 1, j) : position_bias(P, h, p, st_pos[j]);
      x[j] = P->logit_scale * (rot ? dot_double(qr.data(), Kr.data() + (size_t)j * d, d)
                                   : dot_half(q + (size_t)r * d, st_K + (size_t)j * d, d)) + bias;
      y[j] = (x[j] + ko_noise(P, b, l, h, p, st_pos[j])) / tau;
    }
    softmax_inplace(x.data(), a.data(), m);
    for (int c = 0; c < d; ++c) {
      double s = 0.0;
      for (int j = 0; j < m; ++j) s += a[j] * h2d(st_V[(size_t)j * d + c]);
      out[(size_t)r * d + c] = s;
    }
    softmax_inplace(y.data(), z.data(), m);
    for (int j = 0; j < m; ++j) z_out[j] += z[j] / (double)g;
  }
  for (int j = 0; j < m; ++j) st_acc[j] += z_out[j];
}

// Generation phase, eviction half: apply the selection and close the gaps
// (order of the survivors is preserved).  force_evict_pos >= 0 imposes the
// entry to drop (lock-step harness); -1 lets the selection decide.
static void decode_evict_unit(const ko_params* P, int32_t step, int32_t n_prompt,
                              int32_t force_evict_pos,
                              int32_t* st_len, int32_t* st_pos, double* st_acc,
                              uint16_t* st_K, uint16_t* st_V, int32_t* evicted_pos) {
  const int d = P->head_dim;
  const int m = *st_len;
  const int p = n_prompt + step - 1;
  std::vector<uint8_t> keep(m, 1);
  if (force_evict_pos >= 0) {
    for (int j = 0; j < m; ++j) if (st_pos[j] == force_evict_pos) keep[j] = 0;
  } else {
    ko_select(st_pos, st_acc, m, P->budget_k, P->recent_w, p, keep.data());
  }
  *evicted_pos = -1;
  int len = 0;
  for (int j = 0; j < m; ++j) {
    if (!keep[j]) { *evicted_pos = st_pos[j]; continue; }
    if (len != j) {
      st_pos[len] = st_pos[j];
      st_acc[len] = st_acc[j];
      std::memmove(st_K + (size_t)len * d, st_K + (size_t)j * d, sizeof(uint16_t) * d);
      std::memmove(st_V + (size_t)len * d, st_V + (size_t)j * d, sizeof(uint16_t) * d);
    }
    ++len;
  }
  *st_len = len;
}

// ---------------------------------------------------------------------------
// Batched entry points: U independent units, OpenMP across units only.
//   lbh: [U][3] = (layer, batch, key/value head) of each unit; with shared key/value heads the q arrays carry
//   the g query heads of the unit's group one after the other.
//   state arrays have capacity cap = k + 1 entries per unit.
// ---------------------------------------------------------------------------
void ko_prefill_score_units(const ko_params* P, int32_t U, const int32_t* lbh, int32_t n,
                            const uint16_t* Q, const uint16_t* K, double* acc_full) {
  const size_t d = (size_t)P->head_dim, g = (size_t)group_size(P);
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    prefill_score_unit(P, lbh[3 * u + 1], lbh[3 * u + 0], lbh[3 * u + 2], n,
                       Q + (size_t)u * g * n * d, K + (size_t)u * n * d, acc_full + (size_t)u * n);
  }
}

void ko_prefill_attend_units(const ko_params* P, int32_t U, const int32_t* lbh, int32_t n,
                             const uint16_t* Q /* [U][g][n][d] */, const uint16_t* K, const uint16_t* V,
                             double* out /* [U][g][n][d] */) {
  const size_t d = (size_t)P->head_dim, g = (size_t)group_size(P);
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    prefill_attend_unit(P, lbh[3 * u + 2], n, Q + (size_t)u * g * n * d, K + (size_t)u * n * d, V + (size_t)u * n * d,
                        out + (size_t)u * g * n * d);
  }
}

void ko_prefill_prune_units(const ko_params* P, int32_t U, int32_t n,
                            const uint16_t* K, const uint16_t* V, const double* acc_full,
                            const uint8_t* keep_override /* nullable [U][n] */,
                            int32_t* st_len, int32_t* st_pos, double* st_acc,
                            uint16_t* st_K, uint16_t* st_V) {
  const size_t d = (size_t)P->head_dim;
  const size_t cap = (size_t)P->budget_k + 1;
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    prefill_prune_unit(P, n, K + (size_t)u * n * d, V + (size_t)u * n * d, acc_full + (size_t)u * n,
                       keep_override ? keep_override + (size_t)u * n : nullptr,
                       st_len + u, st_pos + u * cap, st_acc + u * cap,
                       st_K + u * cap * d, st_V + u * cap * d);
  }
}

void ko_decode_score_units(const ko_params* P, int32_t U, const int32_t* lbh,
                           int32_t step, int32_t n_prompt,
                           const uint16_t* q, const uint16_t* knew, const uint16_t* vnew,
                           int32_t* st_len, int32_t* st_pos, double* st_acc,
                           uint16_t* st_K, uint16_t* st_V,
                           double* out /* [U][g][d] */, double* z /* [U][cap] */) {
  const size_t d = (size_t)P->head_dim, g = (size_t)group_size(P);
  const size_t cap = (size_t)P->budget_k + 1;
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    decode_score_unit(P, lbh[3 * u + 1], lbh[3 * u + 0], lbh[3 * u + 2], step, n_prompt,
                      q + u * g * d, knew + u * d, vnew + u * d,
                      st_len + u, st_pos + u * cap, st_acc + u * cap,
                      st_K + u * cap * d, st_V + u * cap * d, out + u * g * d, z + u * cap);
  }
}

void ko_decode_evict_units(const ko_params* P, int32_t U, int32_t step, int32_t n_prompt,
                           const int32_t* force_evict_pos /* nullable [U] */,
                           int32_t* st_len, int32_t* st_pos, double* st_acc,
                           uint16_t* st_K, uint16_t* st_V, int32_t* evicted_pos /* [U] */) {
  const size_t d = (size_t)P->head_dim;
  const size_t cap = (size_t)P->budget_k + 1;
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    decode_evict_unit(P, step, n_prompt, force_evict_pos ? force_evict_pos[u] : -1,
                      st_len + u, st_pos + u * cap, st_acc + u * cap,
                      st_K + u * cap * d, st_V + u * cap * d, evicted_pos + u);
  }
}

int32_t ko_num_threads(void) {
  int n = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp single
    n = omp_get_num_threads();
  }
#endif
  return n;
}

}  // extern "C"
