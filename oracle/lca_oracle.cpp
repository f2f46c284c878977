// Latent-Condensed Attention (LCA) -- CPU oracle, fp64, plain loops.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of what the
// CUDA library computes.  It shares no code, header, table or helper with the CUDA path and is
// called only from tests, from the smoke check and from the benchmark's cpu_baseline leg.
//
// Every function follows one passage of the paper, in the paper's order and notation
// (1-based token/group indices in the comments, 0-based in the arrays):
//
//   summary query      Alg. 1 (first step), Sec. 4.2: the mean of the last g queries
//   scores, alpha      Sec. 4.2 importance score s_i, Eq. 6
//   weighted pooling   Eq. 7
//   anchor selection   Eq. 8
//   local window       Sec. 4.2 "Preserving Fine-Grained Local Context", Eq. 9
//   fused attention    Eq. 10 (the last steps of Alg. 1), evaluated at every prefix length t
//   decode             Sec. 4.3 "Decoding and Online Cache Update"
//   GQA variant        Sec. 5.4 "Extension to Other Attention Variants"
//
// Readings taken where the paper is silent (each is listed in the design notes):
//   * heads: one alpha per group shared by all heads; the summary query is the mean over the
//     last n positions AND over the heads (GQA: over the query heads of one KV head);
//   * causal prefill: row t is Eq. 10 on the length-t prefix: representatives of the
//     m_t = floor((t-w)/g) groups (0 if t < w) wholly in the distant history, plus every
//     token after them up to t (k_t = t - m_t*g tokens);
//   * arg-max ties: lowest index wins (the comparison is done on s_i, monotone in alpha_i);
//   * K_loc has exactly k rows (Eq. 9), so that m*g + k = L;
//   * rep_logit_bias is added to the logit of every representative (0 = Alg. 1 as printed;
//     ln g = the multiplicity-weighted form that the proof of Theorem 1 analyses).
//
// All arithmetic is double.  Inputs arrive as double (the caller widens bf16 bits exactly).
// The only rounding is lca_oracle_round_bf16, applied by the caller when a representative is
// stored in the bf16 cache.
//
// Parity status: the paper prints no worked numeric example of c_rep or of an attention
// output, so those values are pinned through reductions and invariants only (dense attention
// at g=1 and at w>=L, a per-prefix brute force of Alg. 1, Proposition 1, mean pooling at
// q_bar=0, the Theorem 1 bound, the printed cache sizes); see tests/test_oracle_pins.py.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#include <limits>
#include <algorithm>
#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

int lca_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// Round a double to the nearest bfloat16 (ties to even) and return its 16 bits.
// Done directly from double so that no intermediate float rounding occurs.
uint16_t lca_oracle_round_bf16_scalar(double x) {
  if (std::isnan(x)) return 0x7fc0;
  if (std::isinf(x)) return x > 0 ? 0x7f80 : 0xff80;
  if (x == 0.0) return std::signbit(x) ? 0x8000 : 0x0000;
  int e;
  std::frexp(x, &e);                 // |x| = f * 2^e, f in [0.5, 1)
  int ex = e - 1;                    // |x| in [2^ex, 2^(ex+1))
  if (ex < -126) ex = -126;          // subnormal range of bf16 shares float's exponent floor
  double quantum = std::ldexp(1.0, ex - 7);   // 8 significant bits
  double r = std::nearbyint(x / quantum) * quantum;   // default mode: ties to even
  float f = (float)r;                // exact: r has <= 8 significant bits (or overflows to inf)
  if (std::fabs(r) >= std::ldexp(1.0, 128)) f = r > 0 ? INFINITY : -INFINITY;
  uint32_t u;
  std::memcpy(&u, &f, 4);
  return (uint16_t)(u >> 16);
}

void lca_oracle_round_bf16(const double* x, int64_t n, uint16_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = lca_oracle_round_bf16_scalar(x[i]);
}

// Group / window arithmetic of Sec. 4.2:  m = floor((L-w)/g), r = (L-w) mod g, k = w + r.
// When L < w + g there is no complete group and the method falls back to plain attention
// (Sec. 4.3, last paragraph of "Prefilling with Fused Context"): m = 0, k = L.
void lca_oracle_partition(int64_t L, int64_t w, int64_t g, int64_t* m, int64_t* k) {
  if (L < w + g) { *m = 0; *k = L; return; }
  *m = (L - w) / g;
  int64_t r = (L - w) % g;
  *k = w + r;
}

// Summary query of Alg. 1: q_bar = Avg(q_{L-n+1} .. q_L), n = n_summary_q (default g), here also
// averaged over the `heads` query heads that share the key/value stream.
//   q: [n_rows, heads, d]  -- the LAST n_rows query positions only
void lca_oracle_summary_query(const double* q, int64_t n_rows, int64_t heads, int64_t d,
                              double* qbar) {
  for (int64_t c = 0; c < d; ++c) qbar[c] = 0.0;
  for (int64_t r = 0; r < n_rows; ++r)
    for (int64_t h = 0; h < heads; ++h)
      for (int64_t c = 0; c < d; ++c) qbar[c] += q[(r * heads + h) * d + c];
  double cnt = (double)(n_rows * heads);
  for (int64_t c = 0; c < d; ++c) qbar[c] /= cnt;
}

// The condensation steps of Alg. 1 (scores, Eq. 6-8) for one key/value stream.
//   key  [L, dk]  the vectors the score is taken against (MLA: k_i = [c_i | k^R_i], dk = 576;
//                 GQA: the key of this KV head)
//   pool [L, dp]  the vectors that are pooled (MLA: c_i^KV; GQA: the value of this KV head)
//   qbar [dk]
// Outputs for j = 0..m-1:
//   scores [m*g]   s_i = scale * qbar . key_i
//   alpha  [m*g]   Eq. 6
//   pooled [m, dp] Eq. 7 (unrounded)
//   anchor [m]     Eq. 8, absolute 0-based token index, lowest index on ties
void lca_oracle_condense_stream(const double* key, int64_t dk, const double* pool, int64_t dp,
                                const double* qbar, int64_t L, int64_t g, int64_t w,
                                double scale, double* scores, double* alpha, double* pooled,
                                int32_t* anchor) {
  int64_t m, k;
  lca_oracle_partition(L, w, g, &m, &k);
#pragma omp parallel for schedule(static)
  for (int64_t j = 0; j < m; ++j) {
    // G_j = {j*g, ..., (j+1)*g - 1}
    double smax = -std::numeric_limits<double>::infinity();
    int64_t imax = j * g;
    for (int64_t i = j * g; i < (j + 1) * g; ++i) {
      double s = 0.0;
      for (int64_t c = 0; c < dk; ++c) s += qbar[c] * key[i * dk + c];
      s *= scale;
      scores[i] = s;
      if (s > smax) { smax = s; imax = i; }      // strict ">" keeps the lowest index on ties
    }
    double z = 0.0;
    for (int64_t i = j * g; i < (j + 1) * g; ++i) z += std::exp(scores[i] - smax);
    for (int64_t i = j * g; i < (j + 1) * g; ++i) alpha[i] = std::exp(scores[i] - smax) / z;
    for (int64_t c = 0; c < dp; ++c) {
      double acc = 0.0;
      for (int64_t i = j * g; i < (j + 1) * g; ++i) acc += alpha[i] * pool[i * dp + c];
      pooled[j * dp + c] = acc;
    }
    anchor[j] = (int32_t)imax;
  }
}

// Number of representatives / first local token seen by the query at 0-based position p
// (prefix length t = p + 1):  m_t = floor((t - w)/g) if t >= w + g else 0.
static inline int64_t reps_visible(int64_t p, int64_t w, int64_t g) {
  int64_t t = p + 1;
  if (t < w + g) return 0;
  return (t - w) / g;
}

// Eq. 10 at prefix length t for a list of query positions, one key/value stream.
//   q        [n_rows, heads, dk]   queries of the listed positions
//   pos      [n_rows]              0-based positions p (prefix length t = p+1)
//   key/val  [L, dk] / [L, dv]     per-token keys and values (MLA: [c|k^R] and c)
//   rkey/rval[m, dk] / [m, dv]     representative keys / values (MLA: [c_rep|k^R_anchor], c_rep)
//   out      [n_rows, heads, dv],  lse [n_rows, heads] (natural log of the softmax denominator
//                                  times exp(max), i.e. log sum exp of the logits)
void lca_oracle_attend_rows(const double* q, const int64_t* pos, int64_t n_rows, int64_t heads,
                            const double* key, const double* val, int64_t L,
                            const double* rkey, const double* rval, int64_t m,
                            int64_t dk, int64_t dv, int64_t g, int64_t w, double scale,
                            double rep_logit_bias, double* out, double* lse) {
  (void)L; (void)m;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int64_t r = 0; r < n_rows; ++r) {
    for (int64_t h = 0; h < heads; ++h) {
      const double* qv = q + (r * heads + h) * dk;
      int64_t p = pos[r];
      int64_t mt = reps_visible(p, w, g);      // representatives j < mt
      int64_t first = mt * g;                  // local tokens first..p
      int64_t n = mt + (p - first + 1);
      std::vector<double> logit((size_t)n);
      double lmax = -std::numeric_limits<double>::infinity();
      for (int64_t j = 0; j < mt; ++j) {
        double s = 0.0;
        for (int64_t c = 0; c < dk; ++c) s += qv[c] * rkey[j * dk + c];
        s = s * scale + rep_logit_bias;
        logit[(size_t)j] = s;
        lmax = std::max(lmax, s);
      }
      for (int64_t i = first; i <= p; ++i) {
        double s = 0.0;
        for (int64_t c = 0; c < dk; ++c) s += qv[c] * key[i * dk + c];
        s *= scale;
        logit[(size_t)(mt + i - first)] = s;
        lmax = std::max(lmax, s);
      }
      double z = 0.0;
      for (int64_t x = 0; x < n; ++x) { logit[(size_t)x] = std::exp(logit[(size_t)x] - lmax); z += logit[(size_t)x]; }
      double* o = out + (r * heads + h) * dv;
      for (int64_t c = 0; c < dv; ++c) o[c] = 0.0;
      for (int64_t j = 0; j < mt; ++j) {
        double pj = logit[(size_t)j] / z;
        for (int64_t c = 0; c < dv; ++c) o[c] += pj * rval[j * dv + c];
      }
      for (int64_t i = first; i <= p; ++i) {
        double pi = logit[(size_t)(mt + i - first)] / z;
        for (int64_t c = 0; c < dv; ++c) o[c] += pi * val[i * dv + c];
      }
      if (lse) lse[r * heads + h] = lmax + std::log(z);
    }
  }
}

// Decode step (Sec. 4.3): one query per head attends to every row of the condensed cache:
// the first n_rep rows are representatives (their logits get rep_logit_bias), the rest are
// the recent tokens kept in full.
//   q [heads, dk], ckey [rows, dk], cval [rows, dv]
void lca_oracle_decode(const double* q, int64_t heads, const double* ckey, const double* cval,
                       int64_t rows, int64_t n_rep, int64_t dk, int64_t dv, double scale,
                       double rep_logit_bias, double* out, double* lse) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t h = 0; h < heads; ++h) {
    const double* qv = q + h * dk;
    std::vector<double> logit((size_t)rows);
    double lmax = -std::numeric_limits<double>::infinity();
    for (int64_t x = 0; x < rows; ++x) {
      double s = 0.0;
      for (int64_t c = 0; c < dk; ++c) s += qv[c] * ckey[x * dk + c];
      s *= scale;
      if (x < n_rep) s += rep_logit_bias;
      logit[(size_t)x] = s;
      lmax = std::max(lmax, s);
    }
    double z = 0.0;
    for (int64_t x = 0; x < rows; ++x) { logit[(size_t)x] = std::exp(logit[(size_t)x] - lmax); z += logit[(size_t)x]; }
    double* o = out + h * dv;
    for (int64_t c = 0; c < dv; ++c) o[c] = 0.0;
    for (int64_t x = 0; x < rows; ++x) {
      double px = logit[(size_t)x] / z;
      for (int64_t c = 0; c < dv; ++c) o[c] += px * cval[x * dv + c];
    }
    if (lse) lse[h] = lmax + std::log(z);
  }
}

}  // extern "C"
