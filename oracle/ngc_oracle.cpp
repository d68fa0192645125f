/*
 * CPU oracle for the Neural Garbage Collection hot path -- TEST INFRASTRUCTURE ONLY.
 * See ngc_oracle.h for the contract.  Plain sequential C++17; OpenMP is used
 * only across independent lists / sequences / strips.  Floating point is
 * double (long double for the log-probability sums) except where the sampling
 * contract fixes single precision operation by operation.
 * Build: g++ -O2 -std=c++17 -fopenmp -ffp-contract=off -fno-fast-math -shared -fPIC
 */
#include "ngc_oracle.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

/* ---- element access ---------------------------------------------------- */

inline double widen(const void* base, int64_t idx, int dtype) {
  if (dtype == 0) return (double)((const float*)base)[idx];
  uint32_t bits = (uint32_t)((const uint16_t*)base)[idx] << 16;   /* bf16 = top half of fp32 */
  float f;
  std::memcpy(&f, &bits, 4);
  return (double)f;
}
inline int elt_size(int dtype) { return dtype == 0 ? 4 : 2; }

inline int lists_G(int lists, int L, int Hkv) { return lists == 0 ? 1 : (lists == 1 ? L : L * Hkv); }
inline int list_of(int lists, int l, int h, int Hkv) {
  return lists == 0 ? 0 : (lists == 1 ? l : l * Hkv + h);
}

/* ---- Philox4x32-10 ------------------------------------------------------ */

inline void mulhilo(uint32_t a, uint32_t b, uint32_t* hi, uint32_t* lo) {
  uint64_t p = (uint64_t)a * (uint64_t)b;
  *hi = (uint32_t)(p >> 32);
  *lo = (uint32_t)p;
}

void philox(const uint32_t c_in[4], const uint32_t k_in[2], uint32_t out[4]) {
  uint32_t c0 = c_in[0], c1 = c_in[1], c2 = c_in[2], c3 = c_in[3];
  uint32_t k0 = k_in[0], k1 = k_in[1];
  for (int r = 0; r < 10; ++r) {
    uint32_t hi0, lo0, hi1, lo1;
    mulhilo(0xD2511F53u, c0, &hi0, &lo0);
    mulhilo(0xCD9E8D57u, c2, &hi1, &lo1);
    uint32_t n0 = hi1 ^ c1 ^ k0;
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c3 ^ k1;
    uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;   /* key schedule: golden-ratio and sqrt(3)-1 Weyl increments */
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* ---- the fixed fp32 logarithm and the Gumbel transform ------------------- */

float dlog(float x) {
  uint32_t bits;
  std::memcpy(&bits, &x, 4);
  int e = (int)(bits >> 23) - 127;
  uint32_t mb = (bits & 0x007FFFFFu) | 0x3F800000u;
  float m;
  std::memcpy(&m, &mb, 4);                    /* m in [1,2) */
  if (m >= 1.41421354f) { m = m * 0.5f; e += 1; }   /* m in [sqrt(1/2), sqrt(2)) */
  float z = (m - 1.0f) / (m + 1.0f);
  float w = z * z;
  /* log m = 2 atanh z = z * (2 + 2/3 w + 2/5 w^2 + 2/7 w^3 + 2/9 w^4 + ...) */
  float p = 2.0f / 9.0f;
  p = std::fmaf(p, w, 2.0f / 7.0f);
  p = std::fmaf(p, w, 2.0f / 5.0f);
  p = std::fmaf(p, w, 2.0f / 3.0f);
  p = std::fmaf(p, w, 2.0f);
  float r = z * p;
  return std::fmaf((float)e, 0.693147180559945f, r);
}

inline float uniform01(uint32_t x) {
  /* odd multiples of 2^-24: (2*(x>>9)+1) * 2^-24, exact in fp32, never 0 or 1 */
  return (float)(2u * (x >> 9) + 1u) * 5.9604644775390625e-08f;
}

inline float gumbel(uint32_t x) {
  float u = uniform01(x);
  float t = -dlog(u);
  return -dlog(t);
}

float perturbed_key(float logit, uint64_t seed, uint64_t round, uint32_t list, uint32_t i, int greedy) {
  if (greedy) return logit;
  uint32_t ctr[4] = {i >> 2, list, (uint32_t)round, (uint32_t)(round >> 32)};
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t out[4];
  philox(ctr, key, out);
  return logit + gumbel(out[i & 3u]);
}

/* ---- Eq. (1) helpers ------------------------------------------------------ */

struct ListView {
  const float* s;        /* logits of the list */
  const int32_t* sigma;  /* kept_order of the list */
  int n, P, K;           /* units, protected, budget */
};

bool list_view(const float* logits, const int32_t* n, const int32_t* n_protect, const int32_t* budget,
               const int32_t* kept_order, int G, int n_max, int k_max, int64_t outer, int gi, ListView* lv) {
  lv->n = n[outer];
  lv->P = n_protect ? n_protect[outer] : 0;
  lv->K = budget[outer];
  lv->s = logits + (outer * G + gi) * (int64_t)n_max;
  lv->sigma = kept_order + (outer * G + gi) * (int64_t)k_max;
  return lv->P >= 0 && lv->P <= lv->K && lv->K <= lv->n && lv->n <= n_max && lv->K - lv->P <= k_max;
}

}  // namespace

extern "C" {

int ngc_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void ngc_oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) { philox(ctr, key, out); }
float ngc_oracle_dlog(float x) { return dlog(x); }
float ngc_oracle_uniform(uint32_t x) { return uniform01(x); }
float ngc_oracle_gumbel(uint32_t x) { return gumbel(x); }
float ngc_oracle_perturbed_key(float logit, uint64_t seed, uint64_t round, uint32_t list, uint32_t i, int greedy) {
  return perturbed_key(logit, seed, round, list, i, greedy);
}

/* Section 4.3: add Gumbel noise to the logits, keep the K largest perturbed values. */
int ngc_oracle_sample_evict(const float* logits, const int32_t* n, const int32_t* n_protect,
                            const int32_t* budget, int B, int G, int n_max, int k_max,
                            uint64_t seed, uint64_t round, uint32_t list_base, int greedy,
                            int32_t* kept_order, int32_t* kept_sorted, uint8_t* keep_mask,
                            int32_t* status) {
  int worst = 0;
#pragma omp parallel for schedule(dynamic) reduction(max : worst)
  for (int64_t li = 0; li < (int64_t)B * G; ++li) {
    int b = (int)(li / G);
    const float* s = logits + li * n_max;
    int32_t* ko = kept_order + li * k_max;
    int32_t* ks = kept_sorted + li * k_max;
    uint8_t* km = keep_mask ? keep_mask + li * n_max : nullptr;
    for (int j = 0; j < k_max; ++j) { ko[j] = -1; ks[j] = -1; }
    if (km) std::memset(km, 0, (size_t)n_max);
    int nb = n[b], P = n_protect ? n_protect[b] : 0, K = budget[b];
    int st = 0;
    if (!(P >= 0 && P <= K && K <= nb && nb <= n_max && K <= k_max)) st = 1;
    if (!st)
      for (int i = P; i < nb; ++i)
        if (std::isnan(s[i])) st = 2;
    if (status) status[li] = st;
    if (st) { worst = std::max(worst, st); continue; }

    /* candidates and their perturbed keys */
    std::vector<std::pair<float, int32_t>> cand;
    cand.reserve((size_t)(nb - P));
    for (int i = P; i < nb; ++i)
      cand.emplace_back(perturbed_key(s[i], seed, round, list_base + (uint32_t)li, (uint32_t)i, greedy), i);
    /* total order: larger key first, equal keys -> smaller index first */
    std::sort(cand.begin(), cand.end(), [](const std::pair<float, int32_t>& a, const std::pair<float, int32_t>& c) {
      if (a.first != c.first) return a.first > c.first;
      return a.second < c.second;
    });
    int Kp = K - P;
    std::vector<uint8_t> mask((size_t)nb, 0);
    for (int i = 0; i < P; ++i) mask[i] = 1;
    for (int j = 0; j < Kp; ++j) { ko[j] = cand[j].second; mask[cand[j].second] = 1; }
    int c = 0;
    for (int i = 0; i < nb; ++i)
      if (mask[i]) ks[c++] = i;
    if (km) std::memcpy(km, mask.data(), (size_t)nb);
  }
  return worst;
}

/* Eq. (1), literally: for step j the partition function runs over every
 * candidate not selected in steps 1..j-1. */
int ngc_oracle_evict_logprob(const float* logits, const int32_t* n, const int32_t* n_protect,
                             const int32_t* budget, const int32_t* kept_order,
                             int n_batches, int B, int G, int n_max, int k_max, double* logp) {
  int worst = 0;
#pragma omp parallel for schedule(dynamic) reduction(max : worst)
  for (int64_t li = 0; li < (int64_t)n_batches * B * G; ++li) {
    int64_t outer = li / G;
    int gi = (int)(li % G);
    ListView lv;
    logp[li] = std::numeric_limits<double>::quiet_NaN();
    if (!list_view(logits, n, n_protect, budget, kept_order, G, n_max, k_max, outer, gi, &lv)) { worst = 1; continue; }
    int Kp = lv.K - lv.P;
    bool ok = true;
    std::vector<uint8_t> gone((size_t)lv.n, 0);
    for (int j = 0; j < Kp && ok; ++j) {
      int t = lv.sigma[j];
      if (t < lv.P || t >= lv.n || gone[t]) ok = false; else gone[t] = 1;
    }
    if (!ok) { worst = std::max(worst, 3); continue; }
    std::fill(gone.begin(), gone.end(), 0);
    long double total = 0.0L;
    for (int j = 0; j < Kp; ++j) {
      /* log sum_{t not in {sigma_1..sigma_{j-1}}} exp(s_t), shifted by the max for range */
      long double mx = -std::numeric_limits<long double>::infinity();
      for (int t = lv.P; t < lv.n; ++t)
        if (!gone[t]) mx = std::max(mx, (long double)lv.s[t]);
      long double z = 0.0L;
      for (int t = lv.P; t < lv.n; ++t)
        if (!gone[t]) z += expl((long double)lv.s[t] - mx);
      long double lse = mx + logl(z);
      total += (long double)lv.s[lv.sigma[j]] - lse;
      gone[lv.sigma[j]] = 1;
    }
    logp[li] = (double)total;
  }
  return worst;
}

/* Derivative of Eq. (1) with respect to the logits, term by term:
 *   d/ds_i [ s_sigma_j - log sum_{t in A_j} exp s_t ] = [i == sigma_j] - [i in A_j] exp(s_i) / sum_{t in A_j} exp s_t ,
 * A_j = candidates not drawn before step j.  One softmax over A_j per step, O(K*N).
 * grad_logits[li][t] = grad_logp[li] * d logp / d s_t (grad_logp NULL = 1); protected units and
 * units beyond n[b] get 0; a list that fails validation gets NaN on its first n_max entries. */
int ngc_oracle_evict_logprob_grad(const float* logits, const int32_t* n, const int32_t* n_protect,
                                  const int32_t* budget, const int32_t* kept_order, const double* grad_logp,
                                  int n_batches, int B, int G, int n_max, int k_max, double* grad_logits) {
  int worst = 0;
#pragma omp parallel for schedule(dynamic) reduction(max : worst)
  for (int64_t li = 0; li < (int64_t)n_batches * B * G; ++li) {
    int64_t outer = li / G;
    int gi = (int)(li % G);
    ListView lv;
    double* g = grad_logits + li * n_max;
    for (int t = 0; t < n_max; ++t) g[t] = std::numeric_limits<double>::quiet_NaN();
    if (!list_view(logits, n, n_protect, budget, kept_order, G, n_max, k_max, outer, gi, &lv)) { worst = 1; continue; }
    int Kp = lv.K - lv.P;
    bool ok = true;
    std::vector<uint8_t> gone((size_t)lv.n, 0);
    for (int j = 0; j < Kp && ok; ++j) {
      int t = lv.sigma[j];
      if (t < lv.P || t >= lv.n || gone[t]) ok = false; else gone[t] = 1;
    }
    if (!ok) { worst = std::max(worst, 3); continue; }
    std::fill(gone.begin(), gone.end(), 0);
    std::vector<long double> acc((size_t)n_max, 0.0L);
    for (int j = 0; j < Kp; ++j) {
      long double mx = -std::numeric_limits<long double>::infinity();
      for (int t = lv.P; t < lv.n; ++t)
        if (!gone[t]) mx = std::max(mx, (long double)lv.s[t]);
      long double z = 0.0L;
      for (int t = lv.P; t < lv.n; ++t)
        if (!gone[t]) z += expl((long double)lv.s[t] - mx);
      for (int t = lv.P; t < lv.n; ++t)
        if (!gone[t]) acc[t] -= expl((long double)lv.s[t] - mx) / z;      /* softmax over A_j */
      acc[lv.sigma[j]] += 1.0L;
      gone[lv.sigma[j]] = 1;
    }
    double up = grad_logp ? grad_logp[li] : 1.0;
    for (int t = 0; t < n_max; ++t) g[t] = (double)(acc[t] * (long double)up);
  }
  return worst;
}

/* Remaining-mass scan: rem_j = sum of exp(s_t) over candidates still present
 * at step j = (mass never selected) + (mass of sigma_j..sigma_K).  Built from
 * the tail by addition, so no cancellation when little mass remains. */
int ngc_oracle_evict_logprob_scan(const float* logits, const int32_t* n, const int32_t* n_protect,
                                  const int32_t* budget, const int32_t* kept_order,
                                  int n_batches, int B, int G, int n_max, int k_max, double* logp) {
  int worst = 0;
#pragma omp parallel for schedule(dynamic) reduction(max : worst)
  for (int64_t li = 0; li < (int64_t)n_batches * B * G; ++li) {
    int64_t outer = li / G;
    int gi = (int)(li % G);
    ListView lv;
    logp[li] = std::numeric_limits<double>::quiet_NaN();
    if (!list_view(logits, n, n_protect, budget, kept_order, G, n_max, k_max, outer, gi, &lv)) { worst = 1; continue; }
    int Kp = lv.K - lv.P;
    std::vector<uint8_t> sel((size_t)lv.n, 0);
    bool ok = true;
    for (int j = 0; j < Kp && ok; ++j) {
      int t = lv.sigma[j];
      if (t < lv.P || t >= lv.n || sel[t]) ok = false; else sel[t] = 1;
    }
    if (!ok) { worst = std::max(worst, 3); continue; }
    if (Kp == 0) { logp[li] = 0.0; continue; }
    long double mx = -std::numeric_limits<long double>::infinity();
    for (int t = lv.P; t < lv.n; ++t) mx = std::max(mx, (long double)lv.s[t]);
    long double rem = 0.0L;
    for (int t = lv.P; t < lv.n; ++t)
      if (!sel[t]) rem += expl((long double)lv.s[t] - mx);
    long double total = 0.0L;
    for (int j = Kp - 1; j >= 0; --j) {
      long double sj = (long double)lv.s[lv.sigma[j]] - mx;
      rem += expl(sj);
      total += sj - logl(rem);
    }
    logp[li] = (double)total;
  }
  return worst;
}

/* Physical eviction, out of place: gather the kept tokens in ascending order. */
int ngc_oracle_compact_kv(const void* k, const void* v, const int64_t* seq_off, const int32_t* lens,
                          int L, int B, int Hkv, int d, int dtype,
                          const int32_t* kept_sorted, const int32_t* budget, int k_max,
                          int lists, int block,
                          void* k_out, void* v_out, int32_t* new_lens) {
  const int G = lists_G(lists, L, Hkv);
  const int64_t R = seq_off[B];
  const size_t row_bytes = (size_t)d * elt_size(dtype);
  int rc = 0;
  /* token lists per (b, gi) */
  std::vector<std::vector<int32_t>> tokens((size_t)B * G);
  for (int b = 0; b < B; ++b) {
    int len = lens[b];
    int n_units = (len + block - 1) / block;
    int K = budget[b];
    for (int gi = 0; gi < G; ++gi) {
      const int32_t* ks = kept_sorted + ((int64_t)b * G + gi) * k_max;
      std::vector<int32_t>& tk = tokens[(size_t)b * G + gi];
      int prev = -1;
      for (int j = 0; j < K; ++j) {
        int u = ks[j];
        if (K > k_max || u <= prev || u >= n_units) { rc = 3; break; }
        prev = u;
        for (int t = u * block; t < std::min((u + 1) * block, len); ++t) tk.push_back(t);
      }
    }
    if (rc) return rc;
    for (int gi = 1; gi < G; ++gi)
      if (tokens[(size_t)b * G + gi].size() != tokens[(size_t)b * G].size()) return 5;
    new_lens[b] = (int32_t)tokens[(size_t)b * G].size();
  }
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int l = 0; l < L; ++l)
    for (int b = 0; b < B; ++b)
      for (int h = 0; h < Hkv; ++h) {
        const std::vector<int32_t>& tk = tokens[(size_t)b * G + list_of(lists, l, h, Hkv)];
        int64_t base = ((int64_t)(l * Hkv + h) * R + seq_off[b]);
        for (size_t j = 0; j < tk.size(); ++j) {
          std::memcpy((char*)k_out + (base + (int64_t)j) * row_bytes, (const char*)k + (base + tk[j]) * row_bytes, row_bytes);
          std::memcpy((char*)v_out + (base + (int64_t)j) * row_bytes, (const char*)v + (base + tk[j]) * row_bytes, row_bytes);
        }
      }
  return 0;
}

/* out = softmax(scale * q K^T) V over the alive rows, in double. */
int ngc_oracle_decode_attn(void* k, void* v, const int64_t* seq_off, int32_t* lens,
                           int L, int B, int Hq, int Hkv, int d, int dtype,
                           const void* q, const void* new_k, const void* new_v,
                           int layer_begin, int layer_end, double scale, double* out) {
  const int64_t R = seq_off[B];
  const int g = Hq / Hkv;
  const size_t row_bytes = (size_t)d * elt_size(dtype);
  const bool append = new_k != nullptr && new_v != nullptr;
  int rc = 0;
  for (int b = 0; b < B; ++b)
    if (append && lens[b] + 1 > seq_off[b + 1] - seq_off[b]) rc = 4;
  if (rc) return rc;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int l = layer_begin; l < layer_end; ++l)
    for (int b = 0; b < B; ++b) {
      int T = lens[b];
      for (int h = 0; h < Hkv; ++h) {
        int64_t base = ((int64_t)(l * Hkv + h) * R + seq_off[b]);
        if (append) {
          int64_t src = (((int64_t)l * B + b) * Hkv + h);
          std::memcpy((char*)k + (base + T) * row_bytes, (const char*)new_k + src * row_bytes, row_bytes);
          std::memcpy((char*)v + (base + T) * row_bytes, (const char*)new_v + src * row_bytes, row_bytes);
        }
      }
      int Tv = T + (append ? 1 : 0);
      std::vector<double> z((size_t)std::max(Tv, 1));
      for (int hq = 0; hq < Hq; ++hq) {
        int h = hq / g;
        int64_t base = ((int64_t)(l * Hkv + h) * R + seq_off[b]);
        int64_t qo = (((int64_t)l * B + b) * Hq + hq) * d;
        double* o = out + qo;
        for (int c = 0; c < d; ++c) o[c] = 0.0;
        if (Tv == 0) continue;
        double mx = -std::numeric_limits<double>::infinity();
        for (int t = 0; t < Tv; ++t) {
          double acc = 0.0;
          for (int c = 0; c < d; ++c) acc += widen(q, qo + c, dtype) * widen(k, (base + t) * d + c, dtype);
          z[t] = scale * acc;
          mx = std::max(mx, z[t]);
        }
        double den = 0.0;
        for (int t = 0; t < Tv; ++t) { z[t] = std::exp(z[t] - mx); den += z[t]; }
        for (int t = 0; t < Tv; ++t) {
          double p = z[t] / den;
          for (int c = 0; c < d; ++c) o[c] += p * widen(v, (base + t) * d + c, dtype);
        }
      }
    }
  if (append && layer_end == L)
    for (int b = 0; b < B; ++b) lens[b] += 1;
  return 0;
}

/* Section 4.2: psi_t = mean over heads and recent queries of the softmax
 * attention weight on key t; s_j = mean of psi over block j. */
int ngc_oracle_score_evict(const void* k, const int64_t* seq_off, const int32_t* lens,
                           int L, int B, int Hq, int Hkv, int d, int dtype,
                           const void* q_recent, int w, int block, int lists, int log_transform,
                           double* logits, int n_max) {
  const int G = lists_G(lists, L, Hkv);
  const int64_t R = seq_off[B];
  const int g = Hq / Hkv;
  const double inv_sqrt_d = 1.0 / std::sqrt((double)d);
#pragma omp parallel for schedule(dynamic)
  for (int b = 0; b < B; ++b) {
    int T = lens[b];
    if (T <= 0) continue;
    int w_eff = std::min(w, T);              /* queries at negative positions do not exist */
    /* psi per list: sum of attention rows, divided by the number of rows */
    std::vector<std::vector<double>> psi((size_t)G, std::vector<double>((size_t)T, 0.0));
    std::vector<int64_t> rows((size_t)G, 0);
    std::vector<double> z((size_t)T);
    for (int l = 0; l < L; ++l)
      for (int hq = 0; hq < Hq; ++hq) {
        int h = hq / g;
        int gi = list_of(lists, l, h, Hkv);
        int64_t base = ((int64_t)(l * Hkv + h) * R + seq_off[b]);
        for (int j = w - w_eff; j < w; ++j) {
          int pos = T - w + j;                /* absolute position of this query */
          int64_t qo = ((((int64_t)l * B + b) * Hq + hq) * w + j) * d;
          double mx = -std::numeric_limits<double>::infinity();
          for (int t = 0; t <= pos; ++t) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += widen(q_recent, qo + c, dtype) * widen(k, (base + t) * d + c, dtype);
            z[t] = acc * inv_sqrt_d;
            mx = std::max(mx, z[t]);
          }
          double den = 0.0;
          for (int t = 0; t <= pos; ++t) { z[t] = std::exp(z[t] - mx); den += z[t]; }
          for (int t = 0; t <= pos; ++t) psi[gi][t] += z[t] / den;
          rows[gi] += 1;
        }
      }
    int n_units = (T + block - 1) / block;
    for (int gi = 0; gi < G; ++gi) {
      double* out = logits + ((int64_t)b * G + gi) * n_max;
      for (int u = 0; u < n_units && u < n_max; ++u) {
        int t0 = u * block, t1 = std::min(t0 + block, T);
        double acc = 0.0;
        for (int t = t0; t < t1; ++t) acc += psi[gi][t] / (double)rows[gi];
        double s = acc / (double)(t1 - t0);
        out[u] = log_transform ? std::log(s) : s;
      }
    }
  }
  return 0;
}

/* Gradient of the eviction scores with respect to the recent queries and the keys: the chain
 * rule through the block mean, the row average and the softmax of Section 4.2, written out.
 * With u(t) the unit of token t, |u| its size and n_rows the number of attention rows of the list:
 *   dL/dA[r][t]  = grad_logits[u(t)] / |u(t)| / n_rows        (divided by s_u as well when logit = log s)
 *   dL/dz[r][t]  = A[r][t] * (dL/dA[r][t] - sum_t' A[r][t'] dL/dA[r][t'])           (softmax)
 *   dL/dq[r]     = sum_t dL/dz[r][t] k[t] / sqrt(d),   dL/dk[t] += dL/dz[r][t] q[r] / sqrt(d). */
int ngc_oracle_score_evict_grad(const void* k, const int64_t* seq_off, const int32_t* lens,
                                int L, int B, int Hq, int Hkv, int d, int dtype,
                                const void* q_recent, int w, int block, int lists, int log_transform,
                                const double* grad_logits, int n_max, double* grad_q, double* grad_k) {
  const int G = lists_G(lists, L, Hkv);
  const int64_t R = seq_off[B];
  const int g = Hq / Hkv;
  const double inv_sqrt_d = 1.0 / std::sqrt((double)d);
  std::fill(grad_q, grad_q + (int64_t)L * B * Hq * w * d, 0.0);
  std::fill(grad_k, grad_k + (int64_t)L * Hkv * R * d, 0.0);
  std::vector<double> s_lin;                   /* forward scores, linear (needed for the log variant) */
  if (log_transform) {
    s_lin.assign((size_t)B * G * n_max, 0.0);
    ngc_oracle_score_evict(k, seq_off, lens, L, B, Hq, Hkv, d, dtype, q_recent, w, block, lists, 0, s_lin.data(), n_max);
  }
#pragma omp parallel for schedule(dynamic)
  for (int b = 0; b < B; ++b) {
    int T = lens[b];
    if (T <= 0) continue;
    int w_eff = std::min(w, T);
    std::vector<int64_t> rows((size_t)G, 0);
    for (int l = 0; l < L; ++l)
      for (int hq = 0; hq < Hq; ++hq) rows[list_of(lists, l, hq / g, Hkv)] += w_eff;
    /* dL/dA for any row of list gi, per token */
    std::vector<std::vector<double>> dA((size_t)G, std::vector<double>((size_t)T, 0.0));
    for (int gi = 0; gi < G; ++gi)
      for (int t = 0; t < T; ++t) {
        int u = t / block;
        if (u >= n_max) continue;
        int size = std::min((u + 1) * block, T) - u * block;
        double up = grad_logits[((int64_t)b * G + gi) * n_max + u];
        if (log_transform) up /= s_lin[((int64_t)b * G + gi) * n_max + u];
        dA[gi][t] = up / (double)size / (double)rows[gi];
      }
    std::vector<double> a((size_t)T);
    for (int l = 0; l < L; ++l)
      for (int hq = 0; hq < Hq; ++hq) {
        int h = hq / g;
        int gi = list_of(lists, l, h, Hkv);
        int64_t base = ((int64_t)(l * Hkv + h) * R + seq_off[b]);
        for (int j = w - w_eff; j < w; ++j) {
          int pos = T - w + j;
          int64_t qo = ((((int64_t)l * B + b) * Hq + hq) * w + j) * d;
          double mx = -std::numeric_limits<double>::infinity();
          for (int t = 0; t <= pos; ++t) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += widen(q_recent, qo + c, dtype) * widen(k, (base + t) * d + c, dtype);
            a[t] = acc * inv_sqrt_d;
            mx = std::max(mx, a[t]);
          }
          double den = 0.0;
          for (int t = 0; t <= pos; ++t) { a[t] = std::exp(a[t] - mx); den += a[t]; }
          double dot = 0.0;
          for (int t = 0; t <= pos; ++t) { a[t] /= den; dot += a[t] * dA[gi][t]; }
          for (int t = 0; t <= pos; ++t) {
            double dz = a[t] * (dA[gi][t] - dot) * inv_sqrt_d;
            for (int c = 0; c < d; ++c) {
              grad_q[qo + c] += dz * widen(k, (base + t) * d + c, dtype);
              grad_k[(base + t) * d + c] += dz * widen(q_recent, qo + c, dtype);
            }
          }
        }
      }
  }
  return 0;
}

}  // extern "C"
