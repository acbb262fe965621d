// RegTop-k CPU oracle: TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, single-threaded restatement of the paper's sparsifier, written so that it can be
// checked against the paper by eye.  It exists to judge the CUDA library; the library never calls
// it, links it or shares a line with it.  Only the tests, the smoke check and the CPU-baseline leg
// of the benchmark may load this file's shared object.
//
// What follows the paper, and where:
//   accumulate        a = eps + g                                   Algorithm 1 step 3, Algorithm 2 step 7
//   top-k selector    k entries of largest magnitude                Section 2.2 (definition of Top_k)
//   posterior distortion  Delta = (g_prev - w*a_prev) / (w*a)       Eq. (Delta_def), Algorithm 2 step 8
//   regularised score |a| * tanh(|1 + Delta| / mu) on the previous support, |a| elsewhere (C = 1)
//                                                                   Section 4, Algorithm 2 step 9
//   exponent variant  metric |a|^y * regulariser, y <= 1            Remark 3 (appendix)
//   sparsified gradient = mask * a  (raw accumulator values)        Algorithm 2 steps 10-11
//   residual          eps' = a - ghat                               Algorithm 1 step 7, Algorithm 2 step 12
//   server            g = sum_n w_n * ghat_n                        Section 2.2 (aggregation equation)
//   model update      theta' = theta - eta * g                      Section 1 (after Eq. (1))
//   layer-wise masks  Top_{k_l} applied to each layer's slice of the score vector (the layer-wise
//                     sparsification the paper's "Further Related Work" points to); everything else as above
//
// Readings taken where the paper is silent (each listed in the design notes):
//   * ties in the magnitude sort: the lower index wins;
//   * the ranked quantity is |a| * regulariser (a magnitude), so the result of the sort is a mask;
//   * a zero denominator in Delta gives regulariser 1;
//   * exactly k pairs are emitted, in ascending index order, even if fewer than k scores are non-zero;
//   * eps' = a - ghat is evaluated as "+0 on the mask, a elsewhere", which is what a - a and a - 0 give;
//   * tanh in binary32 is the fixed operation sequence of regtopk_oracle_tanh below;
//   * every operation is an individually rounded IEEE binary32 operation in the written order
//     (compile with -ffp-contract=off; never -ffast-math).
//
//   * layer-wise selection: the model vector is cut into contiguous layers, layer l keeps its k_l best entries
//     by the same ranking, and the pairs of all layers are emitted together in ascending index order;
// Pins (tests/test_oracle_*.py): brute force over all subsets on tiny inputs; k = d pass-through;
// round 0 / mu = 0 / mu -> 0 against an independent Top-k with error feedback; the error-feedback
// identity; the toy logistic example (Delta = -1 exactly); the printed iteration-1 column of the
// paper's low-dimensional table; hand-worked distortion examples; tanh and pow against binary64;
// the exponent variant against its binary64 ranking; aggregation and the model update against hand sums.  Multi-round trajectories on the paper's own data cannot be pinned
// (its data and seeds are not published): "parity unpinned" for those curves only.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

struct Scored {
  float score;
  int32_t idx;
};

// Order of the magnitude sort: larger score first; equal scores: lower index first.
inline bool ranks_before(const Scored& x, const Scored& y) {
  if (x.score != y.score) return x.score > y.score;
  return x.idx < y.idx;
}

inline float bf16_bits_to_float(uint16_t h) {
  uint32_t u = static_cast<uint32_t>(h) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return f;
}

inline float grad_at(const void* grad, int grad_dtype, int64_t j) {
  if (grad_dtype == 1) return bf16_bits_to_float(static_cast<const uint16_t*>(grad)[j]);
  return static_cast<const float*>(grad)[j];
}

}  // namespace

extern "C" {

// tanh(x) for x >= 0 as a fixed sequence of binary32 operations.
//   x >= 9.25          -> 1
//   x <  0.25          -> x + x*q,  q = x2*(c3 + x2*(c5 + x2*(c7 + x2*c9))),  x2 = x*x  (odd Taylor terms)
//   otherwise          -> (1 - t)/(1 + t),  t = exp(-2x) = 2^n * P(f),
//                         y = (-2x)*log2(e), n = nearest integer to y (ties to even), f = y - n,
//                         P = degree-7 Taylor polynomial of 2^f in Horner form.
float regtopk_oracle_tanh(float x) {
  if (x >= 9.25f) return 1.0f;
  if (x < 0.25f) {
    const float c3 = -0x1.555556p-2f;  // -1/3
    const float c5 = 0x1.111112p-3f;   //  2/15
    const float c7 = -0x1.ba1ba2p-5f;  // -17/315
    const float c9 = 0x1.664f48p-6f;   //  62/2835
    float x2 = x * x;
    float q = c7 + x2 * c9;
    q = c5 + x2 * q;
    q = c3 + x2 * q;
    q = x2 * q;
    return x + x * q;
  }
  const float log2e = 0x1.715476p+0f;
  // (ln 2)^i / i!, i = 0..7
  const float e0 = 1.0f;
  const float e1 = 0x1.62e430p-1f;
  const float e2 = 0x1.ebfbe0p-3f;
  const float e3 = 0x1.c6b08ep-5f;
  const float e4 = 0x1.3b2ab6p-7f;
  const float e5 = 0x1.5d87fep-10f;
  const float e6 = 0x1.430912p-13f;
  const float e7 = 0x1.ffcbfcp-17f;
  float y = (-2.0f * x) * log2e;
  float n = std::nearbyintf(y);  // default rounding mode: ties to even
  float f = y - n;
  float p = e6 + f * e7;
  p = e5 + f * p;
  p = e4 + f * p;
  p = e3 + f * p;
  p = e2 + f * p;
  p = e1 + f * p;
  p = e0 + f * p;
  float t = std::ldexp(p, static_cast<int>(n));  // exact scaling by 2^n
  return (1.0f - t) / (1.0f + t);
}

// m^p for 0 <= m <= 1 and p >= 1 as a fixed sequence of binary32 operations (used for the exponent
// variant of Remark 3): 0 -> 0, 1 -> 1, otherwise 2^(p * log2 m) with
//   log2 m = e + log2 f, m = 2^e f, f in (sqrt(1/2), sqrt 2]; ln f = 2 s (1 + s2/3 + s2^2/5 + s2^3/7 + s2^4/9),
//   s = (f - 1)/(f + 1), s2 = s*s (Horner); log2 f = ln f * log2(e);
//   2^z as in regtopk_oracle_tanh (n = nearest integer, degree-7 polynomial of 2^(z - n), exact scaling);
//   z < -125 -> 0.
float regtopk_oracle_pow(float m, float p) {
  if (m == 0.0f) return 0.0f;
  if (m >= 1.0f) return 1.0f;
  int e0 = 0;
  if (m < 0x1p-126f) {  // subnormal: scale into the normal range (exact)
    m = m * 0x1p+24f;
    e0 = -24;
  }
  uint32_t b;
  std::memcpy(&b, &m, sizeof b);
  int e = static_cast<int>((b >> 23) & 0xffu) - 127 + e0;
  uint32_t fb = (b & 0x7fffffu) | 0x3f800000u;
  float f;
  std::memcpy(&f, &fb, sizeof f);
  if (f > 0x1.6a09e6p+0f) {  // sqrt(2)
    f = f * 0.5f;
    e += 1;
  }
  float s = (f - 1.0f) / (f + 1.0f);
  float s2 = s * s;
  float q = 0x1.c71c72p-4f;            // 1/9
  q = 0x1.24924ap-3f + s2 * q;         // 1/7
  q = 0x1.99999ap-3f + s2 * q;         // 1/5
  q = 0x1.555556p-2f + s2 * q;         // 1/3
  q = 1.0f + s2 * q;
  float lnf = (2.0f * s) * q;
  float log2f = lnf * 0x1.715476p+0f;  // log2(e)
  float L = static_cast<float>(e) + log2f;
  float z = p * L;
  if (!(z >= -125.0f)) return 0.0f;
  const float e1 = 0x1.62e430p-1f, e2 = 0x1.ebfbe0p-3f, e3 = 0x1.c6b08ep-5f, e4 = 0x1.3b2ab6p-7f;
  const float e5 = 0x1.5d87fep-10f, e6 = 0x1.430912p-13f, e7 = 0x1.ffcbfcp-17f;
  float n = std::nearbyintf(z);
  float fr = z - n;
  float P = e6 + fr * e7;
  P = e5 + fr * P;
  P = e4 + fr * P;
  P = e3 + fr * P;
  P = e2 + fr * P;
  P = e1 + fr * P;
  P = 1.0f + fr * P;
  return std::ldexp(P, static_cast<int>(n));  // n in [-125, 0]: exact scaling
}

// Accumulator and selection score of one worker (Algorithm 2 steps 7-9).
//   grad        d gradient entries, binary32 (grad_dtype 0) or bfloat16 bit patterns (grad_dtype 1)
//   eps         d residual entries carried from the previous round
//   n_prev      number of (index, value) pairs this worker sent in the previous round;
//               0 means "no previous round" (round 0) and gives plain Top-k scores
//   prev_idx, prev_val   those pairs: the previous mask's support and a^{t-1} on it
//   g_prev      d entries: the previous aggregated sparse gradient g^{t-1}
//   mu          regulariser parameter; mu == 0 selects plain Top-k (no regularisation)
//   omega_n     this worker's aggregation weight
//   y           exponent of Remark 3 (selection metric |a|^y * regulariser), 0 < y <= 1; y = 1 is Algorithm 2.
//               Ranking by |a|^y * m is ranking by |a| * m^(1/y); the score is computed in the second form,
//               which leaves the score off the previous support equal to |a|
//   a_out, score_out   d entries each
void regtopk_oracle_scores(int64_t d, const void* grad, int grad_dtype, const float* eps,
                           int64_t n_prev, const int32_t* prev_idx, const float* prev_val,
                           const float* g_prev, float mu, float omega_n, float y, float* a_out,
                           float* score_out) {
  for (int64_t j = 0; j < d; ++j) {
    float a = eps[j] + grad_at(grad, grad_dtype, j);
    a_out[j] = a;
    score_out[j] = std::fabs(a);  // regulariser 1 off the previous support
  }
  if (n_prev > 0 && mu > 0.0f) {
    for (int64_t i = 0; i < n_prev; ++i) {
      int64_t j = prev_idx[i];
      float a = a_out[j];
      float num = g_prev[j] - omega_n * prev_val[i];
      float den = omega_n * a;
      float m;
      if (den == 0.0f) {
        m = 1.0f;
      } else {
        float delta = num / den;
        float r = std::fabs(1.0f + delta);
        float x = r / mu;
        m = regtopk_oracle_tanh(x);
      }
      if (y != 1.0f) m = regtopk_oracle_pow(m, 1.0f / y);
      score_out[j] = std::fabs(a) * m;
    }
  }
}

// One sparsification round of one worker (Algorithm 2; Algorithm 1 when n_prev == 0 or mu == 0).
// eps is updated in place; out_idx/out_val receive exactly k pairs in ascending index order.
// select_mode 0: full sort of all d (score, index) records.  select_mode 1: std::nth_element on the
// same records with the same ordering (used only where a full sort is too slow; proven equal to
// mode 0 by the tests).  Returns 0, or -1 on invalid sizes.
int regtopk_oracle_worker_step(int64_t d, int64_t k, const void* grad, int grad_dtype, float* eps,
                               int64_t n_prev, const int32_t* prev_idx, const float* prev_val,
                               const float* g_prev, float mu, float omega_n, float y, int32_t* out_idx,
                               float* out_val, int select_mode) {
  if (d < 1 || k < 1 || k > d || d > INT32_MAX || !(y > 0.0f && y <= 1.0f)) return -1;
  std::vector<float> a(d), score(d);
  regtopk_oracle_scores(d, grad, grad_dtype, eps, n_prev, prev_idx, prev_val, g_prev, mu, omega_n, y,
                        a.data(), score.data());
  std::vector<Scored> rec(d);
  for (int64_t j = 0; j < d; ++j) rec[j] = Scored{score[j], static_cast<int32_t>(j)};
  if (select_mode == 1) {
    if (k < d) std::nth_element(rec.begin(), rec.begin() + k, rec.end(), ranks_before);
  } else {
    std::sort(rec.begin(), rec.end(), ranks_before);
  }
  std::vector<int32_t> chosen(k);
  for (int64_t i = 0; i < k; ++i) chosen[i] = rec[i].idx;
  std::sort(chosen.begin(), chosen.end());
  for (int64_t j = 0; j < d; ++j) eps[j] = a[j];  // a - 0
  for (int64_t i = 0; i < k; ++i) {
    int32_t j = chosen[i];
    out_idx[i] = j;
    out_val[i] = a[j];  // the raw accumulator, not the score
    eps[j] = 0.0f;      // a - a
  }
  return 0;
}

// Layer-wise form of the same round: the d coordinates are cut into n_seg contiguous layers, layer l being
// [seg_end[l-1], seg_end[l]) (seg_end ascending, seg_end[n_seg-1] == d), and the mask is the union over the layers
// of Top_{seg_k[l]} of the score restricted to that layer (1 <= seg_k[l] <= the layer's size).  Accumulator, posterior
// distortion, regulariser, sent values and residual are those of regtopk_oracle_worker_step; only the selector
// changes.  out_idx/out_val receive sum_l seg_k[l] pairs in ascending index order.  Selection by a full sort of
// each layer's records.  Returns 0, or -1 on invalid sizes.
int regtopk_oracle_worker_step_layered(int64_t d, int64_t n_seg, const int64_t* seg_end, const int64_t* seg_k,
                                       const void* grad, int grad_dtype, float* eps, int64_t n_prev,
                                       const int32_t* prev_idx, const float* prev_val, const float* g_prev,
                                       float mu, float omega_n, float y, int32_t* out_idx, float* out_val) {
  if (d < 1 || d > INT32_MAX || n_seg < 1 || !(y > 0.0f && y <= 1.0f)) return -1;
  int64_t begin = 0;
  for (int64_t l = 0; l < n_seg; ++l) {
    if (seg_end[l] <= begin || seg_k[l] < 1 || seg_k[l] > seg_end[l] - begin) return -1;
    begin = seg_end[l];
  }
  if (begin != d) return -1;
  std::vector<float> a(d), score(d);
  regtopk_oracle_scores(d, grad, grad_dtype, eps, n_prev, prev_idx, prev_val, g_prev, mu, omega_n, y,
                        a.data(), score.data());
  for (int64_t j = 0; j < d; ++j) eps[j] = a[j];  // (a minus 0 wherever no layer sends the entry)
  int64_t out = 0;
  begin = 0;
  for (int64_t l = 0; l < n_seg; ++l) {
    const int64_t end = seg_end[l], kl = seg_k[l];
    std::vector<Scored> rec;
    for (int64_t j = begin; j < end; ++j) rec.push_back(Scored{score[j], static_cast<int32_t>(j)});
    std::sort(rec.begin(), rec.end(), ranks_before);
    std::vector<int32_t> chosen(kl);
    for (int64_t i = 0; i < kl; ++i) chosen[i] = rec[i].idx;
    std::sort(chosen.begin(), chosen.end());
    for (int64_t i = 0; i < kl; ++i) {
      int32_t j = chosen[i];
      out_idx[out] = j;      // layers are index ranges in ascending order, so the whole output ascends
      out_val[out] = a[j];   // the raw accumulator, not the score
      eps[j] = 0.0f;         // a - a
      ++out;
    }
    begin = end;
  }
  return 0;
}

// Server aggregation g = sum_n w_n * ghat_n, workers added in the order n = 0..N-1, each term
// rounded (w_n * val) before it is added.  idx/val are [N][k].
void regtopk_oracle_aggregate(int64_t d, int32_t N, int64_t k, const float* omega,
                              const int32_t* idx, const float* val, float* g_out) {
  for (int64_t j = 0; j < d; ++j) g_out[j] = 0.0f;
  for (int32_t n = 0; n < N; ++n) {
    for (int64_t i = 0; i < k; ++i) {
      float t = omega[n] * val[n * k + i];
      int64_t j = idx[n * k + i];
      g_out[j] = g_out[j] + t;
    }
  }
}

// Model update of distributed SGD, theta^{t+1} = theta^t - eta * g^t (Section 1, after Eq. (1)), in place;
// the product is rounded before the subtraction.
void regtopk_oracle_model_update(int64_t d, float* theta, float eta, const float* g) {
  for (int64_t j = 0; j < d; ++j) {
    float step = eta * g[j];
    theta[j] = theta[j] - step;
  }
}

// Certificate for a claimed mask without sorting: with the scores of regtopk_oracle_scores and a set
// S of k distinct indices, S is the selector's answer exactly when no record outside S ranks before
// the last-ranked record of S.  Returns the number of records (over all d) that rank at or before
// that record; the mask is right iff the return value equals k.  Returns -1 if S is not k distinct
// in-range indices in ascending order.
int64_t regtopk_oracle_mask_certificate(int64_t d, int64_t k, const float* score,
                                        const int32_t* sel_idx) {
  if (k < 1 || k > d) return -1;
  for (int64_t i = 0; i < k; ++i) {
    if (sel_idx[i] < 0 || sel_idx[i] >= d) return -1;
    if (i > 0 && sel_idx[i] <= sel_idx[i - 1]) return -1;
  }
  Scored last{score[sel_idx[0]], sel_idx[0]};
  for (int64_t i = 1; i < k; ++i) {
    Scored r{score[sel_idx[i]], sel_idx[i]};
    if (ranks_before(last, r)) last = r;
  }
  int64_t count = 0;
  for (int64_t j = 0; j < d; ++j) {
    Scored r{score[j], static_cast<int32_t>(j)};
    if (!ranks_before(last, r)) ++count;  // r ranks before last, or is last
  }
  return count;
}

}  // extern "C"
