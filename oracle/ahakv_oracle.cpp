// AhaKV eviction oracle -- TEST INFRASTRUCTURE, not a product path.
//
// A plain, slow, double-precision CPU statement of what the eviction step of
// AhaKV (arXiv 2506.03762) computes for one layer: SG-softmax over the last r
// query rows, Recent Accumulation, value-prior refinement, budgeted selection
// and the gather of the surviving K/V rows.  It exists so that the CUDA path
// can be checked element by element; nothing in the product may call it, and
// it shares no code, header, table or constant with the CUDA path.
//
// Every function below takes the paper's steps in the paper's order with no
// blocking, fusion or reordering.  The only parallelism is one std::thread per
// independent (sequence, KV head) unit.
//
// Readings of the paper taken here (the paper is silent or garbled on them):
//   * Eq. 9 lost its exponential in print; it is e^{lambda x_i} / sum_j e^{lambda x_j},
//     the only form from which Eq. 10 follows.
//   * lambda multiplies the raw dot product q.k and replaces 1/sqrt(d)
//     (Eq. 8 holds only for unscaled logits of variance d; Eq. 12 follows).
//   * log is the natural logarithm (Appendix A works with e^x).
//   * In Eq. 12, k is the total budget B and i is the number of tokens the row
//     has seen (its logical position + 1); when i <= k the formula is not
//     real-valued and 1/sqrt(d) is used instead.
//   * Eq. 5 is read as exactly r rows: the last r query positions.
//   * Avgpool (Eq. 13): stride 1, odd width w, same length; edge windows are
//     truncated and divided by the count of in-range elements (or by w when
//     the zero-pad flag is set).  max(gamma) in Eq. 14 runs over all n tokens.
//   * Algorithm 1 line 11 takes TopK of the refined score (line 10), over the
//     tokens outside the recent window, so that |S| = B exactly.
//   * Ties: higher score first, then lower index.  Kept rows stay in ascending
//     original position.
//   * GQA: the score of a KV head is the mean (or, with the group-max flag, the
//     maximum) over its query heads of the per-head accumulated score.
//     PARITY UNPINNED by the paper: it never mentions grouped queries.  The
//     pooling edge rule and the tie order are unpinned by the paper as well.
//
// Layouts (all dense, row-major, d contiguous):
//   q_obs [B, Hq, r, d]   k, v [B, Hkv, n, d]   score [B, Hkv, n]
//   kept_idx [B, Hkv, n_keep]   k_out, v_out [B, Hkv, n_keep, d]
// with n_keep = min(n, budget).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <thread>
#include <vector>

extern "C" {

enum { ORACLE_F32 = 0, ORACLE_F16 = 1, ORACLE_BF16 = 2 };
enum { ORACLE_SCALE_FIXED = 0, ORACLE_SCALE_ADAPTIVE_ROW = 1, ORACLE_SCALE_ADAPTIVE_CALL = 2 };
enum { ORACLE_FLAG_VALUE_PRIOR = 1, ORACLE_FLAG_POOL_ZERO_PAD = 2, ORACLE_FLAG_GROUP_MAX = 4 };

typedef struct {
  int32_t batch, n_q_heads, n_kv_heads, head_dim;
  int32_t n_ctx;          // n: rows in K and V
  int64_t n_total;        // logical tokens seen so far (>= n_ctx)
  int32_t obs_window;     // r
  int32_t recent_window;  // B_r
  int32_t budget;         // B = B_r + B_s
  int32_t dtype;          // of q, k, v
  int32_t scale_mode;
  double scale;           // lambda when scale_mode == FIXED
  int32_t pool_kernel;    // odd width of the mean filter
  uint32_t flags;
  // Optional: the logical positions of the r observation rows, strictly ascending, each inside the cache
  // ([n_total - n_ctx, n_total)).  NULL = the last r positions (Eq. 5).  With positions given, row i sees the
  // cache rows up to its own position (Eq. 1's causal mask) and Eq. 12 counts the tokens up to it.
  const int64_t* obs_pos;
} oracle_params;

}  // extern "C"

namespace {

// ---- exact widening of the storage types to double ------------------------
double half_bits_to_double(uint16_t h) {
  const int sign = (h >> 15) & 1, e = (h >> 10) & 0x1f, m = h & 0x3ff;
  double v;
  if (e == 0) v = std::ldexp((double)m, -24);                       // subnormal
  else if (e == 31) v = m ? std::nan("") : INFINITY;
  else v = std::ldexp((double)(m | 0x400), e - 25);
  return sign ? -v : v;
}
double bf16_bits_to_double(uint16_t b) {
  const uint32_t u = (uint32_t)b << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return (double)f;
}
double load_elem(const void* p, int dtype, size_t idx) {
  switch (dtype) {
    case ORACLE_F32: return (double)((const float*)p)[idx];
    case ORACLE_F16: return half_bits_to_double(((const uint16_t*)p)[idx]);
    default: return bf16_bits_to_double(((const uint16_t*)p)[idx]);
  }
}
size_t elem_size(int dtype) { return dtype == ORACLE_F32 ? 4 : 2; }

bool positions_ok(const oracle_params* p) {
  if (!p->obs_pos) return true;
  for (int i = 0; i < p->obs_window; ++i) {
    if (p->obs_pos[i] < p->n_total - p->n_ctx || p->obs_pos[i] >= p->n_total) return false;
    if (i > 0 && p->obs_pos[i] <= p->obs_pos[i - 1]) return false;
  }
  return true;
}

bool params_ok(const oracle_params* p) {
  return p && p->batch > 0 && p->n_q_heads > 0 && p->n_kv_heads > 0 && p->head_dim > 0 &&
         p->n_q_heads % p->n_kv_heads == 0 && p->n_ctx > 0 && p->n_total >= p->n_ctx &&
         p->obs_window >= 1 && p->obs_window <= p->n_ctx && p->budget >= 1 &&
         p->recent_window >= 0 && p->recent_window <= p->budget && p->dtype >= 0 && p->dtype <= 2 &&
         p->scale_mode >= 0 && p->scale_mode <= 2 && p->pool_kernel >= 1 && (p->pool_kernel & 1) &&
         positions_ok(p);
}

// Eq. 12: lambda = sqrt(2 log(i/k) / d); outside its domain fall back to 1/sqrt(d).
double eq12_lambda(double i_tokens, double k_budget, int d) {
  const double ratio = i_tokens / k_budget;
  if (!(ratio > 1.0)) return 1.0 / std::sqrt((double)d);
  return std::sqrt(2.0 * std::log(ratio) / (double)d);
}

// Logical position of observation row i (0-based among the r rows): the last r positions unless given.
int64_t row_position(const oracle_params* p, int i) {
  return p->obs_pos ? p->obs_pos[i] : p->n_total - p->obs_window + i;
}

// lambda for observation row i; at logical position p_i it has seen p_i + 1 tokens.
double row_lambda(const oracle_params* p, int i) {
  switch (p->scale_mode) {
    case ORACLE_SCALE_FIXED: return p->scale;
    case ORACLE_SCALE_ADAPTIVE_ROW:
      return eq12_lambda((double)(row_position(p, i) + 1), (double)p->budget, p->head_dim);
    default: return eq12_lambda((double)p->n_total, (double)p->budget, p->head_dim);
  }
}

// Step 1 of every unit: widen the stored elements to double, exactly.
std::vector<double> widen(const void* p, int dtype, size_t off, size_t count) {
  std::vector<double> out(count);
  for (size_t t = 0; t < count; ++t) out[t] = load_elem(p, dtype, off + t);
  return out;
}

// SG-softmax of one observation row against the keys it may see (Eq. 1 with the
// causal mask, Eq. 9 for the gain).  qrow [d] and kmat [n, d] are already
// widened.  a[j] = 0 for masked columns.
void attention_row(const oracle_params* p, const double* qrow, const double* kmat, int i,
                   std::vector<double>& a) {
  const int n = p->n_ctx, d = p->head_dim;
  // row i sees the cache columns up to its own position: n - r + i for the last r positions
  const int last = (int)(row_position(p, i) - (p->n_total - p->n_ctx));
  const double lam = row_lambda(p, i);
  a.assign(n, 0.0);
  std::vector<double> x(last + 1);
  double m = -INFINITY;
  for (int j = 0; j <= last; ++j) {
    double w = 0.0;
    for (int c = 0; c < d; ++c) w += qrow[c] * kmat[(size_t)j * d + c];
    x[j] = lam * w;
    m = std::max(m, x[j]);
  }
  double Z = 0.0;
  for (int j = 0; j <= last; ++j) Z += std::exp(x[j] - m);
  for (int j = 0; j <= last; ++j) a[j] = std::exp(x[j] - m) / Z;
}

std::vector<double> widen_q_head(const oracle_params* p, const void* q_obs, int b, int hq) {
  const size_t per_head = (size_t)p->obs_window * p->head_dim;
  return widen(q_obs, p->dtype, ((size_t)b * p->n_q_heads + hq) * per_head, per_head);
}
std::vector<double> widen_kv_head(const oracle_params* p, const void* kv, int b, int h) {
  const size_t per_head = (size_t)p->n_ctx * p->head_dim;
  return widen(kv, p->dtype, ((size_t)b * p->n_kv_heads + h) * per_head, per_head);
}

// Recent Accumulation (Eq. 5) for one KV head, pooled over its query heads.
void accumulated_score_unit(const oracle_params* p, const void* q_obs, const void* k, int b, int h,
                            double* S /*[n]*/) {
  const int n = p->n_ctx, r = p->obs_window, d = p->head_dim, G = p->n_q_heads / p->n_kv_heads;
  const std::vector<double> kmat = widen_kv_head(p, k, b, h);
  std::vector<double> a, Sq(n);
  for (int j = 0; j < n; ++j) S[j] = 0.0;
  for (int g = 0; g < G; ++g) {
    const std::vector<double> qmat = widen_q_head(p, q_obs, b, h * G + g);
    std::fill(Sq.begin(), Sq.end(), 0.0);
    for (int i = 0; i < r; ++i) {
      attention_row(p, qmat.data() + (size_t)i * d, kmat.data(), i, a);
      for (int j = 0; j < n; ++j) Sq[j] += a[j];
    }
    for (int j = 0; j < n; ++j) {
      if (p->flags & ORACLE_FLAG_GROUP_MAX) S[j] = (g == 0) ? Sq[j] : std::max(S[j], Sq[j]);
      else S[j] += Sq[j] / (double)G;
    }
  }
}

// Value prior (Eq. 13-14): nu_j = |V_j|^2, gamma = mean filter of nu, gamma_bar = gamma / max gamma.
void value_prior_unit(const oracle_params* p, const void* v, int b, int h, double* gbar /*[n]*/) {
  const int n = p->n_ctx, d = p->head_dim, half = p->pool_kernel / 2;
  const std::vector<double> vmat = widen_kv_head(p, v, b, h);
  std::vector<double> nu(n), gamma(n);
  for (int j = 0; j < n; ++j) {
    double s = 0.0;
    for (int c = 0; c < d; ++c) s += vmat[(size_t)j * d + c] * vmat[(size_t)j * d + c];
    nu[j] = s;
  }
  for (int j = 0; j < n; ++j) {
    double s = 0.0;
    int cnt = 0;
    for (int t = j - half; t <= j + half; ++t)
      if (t >= 0 && t < n) { s += nu[t]; ++cnt; }
    gamma[j] = s / (double)((p->flags & ORACLE_FLAG_POOL_ZERO_PAD) ? p->pool_kernel : cnt);
  }
  const double gmax = *std::max_element(gamma.begin(), gamma.end());
  for (int j = 0; j < n; ++j) gbar[j] = gamma[j] / gmax;
}

// Eviction score of one unit: Eq. 5, then Eq. 15 when the value prior is on,
// then the carried score F_{t-1} of Algorithm 1's generation phase when given.
void score_unit(const oracle_params* p, const void* q_obs, const void* k, const void* v,
                const double* score_prev, double* raw, double* score, int b, int h) {
  const int n = p->n_ctx;
  const size_t off = ((size_t)b * p->n_kv_heads + h) * (size_t)n;
  std::vector<double> S(n), gbar;
  accumulated_score_unit(p, q_obs, k, b, h, S.data());
  if (raw) std::copy(S.begin(), S.end(), raw + off);
  if (p->flags & ORACLE_FLAG_VALUE_PRIOR) {
    gbar.resize(n);
    value_prior_unit(p, v, b, h, gbar.data());
    for (int j = 0; j < n; ++j) S[j] = gbar[j] * S[j];
  }
  if (score_prev)
    for (int j = 0; j < n; ++j) S[j] += score_prev[off + j];
  std::copy(S.begin(), S.end(), score + off);
}

// Algorithm 1: keep the recent B_r tokens, TopK(B_s) of the rest, ascending.
void select_unit(const oracle_params* p, const double* score /*[n]*/, int32_t* kept /*[n_keep]*/) {
  const int n = p->n_ctx, Bud = p->budget, Br = p->recent_window;
  if (n <= Bud) {
    for (int j = 0; j < n; ++j) kept[j] = j;
    return;
  }
  const int Bs = Bud - Br, n_cand = n - Br;
  std::vector<int32_t> order(n_cand);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) {
    if (score[x] != score[y]) return score[x] > score[y];
    return x < y;
  });
  std::vector<int32_t> S(order.begin(), order.begin() + Bs);
  for (int j = n - Br; j < n; ++j) S.push_back(j);
  std::sort(S.begin(), S.end());
  std::copy(S.begin(), S.end(), kept);
}

template <class F>
void for_each_unit(const oracle_params* p, int nthreads, F f) {
  const int units = p->batch * p->n_kv_heads;
  int T = nthreads > 0 ? nthreads : (int)std::thread::hardware_concurrency();
  T = std::max(1, std::min(T, units));
  if (T == 1) {
    for (int u = 0; u < units; ++u) f(u / p->n_kv_heads, u % p->n_kv_heads);
    return;
  }
  std::vector<std::thread> pool;
  for (int t = 0; t < T; ++t)
    pool.emplace_back([=]() {
      for (int u = t; u < units; u += T) f(u / p->n_kv_heads, u % p->n_kv_heads);
    });
  for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

// Eq. 12 as printed (natural log); 1/sqrt(d) when n_total <= budget.
double ahakv_oracle_lambda(int64_t n_total, int32_t budget, int32_t head_dim) {
  return eq12_lambda((double)n_total, (double)budget, head_dim);
}

// The r x n attention matrix of one query head (b, hq), row-major, masked
// columns zero.  For tests on small shapes.
int ahakv_oracle_attention(const oracle_params* p, const void* q_obs, const void* k, int32_t b,
                           int32_t hq, double* a_out /*[r, n]*/) {
  if (!params_ok(p) || b < 0 || b >= p->batch || hq < 0 || hq >= p->n_q_heads) return 1;
  const int G = p->n_q_heads / p->n_kv_heads;
  const std::vector<double> qmat = widen_q_head(p, q_obs, b, hq), kmat = widen_kv_head(p, k, b, hq / G);
  std::vector<double> a;
  for (int i = 0; i < p->obs_window; ++i) {
    attention_row(p, qmat.data() + (size_t)i * p->head_dim, kmat.data(), i, a);
    std::copy(a.begin(), a.end(), a_out + (size_t)i * p->n_ctx);
  }
  return 0;
}

// Eq. 6: H_i = -sum_j a_ij log a_ij for each observation row of head (b, hq).
int ahakv_oracle_row_entropy(const oracle_params* p, const void* q_obs, const void* k, int32_t b,
                             int32_t hq, double* H_out /*[r]*/) {
  if (!params_ok(p) || b < 0 || b >= p->batch || hq < 0 || hq >= p->n_q_heads) return 1;
  const int G = p->n_q_heads / p->n_kv_heads;
  const std::vector<double> qmat = widen_q_head(p, q_obs, b, hq), kmat = widen_kv_head(p, k, b, hq / G);
  std::vector<double> a;
  for (int i = 0; i < p->obs_window; ++i) {
    attention_row(p, qmat.data() + (size_t)i * p->head_dim, kmat.data(), i, a);
    double H = 0.0;
    for (double x : a)
      if (x > 0.0) H -= x * std::log(x);
    H_out[i] = H;
  }
  return 0;
}

// score [B,Hkv,n] (refined, plus score_prev when given); raw (nullable) receives
// the accumulated score before the value prior.
int ahakv_oracle_score(const oracle_params* p, const void* q_obs, const void* k, const void* v,
                       const double* score_prev, double* raw, double* score, int32_t nthreads) {
  if (!params_ok(p)) return 1;
  for_each_unit(p, nthreads,
                [=](int b, int h) { score_unit(p, q_obs, k, v, score_prev, raw, score, b, h); });
  return 0;
}

int ahakv_oracle_select(const oracle_params* p, const double* score, int32_t* kept_idx) {
  if (!params_ok(p)) return 1;
  const int n_keep = std::min(p->n_ctx, p->budget);
  for (int u = 0; u < p->batch * p->n_kv_heads; ++u)
    select_unit(p, score + (size_t)u * p->n_ctx, kept_idx + (size_t)u * n_keep);
  return 0;
}

// K <- K_S, V <- V_S (Algorithm 1, generation line 1) and the same gather of the score.
int ahakv_oracle_compact(const oracle_params* p, const void* k, const void* v, const double* score,
                         const int32_t* kept_idx, void* k_out, void* v_out, double* score_out) {
  if (!params_ok(p)) return 1;
  const int n = p->n_ctx, n_keep = std::min(n, p->budget);
  const size_t row = (size_t)p->head_dim * elem_size(p->dtype);
  for (int u = 0; u < p->batch * p->n_kv_heads; ++u)
    for (int t = 0; t < n_keep; ++t) {
      const int32_t j = kept_idx[(size_t)u * n_keep + t];
      if (j < 0 || j >= n) return 2;
      std::memcpy((char*)k_out + ((size_t)u * n_keep + t) * row, (const char*)k + ((size_t)u * n + j) * row, row);
      std::memcpy((char*)v_out + ((size_t)u * n_keep + t) * row, (const char*)v + ((size_t)u * n + j) * row, row);
      if (score && score_out) score_out[(size_t)u * n_keep + t] = score[(size_t)u * n + j];
    }
  return 0;
}

// One whole eviction step: score, select, compact.  score_full (nullable)
// receives the refined score over all n tokens.
int ahakv_oracle_evict(const oracle_params* p, const void* q_obs, const void* k, const void* v,
                       const double* score_prev, void* k_out, void* v_out, double* score_out,
                       int32_t* kept_idx, double* score_full, int32_t nthreads) {
  if (!params_ok(p)) return 1;
  std::vector<double> local;
  double* s = score_full;
  if (!s) {
    local.resize((size_t)p->batch * p->n_kv_heads * p->n_ctx);
    s = local.data();
  }
  int rc = ahakv_oracle_score(p, q_obs, k, v, score_prev, nullptr, s, nthreads);
  if (rc) return rc;
  rc = ahakv_oracle_select(p, s, kept_idx);
  if (rc) return rc;
  return ahakv_oracle_compact(p, k, v, s, kept_idx, k_out, v_out, score_out);
}

}  // extern "C"
