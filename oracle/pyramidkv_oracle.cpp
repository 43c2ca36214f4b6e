// PyramidKV prefill KV-cache compression: CPU ORACLE.
//
// TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  This file is the slow, plain
// restatement of what the compression step computes, written from the paper's
// definitions.  It shares no code with the CUDA library and must never be
// called by it.  Only the tests, the smoke check and the benchmark's CPU
// baseline may use it.
//
// Steps, in the paper's order (Section 4.2):
//   budgets   Section 4.2.1, Eq. 1   pyramidal per-layer budgets k^l (and the appendix's geometric decay)
//   logits    Section 4.2.2, Eq. 2   A^h = softmax(Q^h K^hT / sqrt(d_k)), window rows only
//   scores    Section 4.2.2, Eq. 3   s_i = sum over window rows j of A[j][i]
//   pool      Section 4.2.2          a pooling layer applied to the scores (max, odd width)
//   select    Section 4.2.2          top k^l per head, plus the last alpha tokens always
//   gather    Appendix (eviction by gather): copy the kept rows into a new tensor
//   paged     Appendix (paged attention): the same rows placed in pages through a per-layer block table
//
// Where the paper is silent the readings are: the budget B counts the alpha
// window rows, the pyramid is laid over B - alpha; real budgets are floored and
// the leftover units go one each to the lowest layers; the window rows are
// causal among themselves; GQA scores are the mean over the query heads of a
// group; pooling is a centred max clipped at both ends; ties are broken by
// (value descending, position ascending); kept positions are emitted ascending.
// Variants reachable through arguments: a mean pool (zeros outside the prefix,
// divided by the full width, in float) and binary16 inputs.
//
// Arithmetic: every floating-point accumulation is in double; scores are
// rounded once to float at the end of the score step, and the pool and the
// selection work on those floats.
//
// Pins (tests/test_oracle_*.py): budget closed forms and sums; softmax mass
// invariant; Q = 0 closed form; library softmax / max_pool1d / avg_pool1d / sort
// on small inputs; brute-force subset search; identity when the context fits the
// budget; every finite 16-bit pattern against the library's widening.
// Absolute score values on random data have no value printed in the paper.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline double widen_bf16(uint16_t bits) {
  uint32_t w = static_cast<uint32_t>(bits) << 16;
  float f;
  std::memcpy(&f, &w, sizeof f);
  return static_cast<double>(f);
}

// IEEE 754 binary16: 1 sign bit, 5 exponent bits (bias 15), 10 fraction bits.  Every value is exact in double.
inline double widen_fp16(uint16_t bits) {
  const int sign = bits >> 15, e = (bits >> 10) & 31, frac = bits & 1023;
  double mag;
  if (e == 0) mag = std::ldexp(static_cast<double>(frac), -24);                 // zero and subnormals
  else if (e == 31) mag = frac ? std::nan("") : HUGE_VAL;
  else mag = std::ldexp(1.0 + static_cast<double>(frac) / 1024.0, e - 15);
  return sign ? -mag : mag;
}

// Element (row, c) of a [rows][d] matrix stored as float (dtype 0), bfloat16 bits (dtype 1) or binary16 bits
// (dtype 2).
inline double elem(const void* base, int dtype, int64_t index) {
  if (dtype == 0) return static_cast<double>(static_cast<const float*>(base)[index]);
  if (dtype == 2) return widen_fp16(static_cast<const uint16_t*>(base)[index]);
  return widen_bf16(static_cast<const uint16_t*>(base)[index]);
}

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------
// Section 4.2.1, Eq. 1.  k_total = m (B - alpha) is the budget that remains
// after the alpha instruction tokens are set aside in every layer.
//   k^{m-1} = k_total / (beta m),  k^0 = 2 k_total / m - k^{m-1},
//   k^l     = k^0 - (k^0 - k^{m-1}) l / (m - 1).
// Substituting gives  k^l = k_total [ (2 beta - 1)(m - 1) - (2 beta - 2) l ] / (beta m (m - 1)).
// beta is snapped to a multiple of 1/1024 so the whole schedule is integer
// arithmetic: floor each k^l, then hand the leftover units to layers 0, 1, ...
// Returns 0, or -1 for arguments the schedule is not defined for.
int orc_layer_budgets(int m, int avg_budget, int alpha, double beta, int32_t* k_out) {
  if (m < 1 || alpha < 1 || avg_budget < alpha || !(beta >= 1.0) || beta > 1.0e6) return -1;
  const int64_t k_total = static_cast<int64_t>(m) * (avg_budget - alpha);
  if (m == 1) {
    k_out[0] = static_cast<int32_t>(k_total);
    return 0;
  }
  const int64_t bq = std::llround(beta * 1024.0);          // beta = bq / 1024
  const __int128 den = static_cast<__int128>(bq) * m * (m - 1);
  int64_t assigned = 0;
  for (int l = 0; l < m; ++l) {
    const __int128 num = static_cast<__int128>(2 * bq - 1024) * (m - 1) -
                         static_cast<__int128>(2 * bq - 2048) * l;
    const int64_t kl = static_cast<int64_t>((static_cast<__int128>(k_total) * num) / den);
    k_out[l] = static_cast<int32_t>(kl);
    assigned += kl;
  }
  int64_t left = k_total - assigned;                        // 0 <= left < m
  for (int l = 0; l < m && left > 0; ++l, --left) k_out[l] += 1;
  return 0;
}

// ---------------------------------------------------------------------------
// Appendix "Allocation Strategies": a geometric (equivalently, exponential in the
// layer index) decay in place of Eq. 1's arithmetic one.  The paper names the
// strategy without a formula; the reading keeps Eq. 1's two constraints and changes
// only the shape between them:
//   real budgets with a constant ratio rho >= 1 between consecutive layers,
//   x_l = x_{m-1} rho^(m-1-l),   sum_l x_l = k_total,   x_{m-1} = k_total / (beta m),
// which makes rho the root of  1 + rho + ... + rho^(m-1) = beta m  (unique for rho >= 1;
// beta = 1 gives rho = 1, the uniform split).  The root is found by bisection and then
// snapped to the nearest multiple of 2^-20, so that two implementations agree on it
// bit for bit; with the snapped rho the shares are  x_l = k_total rho^(m-1-l) / sum_j rho^j
// (powers by repeated multiplication, the sum taken from j = 0 upward, all in double).
// Flooring and the leftover units follow the linear schedule's rule.
// Returns 0, or -1 for arguments the schedule is not defined for.
int orc_layer_budgets_geometric(int m, int avg_budget, int alpha, double beta, int32_t* k_out) {
  if (m < 1 || alpha < 1 || avg_budget < alpha || !(beta >= 1.0) || beta > 1.0e6) return -1;
  const int64_t k_total = static_cast<int64_t>(m) * (avg_budget - alpha);
  const int64_t bq = std::llround(beta * 1024.0);          // beta = bq / 1024
  double rho = 1.0;
  if (m > 1 && bq > 1024) {
    const double target = static_cast<double>(bq) / 1024.0 * m;
    double lo = 1.0, hi = target;                          // 1 + rho <= sum, so the root is below beta m
    for (int it = 0; it < 200; ++it) {
      const double mid = 0.5 * (lo + hi);
      double sum = 0.0, pw = 1.0;
      for (int j = 0; j < m; ++j) { sum += pw; pw *= mid; }
      if (sum < target) lo = mid; else hi = mid;
    }
    rho = std::round(0.5 * (lo + hi) * 1048576.0) / 1048576.0;
  }
  std::vector<double> power(m);
  double total = 0.0;
  for (int j = 0; j < m; ++j) {
    power[j] = j == 0 ? 1.0 : power[j - 1] * rho;
    total += power[j];
  }
  int64_t assigned = 0;
  for (int l = 0; l < m; ++l) {
    const int64_t kl = static_cast<int64_t>(std::floor(static_cast<double>(k_total) * power[m - 1 - l] / total));
    k_out[l] = static_cast<int32_t>(kl);
    assigned += kl;
  }
  int64_t left = k_total - assigned;
  for (int l = 0; l < m && left > 0; ++l, --left) k_out[l] += 1;
  return 0;
}

// Number of rows kept for a sequence of n tokens in a layer with budget k_layer.
// A context that fits the average budget is not compressed at all.
int orc_kept_count(int avg_budget, int alpha, int k_layer, int n) {
  if (n <= avg_budget) return n;
  const int prefix = n - alpha;
  return std::min(k_layer, prefix) + alpha;
}

// ---------------------------------------------------------------------------
// Section 4.2.2, Eq. 2 and Eq. 3, one sequence.
//   q   [H_q][alpha][d]   window queries (the last alpha positions), contiguous
//   k   [H_kv][n][d]      keys, contiguous
//   dtype 0 = float, 1 = bfloat16 bit patterns, 2 = binary16 bit patterns
// Window row j sits at absolute position P + j (P = n - alpha) and, the model
// being autoregressive, sees keys 0 .. P + j.  Each row is a softmax over what
// it sees.  The score of prefix key i < P is the sum over the alpha rows of
// A[j][i]; with several query heads per KV head the group's scores are averaged.
//   scores      [H_kv][P]   float, rounded once from double
//   window_mass [H_kv]      double, may be null: the same sum taken over the
//                           window columns i >= P, so that for every head
//                           sum_i scores + window_mass = alpha.
//   row_lse     [H_q][alpha] double, may be null: log of each row's softmax denominator,
//                           log sum_{i <= P+j} exp(logit[i]) (what a prefill attention kernel keeps).
void orc_window_scores_lse(const void* q, const void* k, int dtype, int num_q_heads, int num_kv_heads,
                           int d, int alpha, int n, float* scores, double* window_mass, double* row_lse) {
  const int group = num_q_heads / num_kv_heads;
  const int P = n - alpha;
  const double scale = 1.0 / std::sqrt(static_cast<double>(d));
  for (int h = 0; h < num_kv_heads; ++h) {
    // Keys of this head, widened once.
    std::vector<double> kd(static_cast<size_t>(n) * d);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < static_cast<int64_t>(n) * d; ++t)
      kd[t] = elem(k, dtype, static_cast<int64_t>(h) * n * d + t);

    std::vector<double> acc(n, 0.0);                       // sum over rows of A[row][i]
    std::vector<double> logit(n);
    std::vector<double> qd(d);
    for (int g = 0; g < group; ++g) {
      const int hq = h * group + g;
      for (int j = 0; j < alpha; ++j) {
        for (int c = 0; c < d; ++c)
          qd[c] = elem(q, dtype, (static_cast<int64_t>(hq) * alpha + j) * d + c);
        const int visible = P + j + 1;                     // keys 0 .. P + j
        // Eq. 2: logits of this row.
#pragma omp parallel for schedule(static)
        for (int i = 0; i < visible; ++i) {
          const double* kr = &kd[static_cast<size_t>(i) * d];
          double dot = 0.0;
          for (int c = 0; c < d; ++c) dot += qd[c] * kr[c];
          logit[i] = dot * scale;
        }
        // Row softmax over the visible keys.
        double mx = -std::numeric_limits<double>::infinity();
        for (int i = 0; i < visible; ++i) mx = std::max(mx, logit[i]);
#pragma omp parallel for schedule(static)
        for (int i = 0; i < visible; ++i) logit[i] = std::exp(logit[i] - mx);
        double z = 0.0;
        for (int i = 0; i < visible; ++i) z += logit[i];
        if (row_lse) row_lse[static_cast<int64_t>(hq) * alpha + j] = mx + std::log(z);
        // Eq. 3: add this row's attention to every key it sees.
#pragma omp parallel for schedule(static)
        for (int i = 0; i < visible; ++i) acc[i] += logit[i] / z;
      }
    }
    const double inv_group = 1.0 / static_cast<double>(group);
    for (int i = 0; i < P; ++i)
      scores[static_cast<int64_t>(h) * P + i] = static_cast<float>(acc[i] * inv_group);
    if (window_mass) {
      double wm = 0.0;
      for (int i = P; i < n; ++i) wm += acc[i];
      window_mass[h] = wm * inv_group;
    }
  }
}

void orc_window_scores(const void* q, const void* k, int dtype, int num_q_heads, int num_kv_heads,
                       int d, int alpha, int n, float* scores, double* window_mass) {
  orc_window_scores_lse(q, k, dtype, num_q_heads, num_kv_heads, d, alpha, n, scores, window_mass, nullptr);
}

// ---------------------------------------------------------------------------
// Section 4.2.2: the pooling layer.  Centred max of odd width w, stride 1,
// clipped to [0, P): out[i] = max over |t| <= (w-1)/2 with 0 <= i+t < P of in[i+t].
int orc_pool_max(const float* in, int P, int w, float* out) {
  if (w < 1 || (w % 2) == 0) return -1;
  const int r = (w - 1) / 2;
  for (int i = 0; i < P; ++i) {
    float best = in[i];
    for (int t = -r; t <= r; ++t) {
      const int x = i + t;
      if (x >= 0 && x < P) best = std::max(best, in[x]);
    }
    out[i] = best;
  }
  return 0;
}

// The same layer as a mean (the variant the section's "pooling layer" also admits): centred window of odd
// width w, stride 1, positions outside [0, P) count as zeros, the sum is always divided by w.  The result
// decides a top-k, so its precision is part of the definition: float additions from the left-most
// window position to the right-most, then one float division by w.
int orc_pool_avg(const float* in, int P, int w, float* out) {
  if (w < 1 || (w % 2) == 0) return -1;
  const int r = (w - 1) / 2;
  for (int i = 0; i < P; ++i) {
    float sum = 0.0f;
    for (int t = -r; t <= r; ++t) {
      const int x = i + t;
      if (x >= 0 && x < P) sum = sum + in[x];
    }
    out[i] = sum / static_cast<float>(w);
  }
  return 0;
}

// ---------------------------------------------------------------------------
// Section 4.2.2: keep the k highest-scored prefix positions.  Order all P
// positions by (value descending, position ascending), keep the first
// min(k, P), and list them in ascending position.  Returns how many were kept.
int orc_select_topk(const float* pooled, int P, int k, int32_t* idx_out) {
  const int keep = std::max(0, std::min(k, P));
  std::vector<int32_t> order(P);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(),
                   [&](int32_t a, int32_t b) { return pooled[a] > pooled[b]; });
  std::vector<int32_t> kept(order.begin(), order.begin() + keep);
  std::sort(kept.begin(), kept.end());
  std::copy(kept.begin(), kept.end(), idx_out);
  return keep;
}

// ---------------------------------------------------------------------------
// One layer, one sequence: scores -> pool -> top-k per KV head -> window rows
// appended -> rows of K and V copied out.
//   k_layer     budget k^l of this layer (prefix rows to keep)
//   kept        out [H_kv][c]  kept positions, ascending, c = orc_kept_count(...)
//   k_out,v_out out [H_kv][c][d] in the input dtype (bit copies), may be null
//   scores_out  out [H_kv][P] float, may be null
// Returns c.
int orc_compress_layer(const void* q, const void* k, const void* v, int dtype, int num_q_heads,
                       int num_kv_heads, int d, int alpha, int pool_w, int pool_kind, int avg_budget, int k_layer,
                       int n, int32_t* kept, void* k_out, void* v_out, float* scores_out) {
  const int P = n - alpha;
  const int c = orc_kept_count(avg_budget, alpha, k_layer, n);
  const size_t esz = dtype == 0 ? 4 : 2;
  std::vector<float> scores(static_cast<size_t>(num_kv_heads) * P);
  const bool keep_all = n <= avg_budget;
  if (!keep_all || scores_out)
    orc_window_scores(q, k, dtype, num_q_heads, num_kv_heads, d, alpha, n, scores.data(), nullptr);
  if (scores_out) std::copy(scores.begin(), scores.end(), scores_out);
  std::vector<float> pooled(P);
  for (int h = 0; h < num_kv_heads; ++h) {
    int32_t* row = kept + static_cast<int64_t>(h) * c;
    int cnt = 0;
    if (keep_all) {
      for (int i = 0; i < P; ++i) row[cnt++] = i;
    } else {
      if (pool_kind == 1) orc_pool_avg(scores.data() + static_cast<int64_t>(h) * P, P, pool_w, pooled.data());
      else orc_pool_max(scores.data() + static_cast<int64_t>(h) * P, P, pool_w, pooled.data());
      cnt = orc_select_topk(pooled.data(), P, k_layer, row);
    }
    for (int i = P; i < n; ++i) row[cnt++] = i;             // instruction tokens, always kept
    for (int r = 0; r < c && (k_out || v_out); ++r) {
      const size_t src = (static_cast<size_t>(h) * n + row[r]) * d * esz;
      const size_t dst = (static_cast<size_t>(h) * c + r) * d * esz;
      if (k_out) std::memcpy(static_cast<char*>(k_out) + dst, static_cast<const char*>(k) + src, d * esz);
      if (v_out) std::memcpy(static_cast<char*>(v_out) + dst, static_cast<const char*>(v) + src, d * esz);
    }
  }
  return c;
}

// ---------------------------------------------------------------------------
// Softmax attention of the window queries over a set of cached rows (used to
// check that a cache that keeps everything reproduces full attention).
//   pos [c] original positions of the cached rows of one KV head;
//   kc, vc [c][d] the cached rows; q [alpha][d] one query head's window rows.
//   out [alpha][d] double.  Row j attends to cached rows with pos <= P + j.
void orc_window_attention(const void* q, const void* kc, const void* vc, const int32_t* pos,
                          int dtype, int d, int alpha, int n, int c, double* out) {
  const int P = n - alpha;
  const double scale = 1.0 / std::sqrt(static_cast<double>(d));
  std::vector<double> w(c);
  for (int j = 0; j < alpha; ++j) {
    double mx = -std::numeric_limits<double>::infinity();
    for (int r = 0; r < c; ++r) {
      if (pos[r] > P + j) { w[r] = -std::numeric_limits<double>::infinity(); continue; }
      double dot = 0.0;
      for (int t = 0; t < d; ++t)
        dot += elem(q, dtype, static_cast<int64_t>(j) * d + t) * elem(kc, dtype, static_cast<int64_t>(r) * d + t);
      w[r] = dot * scale;
      mx = std::max(mx, w[r]);
    }
    double z = 0.0;
    for (int r = 0; r < c; ++r) { w[r] = std::exp(w[r] - mx); z += w[r]; }
    for (int t = 0; t < d; ++t) {
      double o = 0.0;
      for (int r = 0; r < c; ++r) o += (w[r] / z) * elem(vc, dtype, static_cast<int64_t>(r) * d + t);
      out[static_cast<int64_t>(j) * d + t] = o;
    }
  }
}

// ---------------------------------------------------------------------------
// Section 4.1: inference after compression uses only the kept rows.  One new token's query attends to
// every cached row of its KV head (no mask: all of them precede it).
//   q [d]; kc, vc [c][d]; out [d] double.
void orc_decode_attention(const void* q, const void* kc, const void* vc, int dtype, int d, int c, double* out) {
  const double scale = 1.0 / std::sqrt(static_cast<double>(d));
  std::vector<double> w(c);
  double mx = -std::numeric_limits<double>::infinity();
  for (int r = 0; r < c; ++r) {
    double dot = 0.0;
    for (int t = 0; t < d; ++t) dot += elem(q, dtype, t) * elem(kc, dtype, static_cast<int64_t>(r) * d + t);
    w[r] = dot * scale;
    mx = std::max(mx, w[r]);
  }
  double z = 0.0;
  for (int r = 0; r < c; ++r) { w[r] = std::exp(w[r] - mx); z += w[r]; }
  for (int t = 0; t < d; ++t) {
    double o = 0.0;
    for (int r = 0; r < c; ++r) o += (w[r] / z) * elem(vc, dtype, static_cast<int64_t>(r) * d + t);
    out[t] = o;
  }
}

// Appendix on the attention recall rate: share of the window rows' attention that lands on kept keys,
// averaged over the alpha rows and the group's query heads.  scores [P] are the Eq. 3 scores of one KV
// head (they already hold the group mean of the row sums), kept [c] its kept positions (window included).
double orc_attention_recall(const float* scores, int P, int alpha, const int32_t* kept, int c) {
  double all = 0.0, on_kept = 0.0;
  for (int i = 0; i < P; ++i) all += scores[i];
  for (int r = 0; r < c; ++r)
    if (kept[r] < P) on_kept += scores[kept[r]];
  const double window_mass = alpha - all;                 // every row's attention sums to one
  return (on_kept + window_mass) / alpha;
}

// ---------------------------------------------------------------------------
// Appendix on paged attention: a per-layer block table per sequence, so that each layer's cache lives in
// pages of its own and can be found "without the use of fixed memory offsets".  Layout used here: a pool
// of pages, each holding page_size rows of one KV head; row r of a head's kept list sits in the page
// table[r / page_size] at slot r % page_size.
int orc_pages_needed(int avg_budget, int alpha, int k_layer, int n, int page_size) {
  if (page_size < 1) return -1;
  const int c = orc_kept_count(avg_budget, alpha, k_layer, n);
  return (c + page_size - 1) / page_size;
}

// rows [c][row_bytes] of one head -> pool [num_pages][page_size][row_bytes] through table [ceil(c/page_size)].
// Returns 0, or -1 when a table entry names a page outside the pool (nothing is written then).
int orc_scatter_paged(const void* rows, int c, int row_bytes, int page_size, const int32_t* table, int num_pages,
                      void* pool) {
  const int pages = (c + page_size - 1) / page_size;
  for (int j = 0; j < pages; ++j)
    if (table[j] < 0 || table[j] >= num_pages) return -1;
  for (int r = 0; r < c; ++r) {
    const size_t dst = (static_cast<size_t>(table[r / page_size]) * page_size + (r % page_size)) * row_bytes;
    std::memcpy(static_cast<char*>(pool) + dst, static_cast<const char*>(rows) + static_cast<size_t>(r) * row_bytes,
                row_bytes);
  }
  return 0;
}

// The inverse walk: the c rows of one head, in list order, read back through its table.
int orc_read_paged(const void* pool, int c, int row_bytes, int page_size, const int32_t* table, int num_pages,
                   void* rows) {
  const int pages = (c + page_size - 1) / page_size;
  for (int j = 0; j < pages; ++j)
    if (table[j] < 0 || table[j] >= num_pages) return -1;
  for (int r = 0; r < c; ++r) {
    const size_t src = (static_cast<size_t>(table[r / page_size]) * page_size + (r % page_size)) * row_bytes;
    std::memcpy(static_cast<char*>(rows) + static_cast<size_t>(r) * row_bytes, static_cast<const char*>(pool) + src,
                row_bytes);
  }
  return 0;
}

int orc_num_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"
