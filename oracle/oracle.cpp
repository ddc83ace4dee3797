// CPU oracle for the batched verification step of speculative decoding.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of what the
// verification step computes.  It is independent of the CUDA path: it shares no header, helper,
// table or constant with it, and nothing in the product path may call it.  Only the test-suite,
// the smoke check and the CPU-baseline leg of the benchmark load this library.
//
// What it follows.  The paper (Sec. 2.2 "Speculative Decoding", Sec. 3 "Overall Efficiency
// Analysis", Sec. 4.2 Eq. 3 / Algorithm 2) fixes only the problem: a lossless draft-then-verify
// step in which every request i of a batch proposes its own number k_i of draft tokens (a single
// chain, the most frequent continuation prefix) and the target model verifies them in one pass.
// It leaves every numeric detail of verification open.  The readings taken here are:
//
//   * request i has n_i committed cache entries (positions 0..n_i-1).  The step feeds k_i+1
//     tokens: the last emitted token (row 0, position n_i) and the k_i drafts (rows 1..k_i,
//     positions n_i+1..n_i+k_i).  Row j attends to positions lo..n_i+j, itself included, with
//     lo = 0, or max(0, n_i+j-W+1) for a sliding window of W visible keys.
//   * scores are sm_scale * <q, k>; q-head h reads kv-head h / (Hq/Hkv); an optional per-head
//     "sink" logit joins the softmax denominator and contributes no value.
//   * logit row j of request i judges draft j+1.  Greedy: the draft must equal the lowest-index
//     maximum of the row (NaN counts as -inf).  Sampled: accept iff u < min(1, p[d]/q[d]) with
//     p = softmax(z/T); on the first rejection the extra token is drawn from norm(max(0, p-q)) by
//     inverse CDF with one uniform; if all drafts pass it is drawn from p of the last row.
//   * commit: the new length is n_i + a_i + 1; pages wholly past it are released in
//     (request, logical page) order; rejected slots in pages still held may be scrubbed to zero.
//
// Arithmetic is fp64 throughout with one plain loop nest per quantity: no tiling, no online
// softmax, no reordering.  bf16 / fp32 inputs are widened exactly at the edge.
//
// Parity pins (tests that tie each function to something other than itself):
//   ov_attn*            brute-force dense masked softmax, hand-worked 2-d example with ln 2 / ln 3
//                       queries, uniform-softmax closed form, needle keys, k=0 == single-query decode
//   ov_accept*          hand-worked greedy and sampled examples, losslessness identity by
//                       enumeration, Monte-Carlo marginal, T -> 0 limit, greedy == autoregressive loop
//   ov_kv_commit        hand-worked paging example, poison test, speculative loop == sequential loop
//   ov_merge_partials   equals the unsplit softmax for random chunkings
//   ov_philox*          the generator's published known-answer vectors, range and grid of the floats,
//                       chi-square and serial-correlation checks, distinct streams per (seed, step, request)
//   ov_budget           hand-worked four-request example, p(1) = g_min and saturation, equal-score split,
//                       50-digit decimal re-evaluation on random batches, budget and floor invariants
//   ov_lm_head          numpy's float64 matrix product on random inputs, a hand-worked 2 x 3 example, rows of
//                       one-hot hidden states that must return the corresponding weight column exactly
// Parity unpinned: the bytes left in rolled-back slots when scrubbing is off (declared unspecified).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

inline double widen(uint16_t bf16_bits) {
  uint32_t u = static_cast<uint32_t>(bf16_bits) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return static_cast<double>(f);
}
inline double widen(double x) { return x; }

// Runs fn(item) for item in [0, n) on `threads` host threads (static interleave).
template <class F>
void parallel_for(int64_t n, int threads, F fn) {
  if (threads <= 1 || n <= 1) {
    for (int64_t i = 0; i < n; ++i) fn(i);
    return;
  }
  std::vector<std::thread> pool;
  int t_used = static_cast<int>(std::min<int64_t>(threads, n));
  for (int t = 0; t < t_used; ++t)
    pool.emplace_back([=]() {
      for (int64_t i = t; i < n; i += t_used) fn(i);
    });
  for (auto& th : pool) th.join();
}

struct Shape {
  int B, Hq, Hkv, D, bs, max_blocks, window;
  double sm_scale;
};

// Address of the D-vector of logical key t of request i, kv-head g.  Committed positions come
// from the paged pool through the block table, positions >= n_i from the staging rows.
template <class E>
const E* key_ptr(const Shape& s, int i, int g, int t, int n_i, int64_t row0, const E* pool,
                 const E* fresh, const int32_t* block_table) {
  if (t < n_i) {
    int64_t blk = block_table[static_cast<int64_t>(i) * s.max_blocks + t / s.bs];
    return pool + ((blk * s.Hkv + g) * s.bs + (t % s.bs)) * static_cast<int64_t>(s.D);
  }
  return fresh + ((row0 + (t - n_i)) * s.Hkv + g) * static_cast<int64_t>(s.D);
}

template <class E>
void attn_one(const Shape& s, const double* sinks, const int32_t* seq_lens, const int64_t* cu_q,
              int i, int h, const E* q, const E* k_new, const E* v_new, const E* k_pool,
              const E* v_pool, const int32_t* block_table, int k_i, double* out, double* lse) {
  const int G = s.Hq / s.Hkv;
  const int g = h / G;
  const int n_i = seq_lens[i];
  const int64_t row0 = cu_q[i];
  std::vector<double> sc;
  for (int j = 0; j <= k_i; ++j) {
    const int p = n_i + j;
    const int lo = s.window > 0 ? std::max(0, p - s.window + 1) : 0;
    const E* qv = q + ((row0 + j) * s.Hq + h) * static_cast<int64_t>(s.D);
    sc.assign(p - lo + 1, 0.0);
    double m = -std::numeric_limits<double>::infinity();
    for (int t = lo; t <= p; ++t) {
      const E* kv = key_ptr(s, i, g, t, n_i, row0, k_pool, k_new, block_table);
      double dot = 0.0;
      for (int d = 0; d < s.D; ++d) dot += widen(qv[d]) * widen(kv[d]);
      sc[t - lo] = s.sm_scale * dot;
      m = std::max(m, sc[t - lo]);
    }
    if (sinks) m = std::max(m, sinks[h]);
    double den = 0.0;
    for (int t = lo; t <= p; ++t) den += std::exp(sc[t - lo] - m);
    if (sinks) den += std::exp(sinks[h] - m);
    double* o = out + ((row0 + j) * s.Hq + h) * static_cast<int64_t>(s.D);
    for (int d = 0; d < s.D; ++d) o[d] = 0.0;
    for (int t = lo; t <= p; ++t) {
      const E* vv = key_ptr(s, i, g, t, n_i, row0, v_pool, v_new, block_table);
      const double wgt = std::exp(sc[t - lo] - m);
      for (int d = 0; d < s.D; ++d) o[d] += wgt * widen(vv[d]);
    }
    for (int d = 0; d < s.D; ++d) o[d] /= den;
    if (lse) lse[(row0 + j) * s.Hq + h] = m + std::log(den);
  }
}

template <class E>
int attn_all(int B, int Hq, int Hkv, int D, int bs, int max_blocks, int window, double sm_scale,
             const double* sinks, const int32_t* seq_lens, const int32_t* draft_lens, const E* q,
             const E* k_new, const E* v_new, const E* k_pool, const E* v_pool,
             const int32_t* block_table, int n_sel, const int32_t* sel, double* out, double* lse,
             int threads) {
  if (B < 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || D <= 0 || bs <= 0) return 1;
  Shape s{B, Hq, Hkv, D, bs, max_blocks, window, sm_scale > 0 ? sm_scale : 1.0 / std::sqrt(double(D))};
  std::vector<int64_t> cu_q(B + 1, 0);
  for (int i = 0; i < B; ++i) cu_q[i + 1] = cu_q[i] + draft_lens[i] + 1;
  const int64_t items = sel ? n_sel : static_cast<int64_t>(B) * Hq;
  parallel_for(items, threads, [&](int64_t it) {
    int i = sel ? sel[2 * it] : static_cast<int>(it / Hq);
    int h = sel ? sel[2 * it + 1] : static_cast<int>(it % Hq);
    attn_one<E>(s, sinks, seq_lens, cu_q.data(), i, h, q, k_new, v_new, k_pool, v_pool, block_table,
                draft_lens[i], out, lse);
  });
  return 0;
}

// Lowest index of the maximum; NaN compares as -inf; an all-NaN / all -inf row gives 0.
int argmax_row(const float* z, int V) {
  int best = 0;
  double bv = -std::numeric_limits<double>::infinity();
  for (int v = 0; v < V; ++v) {
    double x = static_cast<double>(z[v]);
    if (x != x) continue;
    if (x > bv) {
      bv = x;
      best = v;
    }
  }
  return best;
}

void softmax_row(const float* z, int V, double T, std::vector<double>& p) {
  p.resize(V);
  double m = -std::numeric_limits<double>::infinity();
  for (int v = 0; v < V; ++v) m = std::max(m, static_cast<double>(z[v]) / T);
  double den = 0.0;
  for (int v = 0; v < V; ++v) {
    p[v] = std::exp(static_cast<double>(z[v]) / T - m);
    den += p[v];
  }
  for (int v = 0; v < V; ++v) p[v] /= den;
}

// Acceptance probability min(1, p/q) of one draft token under the strict test u < ratio.
double accept_ratio(double p_d, double q_d) {
  if (p_d <= 0.0) return 0.0;           // zero target mass: always reject
  if (q_d <= 0.0) return 1.0;           // drafter claims zero mass but target has some: accept
  return std::min(1.0, p_d / q_d);
}

// Unnormalised recovery weights: max(0, p-q) after a rejection, p itself after a full accept;
// if the residual is identically zero the row falls back to p.
void recovery_weights(const std::vector<double>& p, const double* q_row, int onehot_at, bool bonus,
                      std::vector<double>& r) {
  const int V = static_cast<int>(p.size());
  r.resize(V);
  if (bonus) {
    r = p;
    return;
  }
  double tot = 0.0;
  for (int v = 0; v < V; ++v) {
    double qv = q_row ? q_row[v] : (v == onehot_at ? 1.0 : 0.0);
    r[v] = std::max(0.0, p[v] - qv);
    tot += r[v];
  }
  if (!(tot > 0.0)) r = p;
}

// Inverse CDF with strict '>' so that zero-mass tokens are never chosen; if rounding leaves no
// index the largest index with positive mass is returned.
int inverse_cdf(const std::vector<double>& r, double w) {
  const int V = static_cast<int>(r.size());
  double S = 0.0;
  for (int v = 0; v < V; ++v) S += r[v];
  const double target = w * S;
  double c = 0.0;
  int last_pos = 0;
  for (int v = 0; v < V; ++v) {
    c += r[v];
    if (r[v] > 0.0) last_pos = v;
    if (c > target && r[v] > 0.0) return v;
  }
  return last_pos;
}

}  // namespace

extern "C" {

int ov_hardware_threads() {
  unsigned n = std::thread::hardware_concurrency();
  return n ? static_cast<int>(n) : 1;
}

// Verify attention, bf16 inputs (raw 16-bit patterns).  Layouts:
//   q [total_q, Hq, D]; k_new, v_new [total_q, Hkv, D]; pools [num_blocks, Hkv, bs, D];
//   block_table [B, max_blocks]; out fp64 [total_q, Hq, D]; lse fp64 [total_q, Hq] or NULL.
// sel: optional list of n_sel (request, q_head) pairs to compute; NULL computes everything.
// sm_scale <= 0 selects 1/sqrt(D).  window = 0 means full attention.
int ov_attn_bf16(int B, int Hq, int Hkv, int D, int bs, int max_blocks, int window, double sm_scale,
                 const double* sinks, const int32_t* seq_lens, const int32_t* draft_lens,
                 const uint16_t* q, const uint16_t* k_new, const uint16_t* v_new,
                 const uint16_t* k_pool, const uint16_t* v_pool, const int32_t* block_table,
                 int n_sel, const int32_t* sel, double* out, double* lse, int threads) {
  return attn_all<uint16_t>(B, Hq, Hkv, D, bs, max_blocks, window, sm_scale, sinks, seq_lens,
                            draft_lens, q, k_new, v_new, k_pool, v_pool, block_table, n_sel, sel,
                            out, lse, threads);
}

// Same computation on fp64 inputs, so that hand-worked examples with irrational entries can be
// fed without rounding.
int ov_attn_f64(int B, int Hq, int Hkv, int D, int bs, int max_blocks, int window, double sm_scale,
                const double* sinks, const int32_t* seq_lens, const int32_t* draft_lens,
                const double* q, const double* k_new, const double* v_new, const double* k_pool,
                const double* v_pool, const int32_t* block_table, int n_sel, const int32_t* sel,
                double* out, double* lse, int threads) {
  return attn_all<double>(B, Hq, Hkv, D, bs, max_blocks, window, sm_scale, sinks, seq_lens,
                          draft_lens, q, k_new, v_new, k_pool, v_pool, block_table, n_sel, sel, out,
                          lse, threads);
}

// Plain single-query decode over n+1 keys (the n cached ones and the token's own), written
// separately from attn_one so that "k = 0 reduces to decode" compares two pieces of code.
// k_ctx, v_ctx: [n+1, D] fp64, already gathered in logical order.
int ov_decode_f64(int n_plus_1, int D, double sm_scale, const double* qv, const double* k_ctx,
                  const double* v_ctx, double* out, double* lse) {
  std::vector<double> e(n_plus_1);
  double m = -std::numeric_limits<double>::infinity();
  for (int t = 0; t < n_plus_1; ++t) {
    double dot = 0.0;
    for (int d = 0; d < D; ++d) dot += qv[d] * k_ctx[static_cast<int64_t>(t) * D + d];
    e[t] = sm_scale * dot;
    m = std::max(m, e[t]);
  }
  double den = 0.0;
  for (int t = 0; t < n_plus_1; ++t) {
    e[t] = std::exp(e[t] - m);
    den += e[t];
  }
  for (int d = 0; d < D; ++d) {
    double acc = 0.0;
    for (int t = 0; t < n_plus_1; ++t) acc += e[t] * v_ctx[static_cast<int64_t>(t) * D + d];
    out[d] = acc / den;
  }
  if (lse) *lse = m + std::log(den);
  return 0;
}

// Merge of per-chunk softmax partials (m_s, l_s, O_s), O_s unnormalised: the identity a split-KV
// kernel relies on.  parts_o [S, D], parts_m [S], parts_l [S]; sink may be NaN for "none".
int ov_merge_partials(int S, int D, const double* parts_m, const double* parts_l,
                      const double* parts_o, double sink, double* out, double* lse) {
  double m = -std::numeric_limits<double>::infinity();
  for (int s = 0; s < S; ++s) m = std::max(m, parts_m[s]);
  const bool has_sink = sink == sink;
  if (has_sink) m = std::max(m, sink);
  double den = 0.0;
  for (int s = 0; s < S; ++s) den += std::exp(parts_m[s] - m) * parts_l[s];
  if (has_sink) den += std::exp(sink - m);
  for (int d = 0; d < D; ++d) {
    double acc = 0.0;
    for (int s = 0; s < S; ++s) acc += std::exp(parts_m[s] - m) * parts_o[static_cast<int64_t>(s) * D + d];
    out[d] = acc / den;
  }
  if (lse) *lse = m + std::log(den);
  return 0;
}

// Acceptance on probability rows given directly in fp64 (T already applied): one request.
//   p [k+1, V]; q [k, V] or NULL (one-hot drafter); drafts [k]; u [k]; w [k+1].
//   force_accept >= 0 overrides the accept/reject decisions with that accepted length.
// Outputs: *accept_len, out_tokens[k+1] (-1 padded), ratios[k] (NaN where not evaluated).
int ov_accept_probs_f64(int k, int V, const double* p, const double* q, const int32_t* drafts,
                        const double* u, const double* w, int force_accept, int32_t* accept_len,
                        int32_t* out_tokens, double* ratios) {
  for (int j = 0; j <= k; ++j) out_tokens[j] = -1;
  for (int j = 0; j < k; ++j) ratios[j] = std::numeric_limits<double>::quiet_NaN();
  int a = 0;
  for (int j = 0; j < k; ++j) {
    const int d = drafts[j];
    double ratio = 0.0;
    if (d >= 0 && d < V) {
      const double pd = p[static_cast<int64_t>(j) * V + d];
      const double qd = q ? q[static_cast<int64_t>(j) * V + d] : 1.0;
      ratio = accept_ratio(pd, qd);
    }
    ratios[j] = ratio;
    const bool ok = force_accept >= 0 ? (j < force_accept) : (u[j] < ratio);
    if (!ok) break;
    out_tokens[a++] = d;
  }
  std::vector<double> prow(p + static_cast<int64_t>(a) * V, p + static_cast<int64_t>(a + 1) * V), r;
  const bool bonus = (a == k);
  recovery_weights(prow, (q && !bonus) ? q + static_cast<int64_t>(a) * V : nullptr,
                   bonus ? -1 : drafts[a], bonus, r);
  out_tokens[a] = inverse_cdf(r, w[a]);
  *accept_len = a;
  return 0;
}

// Batched acceptance on fp32 logits.
//   logits [total_q, ld]; draft_tokens [total_d]; draft_probs [total_d, ld] or NULL (one-hot);
//   temperature [B] or NULL (greedy); T_i <= 0 is greedy for that request;
//   u [total_d] (request i, draft j at cu_d[i]+j); w [total_q] (request i, row j at cu_q[i]+j);
//   force_accept [B] or NULL: entries >= 0 force that request's accepted length (sampled only).
// Outputs: accept_len [B]; out_tokens [B, k_max+1] (-1 padded); ratios [total_d] or NULL (NaN where
// the position was not reached or the request is greedy); target_argmax [total_q] or NULL.
int ov_accept(int B, int k_max, const int32_t* draft_lens, const float* logits, int64_t ld, int V,
              const int32_t* draft_tokens, const float* draft_probs, const float* temperature,
              const float* u, const float* w, const int32_t* force_accept, int32_t* accept_len,
              int32_t* out_tokens, double* ratios, int32_t* target_argmax, int threads) {
  std::vector<int64_t> cu_q(B + 1, 0), cu_d(B + 1, 0);
  for (int i = 0; i < B; ++i) {
    if (draft_lens[i] < 0 || draft_lens[i] > k_max) return 1;
    cu_q[i + 1] = cu_q[i] + draft_lens[i] + 1;
    cu_d[i + 1] = cu_d[i] + draft_lens[i];
  }
  if (ratios)
    for (int64_t x = 0; x < cu_d[B]; ++x) ratios[x] = std::numeric_limits<double>::quiet_NaN();
  if (target_argmax)
    parallel_for(cu_q[B], threads, [&](int64_t r) { target_argmax[r] = argmax_row(logits + r * ld, V); });
  parallel_for(B, threads, [&](int64_t i) {
    const int k = draft_lens[i];
    int32_t* outs = out_tokens + i * (k_max + 1);
    for (int j = 0; j <= k_max; ++j) outs[j] = -1;
    const double T = temperature ? static_cast<double>(temperature[i]) : 0.0;
    const int32_t* dr = draft_tokens + cu_d[i];
    int a = 0;
    if (!(T > 0.0)) {
      for (int j = 0; j < k; ++j) {
        if (argmax_row(logits + (cu_q[i] + j) * ld, V) != dr[j]) break;
        outs[a++] = dr[j];
      }
      outs[a] = argmax_row(logits + (cu_q[i] + a) * ld, V);
      accept_len[i] = a;
      return;
    }
    std::vector<double> p, r;
    const int forced = force_accept ? force_accept[i] : -1;
    for (int j = 0; j < k; ++j) {
      const int d = dr[j];
      double ratio = 0.0;
      if (d >= 0 && d < V) {
        softmax_row(logits + (cu_q[i] + j) * ld, V, T, p);
        const double qd = draft_probs ? static_cast<double>(draft_probs[(cu_d[i] + j) * ld + d]) : 1.0;
        ratio = accept_ratio(p[d], qd);
      }
      if (ratios) ratios[cu_d[i] + j] = ratio;
      const bool ok = forced >= 0 ? (j < forced) : (static_cast<double>(u[cu_d[i] + j]) < ratio);
      if (!ok) break;
      outs[a++] = d;
    }
    softmax_row(logits + (cu_q[i] + a) * ld, V, T, p);
    const bool bonus = (a == k);
    std::vector<double> qrow;
    if (!bonus && draft_probs) {
      qrow.resize(V);
      for (int v = 0; v < V; ++v) qrow[v] = static_cast<double>(draft_probs[(cu_d[i] + a) * ld + v]);
    }
    recovery_weights(p, qrow.empty() ? nullptr : qrow.data(), bonus ? -1 : dr[a], bonus, r);
    outs[a] = inverse_cdf(r, static_cast<double>(w[cu_q[i] + a]));
    accept_len[i] = a;
  });
  return 0;
}

// For one request with accepted length a: the recovery CDF around token v, C[v-1], C[v] and the
// total S, plus the weight r[v]; used to judge an extra token chosen in lower precision.
int ov_recovery_interval(int k, int a, const float* logits_row, int V, const float* draft_prob_row,
                         int draft_token, double T, int v, double* c_lo, double* c_hi, double* total,
                         double* r_v) {
  if (v < 0 || v >= V) return 1;
  std::vector<double> p, r, qrow;
  softmax_row(logits_row, V, T, p);
  const bool bonus = (a == k);
  if (!bonus && draft_prob_row) {
    qrow.resize(V);
    for (int x = 0; x < V; ++x) qrow[x] = static_cast<double>(draft_prob_row[x]);
  }
  recovery_weights(p, qrow.empty() ? nullptr : qrow.data(), bonus ? -1 : draft_token, bonus, r);
  double c = 0.0, lo = 0.0, hi = 0.0;
  for (int x = 0; x < V; ++x) {
    if (x == v) lo = c;
    c += r[x];
    if (x == v) hi = c;
  }
  *c_lo = lo;
  *c_hi = hi;
  *total = c;
  *r_v = r[v];
  return 0;
}

// Commit accepted rows and roll back the rest.  bf16 pools (raw 16-bit patterns), updated in place.
//   The first a_i+1 staging rows of request i are stored at positions n_i..n_i+a_i;
//   seq_lens[i] becomes n_i + a_i + 1; every page the step held for positions n_i'..n_i+k_i beyond the
//   last kept page (logical index in [ceil(n_i'/bs), ceil((n_i+k_i+1)/bs)), entry != -1) is released:
//   its id is appended to freed[] and its entry set to -1, scanning requests in ascending order and
//   logical pages in ascending order.  Table entries past the step's positions are not looked at.  With scrub != 0, slots of
//   positions n_i'..n_i+k_i that lie in pages still held are zeroed.
int ov_kv_commit(int B, int Hkv, int D, int bs, int max_blocks, int32_t* seq_lens,
                 const int32_t* draft_lens, const int32_t* accept_len, int32_t* block_table,
                 const uint16_t* k_new, const uint16_t* v_new, uint16_t* k_pool, uint16_t* v_pool,
                 int32_t* freed, int32_t* freed_count, int scrub) {
  int64_t row0 = 0;
  int nf = 0;
  for (int i = 0; i < B; ++i) {
    const int n = seq_lens[i], k = draft_lens[i], a = accept_len[i];
    if (a < 0 || a > k) return 1;
    int32_t* bt = block_table + static_cast<int64_t>(i) * max_blocks;
    for (int j = 0; j <= k; ++j) {
      const int t = n + j;
      const int32_t blk = bt[t / bs];
      if (blk < 0) return 2;
      for (int g = 0; g < Hkv; ++g) {
        const int64_t dst = ((static_cast<int64_t>(blk) * Hkv + g) * bs + (t % bs)) * D;
        const int64_t src = ((row0 + j) * Hkv + g) * D;
        for (int d = 0; d < D; ++d) {
          if (j <= a) {
            k_pool[dst + d] = k_new[src + d];
            v_pool[dst + d] = v_new[src + d];
          } else if (scrub) {
            k_pool[dst + d] = 0;
            v_pool[dst + d] = 0;
          }
        }
      }
    }
    const int n_new = n + a + 1;
    seq_lens[i] = n_new;
    const int keep = (n_new + bs - 1) / bs;
    const int held = std::min(max_blocks, (n + k + 1 + bs - 1) / bs);   // pages the step held: positions 0..n+k
    for (int b = keep; b < held; ++b)
      if (bt[b] >= 0) {
        freed[nf++] = bt[b];
        bt[b] = -1;
      }
    row0 += k + 1;
  }
  *freed_count = nf;
  return 0;
}

// Redundancy-aware budget allocation (Sec. 4.2, Eq. 1-3; Algorithm 2), the step that hands the
// verification step its draft lengths.  For request i: n_i candidate continuations were retrieved,
// c_i of them agree on the most frequent prefix, which is len_i tokens long.
//   score   g_i = (c_i / n_i) * p(n_i),  p(n) = g_min + (1 - g_min) * (1 - e^(1 - n)),  g_i = 0 if n_i = 0
//   budget  B_t = floor(alpha / bz)
//   length  L_i = max(len_i, floor(B_t * g_i / G)),  G = sum_j g_j  (L_i = len_i when G = 0)
// The body of the paper writes e^(1-n), its appendix e^(-n); the body is followed (it makes
// p(1) = g_min, the "minimum confidence under low support" the text describes).  The share is
// rounded down to whole tokens.  max_len > 0 caps L_i (the verification step's K_max); the paper
// has no such cap, pass 0 for none.  g (optional) receives the scores.
int ov_budget(int bz, const int32_t* c, const int32_t* n, const int32_t* len, double alpha, double g_min,
              int max_len, int32_t* L, double* g_out) {
  if (bz < 0 || !(alpha >= 0.0) || !(g_min >= 0.0 && g_min <= 1.0)) return 1;
  std::vector<double> g(static_cast<size_t>(bz), 0.0);
  for (int i = 0; i < bz; ++i) {
    if (n[i] < 0 || c[i] < 0 || c[i] > n[i] || len[i] < 0) return 1;
    if (n[i] == 0) continue;
    const double p = g_min + (1.0 - g_min) * (1.0 - std::exp(1.0 - static_cast<double>(n[i])));
    g[i] = static_cast<double>(c[i]) / static_cast<double>(n[i]) * p;
  }
  double G = 0.0;
  for (int i = 0; i < bz; ++i) G += g[i];
  const double Bt = bz > 0 ? std::floor(alpha / static_cast<double>(bz)) : 0.0;
  for (int i = 0; i < bz; ++i) {
    double share = 0.0;
    if (G > 0.0) share = std::floor(Bt * g[i] / G);
    double Li = std::max(static_cast<double>(len[i]), share);
    if (max_len > 0) Li = std::min(Li, static_cast<double>(max_len));
    L[i] = static_cast<int32_t>(std::min(Li, 2147483647.0));
    if (g_out) g_out[i] = g[i];
  }
  return 0;
}

// Counter-based random numbers for rejection sampling.  The paper takes stochastic verification as given
// (Sec. 2.2) and says nothing about where its uniforms come from; so that both sides of a parity test can
// draw them without passing arrays around, each implements the public Philox4x32-10 generator (Salmon,
// Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC 2011) on its own.
//   block(i, b) = Philox4x32-10(counter = (i, b, step_lo, step_hi), key = (seed_lo, seed_hi))
//   u of draft j (0-based) of request i = word j mod 4 of block(i, j / 4)
//   w of request i                     = word 0 of block(i, 0x80000000)
//   a 32-bit word x becomes the float (x >> 8) * 2^-24, in [0, 1)
void ov_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    const uint64_t p0 = static_cast<uint64_t>(0xD2511F53u) * c0;
    const uint64_t p1 = static_cast<uint64_t>(0xCD9E8D57u) * c2;
    const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n1 = static_cast<uint32_t>(p1);
    const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ k1;
    const uint32_t n3 = static_cast<uint32_t>(p0);
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

int ov_philox_uniforms(uint64_t seed, uint64_t step, int B, const int32_t* draft_lens, float* u, float* w) {
  const uint32_t key[2] = {static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32)};
  int64_t at = 0;
  for (int i = 0; i < B; ++i) {
    if (draft_lens[i] < 0) return 1;
    uint32_t out[4];
    for (int j = 0; j < draft_lens[i]; ++j) {
      const uint32_t ctr[4] = {static_cast<uint32_t>(i), static_cast<uint32_t>(j / 4), static_cast<uint32_t>(step),
                               static_cast<uint32_t>(step >> 32)};
      ov_philox4x32_10(ctr, key, out);
      u[at++] = static_cast<float>(out[j % 4] >> 8) * (1.0f / 16777216.0f);
    }
    const uint32_t ctr[4] = {static_cast<uint32_t>(i), 0x80000000u, static_cast<uint32_t>(step),
                             static_cast<uint32_t>(step >> 32)};
    ov_philox4x32_10(ctr, key, out);
    w[i] = static_cast<float>(out[0] >> 8) * (1.0f / 16777216.0f);
  }
  return 0;
}

// The target model's last layer in front of the acceptance test (a reading: Sec. 2.2 says only that the
// target model verifies the drafts; its output layer is a plain projection of the final hidden state onto the vocabulary):
// logits[r][v] = sum_h hidden[r][h] * weight[v][h], bf16 inputs widened exactly, fp64 sum in index order.
int ov_lm_head(int rows, int H, int V, const uint16_t* hidden, const uint16_t* weight, double* logits, int threads) {
  if (rows < 0 || H < 1 || V < 1 || !hidden || !weight || !logits) return 1;
  const int T = std::max(1, std::min(threads > 0 ? threads : ov_hardware_threads(), std::max(1, rows)));
  std::vector<std::thread> pool;
  for (int t = 0; t < T; ++t)
    pool.emplace_back([=] {
      for (int r = t; r < rows; r += T)
        for (int v = 0; v < V; ++v) {
          double acc = 0.0;
          for (int h = 0; h < H; ++h) acc += widen(hidden[(size_t)r * H + h]) * widen(weight[(size_t)v * H + h]);
          logits[(size_t)r * V + v] = acc;
        }
    });
  for (auto& th : pool) th.join();
  return 0;
}

}  // extern "C"
