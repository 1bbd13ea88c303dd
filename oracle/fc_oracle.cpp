// FlowCache hot-path ORACLE — test infrastructure, not product code.
//
// Plain C++17, fp64 arithmetic, no BLAS, no blocking or fusion: each function
// is the paper's definition written out so that it can be checked against the
// text by eye.  Threads only split independent units (chunks, heads, rows).
// Nothing here is shared with, or called by, the CUDA library.
#include "fc_oracle.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <limits>
#include <numeric>
#include <thread>
#include <vector>

namespace {

inline double widen(const void* base, int dtype, int64_t i) {
  if (dtype == FCO_F32) return (double)static_cast<const float*>(base)[i];
  uint32_t bits = (uint32_t)static_cast<const uint16_t*>(base)[i] << 16;
  float f;
  std::memcpy(&f, &bits, sizeof f);
  return (double)f;
}

template <class F>
void parallel_for(int64_t n, int n_threads, F body) {
  if (n_threads <= 0) n_threads = fco_hardware_threads();
  n_threads = (int)std::min<int64_t>(n_threads, std::max<int64_t>(n, 1));
  if (n_threads <= 1) {
    for (int64_t i = 0; i < n; ++i) body(i);
    return;
  }
  std::vector<std::thread> pool;
  for (int t = 0; t < n_threads; ++t)
    pool.emplace_back([=] {
      for (int64_t i = t; i < n; i += n_threads) body(i);
    });
  for (auto& th : pool) th.join();
}

// Physical row of logical key/value token j (segment table or token map).
inline int64_t physical_row(int64_t j, const int32_t* seg_logical_off,
                            const int32_t* seg_phys_off, int n_seg,
                            const int32_t* token_index_head) {
  if (token_index_head) return token_index_head[j];
  for (int s = 0; s < n_seg; ++s)
    if (j >= seg_logical_off[s] && j < seg_logical_off[s + 1])
      return (int64_t)seg_phys_off[s] + (j - seg_logical_off[s]);
  return -1;
}

}  // namespace

extern "C" int fco_hardware_threads(void) {
  unsigned n = std::thread::hardware_concurrency();
  return n ? (int)n : 1;
}

// ---------------------------------------------------------------------------
// Eq. 5 (relative L1 of chunk i between consecutive steps; the denominator is
// the earlier state) and Eq. 8 (accumulate, compare with eps, reset).
// ---------------------------------------------------------------------------
extern "C" int fco_chunk_decide(const void* cur, const void* prev, int dtype,
                                const int64_t* chunk_elem_off, int n_chunks,
                                const int32_t* chunk_step, int warmup_m,
                                float eps, const uint8_t* force, float* acc,
                                float* l1rel, uint8_t* recompute,
                                int32_t* active_ids, int32_t* n_active,
                                int n_threads) {
  if (!chunk_elem_off || !chunk_step || !acc || !recompute || n_chunks < 0)
    return -1;
  if (dtype != FCO_BF16 && dtype != FCO_F32) return -2;
  std::vector<double> r(n_chunks, 0.0);
  parallel_for(n_chunks, n_threads, [&](int64_t c) {
    double num = 0.0, den = 0.0;
    for (int64_t e = chunk_elem_off[c]; e < chunk_elem_off[c + 1]; ++e) {
      double x_prev = widen(prev, dtype, e), x_cur = widen(cur, dtype, e);
      num += std::fabs(x_cur - x_prev);
      den += std::fabs(x_prev);
    }
    if (den > 0.0)
      r[c] = num / den;
    else
      r[c] = num > 0.0 ? std::numeric_limits<double>::infinity() : 0.0;
  });
  int32_t count = 0;
  for (int c = 0; c < n_chunks; ++c) {
    float rf = (float)r[c];
    if (l1rel) l1rel[c] = rf;
    volatile float s = acc[c] + rf;  // fp32 sum, as the accumulator is fp32
    bool warm = chunk_step[c] < warmup_m;
    bool forced = force && force[c];
    if (warm || forced || s > eps) {  // cases 1 and 2 of Eq. 8
      recompute[c] = 1;
      acc[c] = 0.0f;
      if (active_ids) active_ids[count] = c;
      ++count;
    } else {  // case 3 of Eq. 8
      recompute[c] = 0;
      acc[c] = s;
    }
  }
  if (n_active) *n_active = count;
  return 0;
}

// ---------------------------------------------------------------------------
// The uniform ("traditional reuse") policy of the caption of Fig. 3: all chunks
// of a timestep share ONE compute / reuse status, except chunks that must be
// computed anyway (newly initialised: still in warm-up, or forced).  The shared
// indicator is Eq. 4 taken over all sharing chunks as one tensor; the shared
// accumulator follows Eq. 8.
// ---------------------------------------------------------------------------
extern "C" int fco_chunk_decide_uniform(const void* cur, const void* prev, int dtype,
                                        const int64_t* chunk_elem_off, int n_chunks,
                                        const int32_t* chunk_step, int warmup_m,
                                        float eps, const uint8_t* force, float* acc,
                                        float* l1rel, uint8_t* recompute,
                                        int32_t* active_ids, int32_t* n_active,
                                        int n_threads) {
  if (!chunk_elem_off || !chunk_step || !acc || !recompute || n_chunks < 0)
    return -1;
  if (dtype != FCO_BF16 && dtype != FCO_F32) return -2;
  std::vector<double> num(n_chunks, 0.0), den(n_chunks, 0.0);
  parallel_for(n_chunks, n_threads, [&](int64_t c) {
    for (int64_t e = chunk_elem_off[c]; e < chunk_elem_off[c + 1]; ++e) {
      double x_prev = widen(prev, dtype, e), x_cur = widen(cur, dtype, e);
      num[c] += std::fabs(x_cur - x_prev);
      den[c] += std::fabs(x_prev);
    }
  });
  auto ratio = [](double n, double d) {
    if (d > 0.0) return n / d;
    return n > 0.0 ? std::numeric_limits<double>::infinity() : 0.0;
  };
  // the chunks that share the decision, and their common indicator
  double num_all = 0.0, den_all = 0.0;
  int first_sharing = -1;
  std::vector<uint8_t> own(n_chunks, 0);
  for (int c = 0; c < n_chunks; ++c) {
    own[c] = (chunk_step[c] < warmup_m) || (force && force[c]);
    if (own[c]) continue;
    if (first_sharing < 0) first_sharing = c;
    num_all += num[c];
    den_all += den[c];
  }
  bool shared_compute = true;
  float acc_next = 0.0f;
  float r_shared = 0.0f;
  if (first_sharing >= 0) {
    r_shared = (float)ratio(num_all, den_all);
    volatile float s = acc[first_sharing] + r_shared;  // fp32, as in Eq. 8's accumulator
    shared_compute = s > eps;
    acc_next = shared_compute ? 0.0f : s;
  }
  int32_t count = 0;
  for (int c = 0; c < n_chunks; ++c) {
    if (l1rel) l1rel[c] = own[c] ? (float)ratio(num[c], den[c]) : r_shared;
    recompute[c] = (own[c] || shared_compute) ? 1 : 0;
    acc[c] = acc_next;
    if (recompute[c]) {
      if (active_ids) active_ids[count] = c;
      ++count;
    }
  }
  if (n_active) *n_active = count;
  return 0;
}

// ---------------------------------------------------------------------------
// Sec. 3.2 (text after Eq. 8): a chunk that is not recomputed is served from
// its cached activations.  The cache holds, per chunk, the residual between the
// output and the input of the last computed forward; a reused chunk's output is
// its current input plus that residual.  Arithmetic is in fp32 and rounded once
// to the storage type (the result is a stored code: both sides of a parity test
// must round the same fp32 value).
// ---------------------------------------------------------------------------
namespace {
inline float load_f32(const void* base, int dtype, int64_t i) {
  if (dtype == FCO_F32) return static_cast<const float*>(base)[i];
  uint32_t bits = (uint32_t)static_cast<const uint16_t*>(base)[i] << 16;
  float f;
  std::memcpy(&f, &bits, sizeof f);
  return f;
}
inline void store_rounded(void* base, int dtype, int64_t i, float v) {
  if (dtype == FCO_F32) {
    static_cast<float*>(base)[i] = v;
    return;
  }
  uint32_t u;
  std::memcpy(&u, &v, sizeof u);
  uint16_t out;
  if ((u & 0x7fffffffu) > 0x7f800000u) {
    out = (uint16_t)((u >> 16) | 0x0040u);  // NaN stays NaN (quiet)
  } else {
    // round to nearest, ties to even, on the 16 bits that are dropped
    uint32_t lsb = (u >> 16) & 1u;
    out = (uint16_t)((u + 0x7fffu + lsb) >> 16);
  }
  static_cast<uint16_t*>(base)[i] = out;
}
}  // namespace

extern "C" int fco_chunk_cache_apply(const void* x_in, void* y_io, void* cache, int dtype,
                                     const int64_t* chunk_elem_off, int n_chunks,
                                     const uint8_t* recompute, int n_threads) {
  if (!chunk_elem_off || !recompute || n_chunks < 0) return -1;
  if (dtype != FCO_BF16 && dtype != FCO_F32) return -2;
  parallel_for(n_chunks, n_threads, [&](int64_t c) {
    for (int64_t e = chunk_elem_off[c]; e < chunk_elem_off[c + 1]; ++e) {
      const float x = load_f32(x_in, dtype, e);
      if (recompute[c]) {
        // the forward ran: remember what it added to its input
        volatile float delta = load_f32(y_io, dtype, e) - x;
        store_rounded(cache, dtype, e, delta);
      } else {
        // the forward was skipped: input plus the remembered residual
        volatile float y = x + load_f32(cache, dtype, e);
        store_rounded(y_io, dtype, e, y);
      }
    }
  });
  return 0;
}

// ---------------------------------------------------------------------------
// Sec. 3.3: queries of the chunks being denoised attend to the compressed
// clean-chunk region followed by the denoising region; chunk c sees a logical
// prefix of kv_visible_len[c] tokens.  Textbook softmax attention per row.
// ---------------------------------------------------------------------------
extern "C" int fco_chunk_attention(
    const fco_attn_desc* desc, const void* Q, const void* K, const void* V,
    int dtype, const int32_t* q_chunk_row_off, const int32_t* kv_visible_len,
    const int32_t* seg_logical_off, const int32_t* seg_phys_off, int n_seg,
    const int32_t* kv_token_index, int64_t kv_index_hs,
    const int32_t* active_ids, int n_active, const int32_t* sample_rows,
    int n_sample, double* O, int64_t o_hs, int64_t o_rs, double* lse,
    int n_threads) {
  if (!desc || !Q || !K || !V || !q_chunk_row_off || !kv_visible_len || !O)
    return -1;
  if (dtype != FCO_BF16 && dtype != FCO_F32) return -2;
  if (!kv_token_index && (!seg_logical_off || !seg_phys_off || n_seg <= 0))
    return -3;
  const int H_q = desc->H_q, H_kv = desc->H_kv, d = desc->d, W = desc->W;
  if (H_q <= 0 || H_kv <= 0 || H_q % H_kv || d <= 0 || W <= 0) return -4;
  const int group = H_q / H_kv;
  const double scale = desc->scale != 0.0 ? desc->scale : 1.0 / std::sqrt((double)d);

  std::vector<uint8_t> is_active(W, 0);
  for (int a = 0; a < n_active; ++a) {
    if (active_ids[a] < 0 || active_ids[a] >= W) return -5;
    is_active[active_ids[a]] = 1;
  }
  // The list of (query row, output slot) pairs to evaluate.
  std::vector<int32_t> rows, slots, chunk_of;
  auto chunk_of_row = [&](int32_t r) {
    for (int c = 0; c < W; ++c)
      if (r >= q_chunk_row_off[c] && r < q_chunk_row_off[c + 1]) return c;
    return -1;
  };
  if (sample_rows) {
    for (int s = 0; s < n_sample; ++s) {
      int c = chunk_of_row(sample_rows[s]);
      if (c < 0) return -6;
      if (!is_active[c]) continue;
      rows.push_back(sample_rows[s]);
      slots.push_back(s);
      chunk_of.push_back(c);
    }
  } else {
    for (int c = 0; c < W; ++c) {
      if (!is_active[c]) continue;
      for (int32_t r = q_chunk_row_off[c]; r < q_chunk_row_off[c + 1]; ++r) {
        rows.push_back(r);
        slots.push_back(r);
        chunk_of.push_back(c);
      }
    }
  }
  const int64_t n_rows = (int64_t)rows.size();
  const int64_t lse_hs = sample_rows ? n_sample : q_chunk_row_off[W];
  const int64_t out_hs = sample_rows ? (int64_t)n_sample * d : o_hs;
  const int64_t out_rs = sample_rows ? d : o_rs;

  parallel_for(n_rows * H_q, n_threads, [&](int64_t item) {
    const int h = (int)(item / n_rows);
    const int64_t idx = item % n_rows;
    const int h_kv = h / group;
    const int32_t r = rows[idx];
    const int32_t n_vis = kv_visible_len[chunk_of[idx]];
    const int32_t* tok_map =
        kv_token_index ? kv_token_index + (int64_t)h_kv * kv_index_hs : nullptr;
    double* out = O + (int64_t)h * out_hs + (int64_t)slots[idx] * out_rs;
    std::vector<double> s(std::max(n_vis, 0));
    std::vector<int64_t> phys(std::max(n_vis, 0));
    std::vector<double> q(d);
    for (int e = 0; e < d; ++e)
      q[e] = widen(Q, dtype, (int64_t)h * desc->q_hs + (int64_t)r * desc->q_rs + e);
    double s_max = -std::numeric_limits<double>::infinity();
    for (int32_t j = 0; j < n_vis; ++j) {
      phys[j] = physical_row(j, seg_logical_off, seg_phys_off, n_seg, tok_map);
      double dot = 0.0;
      for (int e = 0; e < d; ++e)
        dot += q[e] * widen(K, dtype, (int64_t)h_kv * desc->k_hs + phys[j] * desc->k_rs + e);
      s[j] = dot * scale;
      s_max = std::max(s_max, s[j]);
    }
    double denom = 0.0;
    for (int32_t j = 0; j < n_vis; ++j) {
      s[j] = std::exp(s[j] - s_max);
      denom += s[j];
    }
    // o = sum_j p_j v_j, one value row at a time (every component still adds its terms in the order j = 0, 1, ...)
    std::vector<double> o(d, 0.0);
    for (int32_t j = 0; j < n_vis; ++j) {
      const int64_t v_row = (int64_t)h_kv * desc->v_hs + phys[j] * desc->v_rs;
      for (int e = 0; e < d; ++e) o[e] += s[j] * widen(V, dtype, v_row + e);
    }
    for (int e = 0; e < d; ++e) out[e] = n_vis > 0 ? o[e] / denom : 0.0;
    if (lse)
      lse[(int64_t)h * lse_hs + slots[idx]] =
          n_vis > 0 ? s_max + std::log(denom)
                    : -std::numeric_limits<double>::infinity();
  });
  return 0;
}

// ---------------------------------------------------------------------------
// Eqs. 9-12 and the appendix identity for the column means of the cosine
// matrix.
// ---------------------------------------------------------------------------
extern "C" int fco_kv_score(const fco_score_desc* desc, const void* Q_obs,
                            const void* K_cand, int dtype, double* imp_accum,
                            int accum_phase, int n_steps, double* imp,
                            double* imp_pooled, double* red, float* score,
                            int n_threads) {
  if (!desc || !Q_obs || !K_cand) return -1;
  if (dtype != FCO_BF16 && dtype != FCO_F32) return -2;
  const int H_q = desc->H_q, H_kv = desc->H_kv, d = desc->d;
  const int L_q = desc->L_q, L_k = desc->L_k, pool_k = desc->pool_k;
  if (H_q <= 0 || H_kv <= 0 || H_q % H_kv || d <= 0 || L_q <= 0 || L_k <= 0)
    return -4;
  if (pool_k < 1 || pool_k % 2 == 0) return -5;
  if (accum_phase < 0 || accum_phase > 2) return -6;
  if (accum_phase != 0 && (!imp_accum || n_steps <= 0)) return -7;
  if (accum_phase != 1 && !score) return -8;
  const int group = H_q / H_kv;
  const double scale = desc->scale != 0.0 ? desc->scale : 1.0 / std::sqrt((double)d);
  const double lambda = desc->lambda;
  int red_mode = desc->red_mode;
  if (red_mode == FCO_RED_AUTO)
    red_mode = L_k <= 4096 ? FCO_RED_PLAIN : FCO_RED_MEANKEY;

  std::vector<double> imp_all((size_t)H_kv * L_k, 0.0);
  // Eq. 9: softmax over the candidate keys for every (query head, query row),
  // then the mean over rows and over the query heads of the group.
  parallel_for(H_kv, n_threads, [&](int64_t hk) {
    double* imp_h = imp_all.data() + hk * L_k;
    std::vector<double> p(L_k);
    for (int g = 0; g < group; ++g) {
      const int hq = (int)hk * group + g;
      for (int i = 0; i < L_q; ++i) {
        double s_max = -std::numeric_limits<double>::infinity();
        for (int j = 0; j < L_k; ++j) {
          double dot = 0.0;
          for (int e = 0; e < d; ++e)
            dot += widen(Q_obs, dtype, (int64_t)hq * desc->q_hs + (int64_t)i * desc->q_rs + e) *
                   widen(K_cand, dtype, hk * desc->k_hs + (int64_t)j * desc->k_rs + e);
          p[j] = dot * scale;
          s_max = std::max(s_max, p[j]);
        }
        double denom = 0.0;
        for (int j = 0; j < L_k; ++j) {
          p[j] = std::exp(p[j] - s_max);
          denom += p[j];
        }
        for (int j = 0; j < L_k; ++j) imp_h[j] += p[j] / denom;
      }
    }
    for (int j = 0; j < L_k; ++j) imp_h[j] /= (double)(L_q * group);
  });

  if (accum_phase != 0)
    for (size_t t = 0; t < imp_all.size(); ++t) imp_accum[t] += imp_all[t];
  if (accum_phase == 1) return 0;
  if (accum_phase == 2)
    for (size_t t = 0; t < imp_all.size(); ++t)
      imp_all[t] = imp_accum[t] / (double)n_steps;

  parallel_for(H_kv, n_threads, [&](int64_t hk) {
    const double* imp_h = imp_all.data() + hk * L_k;
    // Eq. 10: stride-1 max-pool, window pool_k, -inf padding of pool_k/2.
    std::vector<double> pooled(L_k);
    const int half = pool_k / 2;
    for (int j = 0; j < L_k; ++j) {
      double m = -std::numeric_limits<double>::infinity();
      for (int u = -half; u <= half; ++u)
        if (j + u >= 0 && j + u < L_k) m = std::max(m, imp_h[j + u]);
      pooled[j] = m;
    }
    // Eq. 11: l2-normalise the keys, cosine matrix, zero diagonal, column mean.
    std::vector<double> khat((size_t)L_k * d);
    for (int j = 0; j < L_k; ++j) {
      double nrm2 = 0.0;
      for (int e = 0; e < d; ++e) {
        double x = widen(K_cand, dtype, hk * desc->k_hs + (int64_t)j * desc->k_rs + e);
        khat[(size_t)j * d + e] = x;
        nrm2 += x * x;
      }
      double inv = 1.0 / std::max(std::sqrt(nrm2), 1e-12);
      for (int e = 0; e < d; ++e) khat[(size_t)j * d + e] *= inv;
    }
    std::vector<double> col_mean(L_k, 0.0);
    if (red_mode == FCO_RED_MAXSIM) {
      // Variant outside the paper (it does not collapse to a mean key): the similarity of token j to its most
      // similar OTHER token takes the place of the column mean; the diagonal is excluded, not zeroed.
      for (int j = 0; j < L_k; ++j) {
        double best = L_k > 1 ? -std::numeric_limits<double>::infinity() : 0.0;
        for (int i = 0; i < L_k; ++i) {
          if (i == j) continue;
          double dot = 0.0;
          for (int e = 0; e < d; ++e)
            dot += khat[(size_t)i * d + e] * khat[(size_t)j * d + e];
          best = std::max(best, dot);
        }
        col_mean[j] = best;
      }
    } else if (red_mode == FCO_RED_PLAIN) {
      for (int j = 0; j < L_k; ++j) {
        double acc = 0.0;
        for (int i = 0; i < L_k; ++i) {
          if (i == j) continue;  // S_ii = 0
          double dot = 0.0;
          for (int e = 0; e < d; ++e)
            dot += khat[(size_t)i * d + e] * khat[(size_t)j * d + e];
          acc += dot;
        }
        col_mean[j] = acc / (double)L_k;
      }
    } else {
      // Appendix identity: mean_i (khat_i . khat_j) = (mean_i khat_i) . khat_j;
      // the zeroed diagonal removes |khat_j|^2 / L_k from column j.
      std::vector<double> mean_key(d, 0.0);
      for (int i = 0; i < L_k; ++i)
        for (int e = 0; e < d; ++e) mean_key[e] += khat[(size_t)i * d + e];
      for (int e = 0; e < d; ++e) mean_key[e] /= (double)L_k;
      for (int j = 0; j < L_k; ++j) {
        double dot = 0.0, self = 0.0;
        for (int e = 0; e < d; ++e) {
          dot += mean_key[e] * khat[(size_t)j * d + e];
          self += khat[(size_t)j * d + e] * khat[(size_t)j * d + e];
        }
        col_mean[j] = dot - self / (double)L_k;
      }
    }
    // softmax over the tokens of this head
    double c_max = *std::max_element(col_mean.begin(), col_mean.end());
    double denom = 0.0;
    std::vector<double> red_h(L_k);
    for (int j = 0; j < L_k; ++j) {
      red_h[j] = std::exp(col_mean[j] - c_max);
      denom += red_h[j];
    }
    for (int j = 0; j < L_k; ++j) red_h[j] /= denom;
    // Eq. 12
    for (int j = 0; j < L_k; ++j) {
      if (imp) imp[hk * L_k + j] = imp_h[j];
      if (imp_pooled) imp_pooled[hk * L_k + j] = pooled[j];
      if (red) red[hk * L_k + j] = red_h[j];
      score[hk * L_k + j] = (float)(lambda * pooled[j] - (1.0 - lambda) * red_h[j]);
    }
  });
  return 0;
}

// ---------------------------------------------------------------------------
// Eq. 11 before its softmax, for chosen columns only: the column statistic of the
// cosine-similarity matrix by its plain definition (every other token visited),
// so that large caches can be checked on a sample of columns.
// ---------------------------------------------------------------------------
extern "C" int fco_key_similarity_columns(const void* K_cand, int dtype, int n_heads,
                                          int L_k, int d, int64_t k_hs, int64_t k_rs,
                                          const int32_t* cols, int n_cols, int red_mode,
                                          double* out, int n_threads) {
  if (!K_cand || !cols || !out || n_heads <= 0 || L_k <= 0 || d <= 0 || n_cols < 0) return -1;
  if (dtype != FCO_BF16 && dtype != FCO_F32) return -2;
  if (red_mode != FCO_RED_PLAIN && red_mode != FCO_RED_MAXSIM) return -3;
  for (int c = 0; c < n_cols; ++c)
    if (cols[c] < 0 || cols[c] >= L_k) return -4;
  parallel_for((int64_t)n_heads * n_cols, n_threads, [&](int64_t item) {
    const int64_t h = item / n_cols;
    const int j = cols[item % n_cols];
    auto unit_key = [&](int t, std::vector<double>& v) {
      double nrm2 = 0.0;
      for (int e = 0; e < d; ++e) {
        v[e] = widen(K_cand, dtype, h * k_hs + (int64_t)t * k_rs + e);
        nrm2 += v[e] * v[e];
      }
      const double inv = 1.0 / std::max(std::sqrt(nrm2), 1e-12);
      for (int e = 0; e < d; ++e) v[e] *= inv;
    };
    std::vector<double> kj(d), ki(d);
    unit_key(j, kj);
    double sum = 0.0;
    double best = L_k > 1 ? -std::numeric_limits<double>::infinity() : 0.0;
    for (int i = 0; i < L_k; ++i) {
      if (i == j) continue;  // S_jj = 0 (sum) / excluded (max)
      unit_key(i, ki);
      double dot = 0.0;
      for (int e = 0; e < d; ++e) dot += ki[e] * kj[e];
      sum += dot;
      best = std::max(best, dot);
    }
    out[item] = red_mode == FCO_RED_PLAIN ? sum / (double)L_k : best;
  });
  return 0;
}

// ---------------------------------------------------------------------------
// Top-B per head and retention of the selected rows.
// ---------------------------------------------------------------------------
extern "C" int fco_kv_select_compact(const float* score, int n_heads, int L_k,
                                     int B, const void* K_src,
                                     const void* V_src, void* K_dst,
                                     void* V_dst, int elem_bytes, int d,
                                     int64_t src_hs, int64_t src_rs,
                                     int64_t dst_hs, int64_t dst_rs,
                                     int32_t* kept_idx, int32_t* n_kept,
                                     int n_threads) {
  if (!score || !kept_idx || n_heads <= 0 || L_k < 0 || B < 0) return -1;
  const bool copy = K_src || V_src || K_dst || V_dst;
  if (copy && (!K_src || !V_src || !K_dst || !V_dst || d <= 0 || elem_bytes <= 0))
    return -2;
  const int n_keep = std::min(B, L_k);
  if (n_kept) *n_kept = n_keep;
  parallel_for(n_heads, n_threads, [&](int64_t h) {
    const float* s = score + h * L_k;
    auto rank_value = [&](int j) {
      return std::isnan(s[j]) ? -std::numeric_limits<float>::infinity() : s[j];
    };
    std::vector<int32_t> order(L_k);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
      return rank_value(a) > rank_value(b);  // stable => index ascending on ties
    });
    std::vector<int32_t> kept(order.begin(), order.begin() + n_keep);
    std::sort(kept.begin(), kept.end());
    for (int r = 0; r < n_keep; ++r) kept_idx[h * n_keep + r] = kept[r];
    if (!copy) return;
    const size_t row_bytes = (size_t)d * elem_bytes;
    for (int r = 0; r < n_keep; ++r) {
      const size_t src = ((size_t)h * src_hs + (size_t)kept[r] * src_rs) * elem_bytes;
      const size_t dst = ((size_t)h * dst_hs + (size_t)r * dst_rs) * elem_bytes;
      std::memcpy((char*)K_dst + dst, (const char*)K_src + src, row_bytes);
      std::memcpy((char*)V_dst + dst, (const char*)V_src + src, row_bytes);
    }
  });
  return 0;
}

// ---------------------------------------------------------------------------
// Selection at a coarser key granularity (the key-granularity ablation of the
// paper's Table 4: frame- or chunk-level keys instead of tokens) and with a
// protected tail.  Units of `unit` consecutive tokens are kept or dropped as a
// whole; a unit's score is the mean of its tokens' scores (fp64 sum in token
// order, rounded to fp32: the selection compares fp32 values as the token-level
// one does).  The last ceil(n_protect / unit) units (the newest tokens) are kept
// whatever their score.  Order among the others: score descending, unit index
// ascending, NaN as -inf.  kept_idx lists the tokens of the kept units ascending.
// ---------------------------------------------------------------------------
extern "C" int fco_kv_select_units(const float* score, int n_heads, int L_k, int B, int unit,
                                   int n_protect, int32_t* kept_idx, int32_t* n_kept,
                                   int n_threads) {
  if (!score || !kept_idx || n_heads <= 0 || L_k <= 0 || B <= 0 || unit <= 0 || n_protect < 0) return -1;
  if (L_k % unit || B % unit) return -2;
  const int n_units = L_k / unit, keep_units = std::min(B / unit, n_units);
  const int protect_units = std::min((n_protect + unit - 1) / unit, keep_units);
  if (n_kept) *n_kept = keep_units * unit;
  parallel_for(n_heads, n_threads, [&](int64_t h) {
    const float* s = score + h * L_k;
    std::vector<float> us(n_units);
    for (int u = 0; u < n_units; ++u) {
      double acc = 0.0;
      for (int t = 0; t < unit; ++t) acc += (double)s[(int64_t)u * unit + t];
      us[u] = (float)(acc / (double)unit);
    }
    auto rank_value = [&](int u) {
      return std::isnan(us[u]) ? -std::numeric_limits<float>::infinity() : us[u];
    };
    std::vector<int32_t> order(n_units - protect_units);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
      return rank_value(a) > rank_value(b);  // stable => index ascending on ties
    });
    std::vector<int32_t> kept(order.begin(), order.begin() + (keep_units - protect_units));
    for (int u = n_units - protect_units; u < n_units; ++u) kept.push_back(u);
    std::sort(kept.begin(), kept.end());
    for (int r = 0; r < keep_units; ++r)
      for (int t = 0; t < unit; ++t)
        kept_idx[h * (int64_t)keep_units * unit + (int64_t)r * unit + t] = kept[r] * unit + t;
  });
  return 0;
}

