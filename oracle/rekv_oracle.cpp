/*
 * CPU oracle for the in-context video KV-cache retrieval hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, double-precision
 * statement of what the five steps compute; the CUDA library never includes,
 * links or calls it, and it shares no code with the CUDA path.  Only the test
 * suite, the smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * Steps, in the paper's order (Section "ReKV", internal retrieval):
 *   1. frame representative  = mean of the frame's N_f key vectors, heads
 *      concatenated                     (internal-retrieval paragraph)
 *   2. question vector       = mean of the question's N_q query vectors;
 *      score = cosine similarity, tau=1 (Eq. 2 with tau = 1)
 *   3. keep the r most similar frames   (Eq. 2 paragraph, "r most relevant")
 *   4. the retrieved K/V, R, are brought together as the context
 *   5. O = Attn(Q, R_k, R_v)            (Eq. 3)
 *   2'. external retrieval: the same cosine on embeddings from a CLIP-like
 *      encoder, divided by the temperature tau; one selection for all layers
 *                                         (Eq. 2, external-retrieval paragraph)
 *   5'. the whole of Eq. 3: O = Attn(W_Q X, [R_k, W_K X], [R_v, W_V X]) -- the
 *      question's (and generated tokens') own K/V follow the retrieved context,
 *      causally; rotary position embedding with the retrieved tokens taken as
 *      consecutive tokens                 (Eq. 3, "Positional Encoding")
 *
 * Readings where the paper is silent (each also listed in the design notes):
 *   - GQA: the G query heads of one KV group are averaged so that question
 *     and frame vectors share D' = H_kv * D.
 *   - norms are clamped at 1e-8; NaN scores rank below every number.
 *   - the last W visible frames (the recent window) are always in the
 *     context and are not candidates for retrieval.
 *   - ties go to the lower frame index; selected frames are emitted in
 *     ascending frame order (temporal order).
 *   - Attn = softmax(Q K^T / sqrt(D)) V, no mask (all context precedes the
 *     question), query head h reads KV head floor(h / G).
 *
 *   - Eq. 3 in full: the retrieved tokens take positions 0 .. n_ctx-1 in
 *     context order, the tokens of X continue at n_ctx; a query of X sees all
 *     of R and the tokens of X up to itself.  Rotary embedding pairs dimension
 *     i with i + D/2 (angle = position * theta^(-2i/D)); rotated queries and
 *     keys are rounded to bf16 once, as a bf16 model holds them.
 *
 * Arithmetic: bf16 inputs are widened exactly; every sum is a double; each
 * stored result is rounded once (to float, and for attention also to bf16).
 *
 * Parity pins: every function below is pinned by tests/test_oracle_pins.py
 * (closed forms, brute force, library routines, invariants).  The paper's
 * accuracy / recall / latency tables need its datasets and weights and stay
 * "parity unpinned".
 */
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

namespace {

inline double bf16_to_double(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return (double)f;
}

inline uint16_t float_to_bf16_rne(float x) {
  uint32_t u;
  std::memcpy(&u, &x, 4);
  if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return (uint16_t)((u >> 16) | 0x40);  // NaN
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

}  // namespace

extern "C" {

/* Step 1.  k: one layer of one frame, token-major [n_tokens][n_kv_heads][head_dim] bf16.
 * rep[h*head_dim + d] = (1/N_f) * sum_t k[t][h][d], rounded once to float. */
void oracle_pool_frame(const uint16_t* k, int n_tokens, int n_kv_heads, int head_dim, float* rep) {
  const int dp = n_kv_heads * head_dim;
  for (int c = 0; c < dp; ++c) {
    double s = 0.0;
    for (int t = 0; t < n_tokens; ++t) s += bf16_to_double(k[(long)t * dp + c]);
    rep[c] = (float)(s / (double)n_tokens);
  }
}

/* Step 2a.  q: one layer of one question, [n_q][n_q_heads][head_dim] bf16.
 * qa[g*head_dim + d] = mean over the question's tokens and over the G query heads of KV group g. */
void oracle_question_vector(const uint16_t* q, int n_q, int n_q_heads, int n_kv_heads, int head_dim, double* qa) {
  const int G = n_q_heads / n_kv_heads;
  std::vector<double> qbar((size_t)n_q_heads * head_dim, 0.0);
  for (int h = 0; h < n_q_heads; ++h)
    for (int d = 0; d < head_dim; ++d) {
      double s = 0.0;
      for (int n = 0; n < n_q; ++n) s += bf16_to_double(q[((long)n * n_q_heads + h) * head_dim + d]);
      qbar[(size_t)h * head_dim + d] = s / (double)n_q;
    }
  for (int g = 0; g < n_kv_heads; ++g)
    for (int d = 0; d < head_dim; ++d) {
      double s = 0.0;
      for (int j = 0; j < G; ++j) s += qbar[(size_t)(g * G + j) * head_dim + d];
      qa[g * head_dim + d] = s / (double)G;
    }
}

/* Step 2b.  scores[f] = <qa, rep_f> / (max(|qa|,eps) * max(|rep_f|,eps)), tau = 1.
 * reps: [n_frames][n_kv_heads*head_dim] float (as stored by step 1). */
void oracle_score(const uint16_t* q, int n_q, int n_q_heads, int n_kv_heads, int head_dim, const float* reps,
                  int n_frames, float* scores) {
  const int dp = n_kv_heads * head_dim;
  const double eps = 1e-8;
  std::vector<double> qa(dp);
  oracle_question_vector(q, n_q, n_q_heads, n_kv_heads, head_dim, qa.data());
  double qn = 0.0;
  for (int c = 0; c < dp; ++c) qn += qa[c] * qa[c];
  qn = std::max(std::sqrt(qn), eps);
  for (int f = 0; f < n_frames; ++f) {
    const float* r = reps + (long)f * dp;
    double dot = 0.0, rn = 0.0;
    for (int c = 0; c < dp; ++c) {
      dot += qa[c] * (double)r[c];
      rn += (double)r[c] * (double)r[c];
    }
    rn = std::max(std::sqrt(rn), eps);
    scores[f] = (float)(dot / (qn * rn));
  }
}

/* External retrieval (Eq. 2 with its temperature): Sim(v, q) = <v, q> / (tau |v| |q|) between the question's
 * embedding q [dim] and frame embeddings embs [n_frames][dim] (floats, from a CLIP-like encoder outside this
 * library); with b > 1 the vector of a block is the mean of its b frame vectors (kept in double) and
 * n_items counts complete blocks.  Norms are clamped at 1e-8 as in the internal variant. */
void oracle_score_external(const float* q, const float* embs, int dim, int n_items, int b, double tau,
                           float* scores) {
  const double eps = 1e-8;
  double qn = 0.0;
  for (int c = 0; c < dim; ++c) qn += (double)q[c] * (double)q[c];
  qn = std::max(std::sqrt(qn), eps);
  std::vector<double> v(dim);
  for (int j = 0; j < n_items; ++j) {
    for (int c = 0; c < dim; ++c) {
      double s = 0.0;
      for (int f = 0; f < b; ++f) s += (double)embs[((long)j * b + f) * dim + c];
      v[c] = s / (double)b;
    }
    double dot = 0.0, vn = 0.0;
    for (int c = 0; c < dim; ++c) {
      dot += (double)q[c] * v[c];
      vn += v[c] * v[c];
    }
    vn = std::max(std::sqrt(vn), eps);
    scores[j] = (float)(dot / (tau * qn * vn));
  }
}

/* Step 2, block variant (Eq. 2 paragraph: b consecutive frames form a block whose vector is the average of the
 * frames' vectors).  Block j averages the representatives of frames [j*b, (j+1)*b); only complete blocks exist.
 * scores[j] = cosine(question vector, block vector), tau = 1.  The block mean is kept in double. */
void oracle_score_blocks(const uint16_t* q, int n_q, int n_q_heads, int n_kv_heads, int head_dim, const float* reps,
                         int n_blocks, int b, float* scores) {
  const int dp = n_kv_heads * head_dim;
  const double eps = 1e-8;
  std::vector<double> qa(dp), bv(dp);
  oracle_question_vector(q, n_q, n_q_heads, n_kv_heads, head_dim, qa.data());
  double qn = 0.0;
  for (int c = 0; c < dp; ++c) qn += qa[c] * qa[c];
  qn = std::max(std::sqrt(qn), eps);
  for (int j = 0; j < n_blocks; ++j) {
    for (int c = 0; c < dp; ++c) {
      double s = 0.0;
      for (int f = 0; f < b; ++f) s += (double)reps[((long)j * b + f) * dp + c];
      bv[c] = s / (double)b;
    }
    double dot = 0.0, rn = 0.0;
    for (int c = 0; c < dp; ++c) {
      dot += qa[c] * bv[c];
      rn += bv[c] * bv[c];
    }
    rn = std::max(std::sqrt(rn), eps);
    scores[j] = (float)(dot / (qn * rn));
  }
}

/* Step 3.  Candidates are frames [0, n_visible - window).  Order by (score descending, index
 * ascending), keep k_eff = min(k, #candidates), write them in ascending index order, pad idx_out
 * (length k) with -1.  *gap_out = score of the last kept minus score of the best rejected
 * (+inf if nothing is rejected or nothing kept).  Returns k_eff. */
int oracle_select(const float* scores, int n_visible, int window, int k, int32_t* idx_out, double* gap_out) {
  int n_cand = std::max(n_visible - window, 0);
  int k_eff = std::max(std::min(k, n_cand), 0);
  std::vector<int32_t> order(n_cand);
  for (int i = 0; i < n_cand; ++i) order[i] = i;
  auto key = [&](int i) {
    float s = scores[i];
    return std::isnan(s) ? -std::numeric_limits<double>::infinity() : (double)s;
  };
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
    double sa = key(a), sb = key(b);
    if (sa != sb) return sa > sb;
    return a < b;
  });
  double gap = std::numeric_limits<double>::infinity();
  if (k_eff > 0 && k_eff < n_cand) gap = key(order[k_eff - 1]) - key(order[k_eff]);
  if (gap_out) *gap_out = gap;
  std::vector<int32_t> sel(order.begin(), order.begin() + k_eff);
  std::sort(sel.begin(), sel.end());
  for (int i = 0; i < k; ++i) idx_out[i] = i < k_eff ? sel[i] : -1;
  return k_eff;
}

/* Step 4.  cache: one layer's K (or V), token-major frames [n_frames][n_tokens][n_kv_heads][head_dim].
 * Context frame list = idx[0..k_eff) (ascending) followed by frames max(n_visible-window,0) .. n_visible-1.
 * ctx: [n_kv_heads][n_ctx_frames*n_tokens][head_dim].  Returns the number of context frames. */
int oracle_gather(const uint16_t* cache, int n_tokens, int n_kv_heads, int head_dim, const int32_t* idx, int k_eff,
                  int n_visible, int window, uint16_t* ctx) {
  std::vector<int> frames;
  for (int i = 0; i < k_eff; ++i) frames.push_back(idx[i]);
  for (int f = std::max(n_visible - window, 0); f < n_visible; ++f) frames.push_back(f);
  const int nf = (int)frames.size();
  const long n_ctx = (long)nf * n_tokens;
  for (int h = 0; h < n_kv_heads; ++h)
    for (int j = 0; j < nf; ++j)
      for (int t = 0; t < n_tokens; ++t)
        for (int d = 0; d < head_dim; ++d)
          ctx[((long)h * n_ctx + (long)j * n_tokens + t) * head_dim + d] =
              cache[(((long)frames[j] * n_tokens + t) * n_kv_heads + h) * head_dim + d];
  return nf;
}

/* Step 5.  q: [n_q][n_q_heads][head_dim]; k_ctx, v_ctx: [n_kv_heads][n_ctx][head_dim]; all bf16.
 * out_f32 (and out_bf16, nullable): [n_q][n_q_heads][head_dim].
 * probs (nullable): [n_q][n_q_heads][n_ctx] doubles, the softmax rows, for the row-sum pin. */
void oracle_attend(const uint16_t* q, int n_q, int n_q_heads, int n_kv_heads, int head_dim, const uint16_t* k_ctx,
                   const uint16_t* v_ctx, long n_ctx, float* out_f32, uint16_t* out_bf16, double* probs) {
  const int G = n_q_heads / n_kv_heads;
  const double scale = 1.0 / std::sqrt((double)head_dim);
  const long rows = (long)n_q * n_q_heads;
#pragma omp parallel for schedule(dynamic, 1)
  for (long row = 0; row < rows; ++row) {
    const int h = (int)(row % n_q_heads);
    const int g = h / G;
    const uint16_t* qv = q + row * head_dim;
    const uint16_t* kh = k_ctx + (long)g * n_ctx * head_dim;
    const uint16_t* vh = v_ctx + (long)g * n_ctx * head_dim;
    std::vector<double> qd(head_dim), logit((size_t)n_ctx), acc(head_dim, 0.0);
    for (int d = 0; d < head_dim; ++d) qd[d] = bf16_to_double(qv[d]);
    double m = -std::numeric_limits<double>::infinity();
    for (long j = 0; j < n_ctx; ++j) {
      double s = 0.0;
      for (int d = 0; d < head_dim; ++d) s += qd[d] * bf16_to_double(kh[j * head_dim + d]);
      logit[j] = s * scale;
      m = std::max(m, logit[j]);
    }
    double z = 0.0;
    for (long j = 0; j < n_ctx; ++j) {
      logit[j] = std::exp(logit[j] - m);
      z += logit[j];
    }
    for (long j = 0; j < n_ctx; ++j) {
      const double p = logit[j] / z;
      if (probs) probs[row * n_ctx + j] = p;
      for (int d = 0; d < head_dim; ++d) acc[d] += p * bf16_to_double(vh[j * head_dim + d]);
    }
    for (int d = 0; d < head_dim; ++d) {
      const float o = (float)acc[d];
      out_f32[row * head_dim + d] = o;
      if (out_bf16) out_bf16[row * head_dim + d] = float_to_bf16_rne(o);
    }
  }
}

/* Rotary position embedding (RoFormer) of one vector of D dims at integer position pos:
 * pair i = (x[i], x[i + D/2]) is turned by the angle pos * theta^(-2i/D).  Doubles in and out. */
void oracle_rope(const double* x, int head_dim, long pos, double theta, double* out) {
  const int half = head_dim / 2;
  for (int i = 0; i < half; ++i) {
    const double angle = (double)pos * std::pow(theta, -2.0 * (double)i / (double)head_dim);
    const double c = std::cos(angle), s = std::sin(angle);
    out[i] = x[i] * c - x[i + half] * s;
    out[i + half] = x[i + half] * c + x[i] * s;
  }
}

/* Eq. 3 in full.  q: [n_q][n_q_heads][D] (the rows of X being computed); k_ctx, v_ctx:
 * [n_kv_heads][n_ctx][D] (R, in context order); k_self, v_self: [n_self][n_kv_heads][D], the K/V of X
 * token-major as the model emits them, n_self >= n_q: query row n is token n_self - n_q + n of X
 * (n_self == n_q: the question itself; n_q == 1: a decode step after n_self - 1 earlier tokens).
 * Row n sees every token of R and the tokens 0 .. n_self - n_q + n of X.  rope_theta > 0 applies the
 * rotary embedding: R at positions 0 .. n_ctx-1, X at n_ctx + its token index; rotated vectors are
 * rounded to bf16.  rope_theta == 0: no positional term.  Outputs as oracle_attend. */
void oracle_attend_full(const uint16_t* q, int n_q, int n_q_heads, int n_kv_heads, int head_dim, const uint16_t* k_ctx,
                        const uint16_t* v_ctx, long n_ctx, const uint16_t* k_self, const uint16_t* v_self, int n_self,
                        double rope_theta, int static_ctx, float* out_f32, uint16_t* out_bf16) {
  /* static_ctx != 0: the static variant named in the "Positional Encoding" paragraph (taken from Inf-LLM): all
   * retrieved tokens are assigned the same position.  Reading: every context token has position 0 and token s of X
   * has position 1 + s (X follows the context's single position).  static_ctx == 0: consecutive positions. */
  const int G = n_q_heads / n_kv_heads;
  const double scale = 1.0 / std::sqrt((double)head_dim);
  const long rows = (long)n_q * n_q_heads;
  auto load = [&](const uint16_t* src, long pos, std::vector<double>& dst) {
    std::vector<double> raw(head_dim);
    for (int d = 0; d < head_dim; ++d) raw[d] = bf16_to_double(src[d]);
    if (rope_theta > 0.0) {
      std::vector<double> rot(head_dim);
      oracle_rope(raw.data(), head_dim, pos, rope_theta, rot.data());
      for (int d = 0; d < head_dim; ++d) dst[d] = bf16_to_double(float_to_bf16_rne((float)rot[d]));
    } else {
      dst = raw;
    }
  };
#pragma omp parallel for schedule(dynamic, 1)
  for (long row = 0; row < rows; ++row) {
    const int n = (int)(row / n_q_heads), h = (int)(row % n_q_heads);
    const int g = h / G;
    const int x_tok = n_self - n_q + n;        // this row's token index inside X
    const long n_seen = n_ctx + x_tok + 1;     // all of R, then X up to and including itself
    std::vector<double> qd(head_dim), kd(head_dim), logit((size_t)n_seen), acc(head_dim, 0.0);
    load(q + row * head_dim, static_ctx ? 1 + x_tok : n_ctx + x_tok, qd);
    double m = -std::numeric_limits<double>::infinity();
    for (long j = 0; j < n_seen; ++j) {
      const uint16_t* kj = j < n_ctx ? k_ctx + ((long)g * n_ctx + j) * head_dim
                                     : k_self + ((j - n_ctx) * n_kv_heads + g) * head_dim;
      load(kj, static_ctx ? (j < n_ctx ? 0 : 1 + (j - n_ctx)) : j, kd);
      double s = 0.0;
      for (int d = 0; d < head_dim; ++d) s += qd[d] * kd[d];
      logit[j] = s * scale;
      m = std::max(m, logit[j]);
    }
    double z = 0.0;
    for (long j = 0; j < n_seen; ++j) {
      logit[j] = std::exp(logit[j] - m);
      z += logit[j];
    }
    for (long j = 0; j < n_seen; ++j) {
      const uint16_t* vj = j < n_ctx ? v_ctx + ((long)g * n_ctx + j) * head_dim
                                     : v_self + ((j - n_ctx) * n_kv_heads + g) * head_dim;
      const double p = logit[j] / z;
      for (int d = 0; d < head_dim; ++d) acc[d] += p * bf16_to_double(vj[d]);
    }
    for (int d = 0; d < head_dim; ++d) {
      const float o = (float)acc[d];
      out_f32[row * head_dim + d] = o;
      if (out_bf16) out_bf16[row * head_dim + d] = float_to_bf16_rne(o);
    }
  }
}

/* Quantised host tier (the paper's "Limitations and Future Work" names quantisation as the way to shrink the
 * offloaded cache; no formula is given, this is the reading built here).  A page row -- the 128 dims of one
 * token of one KV head, K or V -- is stored as 128 FP8 E4M3 codes (1 sign, 4 exponent bits with bias 7,
 * 3 mantissa bits; largest finite value 448, subnormal step 2^-9, no infinities) and one float scale:
 *   scale = amax / 448 (1 if the row is all zero), code = round-to-nearest-even(x / scale) saturated at +-448,
 * and read back as bf16_rne(value(code) * scale).  oracle_e4m3_encode is that rounding for one float. */
uint8_t oracle_e4m3_encode(float x) {
  const uint8_t sign = std::signbit(x) ? 0x80 : 0x00;
  double a = std::fabs((double)x);
  if (!(a == a)) return (uint8_t)(sign | 0x7F);  // NaN
  if (a >= 464.0) return (uint8_t)(sign | 0x7E); // beyond the midpoint above 448: saturates (so do 448..464)
  if (a < std::ldexp(1.0, -6)) {                 // subnormal range: multiples of 2^-9
    const double q = std::nearbyint(a * 512.0);  // ties to even (default rounding mode)
    return (uint8_t)(sign | (uint8_t)q);         // q == 8 is the smallest normal, code 0x08
  }
  int e;
  std::frexp(a, &e);                             // a = f * 2^e, f in [0.5, 1)
  e -= 1;                                        // a = m * 2^e, m in [1, 2)
  double m = std::nearbyint(std::ldexp(a, -e) * 8.0);  // 8..16
  if (m == 16.0) {
    m = 8.0;
    e += 1;
  }
  if (e > 8 || (e == 8 && m > 14.0)) return (uint8_t)(sign | 0x7E);  // 448 = 1.75 * 2^8
  return (uint8_t)(sign | ((uint8_t)(e + 7) << 3) | (uint8_t)(m - 8.0));
}

double oracle_e4m3_decode(uint8_t c) {
  const int e = (c >> 3) & 0xF, m = c & 7;
  const double v = e == 0 ? std::ldexp((double)m, -9) : std::ldexp(1.0 + m / 8.0, e - 7);
  return (c & 0x80) ? -v : v;
}

/* rows x 128 bf16 in, the same shape out: each row through the quantised host tier and back. */
void oracle_fp8_roundtrip(const uint16_t* x, long rows, int dim, uint16_t* out, float* scales /* nullable */) {
  for (long r = 0; r < rows; ++r) {
    float amax = 0.f;
    for (int d = 0; d < dim; ++d) amax = std::max(amax, std::fabs((float)bf16_to_double(x[r * dim + d])));
    const float scale = amax > 0.f ? amax / 448.0f : 1.0f;
    if (scales) scales[r] = scale;
    for (int d = 0; d < dim; ++d) {
      const float v = (float)bf16_to_double(x[r * dim + d]);
      const uint8_t c = oracle_e4m3_encode(v / scale);
      out[r * dim + d] = float_to_bf16_rne((float)oracle_e4m3_decode(c) * scale);
    }
  }
}

/* Bytes of K/V cache for a stream: 2 (K and V) * L * T * M * H * D * bytes_per_element
 * (the appendix's cache-size expression; fp16/bf16 -> 2 bytes). */
double oracle_kv_cache_bytes(int n_layers, long n_frames, int tokens_per_frame, int n_kv_heads, int head_dim,
                             int bytes_per_element) {
  return 2.0 * (double)n_layers * (double)n_frames * (double)tokens_per_frame * (double)n_kv_heads *
         (double)head_dim * (double)bytes_per_element;
}

}  // extern "C"
