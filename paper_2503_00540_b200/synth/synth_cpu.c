/*
 * Host-side fillers for the seeded synthetic inputs (see rekv_synth.h).
 * Plain C, OpenMP over tokens.  No method arithmetic lives here.
 */
#include "rekv_synth.h"

/* One frame's K or V for layers [layer0, layer0+n_layers), token-major as a
 * decoder emits it: out[l - layer0][t][h][d], bf16 bits.
 * which: REKV_SYNTH_K or REKV_SYNTH_V.  off_scale: 0.0f (plain N(0,1)) or 0.5f. */
void rekv_synth_fill_frame_cpu(uint64_t seed, int which, int frame, int layer0, int n_layers,
                               int n_tokens, int n_kv_heads, int head_dim, float off_scale,
                               uint16_t* out) {
  const uint64_t kn = rekv_synth_key(seed, (uint32_t)which);
  const uint64_t ko = rekv_synth_key(seed, (uint32_t)(which + 2));
  const long per_layer = (long)n_tokens * n_kv_heads * head_dim;
#pragma omp parallel for collapse(2) schedule(static)
  for (int l = 0; l < n_layers; ++l)
    for (int t = 0; t < n_tokens; ++t)
      for (int h = 0; h < n_kv_heads; ++h)
        for (int d = 0; d < head_dim; ++d) {
          uint32_t L = (uint32_t)(layer0 + l);
          float z = rekv_synth_z(kn, rekv_synth_counter(L, (uint32_t)frame, (uint32_t)t, (uint32_t)h, (uint32_t)d));
          float o = rekv_synth_z(ko, rekv_synth_counter(L, (uint32_t)frame, 0, (uint32_t)h, (uint32_t)d));
          out[l * per_layer + ((long)t * n_kv_heads + h) * head_dim + d] = rekv_synth_bf16(z + off_scale * o);
        }
}

/* One question's queries for layers [layer0, layer0+n_layers): out[l][t][h][d], bf16 bits. */
void rekv_synth_fill_q_cpu(uint64_t seed, int question, int layer0, int n_layers, int n_tokens,
                           int n_q_heads, int head_dim, uint16_t* out) {
  const uint64_t kq = rekv_synth_key(seed, REKV_SYNTH_Q);
  const long per_layer = (long)n_tokens * n_q_heads * head_dim;
#pragma omp parallel for collapse(2) schedule(static)
  for (int l = 0; l < n_layers; ++l)
    for (int t = 0; t < n_tokens; ++t)
      for (int h = 0; h < n_q_heads; ++h)
        for (int d = 0; d < head_dim; ++d)
          out[l * per_layer + ((long)t * n_q_heads + h) * head_dim + d] =
              rekv_synth_q(kq, (uint32_t)(layer0 + l), (uint32_t)question, (uint32_t)t, (uint32_t)h, (uint32_t)d);
}

/* Exposed so that Python can draw seeded integers (question lengths) from the same mixer. */
uint64_t rekv_synth_mix64_c(uint64_t x) { return rekv_synth_mix64(x); }
