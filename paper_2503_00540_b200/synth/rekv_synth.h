/*
 * Seeded, stateless synthetic-input generator for the retrieval hot path.
 *
 * This header holds NONE of the method's arithmetic (no pooling, scoring,
 * selection or attention).  It only defines how a synthetic K/V cache and
 * synthetic question queries are drawn, so that the CUDA path and the CPU
 * oracle can be handed bit-identical bf16 inputs without ever materialising
 * a 100+ GB cache on the host: every element is a pure function of
 * (seed, tensor, layer, frame, token, head, dim).
 *
 * Distribution (stand-in for a Video-LLM's per-frame keys/values):
 *   z      ~ Irwin-Hall(12) - 6 on a 2^-16 grid  (mean 0, variance ~1, |z| < 6)
 *   K,V    = bf16( z(l,f,t,h,d) + 0.5 * z_off(l,f,h,d) )   -- a per-frame,
 *            per-(layer, kv-head, dim) offset of std 0.5, constant over the
 *            frame's tokens, so frame means are separable
 *   Q      = bf16( z(l,q,t,h,d) )
 * Every operation is exact in fp32 (integer sum < 2^24, power-of-two scale,
 * one add, one round-to-nearest-even), so host and device agree bit for bit
 * without depending on libm or FMA contraction.
 *
 * Usable from C, C++ and CUDA.
 */
#ifndef REKV_SYNTH_H_
#define REKV_SYNTH_H_

#include <stdint.h>
#include <string.h>

#if defined(__CUDACC__)
#define REKV_SYNTH_HD __host__ __device__ __forceinline__
#else
#define REKV_SYNTH_HD static inline
#endif

enum {
  REKV_SYNTH_K = 1,      /* key noise      */
  REKV_SYNTH_V = 2,      /* value noise    */
  REKV_SYNTH_K_OFF = 3,  /* key   per-frame offset (token index ignored) */
  REKV_SYNTH_V_OFF = 4,  /* value per-frame offset (token index ignored) */
  REKV_SYNTH_Q = 5       /* question queries; "frame" carries the question id */
};

/* splitmix64 finaliser */
REKV_SYNTH_HD uint64_t rekv_synth_mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

/* per-(seed, tensor) stream key */
REKV_SYNTH_HD uint64_t rekv_synth_key(uint64_t seed, uint32_t tensor) {
  return rekv_synth_mix64(rekv_synth_mix64(seed) ^ ((uint64_t)tensor << 56) ^ 0x5EEDull);
}

/* 56-bit element counter: l < 2^10, f < 2^20, t < 2^10, h < 2^8, d < 2^8 */
REKV_SYNTH_HD uint64_t rekv_synth_counter(uint32_t l, uint32_t f, uint32_t t, uint32_t h, uint32_t d) {
  return ((((((uint64_t)l << 20) | f) << 10 | t) << 8 | h) << 8) | d;
}

/* approximately standard-normal sample on a 2^-16 grid, exact in fp32 */
REKV_SYNTH_HD float rekv_synth_z(uint64_t key, uint64_t counter) {
  uint32_t s = 0;
  for (int i = 0; i < 3; ++i) {
    uint64_t u = rekv_synth_mix64(key ^ (counter * 4u + (uint64_t)i));
    s += (uint32_t)(u & 0xFFFF) + (uint32_t)((u >> 16) & 0xFFFF) +
         (uint32_t)((u >> 32) & 0xFFFF) + (uint32_t)(u >> 48);
  }
  /* s in [0, 12*65535]; centre at 6*65535 */
  return (float)((int32_t)s - 393210) * (1.0f / 65536.0f);
}

/* fp32 -> bf16 bits, round to nearest even (inputs here are always finite) */
REKV_SYNTH_HD uint16_t rekv_synth_bf16(float x) {
  uint32_t u;
#if defined(__CUDA_ARCH__)
  u = __float_as_uint(x);
#else
  memcpy(&u, &x, 4);
#endif
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

/* one K or V element; tensor is REKV_SYNTH_K or REKV_SYNTH_V */
REKV_SYNTH_HD uint16_t rekv_synth_kv(uint64_t key_noise, uint64_t key_off, uint32_t l, uint32_t f,
                                     uint32_t t, uint32_t h, uint32_t d) {
  float z = rekv_synth_z(key_noise, rekv_synth_counter(l, f, t, h, d));
  float o = rekv_synth_z(key_off, rekv_synth_counter(l, f, 0, h, d));
  return rekv_synth_bf16(z + 0.5f * o);
}

/* one Q element of question `q` */
REKV_SYNTH_HD uint16_t rekv_synth_q(uint64_t key_q, uint32_t l, uint32_t q, uint32_t t, uint32_t h,
                                    uint32_t d) {
  return rekv_synth_bf16(rekv_synth_z(key_q, rekv_synth_counter(l, q, t, h, d)));
}

#endif /* REKV_SYNTH_H_ */
