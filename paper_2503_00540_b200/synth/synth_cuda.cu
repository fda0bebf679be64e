/*
 * Device-side fillers for the seeded synthetic inputs (see rekv_synth.h).
 * Same element function as the host fillers, so both produce identical bits.
 * No method arithmetic lives here.
 */
#include <cuda_runtime.h>
#include "rekv_synth.h"

namespace {

__global__ void fill_frame_kernel(uint64_t kn, uint64_t ko, uint32_t frame, uint32_t layer0, long n_elem,
                                  uint32_t n_tokens, uint32_t n_heads, uint32_t head_dim, float off_scale,
                                  uint16_t* __restrict__ out) {
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < n_elem; i += (long)gridDim.x * blockDim.x) {
    uint32_t d = (uint32_t)(i % head_dim);
    long r = i / head_dim;
    uint32_t h = (uint32_t)(r % n_heads);
    r /= n_heads;
    uint32_t t = (uint32_t)(r % n_tokens);
    uint32_t l = layer0 + (uint32_t)(r / n_tokens);
    float z = rekv_synth_z(kn, rekv_synth_counter(l, frame, t, h, d));
    float o = rekv_synth_z(ko, rekv_synth_counter(l, frame, 0, h, d));
    out[i] = rekv_synth_bf16(z + off_scale * o);
  }
}

__global__ void fill_q_kernel(uint64_t kq, uint32_t question, uint32_t layer0, long n_elem, uint32_t n_tokens,
                              uint32_t n_heads, uint32_t head_dim, uint16_t* __restrict__ out) {
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < n_elem; i += (long)gridDim.x * blockDim.x) {
    uint32_t d = (uint32_t)(i % head_dim);
    long r = i / head_dim;
    uint32_t h = (uint32_t)(r % n_heads);
    r /= n_heads;
    uint32_t t = (uint32_t)(r % n_tokens);
    uint32_t l = layer0 + (uint32_t)(r / n_tokens);
    out[i] = rekv_synth_q(kq, l, question, t, h, d);
  }
}

}  // namespace

extern "C" {

/* Device twin of rekv_synth_fill_frame_cpu; `out` is a device pointer; enqueued on `stream`.
 * Returns the cudaError_t of the launch as an int. */
int rekv_synth_fill_frame_cuda(uint64_t seed, int which, int frame, int layer0, int n_layers, int n_tokens,
                               int n_kv_heads, int head_dim, float off_scale, uint16_t* out, void* stream) {
  long n = (long)n_layers * n_tokens * n_kv_heads * head_dim;
  if (n <= 0) return 0;
  int blocks = (int)((n + 255) / 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  fill_frame_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(
      rekv_synth_key(seed, (uint32_t)which), rekv_synth_key(seed, (uint32_t)(which + 2)), (uint32_t)frame,
      (uint32_t)layer0, n, (uint32_t)n_tokens, (uint32_t)n_kv_heads, (uint32_t)head_dim, off_scale, out);
  return (int)cudaGetLastError();
}

int rekv_synth_fill_q_cuda(uint64_t seed, int question, int layer0, int n_layers, int n_tokens, int n_q_heads,
                           int head_dim, uint16_t* out, void* stream) {
  long n = (long)n_layers * n_tokens * n_q_heads * head_dim;
  if (n <= 0) return 0;
  int blocks = (int)((n + 255) / 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  fill_q_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(rekv_synth_key(seed, REKV_SYNTH_Q), (uint32_t)question,
                                                           (uint32_t)layer0, n, (uint32_t)n_tokens,
                                                           (uint32_t)n_q_heads, (uint32_t)head_dim, out);
  return (int)cudaGetLastError();
}

}  // extern "C"
