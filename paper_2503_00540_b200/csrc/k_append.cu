// Step 1: page a frame's K/V into the store and pool its keys into the frame representative
// (internal retrieval: v = 1/N_f * sum_j k_j, heads concatenated), in one pass over the frame.
#include "rekv_internal.cuh"

namespace {

// grid = L * H_kv * 2 (K tiles pool, V tiles only move); 256 threads: 16 row groups x 16 chunks.
// Source rows are 256-byte segments (one head of one token), read as 16-byte chunks; the page is
// written in the swizzled tile layout.  Pooling accumulates in fp32 in a fixed order.
__global__ void __launch_bounds__(256) append_pool_kernel(const uint4* __restrict__ k_in,
                                                          const uint4* __restrict__ v_in, char* __restrict__ page0,
                                                          float* __restrict__ reps, int frame, int L, int Hkv,
                                                          int Nf, int max_frames, long long page_bytes,
                                                          long long store_bytes, char* __restrict__ store,
                                                          int* __restrict__ status) {
  const int kv = blockIdx.x & 1;
  const int h = (blockIdx.x >> 1) % Hkv;
  const int l = (blockIdx.x >> 1) / Hkv;
  const int c = threadIdx.x & 15;   // 16-byte chunk of the 256-byte head row
  const int rg = threadIdx.x >> 4;  // row group
  const uint4* src = (kv ? v_in : k_in) + ((long long)l * Nf * Hkv + h) * 16 + c;
  char* tile = page0 + (long long)l * page_bytes + (long long)(h * 2 + kv) * Nf * 256 + (c >> 3) * (long long)Nf * 128;
  const int cc = c & 7;

  float acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.f;

  // four rows per thread in flight
  for (int t0 = rg; t0 < Nf; t0 += 64) {
    uint4 x[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int t = t0 + 16 * u;
      if (t < Nf) x[u] = __ldg(src + (long long)t * Hkv * 16);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int t = t0 + 16 * u;
      if (t < Nf) {
        char* dst = tile + t * 128 + ((cc ^ (t & 7)) << 4);
        if (!REKV_CHECK(dst >= store && dst + 16 <= store + store_bytes && (reinterpret_cast<uintptr_t>(dst) & 15) == 0,
                        status, 1))
          continue;
        *reinterpret_cast<uint4*>(dst) = x[u];
        if (kv == 0) {
          const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&x[u]);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            float2 f = __bfloat1622float2(p[i]);
            acc[2 * i] += f.x;
            acc[2 * i + 1] += f.y;
          }
        }
      }
    }
  }
  if (kv == 0) {
    __shared__ float red[16][129];
#pragma unroll
    for (int i = 0; i < 8; ++i) red[rg][c * 8 + i] = acc[i];
    __syncthreads();
    if (threadIdx.x < 128) {
      float s = 0.f;
#pragma unroll
      for (int r = 0; r < 16; ++r) s += red[r][threadIdx.x];
      if (REKV_CHECK(frame >= 0 && frame < max_frames && l < L, status, 2))
        reps[((long long)l * max_frames + frame) * (Hkv * 128) + h * 128 + threadIdx.x] = __fdiv_rn(s, (float)Nf);
    }
  }
}

// Test helper: one stored page back to plain [H_kv][N_f][128] K and V.
__global__ void unswizzle_page_kernel(const char* __restrict__ page, uint4* __restrict__ k_out,
                                      uint4* __restrict__ v_out, int Hkv, int Nf) {
  const long long n = (long long)Hkv * 2 * Nf * 16;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    int c = (int)(i & 15);
    long long r = i >> 4;
    int t = (int)(r % Nf);
    r /= Nf;
    int kv = (int)(r & 1);
    int h = (int)(r >> 1);
    const char* tile = page + (long long)(h * 2 + kv) * Nf * 256 + (c >> 3) * (long long)Nf * 128;
    uint4 x = *reinterpret_cast<const uint4*>(tile + t * 128 + (((c & 7) ^ (t & 7)) << 4));
    (kv ? v_out : k_out)[((long long)h * Nf + t) * 16 + c] = x;
  }
}

}  // namespace

cudaError_t rekv_launch_append(rekv_ctx* c, const void* k, const void* v, int frame, cudaStream_t st) {
  const StoreView& s = c->sv;
  char* page0 = s.hbm + rekv_hbm_page_offset(s, frame, 0);
  append_pool_kernel<<<s.L * s.Hkv * 2, 256, 0, st>>>((const uint4*)k, (const uint4*)v, page0, s.reps, frame, s.L,
                                                      s.Hkv, s.Nf, s.max_frames, s.page_bytes,
                                                      (long long)(s.tail > 0 ? s.tail : s.max_frames) * s.L * s.page_bytes,
                                                      s.hbm, c->status);
  c->launches += 1;
  return cudaGetLastError();
}

cudaError_t rekv_launch_unswizzle_page(rekv_ctx* c, const char* page, void* k_out, void* v_out, cudaStream_t st) {
  const StoreView& s = c->sv;
  unswizzle_page_kernel<<<32, 256, 0, st>>>(page, (uint4*)k_out, (uint4*)v_out, s.Hkv, s.Nf);
  c->launches += 1;
  return cudaGetLastError();
}
