// Step 4: bring the retrieved frames' K/V together as the context R of every (layer, question).
//
// The context is a table of page pointers (selected frames in list order, then the recent window).
// Pages resident in HBM are referenced in place; pages that live only in pinned host memory are
// pulled over the host link into an HBM staging page by the same kernel (zero-copy reads of the
// mapped pinned arena, 16 bytes per load, many loads in flight).  A second kernel can write the
// context out contiguously in plain [token][dim] layout.
#include <cuda_fp8.h>

#include "ptx_helpers.cuh"
#include "rekv_internal.cuh"

namespace {

constexpr int PULL_PARTS_HOST = 8;  // CTAs per page when pages may have to cross the host link

// ---- FP8 host tier -----------------------------------------------------------------------------
// Groups of 16 codes [g0, g1) of one host page -> bf16 in the swizzled page layout at dst.  A group is 16
// consecutive dims of one row: two 16-byte chunks of the destination.  The rows' scales are staged in
// shared memory first (coalesced reads of the scale block instead of one small host read per thread).
__device__ __forceinline__ void dequant_groups(const char* __restrict__ src, char* __restrict__ dst, int Hkv, int Nf,
                                               long long g0, long long g1, float* s_scale) {
  const float* scales = reinterpret_cast<const float*>(src + (long long)Hkv * 2 * Nf * 128);
  const long long r0 = g0 >> 3, r1 = (g1 + 7) >> 3;  // rows (tile-major) touched by this range
  for (long long r = r0 + threadIdx.x; r < r1; r += blockDim.x) s_scale[r - r0] = __ldcs(scales + r);
  __syncthreads();
  const uint4* s4 = reinterpret_cast<const uint4*>(src);
  for (long long g = g0 + threadIdx.x; g < g1; g += blockDim.x) {
    const uint4 codes = __ldcs(s4 + g);
    const long long row = g >> 3;
    const int k = (int)(g & 7);                 // dims [16k, 16k + 16)
    const int tile = (int)(row / Nf), r = (int)(row - (long long)tile * Nf);
    const float sc = s_scale[row - r0];
    const unsigned char* cb = reinterpret_cast<const unsigned char*>(&codes);
    uint32_t w[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float lo = __half2float(__half(__nv_cvt_fp8_to_halfraw(cb[2 * e], __NV_E4M3))) * sc;
      const float hi = __half2float(__half(__nv_cvt_fp8_to_halfraw(cb[2 * e + 1], __NV_E4M3))) * sc;
      w[e] = rekv_ptx::pack_bf16(lo, hi);
    }
    char* base = dst + (long long)tile * Nf * 256 + (long long)(k >> 2) * Nf * 128 + (long long)r * 128;
    const int c0 = (2 * k) & 7;
    *reinterpret_cast<uint4*>(base + ((c0 ^ (r & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
    *reinterpret_cast<uint4*>(base + (((c0 + 1) ^ (r & 7)) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
  }
}
constexpr int DEQ_MAX_ROWS = 2048;  // rows of scales a CTA stages (H_kv * 2 * N_f <= 8 * 2 * 208 = 3328 per page, / parts)

// grid = (layers, H_kv * 2 tiles): the ring slot's bf16 pages of one frame -> the frame's FP8 form.
// Eight threads per row (16 dims each); the row maximum comes from three shuffles among them.
__global__ void __launch_bounds__(256) quantize_frame_kernel(const char* __restrict__ pages, char* __restrict__ q8,
                                                             long long page_bytes, long long host_page_bytes, int Hkv,
                                                             int Nf) {
  const int l = blockIdx.x, tile = blockIdx.y;
  const char* page = pages + (long long)l * page_bytes + (long long)tile * Nf * 256;
  char* out = q8 + (long long)l * host_page_bytes;
  float* scales = reinterpret_cast<float*>(out + (long long)Hkv * 2 * Nf * 128);
  const int k = threadIdx.x & 7;
  constexpr int U = 4;  // rows per thread in flight: all their loads are issued before the first reduction
  for (int r0 = 0; r0 < Nf; r0 += 32 * U) {
    uint4 a[U], b[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int r = r0 + u * 32 + (threadIdx.x >> 3);
      a[u] = make_uint4(0, 0, 0, 0);
      b[u] = a[u];
      if (r < Nf) {
        const char* base = page + (long long)(k >> 2) * Nf * 128 + (long long)r * 128;
        const int c0 = (2 * k) & 7;
        a[u] = __ldcs(reinterpret_cast<const uint4*>(base + ((c0 ^ (r & 7)) << 4)));
        b[u] = __ldcs(reinterpret_cast<const uint4*>(base + (((c0 + 1) ^ (r & 7)) << 4)));
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int r = r0 + u * 32 + (threadIdx.x >> 3);
      const uint32_t w[8] = {a[u].x, a[u].y, a[u].z, a[u].w, b[u].x, b[u].y, b[u].z, b[u].w};
      float v[16];
      float amax = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        v[2 * e] = __uint_as_float(w[e] << 16);
        v[2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
        amax = fmaxf(amax, fmaxf(fabsf(v[2 * e]), fabsf(v[2 * e + 1])));
      }
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 4));
      const float sc = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
      uint4 codes;
      unsigned char* cb = reinterpret_cast<unsigned char*>(&codes);
#pragma unroll
      for (int e = 0; e < 16; ++e) cb[e] = __nv_cvt_float_to_fp8(__fdiv_rn(v[e], sc), __NV_SATFINITE, __NV_E4M3);
      if (r < Nf) {
        *reinterpret_cast<uint4*>(out + ((long long)tile * Nf + r) * 128 + k * 16) = codes;
        if (k == 0) scales[(long long)tile * Nf + r] = sc;
      }
    }
  }
}

// one host page -> one bf16 page (test helper path); grid = parts
__global__ void __launch_bounds__(256) dequant_page_kernel(const char* __restrict__ src, char* __restrict__ dst, int Hkv,
                                                           int Nf) {
  __shared__ float s_scale[DEQ_MAX_ROWS];
  const long long n16 = (long long)Hkv * 2 * Nf * 8;
  const long long per = ((n16 + gridDim.x - 1) / gridDim.x + 7) & ~7ll;
  const long long g0 = blockIdx.x * per, g1 = min(g0 + per, n16);
  if (g0 < g1) dequant_groups(src, dst, Hkv, Nf, g0, g1, s_scale);
}

// grid = (ncf * parts, nQ, layer1 - layer0)
__global__ void __launch_bounds__(256) page_table_pull_kernel(StoreView s, const int32_t* __restrict__ idx, int nQ,
                                                              int top_k, int k_eff, int ncf, int n_visible,
                                                              int layer0, int frames_now, int parts, char** __restrict__ tbl,
                                                              int* __restrict__ status,
                                                              unsigned long long* __restrict__ link_bytes) {
  const int j = blockIdx.x / parts, part = blockIdx.x % parts;
  const int qi = blockIdx.y, l = layer0 + blockIdx.z;
  rekv_ptx::grid_dep_wait();
  rekv_ptx::grid_dep_launch();
  int frame;
  if (j < k_eff)
    frame = idx[((long long)l * nQ + qi) * top_k + j];
  else
    frame = n_visible - (ncf - k_eff) + (j - k_eff);
  if (frame < 0 || frame >= n_visible) {
    if (threadIdx.x == 0 && part == 0) atomicExch(status, REKV_ERR_ARG);
    frame = 0;
  }
  const long long slot = ((long long)l * nQ + qi) * ncf + j;
  char* page;
  bool pull = false, from_ring = false;
  if (s.tail == 0) {
    page = s.hbm + rekv_hbm_page_offset(s, frame, l);
  } else {
    // Offloaded context: the context owns its bytes.  A frame that is still in the HBM ring is copied into the
    // staging page as well (HBM to HBM), because the ring slot is recycled by a later append while the context --
    // decode steps reuse it -- must stay what it was at gather time.
    page = s.staging + slot * s.page_bytes;
    pull = true;
    from_ring = frame >= frames_now - s.tail;
  }
  if (threadIdx.x == 0 && part == 0) {
    tbl[slot] = page;
    if (pull && !from_ring) atomicAdd(link_bytes, (unsigned long long)s.host_page_bytes);
  }
  if (!pull) return;
  const char* src = from_ring ? s.hbm + rekv_hbm_page_offset(s, frame, l)
                              : s.host_arenas[frame / s.frames_per_arena] +
                                    ((long long)(frame % s.frames_per_arena) * s.L + l) * s.host_page_bytes;
  if (s.host_fp8 && !from_ring) {  // codes and scales cross the link; the staging page receives bf16
    __shared__ float s_scale[DEQ_MAX_ROWS];
    const long long g16 = (long long)s.Hkv * 2 * s.Nf * 8;
    const long long gper = ((g16 + parts - 1) / parts + 7) & ~7ll;  // whole rows per part
    const long long g0 = part * gper, g1 = min(g0 + gper, g16);
    if (g0 < g1) dequant_groups(src, page, s.Hkv, s.Nf, g0, g1, s_scale);
    return;
  }
  const long long n16 = s.page_bytes >> 4;
  const long long per = (n16 + parts - 1) / parts;
  const long long i0 = part * per, i1 = min(i0 + per, n16);
  const uint4* s4 = reinterpret_cast<const uint4*>(src);
  uint4* d4 = reinterpret_cast<uint4*>(page);
  long long i = i0 + threadIdx.x;
  for (; i + 3 * 256 < i1; i += 4 * 256) {
    uint4 a = __ldcs(s4 + i), b = __ldcs(s4 + i + 256), c = __ldcs(s4 + i + 512), d = __ldcs(s4 + i + 768);
    d4[i] = a;
    d4[i + 256] = b;
    d4[i + 512] = c;
    d4[i + 768] = d;
  }
  for (; i < i1; i += 256) d4[i] = __ldcs(s4 + i);
}

// grid = (ncf, nQ, L): context page j of (layer, question) -> rows [j*Nf, (j+1)*Nf) of the plain
// [H_kv][n_ctx][128] K and V buffers.
__global__ void __launch_bounds__(256) materialize_kernel(char* const* __restrict__ tbl, int nQ, int ncf, int Hkv,
                                                          int Nf, uint4* __restrict__ k_ctx,
                                                          uint4* __restrict__ v_ctx) {
  const int j = blockIdx.x, qi = blockIdx.y, l = blockIdx.z;
  const long long slot = ((long long)l * nQ + qi) * ncf + j;
  const char* page = tbl[slot];
  const long long n_ctx = (long long)ncf * Nf;
  const int n = Hkv * 2 * Nf * 16;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    int c = i & 15;
    int r = i >> 4;
    int t = r % Nf;
    r /= Nf;
    int kv = r & 1, h = r >> 1;
    const char* tile = page + (long long)(h * 2 + kv) * Nf * 256 + (c >> 3) * (long long)Nf * 128;
    uint4 x = *reinterpret_cast<const uint4*>(tile + t * 128 + (((c & 7) ^ (t & 7)) << 4));
    uint4* dst = kv ? v_ctx : k_ctx;
    dst[((((long long)l * nQ + qi) * Hkv + h) * n_ctx + (long long)j * Nf + t) * 16 + c] = x;
  }
}

}  // namespace

cudaError_t rekv_launch_page_table(rekv_ctx* c, const int32_t* idx, int nQ, int top_k, const CtxGeom& geom,
                                   int n_visible, int layer0, int layer1, int frames_now, cudaStream_t st) {
  const int k_eff = geom.k_eff, ncf = geom.ncf;
  if (ncf <= 0 || layer1 <= layer0) return cudaSuccess;
  const int parts = c->sv.tail > 0 ? PULL_PARTS_HOST : 1;
  dim3 grid(ncf * parts, nQ, layer1 - layer0);
  c->launches += 1;
  if (c->sv.tail == 0)
    return rekv_launch_pdl(page_table_pull_kernel, grid, dim3(256), 0, st, c->sv, idx, nQ, top_k, k_eff, ncf, n_visible,
                           layer0, frames_now, parts, c->ctx_tbl, c->status, c->link_bytes);
  page_table_pull_kernel<<<grid, 256, 0, st>>>(c->sv, idx, nQ, top_k, k_eff, ncf, n_visible, layer0, frames_now,
                                               parts, c->ctx_tbl, c->status, c->link_bytes);
  return cudaGetLastError();
}

cudaError_t rekv_launch_quantize_frame(rekv_ctx* c, int frame, cudaStream_t st) {
  const StoreView& s = c->sv;
  const int slot = frame % s.tail;
  quantize_frame_kernel<<<dim3(s.L, s.Hkv * 2), 256, 0, st>>>(s.hbm + rekv_hbm_page_offset(s, frame, 0),
                                                            s.q8_ring + (long long)slot * s.L * s.host_page_bytes,
                                                            s.page_bytes, s.host_page_bytes, s.Hkv, s.Nf);
  c->launches += 1;
  return cudaGetLastError();
}

cudaError_t rekv_launch_dequant_page(rekv_ctx* c, const char* host_page, char* dst_page, cudaStream_t st) {
  dequant_page_kernel<<<8, 256, 0, st>>>(host_page, dst_page, c->sv.Hkv, c->sv.Nf);
  c->launches += 1;
  return cudaGetLastError();
}

cudaError_t rekv_launch_materialize(rekv_ctx* c, int nQ, int ncf, void* k_ctx, void* v_ctx, cudaStream_t st) {
  if (ncf <= 0) return cudaSuccess;
  materialize_kernel<<<dim3(ncf, nQ, c->sv.L), 256, 0, st>>>(c->ctx_tbl, nQ, ncf, c->sv.Hkv, c->sv.Nf, (uint4*)k_ctx,
                                                            (uint4*)v_ctx);
  c->launches += 1;
  return cudaGetLastError();
}
