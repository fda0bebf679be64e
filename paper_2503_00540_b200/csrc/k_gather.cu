// Step 4: bring the retrieved frames' K/V together as the context R of every (layer, question).
//
// The context is a table of page pointers (selected frames in list order, then the recent window).
// Pages resident in HBM are referenced in place; pages that live only in pinned host memory are
// pulled over the host link into an HBM staging page by the same kernel (zero-copy reads of the
// mapped pinned arena, 16 bytes per load, many loads in flight).  A second kernel can write the
// context out contiguously in plain [token][dim] layout.
#include "ptx_helpers.cuh"
#include "rekv_internal.cuh"

namespace {

constexpr int PULL_PARTS_HOST = 8;  // CTAs per page when pages may have to cross the host link

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
  bool pull = false;
  if (s.tail == 0) {
    page = s.hbm + rekv_hbm_page_offset(s, frame, l);
  } else if (frame >= frames_now - s.tail) {
    page = s.hbm + rekv_hbm_page_offset(s, frame, l);
  } else {
    page = s.staging + slot * s.page_bytes;
    pull = true;
  }
  if (threadIdx.x == 0 && part == 0) {
    tbl[slot] = page;
    if (pull) atomicAdd(link_bytes, (unsigned long long)s.page_bytes);
  }
  if (!pull) return;
  const char* src = s.host_arenas[frame / s.frames_per_arena] +
                    ((long long)(frame % s.frames_per_arena) * s.L + l) * s.page_bytes;
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

cudaError_t rekv_launch_materialize(rekv_ctx* c, int nQ, int ncf, void* k_ctx, void* v_ctx, cudaStream_t st) {
  if (ncf <= 0) return cudaSuccess;
  materialize_kernel<<<dim3(ncf, nQ, c->sv.L), 256, 0, st>>>(c->ctx_tbl, nQ, ncf, c->sv.Hkv, c->sv.Nf, (uint4*)k_ctx,
                                                            (uint4*)v_ctx);
  c->launches += 1;
  return cudaGetLastError();
}
