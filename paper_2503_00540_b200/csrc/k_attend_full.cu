// Eq. 3 in full, the pieces around the attention kernel: O = Attn(W_Q X, [R_k, W_K X], [R_v, W_V X]).
//   - rotary position embedding ("Positional Encoding" paragraph): the retrieved tokens are taken as
//     consecutive tokens, so context token j has position j and token s of X has position n_ctx + s.
//     A table of (cos, sin) per (position, pair) is built once per context in double precision;
//     queries are rotated into a workspace, the context's K tiles into rotated copies (one extra pass
//     over K; the attention kernel then reads K from the copies and V from the pages).
//   - the part of the softmax over the tokens of X itself (causal) is computed by self_attend_kernel as
//     a partial (max, sum, numerator) per output row; the attention kernel's epilogue, or the merge
//     kernel for units cut by a CTA boundary, joins it with the part over R.
// Pairing of dimensions: i with i + 64 (head_dim 128), angle = position * theta^(-2i/128).
#include <algorithm>

#include "ptx_helpers.cuh"
#include "rekv_internal.cuh"

namespace {

using namespace rekv_ptx;

__global__ void rope_table_kernel(float2* __restrict__ tab, int n_pos, double theta) {
  const int i = threadIdx.x & 63;
  const long long pos = (long long)blockIdx.x * (blockDim.x >> 6) + (threadIdx.x >> 6);
  if (pos >= n_pos) return;
  const double angle = (double)pos * pow(theta, -2.0 * (double)i / 128.0);
  double s, c;
  sincos(angle, &s, &c);
  tab[pos * 64 + i] = make_float2((float)c, (float)s);
}

// rotates the 8 pairs (lo[e], hi[e]) held as bf16 in two 16-byte chunks; cs: the pairs' (cos, sin),
// two pairs per float4
__device__ __forceinline__ void rotate_chunk(uint4& lo, uint4& hi, const float4 (&cs)[4]) {
  uint32_t* l = reinterpret_cast<uint32_t*>(&lo);
  uint32_t* h = reinterpret_cast<uint32_t*>(&hi);
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    const float x0 = __uint_as_float(l[w] << 16), x1 = __uint_as_float(l[w] & 0xFFFF0000u);
    const float y0 = __uint_as_float(h[w] << 16), y1 = __uint_as_float(h[w] & 0xFFFF0000u);
    // (x, y) -> (x cos - y sin, y cos + x sin); each product rounded once into the sum
    l[w] = pack_bf16(fmaf(x0, cs[w].x, -y0 * cs[w].y), fmaf(x1, cs[w].z, -y1 * cs[w].w));
    h[w] = pack_bf16(fmaf(y0, cs[w].x, x0 * cs[w].y), fmaf(y1, cs[w].z, x1 * cs[w].w));
  }
}
__device__ __forceinline__ void load_cs(float4 (&cs)[4], const float2* __restrict__ tab_row8) {
  const float4* t = reinterpret_cast<const float4*>(tab_row8);
#pragma unroll
  for (int w = 0; w < 4; ++w) cs[w] = __ldg(t + w);
}
__device__ __forceinline__ void rotate_chunk(uint4& lo, uint4& hi, const float2* __restrict__ tab_row8) {
  float4 cs[4];
  load_cs(cs, tab_row8);
  rotate_chunk(lo, hi, cs);
}

// Position of query row n (global row index in the packed batch): n_ctx + (N_s - N_q) + local index.
__device__ __forceinline__ int find_question(const QBatch& qb, int n) {
  int qi = 0;
  while (qi < qb.nQ - 1 && n >= qb.cu[qi + 1]) ++qi;
  return qi;
}

// grid = (ceil(sum_Nq * H_q / 32), L), 256 threads: 8 threads per (token, head) row, one 16-byte chunk of
// each half per thread
__global__ void __launch_bounds__(256) rope_q_kernel(const uint4* __restrict__ q, uint4* __restrict__ q_rot, QBatch qb,
                                                     QBatch sb, int Hq, int n_ctx_tokens,
                                                     const float2* __restrict__ tab, int layer0) {
  const int l = layer0 + blockIdx.y;
  const int row = blockIdx.x * 32 + (threadIdx.x >> 3), c = threadIdx.x & 7;
  if (row >= qb.sumNq * Hq) return;
  const int n = row / Hq;
  const int qi = find_question(qb, n);
  const int nq = qb.cu[qi + 1] - qb.cu[qi], ns = sb.cu[qi + 1] - sb.cu[qi];
  const int pos = n_ctx_tokens + (ns - nq) + (n - qb.cu[qi]);
  const long long base = ((long long)l * qb.sumNq * Hq + row) * 16;  // 16 chunks of 16 bytes per row
  uint4 lo = q[base + c], hi = q[base + 8 + c];
  rotate_chunk(lo, hi, tab + (long long)pos * 64 + c * 8);
  q_rot[base + c] = lo;
  q_rot[base + 8 + c] = hi;
}

// Rotated copies of the context's K tiles.  grid = (ncf, nQ, L), 256 threads.  A K tile of one KV head is
// two 64-dim halves of [N_f rows][128 B] with 16-byte chunks XOR-swizzled by (row & 7): dimension pair
// (i, i + 64) sits at the same swizzled offset of the two halves, so a thread moves one chunk of each.
__global__ void __launch_bounds__(256) rope_stage_kernel(char* const* __restrict__ tbl, char** __restrict__ tbl_k,
                                                         char* __restrict__ k_rot, int nQ, int ncf, int Hkv, int Nf,
                                                         const float2* __restrict__ tab, int layer0) {
  grid_dep_wait();
  const int slot = blockIdx.x, qi = blockIdx.y, l = layer0 + blockIdx.z;
  const long long e = ((long long)l * nQ + qi) * ncf + slot;
  const char* page = tbl[e];
  const long long half_bytes = (long long)Nf * 128;
  char* dst = k_rot + e * Hkv * 2 * half_bytes;
  if (threadIdx.x == 0) tbl_k[e] = dst;
  // a thread takes (row, chunk) positions and walks the KV heads: the (cos, sin) of a position are loaded
  // once for all heads, and four heads' chunks are in flight before the first rotation
  constexpr int U = 4;
  for (int rc = threadIdx.x; rc < Nf * 8; rc += 256) {
    const int c = rc & 7, r = rc >> 3;
    const long long off = (long long)r * 128 + ((c ^ (r & 7)) << 4);
    float4 cs[4];
    load_cs(cs, tab + ((long long)slot * Nf + r) * 64 + c * 8);
    for (int g0 = 0; g0 < Hkv; g0 += U) {
      uint4 lo[U], hi[U];
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (g0 + u < Hkv) {
          const char* src = page + (long long)(g0 + u) * 4 * half_bytes + off;  // the page holds K then V of each KV head
          lo[u] = __ldcs(reinterpret_cast<const uint4*>(src));
          hi[u] = __ldcs(reinterpret_cast<const uint4*>(src + half_bytes));
        }
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (g0 + u < Hkv) {
          rotate_chunk(lo[u], hi[u], cs);
          char* d = dst + (long long)(g0 + u) * 2 * half_bytes + off;
          *reinterpret_cast<uint4*>(d) = lo[u];
          *reinterpret_cast<uint4*>(d + half_bytes) = hi[u];
        }
    }
  }
}

// The softmax part over the tokens of X (causal), on the tensor cores with mma.sync m16n8k16.
// grid = (128-row blocks of the longest question, H_q, L * nQ), 256 threads: a warp owns 16 query rows
// (tokens of the question, one head) and walks X's keys in tiles of 64; the KV head's K (rotated on the
// way in) and V tiles sit in shared memory in the pages' layout -- two 64-dim halves of [64 rows][128 B]
// with the 16-byte chunks XOR-swizzled by (row & 7) -- so ldmatrix reads them without bank conflicts.
// Row n of a question (token N_s - N_q + n of X) sees keys 0 .. N_s - N_q + n.  Writes, per output row,
// the numerator (unnormalised, relative to the row maximum) and (max, sum), log2 domain.
constexpr int SELF_TILE = 64;
__global__ void __launch_bounds__(256) self_attend_kernel(const __nv_bfloat16* __restrict__ q,
                                                          const __nv_bfloat16* __restrict__ k_self,
                                                          const __nv_bfloat16* __restrict__ v_self, QBatch qb, QBatch sb,
                                                          int Hq, int Hkv, int G, int n_ctx_tokens,
                                                          const float2* __restrict__ tab, float scale_log2,
                                                          float* __restrict__ self_o, float* __restrict__ self_ml,
                                                          int layer0) {
  __shared__ __align__(128) unsigned char s_kv[2 * 2 * SELF_TILE * 128];  // K tile, V tile
  const int rb = blockIdx.x, h = blockIdx.y;
  const int l = layer0 + blockIdx.z / qb.nQ, qi = blockIdx.z % qb.nQ;
  const int g = h / G;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int q0 = qb.cu[qi], nq = qb.cu[qi + 1] - q0;
  const int s0 = sb.cu[qi], ns = sb.cu[qi + 1] - s0;
  if (rb * 128 >= nq) return;
  const uint32_t sK = smem_u32(s_kv), sV = sK + 2 * SELF_TILE * 128;
  constexpr uint32_t half_stride = SELF_TILE * 128;

  // this thread's two rows (fragment layout of m16n8k16: rows lane/4 and lane/4 + 8 of the warp's 16)
  const int n_lo = rb * 128 + warp * 16 + (lane >> 2), n_hi = n_lo + 8;
  const bool v_lo = n_lo < nq, v_hi = n_hi < nq;
  const long long row_lo = ((long long)l * qb.sumNq + q0 + (v_lo ? n_lo : 0)) * Hq + h;
  const long long row_hi = ((long long)l * qb.sumNq + q0 + (v_hi ? n_hi : 0)) * Hq + h;
  uint32_t qf[8][4];
  {
    const uint32_t* plo = reinterpret_cast<const uint32_t*>(q + row_lo * 128);
    const uint32_t* phi = reinterpret_cast<const uint32_t*>(q + row_hi * 128);
#pragma unroll
    for (int kb = 0; kb < 8; ++kb) {
      const int w = kb * 8 + (lane & 3);
      qf[kb][0] = v_lo ? __ldg(plo + w) : 0u;
      qf[kb][1] = v_hi ? __ldg(phi + w) : 0u;
      qf[kb][2] = v_lo ? __ldg(plo + w + 4) : 0u;
      qf[kb][3] = v_hi ? __ldg(phi + w + 4) : 0u;
    }
  }
  const int last_lo = ns - nq + n_lo, last_hi = ns - nq + n_hi;        // last key each row sees
  const int last_cta = ns - nq + min(rb * 128 + 127, nq - 1);          // ... and the row block
  const int last_warp = ns - nq + min(rb * 128 + warp * 16 + 15, nq - 1);
  float oacc[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  const int lm = lane >> 3, lr = lane & 7;

  for (int t0 = 0; t0 <= last_cta; t0 += SELF_TILE) {
    __syncthreads();  // the previous tile has been read by every warp
    // K and V rows t0 .. t0+63 of X (zero beyond N_s): 8 threads per row, chunk c of each half per thread
    for (int it = tid; it < SELF_TILE * 8; it += 256) {
      const int c = it & 7, r = it >> 3;
      const int s = t0 + r;
      uint4 klo = make_uint4(0, 0, 0, 0), khi = klo, vlo = klo, vhi = klo;
      if (s < ns) {
        const long long base = (((long long)l * sb.sumNq + s0 + s) * Hkv + g) * 16;  // 16-byte chunks
        const uint4* ks = reinterpret_cast<const uint4*>(k_self) + base;
        const uint4* vs = reinterpret_cast<const uint4*>(v_self) + base;
        klo = __ldg(ks + c);
        khi = __ldg(ks + 8 + c);
        vlo = __ldg(vs + c);
        vhi = __ldg(vs + 8 + c);
        if (tab) rotate_chunk(klo, khi, tab + (long long)(n_ctx_tokens + s) * 64 + c * 8);
      }
      const uint32_t off = r * 128 + ((c ^ (r & 7)) << 4);
      *reinterpret_cast<uint4*>(s_kv + off) = klo;
      *reinterpret_cast<uint4*>(s_kv + half_stride + off) = khi;
      *reinterpret_cast<uint4*>(s_kv + 2 * half_stride + off) = vlo;
      *reinterpret_cast<uint4*>(s_kv + 3 * half_stride + off) = vhi;
    }
    __syncthreads();
    if (t0 > last_warp) continue;  // nothing of this tile is visible to this warp's rows (warp-uniform)
    float sacc[8][4];
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
      sacc[nb][0] = sacc[nb][1] = sacc[nb][2] = sacc[nb][3] = 0.f;
      const int tok = nb * 8 + lr;
#pragma unroll
      for (int kp = 0; kp < 4; ++kp) {
        const int c = kp * 4 + lm;
        const uint32_t addr = sK + (c >> 3) * half_stride + tok * 128 + (((c & 7) ^ (tok & 7)) << 4);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(b0, b1, b2, b3, addr);
        mma_bf16_16816(sacc[nb], qf[2 * kp], b0, b1);
        mma_bf16_16816(sacc[nb], qf[2 * kp + 1], b2, b3);
      }
    }
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
      const int col = t0 + nb * 8 + (lane & 3) * 2;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = col + (e & 1);
        const int last = (e < 2) ? last_lo : last_hi;
        sacc[nb][e] = key <= last ? sacc[nb][e] * scale_log2 : -INFINITY;  // causal (covers keys beyond N_s too)
      }
      mx_lo = fmaxf(mx_lo, fmaxf(sacc[nb][0], sacc[nb][1]));
      mx_hi = fmaxf(mx_hi, fmaxf(sacc[nb][2], sacc[nb][3]));
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    // a row that sees nothing of this tile keeps its state (its maximum stays where it was)
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    const float a_lo = mn_lo == -INFINITY ? 1.f : ex2(m_lo - mn_lo), a_hi = mn_hi == -INFINITY ? 1.f : ex2(m_hi - mn_hi);
    const float sub_lo = mn_lo == -INFINITY ? 0.f : mn_lo, sub_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
    m_lo = mn_lo;
    m_hi = mn_hi;
    l_lo *= a_lo;
    l_hi *= a_hi;
#pragma unroll
    for (int nd = 0; nd < 16; ++nd) {
      oacc[nd][0] *= a_lo;
      oacc[nd][1] *= a_lo;
      oacc[nd][2] *= a_hi;
      oacc[nd][3] *= a_hi;
    }
    uint32_t pf[8][2];
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
      const float p0 = ex2(sacc[nb][0] - sub_lo), p1 = ex2(sacc[nb][1] - sub_lo);
      const float p2 = ex2(sacc[nb][2] - sub_hi), p3 = ex2(sacc[nb][3] - sub_hi);
      l_lo += p0 + p1;
      l_hi += p2 + p3;
      pf[nb][0] = pack_bf16(p0, p1);
      pf[nb][1] = pack_bf16(p2, p3);
    }
#pragma unroll
    for (int kb = 0; kb < 4; ++kb) {
      const uint32_t a[4] = {pf[2 * kb][0], pf[2 * kb][1], pf[2 * kb + 1][0], pf[2 * kb + 1][1]};
      const int tok = kb * 16 + (lm & 1) * 8 + lr;
#pragma unroll
      for (int dp = 0; dp < 8; ++dp) {
        const int c = dp * 2 + (lm >> 1);
        const uint32_t addr = sV + (c >> 3) * half_stride + tok * 128 + (((c & 7) ^ (tok & 7)) << 4);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(b0, b1, b2, b3, addr);
        mma_bf16_16816(oacc[2 * dp], a, b0, b1);
        mma_bf16_16816(oacc[2 * dp + 1], a, b2, b3);
      }
    }
  }
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
#pragma unroll
  for (int nd = 0; nd < 16; ++nd) {
    const int d = nd * 8 + (lane & 3) * 2;
    if (v_lo) *reinterpret_cast<float2*>(self_o + row_lo * 128 + d) = make_float2(oacc[nd][0], oacc[nd][1]);
    if (v_hi) *reinterpret_cast<float2*>(self_o + row_hi * 128 + d) = make_float2(oacc[nd][2], oacc[nd][3]);
  }
  if ((lane & 3) == 0) {
    if (v_lo) {
      self_ml[row_lo * 2] = m_lo;
      self_ml[row_lo * 2 + 1] = l_lo;
    }
    if (v_hi) {
      self_ml[row_hi * 2] = m_hi;
      self_ml[row_hi * 2 + 1] = l_hi;
    }
  }
}

// No retrieved context at all (nothing visible but X): the output is the normalised self part.
__global__ void __launch_bounds__(256) self_finalize_kernel(const float* __restrict__ self_o,
                                                            const float* __restrict__ self_ml,
                                                            __nv_bfloat16* __restrict__ out, long long row0,
                                                            long long rows) {
  const long long row = row0 + (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= row0 + rows) return;
  const float l = self_ml[row * 2 + 1];
  const float inv = l > 0.f ? 1.f / l : 0.f;
  const float4 o = *reinterpret_cast<const float4*>(self_o + row * 128 + lane * 4);
  uint2 packed;
  packed.x = pack_bf16(o.x * inv, o.y * inv);
  packed.y = pack_bf16(o.z * inv, o.w * inv);
  *reinterpret_cast<uint2*>(out + row * 128 + lane * 4) = packed;
}

}  // namespace

cudaError_t rekv_launch_rope_table(rekv_ctx* c, cudaStream_t st) {
  rope_table_kernel<<<(c->rope_positions + 3) / 4, 256, 0, st>>>(c->rope_tab, c->rope_positions,
                                                                (double)c->cfg.rope_theta);
  return cudaGetLastError();
}

// What the attention kernel needs for Eq. 3 in full, in two halves.
// First half, independent of the retrieval: rotated queries (with rotary embedding) and the partial over the tokens
// of X.  Layers [layer0, layer1): q, k_self, v_self are indexed with the absolute layer (a caller that holds one
// layer's rows passes pointers moved back by layer0 layers), as the library's own buffers are.  The part over X
// (latency-bound) goes to the internal stream when something runs beside it on the caller's: the pass over the
// context's keys (consecutive positions), or -- early -- the layer's retrieval kernels.
cudaError_t rekv_launch_attend_full_self(rekv_ctx* c, const void* q, const void* k_self, const void* v_self,
                                         const QBatch& qb, const QBatch& sb, int ncf, cudaStream_t st, int layer0,
                                         int layer1, bool early) {
  const StoreView& s = c->sv;
  const int nl = layer1 - layer0;
  const bool rope = c->cfg.rope_theta > 0.f;
  // positions: context token j at j and token s of X at n_ctx + s; with REKV_FLAG_ROPE_STATIC every context token
  // at 0 -- its rotation is the identity, the stored keys are used as they are -- and token s of X at 1 + s
  const bool static_ctx = rope && (c->cfg.flags & REKV_FLAG_ROPE_STATIC) != 0;
  const int n_ctx_tokens = static_ctx ? 1 : ncf * s.Nf;   // position of X's first token
  const __nv_bfloat16* q_eff = (const __nv_bfloat16*)q;
  if (rope) {
    dim3 grid((qb.sumNq * s.Hq + 31) / 32, nl);
    rope_q_kernel<<<grid, 256, 0, st>>>((const uint4*)q, (uint4*)c->q_rot, qb, sb, s.Hq, n_ctx_tokens, c->rope_tab,
                                        layer0);
    c->launches += 1;
    q_eff = c->q_rot;
  }
  const bool fork = (rope && !static_ctx && ncf > 0) || early;
  cudaStream_t st_self = fork ? c->side : st;
  cudaError_t e;
  if (fork) {
    if ((e = cudaEventRecord(c->ev_main, st)) != cudaSuccess) return e;
    if ((e = cudaStreamWaitEvent(c->side, c->ev_main, 0)) != cudaSuccess) return e;
  }
  int max_nq = 1;
  for (int i = 0; i < qb.nQ; ++i) max_nq = std::max(max_nq, qb.cu[i + 1] - qb.cu[i]);
  self_attend_kernel<<<dim3((max_nq + 127) / 128, s.Hq, nl * qb.nQ), 256, 0, st_self>>>(
      q_eff, (const __nv_bfloat16*)k_self, (const __nv_bfloat16*)v_self, qb, sb, s.Hq, s.Hkv, s.G, n_ctx_tokens,
      rope ? c->rope_tab : nullptr, 1.4426950408889634f / sqrtf(128.f), c->self_o, c->self_ml, layer0);
  c->launches += 1;
  if (fork && (e = cudaEventRecord(c->ev_side, c->side)) != cudaSuccess) return e;
  c->self_forked = fork;
  return cudaGetLastError();
}

// Second half, after the context table is there: rotated copies of the context's keys (consecutive positions), and
// the join with the part over X if that went to the internal stream.
cudaError_t rekv_launch_attend_full_ctx(rekv_ctx* c, const QBatch& qb, int ncf, cudaStream_t st, int layer0,
                                        int layer1) {
  const StoreView& s = c->sv;
  const bool rope = c->cfg.rope_theta > 0.f;
  const bool static_ctx = rope && (c->cfg.flags & REKV_FLAG_ROPE_STATIC) != 0;
  if (rope && !static_ctx && ncf > 0) {
    rope_stage_kernel<<<dim3(ncf, qb.nQ, layer1 - layer0), 256, 0, st>>>(c->ctx_tbl, c->tbl_k, c->k_rot, qb.nQ, ncf,
                                                                        s.Hkv, s.Nf, c->rope_tab, layer0);
    c->launches += 1;
  }
  if (c->self_forked) {
    c->self_forked = false;
    cudaError_t e = cudaStreamWaitEvent(st, c->ev_side, 0);
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

cudaError_t rekv_launch_self_finalize(rekv_ctx* c, const QBatch& qb, void* out, cudaStream_t st, int layer0,
                                      int layer1) {
  const long long per_layer = (long long)qb.sumNq * c->sv.Hq, rows = (layer1 - layer0) * per_layer;
  self_finalize_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(c->self_o, c->self_ml, (__nv_bfloat16*)out,
                                                                   layer0 * per_layer, rows);
  c->launches += 1;
  return cudaGetLastError();
}
