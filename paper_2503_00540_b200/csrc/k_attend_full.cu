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
                                                     const float2* __restrict__ tab) {
  const int l = blockIdx.y;
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
                                                         const float2* __restrict__ tab) {
  grid_dep_wait();
  const int slot = blockIdx.x, qi = blockIdx.y, l = blockIdx.z;
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

// The softmax part over the tokens of X.  grid = (H_q, nQ, L), 256 threads; the CTA holds the KV head's
// keys (rotated on the way in) and values of one 64-token tile of X in shared memory, a warp walks the
// question's query rows of this head: lane s scores key s (and s + 32), the row's running (max, sum) and
// its numerator (4 dims per lane) are combined across tiles through the output arrays (same warp, same
// row, so no other thread touches them).  Writes self_o (unnormalised, relative to the max) and self_ml.
constexpr int SELF_TILE = 64;
__global__ void __launch_bounds__(256) self_attend_kernel(const __nv_bfloat16* __restrict__ q,
                                                          const __nv_bfloat16* __restrict__ k_self,
                                                          const __nv_bfloat16* __restrict__ v_self, QBatch qb, QBatch sb,
                                                          int Hq, int Hkv, int G, int n_ctx_tokens,
                                                          const float2* __restrict__ tab, float scale_log2,
                                                          float* __restrict__ self_o, float* __restrict__ self_ml) {
  __shared__ uint32_t s_k[SELF_TILE][65];  // bf16 pairs; the odd row pitch keeps lane-per-key reads conflict-free
  __shared__ uint2 s_v[SELF_TILE][32];     // 4 bf16 per lane
  __shared__ float s_q[8][128];
  const int h = blockIdx.x, qi = blockIdx.y, l = blockIdx.z;
  const int g = h / G;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = qb.cu[qi], nq = qb.cu[qi + 1] - q0;
  const int s0 = sb.cu[qi], ns = sb.cu[qi + 1] - s0;
  for (int t0 = 0; t0 < ns; t0 += SELF_TILE) {
    const int nt = min(SELF_TILE, ns - t0);
    __syncthreads();
    // keys: 8 threads per token, a 16-byte chunk of each half, rotated at position n_ctx + token
    for (int it = threadIdx.x; it < nt * 8; it += 256) {
      const int c = it & 7, s = it >> 3;
      const uint4* src = reinterpret_cast<const uint4*>(k_self + (((long long)l * sb.sumNq + s0 + t0 + s) * Hkv + g) * 128);
      uint4 lo = src[c], hi = src[8 + c];
      if (tab) rotate_chunk(lo, hi, tab + (long long)(n_ctx_tokens + t0 + s) * 64 + c * 8);
      const uint32_t* a = reinterpret_cast<const uint32_t*>(&lo);
      const uint32_t* b = reinterpret_cast<const uint32_t*>(&hi);
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        s_k[s][c * 4 + w] = a[w];
        s_k[s][32 + c * 4 + w] = b[w];
      }
    }
    for (int it = threadIdx.x; it < nt * 32; it += 256) {
      const int s = it >> 5, d4 = it & 31;
      s_v[s][d4] = *reinterpret_cast<const uint2*>(v_self + (((long long)l * sb.sumNq + s0 + t0 + s) * Hkv + g) * 128 + d4 * 4);
    }
    __syncthreads();
    for (int n = warp; n < nq; n += 8) {
      const int last = ns - nq + n;  // the last token of X this row sees
      if (last < t0) continue;       // (warp-uniform)
      const long long out_row = ((long long)l * qb.sumNq + q0 + n) * Hq + h;
      __syncwarp();
      {
        const uint2 qv = *reinterpret_cast<const uint2*>(q + out_row * 128 + lane * 4);
        s_q[warp][lane * 4] = __uint_as_float(qv.x << 16);
        s_q[warp][lane * 4 + 1] = __uint_as_float(qv.x & 0xFFFF0000u);
        s_q[warp][lane * 4 + 2] = __uint_as_float(qv.y << 16);
        s_q[warp][lane * 4 + 3] = __uint_as_float(qv.y & 0xFFFF0000u);
      }
      __syncwarp();
      float sc[2];
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int s = half * 32 + lane;
        float a0 = 0.f, a1 = 0.f;
        if (s < nt) {
#pragma unroll 16
          for (int w = 0; w < 64; ++w) {
            const uint32_t kk = s_k[s][w];
            a0 = fmaf(s_q[warp][2 * w], __uint_as_float(kk << 16), a0);
            a1 = fmaf(s_q[warp][2 * w + 1], __uint_as_float(kk & 0xFFFF0000u), a1);
          }
        }
        sc[half] = (s < nt && t0 + s <= last) ? (a0 + a1) * scale_log2 : -INFINITY;
      }
      float m_t = fmaxf(sc[0], sc[1]);
      for (int o = 16; o; o >>= 1) m_t = fmaxf(m_t, __shfl_xor_sync(0xffffffffu, m_t, o));
      float m_old = -INFINITY, l_old = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      if (t0 > 0) {
        m_old = self_ml[out_row * 2];
        l_old = self_ml[out_row * 2 + 1];
        acc = *reinterpret_cast<const float4*>(self_o + out_row * 128 + lane * 4);
      }
      const float m_new = fmaxf(m_old, m_t);  // finite: the row sees at least one token of this or an earlier tile
      const float w_old = ex2(m_old - m_new);
      const float p0 = ex2(sc[0] - m_new), p1 = ex2(sc[1] - m_new);
      float l_t = p0 + p1;
      for (int o = 16; o; o >>= 1) l_t += __shfl_xor_sync(0xffffffffu, l_t, o);
      acc.x *= w_old;
      acc.y *= w_old;
      acc.z *= w_old;
      acc.w *= w_old;
      const int n_seen = min(nt, last - t0 + 1);
      for (int s = 0; s < n_seen; ++s) {
        const float pv = __shfl_sync(0xffffffffu, s < 32 ? p0 : p1, s & 31);
        const uint2 vv = s_v[s][lane];
        acc.x = fmaf(pv, __uint_as_float(vv.x << 16), acc.x);
        acc.y = fmaf(pv, __uint_as_float(vv.x & 0xFFFF0000u), acc.y);
        acc.z = fmaf(pv, __uint_as_float(vv.y << 16), acc.z);
        acc.w = fmaf(pv, __uint_as_float(vv.y & 0xFFFF0000u), acc.w);
      }
      *reinterpret_cast<float4*>(self_o + out_row * 128 + lane * 4) = acc;
      if (lane == 0) {
        self_ml[out_row * 2] = m_new;
        self_ml[out_row * 2 + 1] = l_old * w_old + l_t;
      }
    }
  }
}

// No retrieved context at all (nothing visible but X): the output is the normalised self part.
__global__ void __launch_bounds__(256) self_finalize_kernel(const float* __restrict__ self_o,
                                                            const float* __restrict__ self_ml,
                                                            __nv_bfloat16* __restrict__ out, long long rows) {
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
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

// Everything the attention kernel needs for Eq. 3 in full: rotated queries and K copies (with rotary
// embedding) and the partial over the tokens of X.  q_eff receives the query pointer the attention
// kernel must read.
cudaError_t rekv_launch_attend_full_prepare(rekv_ctx* c, const void* q, const void* k_self, const void* v_self,
                                            const QBatch& qb, const QBatch& sb, int ncf, cudaStream_t st) {
  const StoreView& s = c->sv;
  const bool rope = c->cfg.rope_theta > 0.f;
  const int n_ctx_tokens = ncf * s.Nf;
  const __nv_bfloat16* q_eff = (const __nv_bfloat16*)q;
  if (rope) {
    dim3 grid((qb.sumNq * s.Hq + 31) / 32, s.L);
    rope_q_kernel<<<grid, 256, 0, st>>>((const uint4*)q, (uint4*)c->q_rot, qb, sb, s.Hq, n_ctx_tokens, c->rope_tab);
    c->launches += 1;
    q_eff = c->q_rot;
  }
  // the part over X (latency-bound) runs on the side stream beside the pass over the context's keys
  // (bandwidth-bound); both are joined before the attention kernel
  const bool fork = rope && ncf > 0;
  cudaStream_t st_self = fork ? c->side : st;
  cudaError_t e;
  if (fork) {
    if ((e = cudaEventRecord(c->ev_main, st)) != cudaSuccess) return e;
    if ((e = cudaStreamWaitEvent(c->side, c->ev_main, 0)) != cudaSuccess) return e;
  }
  self_attend_kernel<<<dim3(s.Hq, qb.nQ, s.L), 256, 0, st_self>>>(q_eff, (const __nv_bfloat16*)k_self,
                                                                 (const __nv_bfloat16*)v_self, qb, sb, s.Hq, s.Hkv, s.G,
                                                                 n_ctx_tokens, rope ? c->rope_tab : nullptr,
                                                                 1.4426950408889634f / sqrtf(128.f), c->self_o,
                                                                 c->self_ml);
  c->launches += 1;
  if (fork) {
    if ((e = cudaEventRecord(c->ev_side, c->side)) != cudaSuccess) return e;
    rope_stage_kernel<<<dim3(ncf, qb.nQ, s.L), 256, 0, st>>>(c->ctx_tbl, c->tbl_k, c->k_rot, qb.nQ, ncf, s.Hkv, s.Nf,
                                                             c->rope_tab);
    c->launches += 1;
    if ((e = cudaStreamWaitEvent(st, c->ev_side, 0)) != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

cudaError_t rekv_launch_self_finalize(rekv_ctx* c, const QBatch& qb, void* out, cudaStream_t st) {
  const long long rows = (long long)c->sv.L * qb.sumNq * c->sv.Hq;
  self_finalize_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(c->self_o, c->self_ml, (__nv_bfloat16*)out, rows);
  c->launches += 1;
  return cudaGetLastError();
}
