// Steps 2-3: question vector, cosine scores against every frame representative (Eq. 2, tau = 1),
// and the exact top-r selection, per layer and per question.
#include "ptx_helpers.cuh"
#include "rekv_internal.cuh"

namespace {

// ---- question vector: mean over the question's tokens and over the G query heads of each KV group
// grid = (nQ, layers, H_kv), layer = layer0 + blockIdx.y; 1024 threads = 16 token slices x 64 dim pairs (a short
// question is two or three rounds of loads deep): every load instruction of a warp
// covers 128 contiguous bytes of one (token, head) row.  Writes the group's 128 dims of the question
// vector and its partial sum of squares (the score kernel adds the H_kv partials).
constexpr int QM_SLICES = 16;
__global__ void __launch_bounds__(QM_SLICES * 64) qmean_kernel(const __nv_bfloat162* __restrict__ q, QBatch qb, int Hq, int Hkv,
                                                    int G, float* __restrict__ qa, float* __restrict__ qsq,
                                                    int maxQ, int layer0) {
  // launched with programmatic stream serialisation: its blocks are resident when the kernel before it ends (the
  // caller's, which wrote the queries, or the library's own), and wait here for that kernel's results
  rekv_ptx::grid_dep_wait();
  rekv_ptx::grid_dep_launch();
  const int qi = blockIdx.x, l = layer0 + blockIdx.y, g = blockIdx.z;
  const int Dp = Hkv * 128;
  const int n0 = qb.cu[qi], n1 = qb.cu[qi + 1];
  const int d2 = threadIdx.x & 63, slice = threadIdx.x >> 6;
  float sx = 0.f, sy = 0.f;
  for (int n = n0 + slice; n < n1; n += QM_SLICES) {
    const __nv_bfloat162* row = q + (((long long)l * qb.sumNq + n) * Hq + g * G) * 64 + d2;
    for (int j0 = 0; j0 < G; j0 += 8) {  // up to eight independent loads in flight
      __nv_bfloat162 v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (j0 + j < G) v[j] = row[(j0 + j) * 64];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (j0 + j < G) {
          float2 f = __bfloat1622float2(v[j]);
          sx += f.x;
          sy += f.y;
        }
    }
  }
  __shared__ float2 part[QM_SLICES][64];
  __shared__ float red[2];
  part[slice][d2] = make_float2(sx, sy);
  __syncthreads();
  if (threadIdx.x < 64) {
    const float inv = (float)((n1 - n0) * G);
    float ax = 0.f, ay = 0.f;
#pragma unroll
    for (int i = 0; i < QM_SLICES; i += 4) {  // fixed order
      ax += (part[i][d2].x + part[i + 1][d2].x) + (part[i + 2][d2].x + part[i + 3][d2].x);
      ay += (part[i][d2].y + part[i + 1][d2].y) + (part[i + 2][d2].y + part[i + 3][d2].y);
    }
    ax = __fdiv_rn(ax, inv);
    ay = __fdiv_rn(ay, inv);
    float* dst = qa + ((long long)l * maxQ + qi) * Dp + g * 128;
    dst[2 * d2] = ax;
    dst[2 * d2 + 1] = ay;
    float sq = ax * ax + ay * ay;
    for (int o = 16; o; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sq;
  }
  __syncthreads();
  if (threadIdx.x == 0) qsq[((long long)l * maxQ + qi) * Hkv + g] = red[0] + red[1];
}

// ---- cosine scores.  grid = (item chunks, L); an item is a frame, or with block retrieval a block of
// `block` consecutive frames whose vector is the mean of their representatives.  One warp per item: the
// representative rows are read once (float4 per lane, coalesced), the norm and the dot product with
// every question of the batch come from the same registers, reduced with warp shuffles.  The table is
// read once per batch.  n_visible counts items here.
// SCORE_MAX_V4 = float4 per lane (4: D' <= 512, 8: D' <= 1024); fpc = frames per CTA (a multiple of 16), chosen by
// the launcher so that the whole grid is resident at once (no second, mostly empty wave).
template <int SCORE_MAX_V4>
__global__ void __launch_bounds__(256, SCORE_MAX_V4 <= 4 ? 4 : 2)
    score_kernel(const float* __restrict__ reps, const float* __restrict__ qa, const float* __restrict__ qsq, int nQ,
                 int maxQ, int Dp, int Hkv, int max_frames, int n_visible, int q_group, float* __restrict__ scores,
                 int block, int layer0, int fpc, int* __restrict__ status) {
  extern __shared__ float4 s_q[];  // [q_group][Dp/4]
  __shared__ float s_qn[REKV_MAX_QUESTIONS];
  rekv_ptx::grid_dep_wait();
  rekv_ptx::grid_dep_launch();
  const int l = layer0 + blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int f0 = blockIdx.x * fpc;
  const int f1 = min(f0 + fpc, n_visible);
  const int nv4 = Dp / 128;  // float4 per lane
  const float eps = 1e-8f;
  if (threadIdx.x < nQ) {
    float sq = 0.f;
    for (int g = 0; g < Hkv; ++g) sq += qsq[((long long)l * maxQ + threadIdx.x) * Hkv + g];
    s_qn[threadIdx.x] = fmaxf(__fsqrt_rn(sq), eps);
  }

  for (int qg0 = 0; qg0 < nQ; qg0 += q_group) {
    const int qn = min(q_group, nQ - qg0);
    __syncthreads();
    const float4* src = reinterpret_cast<const float4*>(qa + ((long long)l * maxQ + qg0) * Dp);
    for (int i = threadIdx.x; i < qn * (Dp / 4); i += blockDim.x) s_q[i] = src[i];
    __syncthreads();
    // two frames per iteration: twice the loads in flight per warp
    for (int f = f0 + warp * 2; f < f1; f += 16) {
      const bool two = f + 1 < f1;
      if (!REKV_CHECK((long long)(f + (two ? 2 : 1)) * block <= max_frames && f >= 0, status, 11)) continue;
      const float4* row0 = reinterpret_cast<const float4*>(reps + ((long long)l * max_frames + (long long)f * block) * Dp);
      const float4* row1 = row0 + (two ? (long long)block * (Dp / 4) : 0);
      float4 r0[SCORE_MAX_V4], r1[SCORE_MAX_V4];
#pragma unroll
      for (int i = 0; i < SCORE_MAX_V4; ++i)
        if (i < nv4) {
          r0[i] = __ldg(row0 + i * 32 + lane);
          r1[i] = __ldg(row1 + i * 32 + lane);
        }
      if (block > 1) {  // block vector = mean of the block's frame vectors
        for (int j = 1; j < block; ++j) {
#pragma unroll
          for (int i = 0; i < SCORE_MAX_V4; ++i)
            if (i < nv4) {
              const float4 a = __ldg(row0 + (long long)j * (Dp / 4) + i * 32 + lane);
              const float4 b = __ldg(row1 + (long long)j * (Dp / 4) + i * 32 + lane);
              r0[i].x += a.x; r0[i].y += a.y; r0[i].z += a.z; r0[i].w += a.w;
              r1[i].x += b.x; r1[i].y += b.y; r1[i].z += b.z; r1[i].w += b.w;
            }
        }
        const float fb = (float)block;
#pragma unroll
        for (int i = 0; i < SCORE_MAX_V4; ++i)
          if (i < nv4) {
            r0[i].x = __fdiv_rn(r0[i].x, fb); r0[i].y = __fdiv_rn(r0[i].y, fb);
            r0[i].z = __fdiv_rn(r0[i].z, fb); r0[i].w = __fdiv_rn(r0[i].w, fb);
            r1[i].x = __fdiv_rn(r1[i].x, fb); r1[i].y = __fdiv_rn(r1[i].y, fb);
            r1[i].z = __fdiv_rn(r1[i].z, fb); r1[i].w = __fdiv_rn(r1[i].w, fb);
          }
      }
      float n0 = 0.f, n1 = 0.f;
#pragma unroll
      for (int i = 0; i < SCORE_MAX_V4; ++i)
        if (i < nv4) {
          n0 += r0[i].x * r0[i].x + r0[i].y * r0[i].y + r0[i].z * r0[i].z + r0[i].w * r0[i].w;
          n1 += r1[i].x * r1[i].x + r1[i].y * r1[i].y + r1[i].z * r1[i].z + r1[i].w * r1[i].w;
        }
      for (int o = 16; o; o >>= 1) {
        n0 += __shfl_xor_sync(0xffffffffu, n0, o);
        n1 += __shfl_xor_sync(0xffffffffu, n1, o);
      }
      n0 = fmaxf(__fsqrt_rn(n0), eps);
      n1 = fmaxf(__fsqrt_rn(n1), eps);
      for (int qi = 0; qi < qn; ++qi) {
        float d0 = 0.f, d1 = 0.f;
#pragma unroll
        for (int i = 0; i < SCORE_MAX_V4; ++i)
          if (i < nv4) {
            const float4 a = s_q[qi * (Dp / 4) + i * 32 + lane];
            d0 += r0[i].x * a.x + r0[i].y * a.y + r0[i].z * a.z + r0[i].w * a.w;
            d1 += r1[i].x * a.x + r1[i].y * a.y + r1[i].z * a.z + r1[i].w * a.w;
          }
        for (int o = 16; o; o >>= 1) {
          d0 += __shfl_xor_sync(0xffffffffu, d0, o);
          d1 += __shfl_xor_sync(0xffffffffu, d1, o);
        }
        if (lane == 0) {
          const float qn_ = s_qn[qg0 + qi];
          float* dst = scores + ((long long)l * nQ + qg0 + qi) * n_visible + f;
          dst[0] = __fdiv_rn(d0, qn_ * n0);
          if (two) dst[1] = __fdiv_rn(d1, qn_ * n1);
        }
      }
    }
  }
}

// ---- exact top-k by radix select on the score keys (score order, then lower index first).
// Order-preserving 32-bit image of a score: larger score <=> larger key; NaN ranks as -inf, -0 == +0.
__device__ __forceinline__ unsigned score_key(float s) {
  unsigned u = __float_as_uint(s);
  if (s != s) u = 0xFF800000u;
  if (s == 0.f) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// grid = (nQ, L), 512 threads.  Candidates are frames [0, n_cand).  Four 8-bit radix passes over the
// score keys find the k-th largest key T exactly, with the number of candidates above it; one
// ordered compaction then emits, in ascending frame index, every frame above T and the lowest-index
// frames equal to T that are still needed (ties go to the lower index).
// With block retrieval the candidates are blocks; a selected block b_i is written as its `block` frames
// b_i*block .. b_i*block + block-1 (k_eff counts items, top_k counts output slots).
// With tbl != null (cache all in HBM) the block also writes the context table of its (layer, question) -- the
// selected frames' pages then the trailing frames' pages, as the gather kernel would -- so that no further
// launch stands between the selection and the attention.
struct TopkTable {
  char** tbl;            // [L][nQ][ncf] page pointers, or null
  char* hbm;
  long long page_bytes;
  int L, ncf, n_vis_frames;
};
__device__ __forceinline__ void topk_write_table(const TopkTable& t, const int32_t* out, int k_frames, int l, int qi,
                                                 int nQ) {
  if (!t.tbl) return;
  __syncthreads();  // the block's writes of the selection are visible to all its threads
  char** row = t.tbl + ((long long)l * nQ + qi) * t.ncf;
  for (int j = threadIdx.x; j < t.ncf; j += blockDim.x) {
    const int frame = j < k_frames ? out[j] : t.n_vis_frames - (t.ncf - k_frames) + (j - k_frames);
    row[j] = t.hbm + ((long long)frame * t.L + l) * t.page_bytes;
  }
}

__global__ void __launch_bounds__(512) topk_kernel(const float* __restrict__ scores, int nQ, int n_visible,
                                                   int n_cand, int top_k, int k_eff, int32_t* __restrict__ idx_out,
                                                   int block, int layer0, TopkTable tt, int* __restrict__ status) {
  const int qi = blockIdx.x, l = layer0 + blockIdx.y;
  const float* s = scores + ((long long)l * nQ + qi) * n_visible;
  int32_t* out = idx_out + ((long long)l * nQ + qi) * top_k;
  __shared__ unsigned hist[4 * 256];
  __shared__ unsigned s_prefix;
  __shared__ int s_krem;
  __shared__ int warp_gt[16], warp_eq[16];
  __shared__ int s_base_gt, s_base_eq;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  rekv_ptx::grid_dep_wait();
  rekv_ptx::grid_dep_launch();

  for (int j = k_eff * block + threadIdx.x; j < top_k; j += blockDim.x) out[j] = -1;
  if (k_eff <= 0) {
    topk_write_table(tt, out, 0, l, qi, nQ);
    return;
  }
  // up to TK_CACHE * 512 candidates keep their keys in registers: one read of the scores instead of five.  A thread
  // holds TK_CACHE consecutive candidates, so that the ordered compaction at the end is one scan over the threads.
  constexpr int TK_CACHE = 4;
  const bool cached = n_cand <= TK_CACHE * 512;
  unsigned kc[TK_CACHE];
#pragma unroll
  for (int j = 0; j < TK_CACHE; ++j) {
    const int i = threadIdx.x * TK_CACHE + j;
    kc[j] = (cached && i < n_cand) ? score_key(s[i]) : 0u;
  }
  if (threadIdx.x == 0) {
    s_prefix = 0u;
    s_krem = k_eff;
    s_base_gt = 0;
    s_base_eq = 0;
  }
  for (int i = threadIdx.x; i < 4 * 256; i += blockDim.x) hist[i] = 0;  // one histogram per pass, cleared once
  __syncthreads();
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    unsigned* h = hist + 256 * pass;
    const unsigned prefix = s_prefix;
    const unsigned mask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
    if (cached) {
#pragma unroll
      for (int j = 0; j < TK_CACHE; ++j)
        if ((int)threadIdx.x * TK_CACHE + j < n_cand && (kc[j] & mask) == prefix) atomicAdd(&h[(kc[j] >> shift) & 255u], 1u);
    } else {
      for (int i = threadIdx.x; i < n_cand; i += blockDim.x) {
        const unsigned key = score_key(s[i]);
        if ((key & mask) == prefix) atomicAdd(&h[(key >> shift) & 255u], 1u);
      }
    }
    __syncthreads();
    if (warp == 0) {
      // lane owns bins [8*lane, 8*lane+8); suffix sums over lanes locate the bin of the k-th largest
      unsigned b[8], tot = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        b[j] = h[lane * 8 + j];
        tot += b[j];
      }
      unsigned suf = tot;  // inclusive suffix sum over lanes >= this one
      for (int o = 1; o < 32; o <<= 1) {
        unsigned v = __shfl_down_sync(0xffffffffu, suf, o);
        if (lane + o < 32) suf += v;
      }
      const int krem = s_krem;
      const unsigned ball = __ballot_sync(0xffffffffu, (int)suf >= krem);
      const int owner = 31 - __clz(ball);  // highest lane whose suffix still reaches krem
      if (lane == owner) {
        int above = (int)(suf - tot);  // candidates in higher lanes' bins
        int d = 7;
        for (; d > 0; --d) {
          if (above + (int)b[d] >= krem) break;
          above += (int)b[d];
        }
        s_krem = krem - above;
        s_prefix = prefix | ((unsigned)(lane * 8 + d) << shift);
      }
    }
    __syncthreads();
  }
  const unsigned thr = s_prefix;  // key of the k_eff-th largest score
  const int need_eq = s_krem;     // how many candidates equal to it are selected (lowest indices first)
  // Ordered compaction of a stretch of blockDim.x * TK_CACHE candidates starting at i0, thread t holding candidates
  // i0 + t * TK_CACHE + j: counts of "greater" and "equal" per thread, an exclusive scan over the block (shuffles
  // inside a warp, the warps' totals through shared memory), then
  // output position = selected frames before this one = (greater before) + min(equal before, need_eq).
  auto emit = [&](const int i0, const unsigned (&key_in)[TK_CACHE]) {
    int cg = 0, ce = 0;
#pragma unroll
    for (int j = 0; j < TK_CACHE; ++j) {
      const int i = i0 + threadIdx.x * TK_CACHE + j;
      cg += i < n_cand && key_in[j] > thr;
      ce += i < n_cand && key_in[j] == thr;
    }
    int sg = cg, se = ce;  // inclusive scans over the warp
    for (int o = 1; o < 32; o <<= 1) {
      const int vg = __shfl_up_sync(0xffffffffu, sg, o), ve = __shfl_up_sync(0xffffffffu, se, o);
      if (lane >= o) {
        sg += vg;
        se += ve;
      }
    }
    if (lane == 31) {
      warp_gt[warp] = sg;
      warp_eq[warp] = se;
    }
    __syncthreads();
    int og = s_base_gt + sg - cg, oe = s_base_eq + se - ce;  // greater / equal candidates before this thread's
    {
      const int wg = lane < 16 ? warp_gt[lane] : 0, we = lane < 16 ? warp_eq[lane] : 0;
      const unsigned below = lane < warp ? 0xffffffffu : 0u;
      int ag = wg & (int)below, ae = we & (int)below;  // totals of the warps before this one
      for (int o = 16; o; o >>= 1) {
        ag += __shfl_xor_sync(0xffffffffu, ag, o);
        ae += __shfl_xor_sync(0xffffffffu, ae, o);
      }
      og += ag;
      oe += ae;
    }
#pragma unroll
    for (int j = 0; j < TK_CACHE; ++j) {
      const int i = i0 + threadIdx.x * TK_CACHE + j;
      const bool gt = i < n_cand && key_in[j] > thr, eq = i < n_cand && key_in[j] == thr;
      int pos = -1;
      if (gt) pos = og + min(oe, need_eq);
      if (eq && oe < need_eq) pos = og + oe;
      if (pos >= 0 && REKV_CHECK(pos < k_eff && i < n_cand, status, 21))
        for (int jj = 0; jj < block; ++jj) out[pos * block + jj] = i * block + jj;
      og += gt;
      oe += eq;
    }
  };
  if (cached) {
    emit(0, kc);
  } else {
    for (int i0 = 0; i0 < n_cand; i0 += blockDim.x * TK_CACHE) {
      unsigned key[TK_CACHE];
#pragma unroll
      for (int j = 0; j < TK_CACHE; ++j) {
        const int i = i0 + threadIdx.x * TK_CACHE + j;
        key[j] = i < n_cand ? score_key(s[i]) : 0u;
      }
      emit(i0, key);
      __syncthreads();  // everybody has read the warps' totals
      if (threadIdx.x == 0) {
        int tg = 0, te = 0;
        for (int w = 0; w < 16; ++w) {
          tg += warp_gt[w];
          te += warp_eq[w];
        }
        s_base_gt += tg;
        s_base_eq += te;
      }
      __syncthreads();
    }
  }
  topk_write_table(tt, out, k_eff * block, l, qi, nQ);
}

// ---- external retrieval (Eq. 2 with its temperature): cosine of each question embedding with every frame
// embedding (or with the mean of a block's frame embeddings), divided by tau.  grid = ceil(items / 8), 256
// threads, a warp per item: the item's vector is read once into registers (float4 per lane, coalesced) and
// scored against every question of the batch, whose embeddings sit in shared memory in groups.
constexpr int EXT_MAX_V4 = 16;  // float4 per lane: embedding dim <= 2048
__global__ void __launch_bounds__(256) ext_score_kernel(const float* __restrict__ embs, const float* __restrict__ q,
                                                        int nQ, int E, int n_items, int block, int q_group, float tau,
                                                        float* __restrict__ scores) {
  extern __shared__ float4 s_qe[];  // [q_group][E/4]
  __shared__ float s_qn[REKV_MAX_QUESTIONS];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int item = blockIdx.x * 8 + warp;
  const int e4 = E / 4;
  const float eps = 1e-8f;
  float4 r[EXT_MAX_V4];
  float vn = 0.f;
  if (item < n_items) {
#pragma unroll
    for (int i = 0; i < EXT_MAX_V4; ++i)
      if (i * 32 + lane < e4) {
        const float4* row = reinterpret_cast<const float4*>(embs + (long long)item * block * E) + i * 32 + lane;
        float4 a = __ldg(row);
        for (int j = 1; j < block; ++j) {  // block vector = mean of the block's frame vectors
          const float4 b = __ldg(row + (long long)j * e4);
          a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
        }
        if (block > 1) {
          const float fb = (float)block;
          a.x = __fdiv_rn(a.x, fb); a.y = __fdiv_rn(a.y, fb); a.z = __fdiv_rn(a.z, fb); a.w = __fdiv_rn(a.w, fb);
        }
        r[i] = a;
        vn += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
      }
    for (int o = 16; o; o >>= 1) vn += __shfl_xor_sync(0xffffffffu, vn, o);
    vn = fmaxf(__fsqrt_rn(vn), eps);
  }
  for (int qg0 = 0; qg0 < nQ; qg0 += q_group) {
    const int qn = min(q_group, nQ - qg0);
    __syncthreads();
    const float4* src = reinterpret_cast<const float4*>(q + (long long)qg0 * E);
    for (int i = threadIdx.x; i < qn * e4; i += 256) s_qe[i] = src[i];
    __syncthreads();
    for (int qi = warp; qi < qn; qi += 8) {  // the questions' norms
      float sq = 0.f;
      for (int i = lane; i < e4; i += 32) {
        const float4 a = s_qe[qi * e4 + i];
        sq += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
      }
      for (int o = 16; o; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      if (lane == 0) s_qn[qi] = fmaxf(__fsqrt_rn(sq), eps);
    }
    __syncthreads();
    if (item < n_items) {
      for (int qi = 0; qi < qn; ++qi) {
        float d = 0.f;
#pragma unroll
        for (int i = 0; i < EXT_MAX_V4; ++i)
          if (i * 32 + lane < e4) {
            const float4 a = s_qe[qi * e4 + i * 32 + lane];
            d += r[i].x * a.x + r[i].y * a.y + r[i].z * a.z + r[i].w * a.w;
          }
        for (int o = 16; o; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
        if (lane == 0) scores[(long long)(qg0 + qi) * n_items + item] = __fdiv_rn(d, tau * s_qn[qi] * vn);
      }
    }
  }
}

// the external selection is the same in every layer: copies layer 0's [nQ][top_k] block to the others
__global__ void replicate_idx_kernel(int32_t* __restrict__ idx, int per_layer, int L) {
  rekv_ptx::grid_dep_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= per_layer) return;
  const int32_t v = idx[i];
  for (int l = 1; l < L; ++l) idx[(long long)l * per_layer + i] = v;
}

// Launch of the score kernel over frames [0, n_scored) of nl layers.  Frames per CTA grow until the grid fits the
// device in one wave at the kernel's occupancy.
template <int V4>
cudaError_t launch_score_v4(bool pdl, cudaStream_t st, size_t smem, int nl, int n_scored, const float* reps, const float* qa,
                            const float* qsq, int nQ, int maxQ, int Dp, int Hkv, int max_frames, int q_group, float* scores,
                            int block, int layer0, int* status) {
  static PerDeviceOnce attr;
  cudaError_t ea = attr.run([] {
    return cudaFuncSetAttribute(score_kernel<V4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
  });
  if (ea != cudaSuccess) return ea;
  const int sms = rekv_sm_count();
  int occ = 1;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, score_kernel<V4>, 256, smem) != cudaSuccess || occ < 1) occ = 1;
  int per_layer = (sms * occ) / nl;
  if (per_layer < 1) per_layer = 1;
  int fpc = ((n_scored + per_layer - 1) / per_layer + 15) & ~15;
  if (fpc < 16) fpc = 16;
  dim3 grid((n_scored + fpc - 1) / fpc, nl);
  if (pdl)
    return rekv_launch_pdl(score_kernel<V4>, grid, dim3(256), smem, st, reps, qa, qsq, nQ, maxQ, Dp, Hkv, max_frames,
                           n_scored, q_group, scores, block, layer0, fpc, status);
  score_kernel<V4><<<grid, 256, smem, st>>>(reps, qa, qsq, nQ, maxQ, Dp, Hkv, max_frames, n_scored, q_group, scores, block,
                                            layer0, fpc, status);
  return cudaGetLastError();
}
cudaError_t launch_score(bool pdl, cudaStream_t st, size_t smem, int nl, int n_scored, const float* reps, const float* qa,
                         const float* qsq, int nQ, int maxQ, int Dp, int Hkv, int max_frames, int q_group, float* scores,
                         int block, int layer0, int* status) {
  return Dp <= 512 ? launch_score_v4<4>(pdl, st, smem, nl, n_scored, reps, qa, qsq, nQ, maxQ, Dp, Hkv, max_frames, q_group,
                                        scores, block, layer0, status)
                   : launch_score_v4<8>(pdl, st, smem, nl, n_scored, reps, qa, qsq, nQ, maxQ, Dp, Hkv, max_frames, q_group,
                                        scores, block, layer0, status);
}

}  // namespace

cudaError_t rekv_launch_retrieve(rekv_ctx* c, const void* q, const QBatch& qb, int top_k, const CtxGeom& geom,
                                 int n_visible, int layer0, int layer1, int32_t* idx_out, float* scores, cudaStream_t st,
                                 bool write_table) {
  // q, idx_out and scores are indexed with the absolute layer by the kernels; a caller that holds one
  // layer's rows only passes pointers moved back by layer0 layers
  const StoreView& s = c->sv;
  const int maxQ = c->cfg.max_questions;
  const int nl = layer1 - layer0;
  {
    cudaError_t e0 = rekv_launch_pdl(qmean_kernel, dim3(qb.nQ, nl, s.Hkv), dim3(QM_SLICES * 64), 0, st,
                                     (const __nv_bfloat162*)q, qb, s.Hq, s.Hkv, s.G, c->qa, c->qnorm, maxQ, layer0);
    if (e0 != cudaSuccess) return e0;
  }
  int q_group = (int)((96 * 1024) / (s.Dp * sizeof(float)));
  if (q_group > qb.nQ) q_group = qb.nQ;
  size_t smem = (size_t)q_group * s.Dp * sizeof(float);
  // b = 1: every visible frame is scored (the window's scores are reported but not candidates);
  // b > 1: the complete candidate blocks are scored
  const int b = c->cfg.block_frames;
  const int n_scored = b == 1 ? n_visible : geom.n_items;
  if (n_scored > 0) {
    cudaError_t e1 = launch_score(true, st, smem, nl, n_scored, s.reps, c->qa, c->qnorm, qb.nQ, maxQ, s.Dp, s.Hkv,
                                  s.max_frames, q_group, scores, b, layer0, c->status);
    if (e1 != cudaSuccess) return e1;
    c->launches += 1;
  }
  if (top_k > 0) {
    TopkTable tt = {};
    if (write_table) {  // HBM-resident cache: the context table comes out of the same launch
      tt.tbl = c->ctx_tbl;
      tt.hbm = s.hbm;
      tt.page_bytes = s.page_bytes;
      tt.L = s.L;
      tt.ncf = geom.ncf;
      tt.n_vis_frames = n_visible;
    }
    cudaError_t e2 = rekv_launch_pdl(topk_kernel, dim3(qb.nQ, nl), dim3(512), 0, st, scores, qb.nQ, n_scored,
                                     geom.n_items, top_k, geom.k_items, idx_out, b, layer0, tt, c->status);
    if (e2 != cudaSuccess) return e2;
    c->launches += 1;
  }
  c->launches += 1;
  return cudaGetLastError();
}

cudaError_t rekv_launch_retrieve_external(rekv_ctx* c, const float* q_emb, int nQ, int top_k, const CtxGeom& geom,
                                          int n_visible, float tau, int32_t* idx_out, float* scores, cudaStream_t st) {
  const StoreView& s = c->sv;
  const int E = c->cfg.ext_embed_dim, b = c->cfg.block_frames;
  const int n_scored = b == 1 ? n_visible : geom.n_items;
  int q_group = (int)((96 * 1024) / (E * sizeof(float)));
  if (q_group > nQ) q_group = nQ;
  static PerDeviceOnce attr;
  cudaError_t ea = attr.run([] {
    return cudaFuncSetAttribute(ext_score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
  });
  if (ea != cudaSuccess) return ea;
  if (n_scored > 0) {
    ext_score_kernel<<<(n_scored + 7) / 8, 256, (size_t)q_group * E * sizeof(float), st>>>(c->ext_emb, q_emb, nQ, E, n_scored,
                                                                                         b, q_group, tau, scores);
    c->launches += 1;
  }
  if (top_k > 0) {
    cudaError_t e2 = rekv_launch_pdl(topk_kernel, dim3(nQ, 1), dim3(512), 0, st, (const float*)scores, nQ, n_scored,
                                     geom.n_items, top_k, geom.k_items, idx_out, b, 0, TopkTable{}, c->status);
    if (e2 != cudaSuccess) return e2;
    const int per_layer = nQ * top_k;
    if (s.L > 1) {
      cudaError_t e3 = rekv_launch_pdl(replicate_idx_kernel, dim3((per_layer + 255) / 256), dim3(256), 0, st, idx_out,
                                       per_layer, s.L);
      if (e3 != cudaSuccess) return e3;
    }
    c->launches += 2;
  }
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// rekv_score_frames_static: scoring without any allocation.
//
// Some hosts cannot let a library allocate device memory: a serving engine that has handed the whole
// GPU to its own memory pool, or a latency-critical thread for which the implicit device
// synchronisation of cudaMalloc/cudaFree is not acceptable.  For them this entry point runs the
// question-vector and cosine-score kernels of one layer with their intermediate (the fp32 question
// vectors and their partial squared norms) in a fixed array that is part of the library image, so
// nothing is allocated, here or in any routine it calls.
//
// The array lives in every GPU context that loads the library, for the life of the process.  All
// calls on a device share it: it is fully rewritten by each call (nothing in it has to start at
// zero), it keeps the last call's contents afterwards, and two calls whose kernels overlap on the
// GPU (different streams, no ordering between them) race on it.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int STATIC_MAX_QUESTIONS = 16;
constexpr int STATIC_MAX_DP = 1024;                       // H_kv * 128
constexpr int STATIC_QA_FLOATS = STATIC_MAX_QUESTIONS * STATIC_MAX_DP;
constexpr int STATIC_QSQ_FLOATS = STATIC_MAX_QUESTIONS * 8;
// 66 048 bytes: question vectors [16][1024] followed by partial squared norms [16][8]
static __device__ __align__(256) float g_static_scratch[STATIC_QA_FLOATS + STATIC_QSQ_FLOATS];

constexpr int STATIC_MAX_DEVICES = 64;
float* g_static_scratch_addr[STATIC_MAX_DEVICES] = {nullptr};  // device address of the array, per device

}  // namespace

extern "C" int rekv_score_frames_static(const void* q, const int32_t* cu_q, int nQ, int n_q_heads, int n_kv_heads,
                                        int head_dim, const float* reps, int n_frames, float* scores_out, void* stream) {
  if (!q || !cu_q || !reps || !scores_out) {
    rekv_set_error(nullptr, "rekv_score_frames_static: null pointer argument");
    return REKV_ERR_ARG;
  }
  if (head_dim != REKV_HEAD_DIM || n_kv_heads < 1 || n_kv_heads > 8 || n_q_heads < n_kv_heads ||
      n_q_heads % n_kv_heads) {
    rekv_set_error(nullptr, "rekv_score_frames_static: head_dim must be 128 and 1 <= H_kv <= 8 must divide H_q");
    return REKV_ERR_ARG;
  }
  if (nQ < 1 || nQ > STATIC_MAX_QUESTIONS) {
    rekv_set_error(nullptr, "rekv_score_frames_static: at most 16 questions per call (fixed scratch size)");
    return REKV_ERR_ARG;
  }
  if (n_frames < 1) {
    rekv_set_error(nullptr, "rekv_score_frames_static: no frames");
    return REKV_ERR_EMPTY;
  }
  QBatch qb;
  qb.nQ = nQ;
  if (cu_q[0] != 0) {
    rekv_set_error(nullptr, "rekv_score_frames_static: cu_q[0] must be 0");
    return REKV_ERR_ARG;
  }
  for (int i = 0; i < nQ; ++i) {
    if (cu_q[i + 1] <= cu_q[i]) {
      rekv_set_error(nullptr, "rekv_score_frames_static: a question has no tokens");
      return REKV_ERR_ARG;
    }
    qb.cu[i] = cu_q[i];
  }
  qb.cu[nQ] = qb.sumNq = cu_q[nQ];

  // Set-up, once per device, with that device current: in host code the array's name is only a
  // stand-in; the kernels need its device address, which the runtime resolves here.
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) {
    rekv_set_error(nullptr, "rekv_score_frames_static: no current CUDA device (or ordinal >= 64)");
    cudaGetLastError();
    return REKV_ERR_CUDA;
  }
  if (!g_static_scratch_addr[dev]) {
    float* ptr = nullptr;
    e = cudaGetSymbolAddress((void**)&ptr, g_static_scratch);
    if (e != cudaSuccess || !ptr) {
      rekv_set_error(nullptr, "rekv_score_frames_static: cudaGetSymbolAddress failed for the scratch array");
      cudaGetLastError();
      return REKV_ERR_CUDA;
    }
    g_static_scratch_addr[dev] = ptr;
  }
  float* qa = g_static_scratch_addr[dev];
  float* qsq = qa + STATIC_QA_FLOATS;

  const int Dp = n_kv_heads * REKV_HEAD_DIM, G = n_q_heads / n_kv_heads;
  cudaStream_t st = (cudaStream_t)stream;
  qmean_kernel<<<dim3(nQ, 1, n_kv_heads), QM_SLICES * 64, 0, st>>>((const __nv_bfloat162*)q, qb, n_q_heads, n_kv_heads, G, qa, qsq,
                                                         STATIC_MAX_QUESTIONS, 0);
  // the question vectors of one call fit in 64 KB of dynamic shared memory only in groups
  int q_group = (int)((96 * 1024) / (Dp * sizeof(float)));
  if (q_group > nQ) q_group = nQ;
  e = launch_score(false, st, (size_t)q_group * Dp * sizeof(float), 1, n_frames, reps, qa, qsq, nQ, STATIC_MAX_QUESTIONS, Dp,
                   n_kv_heads, n_frames, q_group, scores_out, 1, 0, nullptr);
  if (e != cudaSuccess) {
    rekv_set_error(nullptr, cudaGetErrorString(e));
    return REKV_ERR_CUDA;
  }
  return REKV_OK;
}
