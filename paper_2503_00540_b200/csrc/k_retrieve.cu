// Steps 2-3: question vector, cosine scores against every frame representative (Eq. 2, tau = 1),
// and the exact top-r selection, per layer and per question.
#include "rekv_internal.cuh"

namespace {

// ---- question vector: mean over the question's tokens and over the G query heads of each KV group
// grid = (nQ, L); each thread owns dim pairs.  Also writes |q|.
__global__ void __launch_bounds__(256) qmean_kernel(const __nv_bfloat162* __restrict__ q, QBatch qb, int Hq, int Hkv,
                                                    int G, float* __restrict__ qa, float* __restrict__ qnorm,
                                                    int maxQ) {
  const int qi = blockIdx.x, l = blockIdx.y;
  const int Dp = Hkv * 128;
  const int n0 = qb.cu[qi], n1 = qb.cu[qi + 1];
  float* dst = qa + ((long long)l * maxQ + qi) * Dp;
  float sq = 0.f;
  for (int p = threadIdx.x; p < Dp / 2; p += blockDim.x) {
    const int g = p >> 6, d2 = p & 63;
    float sx = 0.f, sy = 0.f;
    for (int n = n0; n < n1; ++n) {
      const __nv_bfloat162* row = q + (((long long)l * qb.sumNq + n) * Hq + g * G) * 64 + d2;
      for (int j = 0; j < G; ++j) {
        float2 f = __bfloat1622float2(row[j * 64]);
        sx += f.x;
        sy += f.y;
      }
    }
    const float inv = (float)((n1 - n0) * G);
    sx = __fdiv_rn(sx, inv);
    sy = __fdiv_rn(sy, inv);
    dst[2 * p] = sx;
    dst[2 * p + 1] = sy;
    sq += sx * sx + sy * sy;
  }
  __shared__ float red[8];
  for (int o = 16; o; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sq;
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
    for (int w = 0; w < (blockDim.x >> 5); ++w) s += red[w];
    qnorm[l * maxQ + qi] = __fsqrt_rn(s);
  }
}

// ---- cosine scores.  grid = (frame chunks, L); one warp per frame: the representative row is read
// once (float4 per lane, coalesced), its norm and its dot product with every question of the batch
// come from the same registers, reduced with warp shuffles.  The table is read once per batch.
constexpr int SCORE_FRAMES_PER_CTA = 64;
constexpr int SCORE_MAX_V4 = 8;  // float4 per lane: D' <= 1024

__global__ void __launch_bounds__(256) score_kernel(const float* __restrict__ reps, const float* __restrict__ qa,
                                                    const float* __restrict__ qnorm, int nQ, int maxQ, int Dp,
                                                    int max_frames, int n_visible, int q_group,
                                                    float* __restrict__ scores) {
  extern __shared__ float4 s_q[];  // [q_group][Dp/4]
  const int l = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int f0 = blockIdx.x * SCORE_FRAMES_PER_CTA;
  const int f1 = min(f0 + SCORE_FRAMES_PER_CTA, n_visible);
  const int nv4 = Dp / 128;  // float4 per lane
  const float eps = 1e-8f;

  for (int qg0 = 0; qg0 < nQ; qg0 += q_group) {
    const int qn = min(q_group, nQ - qg0);
    __syncthreads();
    const float4* src = reinterpret_cast<const float4*>(qa + ((long long)l * maxQ + qg0) * Dp);
    for (int i = threadIdx.x; i < qn * (Dp / 4); i += blockDim.x) s_q[i] = src[i];
    __syncthreads();
    for (int f = f0 + warp; f < f1; f += 8) {
      const float4* row = reinterpret_cast<const float4*>(reps + ((long long)l * max_frames + f) * Dp);
      float4 r[SCORE_MAX_V4];
      float rn = 0.f;
#pragma unroll
      for (int i = 0; i < SCORE_MAX_V4; ++i)
        if (i < nv4) {
          r[i] = __ldg(row + i * 32 + lane);
          rn += r[i].x * r[i].x + r[i].y * r[i].y + r[i].z * r[i].z + r[i].w * r[i].w;
        }
      for (int o = 16; o; o >>= 1) rn += __shfl_xor_sync(0xffffffffu, rn, o);
      rn = fmaxf(__fsqrt_rn(rn), eps);
      for (int qi = 0; qi < qn; ++qi) {
        float dot = 0.f;
#pragma unroll
        for (int i = 0; i < SCORE_MAX_V4; ++i)
          if (i < nv4) {
            float4 a = s_q[qi * (Dp / 4) + i * 32 + lane];
            dot += r[i].x * a.x + r[i].y * a.y + r[i].z * a.z + r[i].w * a.w;
          }
        for (int o = 16; o; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        if (lane == 0) {
          float qn_ = fmaxf(qnorm[l * maxQ + qg0 + qi], eps);
          scores[((long long)l * nQ + qg0 + qi) * n_visible + f] = __fdiv_rn(dot, qn_ * rn);
        }
      }
    }
  }
}

// ---- exact top-k by radix select on 64-bit keys (score order, then lower index first).
__device__ __forceinline__ unsigned long long topk_key(float s, int idx) {
  unsigned u = __float_as_uint(s);
  if (s != s) u = 0xFF800000u;       // NaN ranks as -inf
  if (s == 0.f) u = 0u;              // -0 == +0
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned)idx);
}

// grid = (nQ, L), 512 threads.  Candidates are frames [0, n_cand).  Eight 8-bit passes find the
// k-th largest key exactly (keys are unique), then an ordered compaction emits the selected frames
// in ascending frame index.
__global__ void __launch_bounds__(512) topk_kernel(const float* __restrict__ scores, int nQ, int n_visible,
                                                   int n_cand, int top_k, int k_eff, int32_t* __restrict__ idx_out) {
  const int qi = blockIdx.x, l = blockIdx.y;
  const float* s = scores + ((long long)l * nQ + qi) * n_visible;
  int32_t* out = idx_out + ((long long)l * nQ + qi) * top_k;
  __shared__ unsigned hist[256];
  __shared__ unsigned long long s_prefix;
  __shared__ int s_krem;
  __shared__ int warp_cnt[16];
  __shared__ int s_base;

  for (int j = k_eff + threadIdx.x; j < top_k; j += blockDim.x) out[j] = -1;
  if (k_eff <= 0) return;

  if (threadIdx.x == 0) {
    s_prefix = 0ull;
    s_krem = k_eff;
    s_base = 0;
  }
  for (int pass = 0; pass < 8; ++pass) {
    const int shift = 56 - 8 * pass;
    for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    const unsigned long long prefix = s_prefix;
    const unsigned long long mask = pass == 0 ? 0ull : (~0ull << (shift + 8));
    for (int i = threadIdx.x; i < n_cand; i += blockDim.x) {
      unsigned long long key = topk_key(s[i], i);
      if ((key & mask) == prefix) atomicAdd(&hist[(unsigned)(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int krem = s_krem;
      int d = 255;
      for (; d > 0; --d) {
        int c = (int)hist[d];
        if (c >= krem) break;
        krem -= c;
      }
      s_krem = krem;
      s_prefix = prefix | ((unsigned long long)d << shift);
    }
    __syncthreads();
  }
  const unsigned long long thr = s_prefix;  // the k_eff-th largest key
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i0 = 0; i0 < n_cand; i0 += blockDim.x) {
    const int i = i0 + threadIdx.x;
    const bool sel = i < n_cand && topk_key(s[i], i) >= thr;
    const unsigned b = __ballot_sync(0xffffffffu, sel);
    if (lane == 0) warp_cnt[warp] = __popc(b);
    __syncthreads();
    int off = s_base;
    for (int w = 0; w < warp; ++w) off += warp_cnt[w];
    if (sel) {
      int pos = off + __popc(b & ((1u << lane) - 1u));
      if (pos < k_eff) out[pos] = i;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int t = 0;
      for (int w = 0; w < 16; ++w) t += warp_cnt[w];
      s_base += t;
    }
    __syncthreads();
  }
}

}  // namespace

cudaError_t rekv_launch_retrieve(rekv_ctx* c, const void* q, const QBatch& qb, int top_k, int k_eff, int n_visible,
                                 int32_t* idx_out, float* scores, cudaStream_t st) {
  const StoreView& s = c->sv;
  const int maxQ = c->cfg.max_questions;
  qmean_kernel<<<dim3(qb.nQ, s.L), 256, 0, st>>>((const __nv_bfloat162*)q, qb, s.Hq, s.Hkv, s.G, c->qa, c->qnorm,
                                                maxQ);
  int q_group = (int)((96 * 1024) / (s.Dp * sizeof(float)));
  if (q_group > qb.nQ) q_group = qb.nQ;
  size_t smem = (size_t)q_group * s.Dp * sizeof(float);
  static bool attr_set = false;
  if (!attr_set) {
    cudaFuncSetAttribute(score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
    attr_set = true;
  }
  dim3 grid((n_visible + SCORE_FRAMES_PER_CTA - 1) / SCORE_FRAMES_PER_CTA, s.L);
  score_kernel<<<grid, 256, smem, st>>>(s.reps, c->qa, c->qnorm, qb.nQ, maxQ, s.Dp, s.max_frames, n_visible, q_group,
                                        scores);
  if (top_k > 0) {
    int n_cand = n_visible - c->cfg.window_frames;
    if (n_cand < 0) n_cand = 0;
    topk_kernel<<<dim3(qb.nQ, s.L), 512, 0, st>>>(scores, qb.nQ, n_visible, n_cand, top_k, k_eff, idx_out);
    c->launches += 1;
  }
  c->launches += 2;
  return cudaGetLastError();
}
