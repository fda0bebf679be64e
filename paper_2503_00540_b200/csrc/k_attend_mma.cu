// Step 5 (Eq. 3): GQA attention of the question tokens over the gathered context, read page by
// page through the context table.  This translation unit holds the mma.sync implementation (the
// portable tensor path) and the split-KV combine kernel.
//
// Work unit = (layer, kv head, split of the context frames, 128-row tile of one question), where a
// question's rows are its N_q tokens x the G query heads of the KV group.  Per context frame the CTA
// brings the head's K and V tiles into shared memory with four contiguous bulk copies (the store's
// swizzled layout is the ldmatrix layout), double-buffered behind mbarriers.
#include "ptx_helpers.cuh"
#include "rekv_internal.cuh"

using namespace rekv_ptx;

namespace {

constexpr int ATT_THREADS = 256;  // 8 warps x 16 rows
constexpr int ATT_ROWS = 128;
constexpr int SUB = 64;           // tokens per softmax sub-tile

struct AttParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  char* const* tbl;
  float* part_o;
  float* part_ml;
  int* status;
  QBatch qb;
  int Hq, Hkv, G, Nf, Npad, ncf, n_splits, MT, layer0;
  float scale_log2;
};

__device__ __forceinline__ void decode_mtile(const QBatch& qb, int G, int mtg, int& qi, int& mt) {
  mt = mtg;
  for (qi = 0; qi < qb.nQ - 1; ++qi) {
    int t = ((qb.cu[qi + 1] - qb.cu[qi]) * G + ATT_ROWS - 1) / ATT_ROWS;
    if (mt < t) break;
    mt -= t;
  }
}

__global__ void __launch_bounds__(ATT_THREADS, 1) attend_mma_kernel(const AttParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  // carve: [stage][K tile | V tile], each tile = 2 halves x Npad rows x 128 B; then 2 mbarriers
  const uint32_t tile_bytes = 2u * p.Npad * 128u;
  const uint32_t half_stride = p.Npad * 128u;
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t s_base = smem_u32(smem);
  const uint32_t bar0 = s_base + 4u * tile_bytes;

  int b = blockIdx.x;
  const int mtg = b % p.MT;
  b /= p.MT;
  const int split = b % p.n_splits;
  b /= p.n_splits;
  const int g = b % p.Hkv;
  const int l = p.layer0 + b / p.Hkv;
  int qi, mt;
  decode_mtile(p.qb, p.G, mtg, qi, mt);
  const int n_q = p.qb.cu[qi + 1] - p.qb.cu[qi];
  const int rows_total = n_q * p.G;
  const int m0 = mt * ATT_ROWS;
  const int f_begin = (int)((long long)split * p.ncf / p.n_splits);
  const int f_end = (int)((long long)(split + 1) * p.ncf / p.n_splits);
  const int n_tiles = f_end - f_begin;
  char* const* pages = p.tbl + ((long long)l * p.qb.nQ + qi) * p.ncf + f_begin;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // zero the pad rows [Nf, Npad) of every tile half once; bulk copies never touch them
  {
    const int pad_rows = p.Npad - p.Nf;
    const int n16 = 2 * 2 * 2 * pad_rows * 8;  // stages x {K,V} x halves x rows x 16-byte chunks
    for (int i = tid; i < n16; i += ATT_THREADS) {
      int c = i & 7;
      int r = (i >> 3) % pad_rows;
      int hh = (i >> 3) / pad_rows;  // 0..7 : (stage, kv, half)
      *reinterpret_cast<uint4*>(smem + (hh >> 1) * tile_bytes + (hh & 1) * half_stride + (p.Nf + r) * 128 + c * 16) =
          make_uint4(0, 0, 0, 0);
    }
  }
  if (tid == 0) {
    mbar_init(bar0, 1);
    mbar_init(bar0 + 8, 1);
    fence_barrier_init();
  }
  __syncthreads();

  const uint32_t half_bytes = (uint32_t)p.Nf * 128u;
  auto issue = [&](int i) {
    const int st = i & 1;
    const char* page = pages[i];
    const char* kt = page + (long long)(g * 2) * p.Nf * 256;
    const uint32_t bar = bar0 + 8 * st;
    const uint32_t dst = s_base + (uint32_t)st * 2u * tile_bytes;
    mbar_expect_tx(bar, 4u * half_bytes);
    bulk_g2s(dst, kt, half_bytes, bar);
    bulk_g2s(dst + half_stride, kt + half_bytes, half_bytes, bar);
    bulk_g2s(dst + tile_bytes, kt + 2 * half_bytes, half_bytes, bar);
    bulk_g2s(dst + tile_bytes + half_stride, kt + 3 * half_bytes, half_bytes, bar);
  };
  if (tid == 0) {
    if (n_tiles > 0) issue(0);
    if (n_tiles > 1) issue(1);
  }

  // ---- Q fragments straight from global (once per unit) ----
  const int r_lo = m0 + warp * 16 + (lane >> 2);
  const int r_hi = r_lo + 8;
  const bool v_lo = r_lo < rows_total, v_hi = r_hi < rows_total;
  const long long q_row0 = ((long long)l * p.qb.sumNq + p.qb.cu[qi]);
  auto q_ptr = [&](int r) {
    int n = r / p.G, j = r - n * p.G;
    return p.q + ((q_row0 + n) * p.Hq + g * p.G + j) * 128;
  };
  uint32_t qf[8][4];
  {
    const uint32_t* plo = reinterpret_cast<const uint32_t*>(q_ptr(v_lo ? r_lo : 0));
    const uint32_t* phi = reinterpret_cast<const uint32_t*>(q_ptr(v_hi ? r_hi : 0));
#pragma unroll
    for (int kb = 0; kb < 8; ++kb) {
      const int w = kb * 8 + (lane & 3);
      qf[kb][0] = v_lo ? __ldg(plo + w) : 0u;
      qf[kb][1] = v_hi ? __ldg(phi + w) : 0u;
      qf[kb][2] = v_lo ? __ldg(plo + w + 4) : 0u;
      qf[kb][3] = v_hi ? __ldg(phi + w + 4) : 0u;
    }
  }

  float oacc[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

  const int lm = lane >> 3, lr = lane & 7;  // ldmatrix: matrix index and row within it
  bool ok = true;

  for (int i = 0; i < n_tiles && ok; ++i) {
    const int st = i & 1;
    if (!mbar_wait_bounded(bar0 + 8 * st, (i >> 1) & 1)) {
      ok = false;
      break;
    }
    const uint32_t sK = s_base + (uint32_t)st * 2u * tile_bytes;
    const uint32_t sV = sK + tile_bytes;

    for (int t0 = 0; t0 < p.Npad; t0 += SUB) {
      const int nblk = min(SUB, p.Npad - t0) >> 3;  // 8-token blocks in this sub-tile (even)
      float sacc[SUB / 8][4];
#pragma unroll
      for (int nb = 0; nb < SUB / 8; ++nb) {
        sacc[nb][0] = sacc[nb][1] = sacc[nb][2] = sacc[nb][3] = 0.f;
        if (nb < nblk) {
          const int tok = t0 + nb * 8 + lr;
#pragma unroll
          for (int kp = 0; kp < 4; ++kp) {
            const int c = kp * 4 + lm;  // 16-byte chunk (8 dims) of the 128-dim row
            const uint32_t addr = sK + (c >> 3) * half_stride + tok * 128 + (((c & 7) ^ (tok & 7)) << 4);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(b0, b1, b2, b3, addr);
            mma_bf16_16816(sacc[nb], qf[2 * kp], b0, b1);
            mma_bf16_16816(sacc[nb], qf[2 * kp + 1], b2, b3);
          }
        }
      }
      // mask pad tokens, scale, row max
      float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
      for (int nb = 0; nb < SUB / 8; ++nb)
        if (nb < nblk) {
          const int col = t0 + nb * 8 + (lane & 3) * 2;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float s = sacc[nb][e] * p.scale_log2;
            if (col + (e & 1) >= p.Nf) s = -INFINITY;
            sacc[nb][e] = s;
          }
          mx_lo = fmaxf(mx_lo, fmaxf(sacc[nb][0], sacc[nb][1]));
          mx_hi = fmaxf(mx_hi, fmaxf(sacc[nb][2], sacc[nb][3]));
        }
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
      const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
      const float a_lo = ex2(m_lo - mn_lo), a_hi = ex2(m_hi - mn_hi);
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
      uint32_t pf[SUB / 8][2];
#pragma unroll
      for (int nb = 0; nb < SUB / 8; ++nb)
        if (nb < nblk) {
          float p0 = ex2(sacc[nb][0] - mn_lo), p1 = ex2(sacc[nb][1] - mn_lo);
          float p2 = ex2(sacc[nb][2] - mn_hi), p3 = ex2(sacc[nb][3] - mn_hi);
          l_lo += p0 + p1;
          l_hi += p2 + p3;
          pf[nb][0] = pack_bf16(p0, p1);
          pf[nb][1] = pack_bf16(p2, p3);
        }
      // O += P V
#pragma unroll
      for (int kb = 0; kb < SUB / 16; ++kb)
        if (2 * kb < nblk) {
          const uint32_t a[4] = {pf[2 * kb][0], pf[2 * kb][1], pf[2 * kb + 1][0], pf[2 * kb + 1][1]};
          const int tok = t0 + kb * 16 + (lm & 1) * 8 + lr;
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
    __syncthreads();
    if (tid == 0 && i + 2 < n_tiles) issue(i + 2);
  }
  if (!ok) {
    // a copy never completed: record it, and give copies still in flight a bounded chance to land
    if (lane == 0) atomicExch(p.status, REKV_ERR_TIMEOUT);
    mbar_wait_bounded(bar0, 0, 1u << 16);
    mbar_wait_bounded(bar0 + 8, 0, 1u << 16);
  }

  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);

  if (p.n_splits == 1) {
    const float i_lo = l_lo > 0.f ? 1.f / l_lo : 0.f, i_hi = l_hi > 0.f ? 1.f / l_hi : 0.f;
    auto o_ptr = [&](int r) {
      int n = r / p.G, j = r - n * p.G;
      return p.out + ((q_row0 + n) * p.Hq + g * p.G + j) * 128;
    };
    uint32_t* olo = reinterpret_cast<uint32_t*>(o_ptr(v_lo ? r_lo : 0));
    uint32_t* ohi = reinterpret_cast<uint32_t*>(o_ptr(v_hi ? r_hi : 0));
#pragma unroll
    for (int nd = 0; nd < 16; ++nd) {
      const int w = nd * 4 + (lane & 3);
      if (v_lo) olo[w] = pack_bf16(oacc[nd][0] * i_lo, oacc[nd][1] * i_lo);
      if (v_hi) ohi[w] = pack_bf16(oacc[nd][2] * i_hi, oacc[nd][3] * i_hi);
    }
  } else {
    const long long unit = blockIdx.x;
    float* po = p.part_o + unit * ATT_ROWS * 128;
    float* pml = p.part_ml + unit * ATT_ROWS * 2;
    const int rl = warp * 16 + (lane >> 2), rh = rl + 8;
#pragma unroll
    for (int nd = 0; nd < 16; ++nd) {
      const int d = nd * 8 + (lane & 3) * 2;
      *reinterpret_cast<float2*>(po + rl * 128 + d) = make_float2(oacc[nd][0], oacc[nd][1]);
      *reinterpret_cast<float2*>(po + rh * 128 + d) = make_float2(oacc[nd][2], oacc[nd][3]);
    }
    if ((lane & 3) == 0) {
      pml[rl * 2] = m_lo;
      pml[rl * 2 + 1] = l_lo;
      pml[rh * 2] = m_hi;
      pml[rh * 2 + 1] = l_hi;
    }
  }
}

// Merge the split-KV partials of one 128-row tile: out = sum_i w_i O_i / sum_i w_i l_i,
// w_i = 2^(m_i - max m).  grid = (MT, Hkv, layers); 4 warps, a warp per row, float4 per lane.
__global__ void __launch_bounds__(128) combine_kernel(const AttParams p) {
  const int mtg = blockIdx.x, g = blockIdx.y, lrel = blockIdx.z;
  const int l = p.layer0 + lrel;
  int qi, mt;
  decode_mtile(p.qb, p.G, mtg, qi, mt);
  const int rows_total = (p.qb.cu[qi + 1] - p.qb.cu[qi]) * p.G;
  const int m0 = mt * ATT_ROWS;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long q_row0 = ((long long)l * p.qb.sumNq + p.qb.cu[qi]);
  for (int r = warp; r < ATT_ROWS && m0 + r < rows_total; r += 4) {
    float M = -INFINITY;
    for (int s = 0; s < p.n_splits; ++s) {
      const long long unit = (((long long)lrel * p.Hkv + g) * p.n_splits + s) * p.MT + mtg;
      M = fmaxf(M, p.part_ml[(unit * ATT_ROWS + r) * 2]);
    }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    for (int s = 0; s < p.n_splits; ++s) {
      const long long unit = (((long long)lrel * p.Hkv + g) * p.n_splits + s) * p.MT + mtg;
      const float m = p.part_ml[(unit * ATT_ROWS + r) * 2], ls = p.part_ml[(unit * ATT_ROWS + r) * 2 + 1];
      const float w = (m == -INFINITY) ? 0.f : ex2(m - M);
      const float4 o = *reinterpret_cast<const float4*>(p.part_o + (unit * ATT_ROWS + r) * 128 + lane * 4);
      acc.x += w * o.x;
      acc.y += w * o.y;
      acc.z += w * o.z;
      acc.w += w * o.w;
      den += w * ls;
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
    const int rr = m0 + r;
    const int n = rr / p.G, j = rr - n * p.G;
    uint2 packed;
    packed.x = pack_bf16(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(p.out + ((q_row0 + n) * p.Hq + g * p.G + j) * 128 + lane * 4) = packed;
  }
}

int total_mtiles(const QBatch& qb, int G) {
  int t = 0;
  for (int i = 0; i < qb.nQ; ++i) t += ((qb.cu[i + 1] - qb.cu[i]) * G + ATT_ROWS - 1) / ATT_ROWS;
  return t;
}

// Split count: fill the 148 SMs evenly (one CTA per SM) with as few splits as reach ~95% of the
// best wave efficiency, bounded by the partial buffer.
int choose_splits(long long base, int ncf, size_t cap_units) {
  if (base >= 8 * 148) return 1;
  int best = 1;
  double best_eff = 0.0;
  const int max_s = ncf < 16 ? ncf : 16;
  for (int s = 1; s <= max_s; ++s) {
    long long ctas = base * s;
    if (s > 1 && (size_t)ctas > cap_units) break;
    double waves = (double)ctas / 148.0;
    double eff = waves / (double)((ctas + 147) / 148);
    if (eff > best_eff * 1.04) {
      best_eff = eff;
      best = s;
    }
  }
  return best;
}

}  // namespace

cudaError_t rekv_launch_attend_mma(rekv_ctx* c, const void* q, const QBatch& qb, int ncf, int layer0, int layer1,
                                   void* out, cudaStream_t st, bool timed, const AttendFullArgs* full) {
  if (full) return cudaErrorNotSupported;  // Eq. 3 in full runs on the tcgen05 kernel only
  const StoreView& s = c->sv;
  AttParams p;
  p.q = (const __nv_bfloat16*)q;
  p.out = (__nv_bfloat16*)out;
  p.tbl = c->ctx_tbl;
  p.part_o = c->part_o;
  p.part_ml = c->part_ml;
  p.status = c->status;
  p.qb = qb;
  p.Hq = s.Hq;
  p.Hkv = s.Hkv;
  p.G = s.G;
  p.Nf = s.Nf;
  p.Npad = (s.Nf + 15) & ~15;
  p.ncf = ncf;
  p.MT = total_mtiles(qb, s.G);
  p.layer0 = layer0;
  p.scale_log2 = 1.4426950408889634f / sqrtf(128.f);
  const long long base = (long long)(layer1 - layer0) * s.Hkv * p.MT;
  p.n_splits = choose_splits(base, ncf, c->part_units);
  const size_t smem = 4u * 2u * p.Npad * 128u + 16 + 1024;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attend_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  if (timed) cudaEventRecord(c->ev_t0, st);
  attend_mma_kernel<<<(unsigned)(base * p.n_splits), ATT_THREADS, smem, st>>>(p);
  if (timed) {
    cudaEventRecord(c->ev_t1, st);
    c->timing_valid = true;
  }
  c->launches += 1;
  if (p.n_splits > 1) {
    combine_kernel<<<dim3(p.MT, s.Hkv, layer1 - layer0), 128, 0, st>>>(p);
    c->launches += 1;
  }
  return cudaGetLastError();
}
