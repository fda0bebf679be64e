// Step 5 (Eq. 3) on the 5th-generation tensor cores: GQA attention of the question tokens over the
// gathered context, read page by page through the context table.
//
// One CTA per SM, persistent over a contiguous range of (unit, context frame) steps ("stream-K"):
// a unit is (layer, kv head, question, pair of 128-row tiles), a row being (question token, query
// head of the KV group).  Each context frame's K and V head tiles are brought in once with
// contiguous bulk copies (the store keeps them in the 128-byte-swizzled operand layout) and applied
// to both row tiles.  Warp roles:
//   warp 0      bulk copies of K/V tiles into a 3-deep shared-memory ring (one lane)
//   warp 1      tcgen05.mma issue (one lane): S = Q K^T into TMEM, O += P V with P read from TMEM
//   warps 2-5   softmax of row tile 0: one thread per row (= TMEM lane), fp32, lazy rescaling of O
//   warps 6-9   softmax of row tile 1 -- the two tiles alternate on the tensor core, so one tile's
//               softmax overlaps the other's matrix products
// TMEM (512 columns): O0 [0,128)  O1 [128,256)  S0/P0 [256,384)  S1/P1 [384,512); P (bf16) overwrites
// the front of its S.  A frame of N_f tokens is processed as one or two token chunks of <= 128.
// A range that does not cover a whole unit leaves (max, sum, O) partials for the combine kernel.
// Every wait is bounded: on expiry the status word is set and the CTA leaves.
#include "ptx_helpers.cuh"
#include "rekv_internal.cuh"

using namespace rekv_ptx;

namespace {

constexpr int TC_THREADS = 320;
constexpr int KV_BUFS = 3;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t Q_TILE_BYTES = 128 * 256;  // 128 rows x 128 dims bf16
constexpr float RESCALE_THRESHOLD = 8.f;      // log2 units: O is rescaled only when the row max grows by > 2^8

struct TcParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  char* const* tbl;
  float* part_o;
  float* part_ml;
  int* status;
  QBatch qb;
  int Hq, Hkv, G, Nf, Npad, NA, NB, ncf, MP, layer0;
  int per;          // (unit, frame) steps per CTA
  long long total;  // units * ncf
  float scale_log2;
};

struct UnitInfo {
  int l, g, qi, m0, rows_q, tiles;
  long long q_row0;
};

__device__ __forceinline__ UnitInfo decode_unit(const TcParams& p, long long u) {
  UnitInfo ui;
  int mpg = (int)(u % p.MP);
  long long r = u / p.MP;
  ui.g = (int)(r % p.Hkv);
  ui.l = p.layer0 + (int)(r / p.Hkv);
  int qi = 0, mp = mpg;
  for (; qi < p.qb.nQ - 1; ++qi) {
    int t = ((p.qb.cu[qi + 1] - p.qb.cu[qi]) * p.G + 255) / 256;
    if (mp < t) break;
    mp -= t;
  }
  ui.qi = qi;
  ui.rows_q = (p.qb.cu[qi + 1] - p.qb.cu[qi]) * p.G;
  ui.m0 = mp * 256;
  ui.tiles = (ui.rows_q - ui.m0 > 128) ? 2 : 1;
  ui.q_row0 = (long long)ui.l * p.qb.sumNq + p.qb.cu[qi];
  return ui;
}

struct Bars {
  uint32_t full[KV_BUFS], empty[KV_BUFS], s_full[2], p_ready[2], pv_done[2];
};

__global__ void __launch_bounds__(TC_THREADS, 1) attend_tc5_kernel(const TcParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t s_base = smem_u32(smem);
  const uint32_t tile_bytes = 2u * p.Npad * 128u;   // one K (or V) head tile: two 64-dim halves
  const uint32_t half_stride = p.Npad * 128u;
  const uint32_t s_q = s_base;                       // two Q row tiles
  const uint32_t s_kv = s_base + 2 * Q_TILE_BYTES;   // ring of KV_BUFS tiles
  const uint32_t s_bar = s_kv + KV_BUFS * tile_bytes;
  Bars bars;
#pragma unroll
  for (int i = 0; i < KV_BUFS; ++i) {
    bars.full[i] = s_bar + 8 * i;
    bars.empty[i] = s_bar + 8 * (KV_BUFS + i);
  }
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    bars.s_full[t] = s_bar + 8 * (2 * KV_BUFS + t);
    bars.p_ready[t] = s_bar + 8 * (2 * KV_BUFS + 2 + t);
    bars.pv_done[t] = s_bar + 8 * (2 * KV_BUFS + 4 + t);
  }
  volatile uint32_t* s_tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + (s_bar - s_base) + 8 * (2 * KV_BUFS + 6));
  volatile uint32_t* s_abort = s_tmem_slot + 1;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- one-time set-up -------------------------------------------------------------------------
  {  // zero the pad rows [Nf, Npad) of every ring tile half; the bulk copies never write them
    const int pad_rows = p.Npad - p.Nf;
    const int n16 = KV_BUFS * 2 * pad_rows * 8;
    for (int i = tid; i < n16; i += TC_THREADS) {
      int c = i & 7;
      int r = (i >> 3) % pad_rows;
      int hh = (i >> 3) / pad_rows;  // (buffer, half)
      *reinterpret_cast<uint4*>(smem + 2 * Q_TILE_BYTES + (hh >> 1) * tile_bytes + (hh & 1) * half_stride +
                                (p.Nf + r) * 128 + c * 16) = make_uint4(0, 0, 0, 0);
    }
  }
  if (tid == 0) {
    for (int i = 0; i < KV_BUFS; ++i) {
      mbar_init(bars.full[i], 1);
      mbar_init(bars.empty[i], 1);
    }
    for (int t = 0; t < 2; ++t) {
      mbar_init(bars.s_full[t], 1);
      mbar_init(bars.p_ready[t], 128);
      mbar_init(bars.pv_done[t], 1);
    }
    *s_abort = 0;
    fence_barrier_init();
  }
  if (warp == 0) {
    tmem_alloc(smem_u32((const void*)s_tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem_slot;
  const uint32_t col_o[2] = {0u, 128u}, col_s[2] = {256u, 384u};

  auto wait = [&](uint32_t bar, uint32_t parity) -> bool {
    for (uint32_t it = 0; it < (1u << 22); ++it) {
      if (mbar_try_wait(bar, parity)) return true;
      if (*s_abort) return false;
      if (it > 2048) __nanosleep(64);
    }
    *s_abort = 1;
    atomicExch(p.status, REKV_ERR_TIMEOUT);
    return false;
  };

  const int cpf = p.NB > 0 ? 2 : 1;                 // token chunks per frame
  const uint32_t half_bytes = (uint32_t)p.Nf * 128u;
  const uint32_t idesc_pv = idesc_bf16(128, 128, 1);

  long long pos = (long long)blockIdx.x * p.per;
  const long long end = min(pos + (long long)p.per, p.total);
  uint32_t ring = 0;    // K/V tiles moved so far (K and V of a frame are consecutive ring entries)
  uint32_t chunk_cnt[2] = {0u, 0u};  // token chunks processed so far, per row tile (barrier phases)

  while (pos < end) {
    const long long u = pos / p.ncf;
    const int f0 = (int)(pos - u * p.ncf);
    const int nfr = (int)min((long long)(p.ncf - f0), end - pos);
    const UnitInfo ui = decode_unit(p, u);
    const int nchunks = nfr * cpf;
    char* const* pages = p.tbl + ((long long)ui.l * p.qb.nQ + ui.qi) * p.ncf + f0;
    const bool whole_unit = (nfr == p.ncf);

    // ---- Q row tiles -> shared memory in the swizzled K-major operand layout -------------------
    if (warp >= 2) {
      const int t = (warp - 2) >> 2;
      const int row = ((warp & 3) << 5) | lane;
      if (t < ui.tiles) {
        const int rr = ui.m0 + t * 128 + row;
        const bool valid = rr < ui.rows_q;
        const int n = rr / p.G, j = rr - n * p.G;
        const uint4* src =
            reinterpret_cast<const uint4*>(p.q + ((ui.q_row0 + (valid ? n : 0)) * p.Hq + ui.g * p.G + (valid ? j : 0)) * 128);
        unsigned char* dst = smem + t * Q_TILE_BYTES + row * 128;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          uint4 x = valid ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
          *reinterpret_cast<uint4*>(dst + (c >> 3) * (Q_TILE_BYTES / 2) + (((c & 7) ^ (row & 7)) << 4)) = x;
        }
      }
      fence_proxy_async();
    }
    __syncthreads();

    if (warp == 0) {
      // ================= copy producer =================
      if (lane == 0) {
        for (int fi = 0; fi < nfr; ++fi) {
          const char* kt = pages[fi] + (long long)(ui.g * 2) * p.Nf * 256;
#pragma unroll
          for (int kv = 0; kv < 2; ++kv) {
            const uint32_t r = ring + 2 * fi + kv;
            const uint32_t b = r % KV_BUFS, use = r / KV_BUFS;
            if (use > 0 && !wait(bars.empty[b], (use - 1) & 1)) break;
            const uint32_t dst = s_kv + b * tile_bytes;
            mbar_expect_tx(bars.full[b], 2u * half_bytes);
            bulk_g2s(dst, kt + (long long)kv * 2 * half_bytes, half_bytes, bars.full[b]);
            bulk_g2s(dst + half_stride, kt + (long long)kv * 2 * half_bytes + half_bytes, half_bytes, bars.full[b]);
          }
          if (*s_abort) break;
        }
      }
      __syncwarp();
    } else if (warp == 1) {
      // ================= MMA issuer =================
      if (lane == 0) {
        bool ok = true;
        auto issue_s = [&](int t, int i) {
          const int fi = i / cpf, part = i - fi * cpf;
          const uint32_t r = ring + 2 * fi, b = r % KV_BUFS;
          const int tok0 = part ? p.NA : 0, N = part ? p.NB : p.NA;
          if (part == 0 && t == 0) ok = ok && wait(bars.full[b], (r / KV_BUFS) & 1);
          if (!ok) return;
          tc_fence_after();
          const uint32_t kb = s_kv + b * tile_bytes + tok0 * 128;
          const uint32_t qb = s_q + t * Q_TILE_BYTES;
          const uint32_t idesc = idesc_bf16(128, N, 0);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint64_t ad = smem_desc_sw128(qb + (kk >> 2) * (Q_TILE_BYTES / 2) + (kk & 3) * 32, 16, 1024);
            const uint64_t bd = smem_desc_sw128(kb + (kk >> 2) * half_stride + (kk & 3) * 32, 16, 1024);
            mma_ss(tmem + col_s[t], ad, bd, idesc, kk > 0);
          }
          tc_commit(bars.s_full[t]);
          if (part == cpf - 1 && t == ui.tiles - 1) tc_commit(bars.empty[b]);  // K tile no longer needed
        };
        auto issue_pv = [&](int t, int i) {
          const int fi = i / cpf, part = i - fi * cpf;
          const uint32_t r = ring + 2 * fi + 1, b = r % KV_BUFS;
          const int tok0 = part ? p.NA : 0, N = part ? p.NB : p.NA;
          if (part == 0 && t == 0) ok = ok && wait(bars.full[b], (r / KV_BUFS) & 1);
          ok = ok && wait(bars.p_ready[t], (chunk_cnt[t] + i) & 1);
          if (!ok) return;
          tc_fence_after();
          const uint32_t vb = s_kv + b * tile_bytes + tok0 * 128;
          for (int kk = 0; kk < N / 16; ++kk) {
            const uint64_t bd = smem_desc_sw128(vb + kk * 2048, half_stride, 1024);
            mma_ts(tmem + col_o[t], tmem + col_s[t] + kk * 8, bd, idesc_pv, (i > 0 || kk > 0));
          }
          tc_commit(bars.pv_done[t]);
          if (part == cpf - 1 && t == ui.tiles - 1) tc_commit(bars.empty[b]);  // V tile no longer needed
        };
        for (int t = 0; t < ui.tiles && ok; ++t) issue_s(t, 0);
        for (int i = 0; i < nchunks && ok; ++i)
          for (int t = 0; t < ui.tiles && ok; ++t) {
            issue_pv(t, i);
            if (i + 1 < nchunks && ok) issue_s(t, i + 1);
          }
      }
      __syncwarp();
    } else {
      // ================= softmax + output, one thread per row =================
      const int t = (warp - 2) >> 2;
      if (t < ui.tiles) {
        const uint32_t lane_base = (uint32_t)((warp & 3) << 5) << 16;
        const int row = ((warp & 3) << 5) | lane;
        const uint32_t t_s = tmem + lane_base + col_s[t];
        const uint32_t t_o = tmem + lane_base + col_o[t];
        float m_used = -INFINITY, l_sum = 0.f;
        bool ok = true;
        for (int i = 0; i < nchunks && ok; ++i) {
          const int part = i % cpf;
          const int tok0 = part ? p.NA : 0, N = part ? p.NB : p.NA;
          const int nv = min(N, p.Nf - tok0);  // valid tokens of this chunk
          const int npc = N >> 4;
          if (!wait(bars.s_full[t], (chunk_cnt[t] + i) & 1)) {
            ok = false;
            break;
          }
          tc_fence_after();
          uint32_t sv[8][16];
#pragma unroll
          for (int pc = 0; pc < 8; ++pc)
            if (pc < npc) tmem_ld16(t_s + pc * 16, sv[pc]);
#pragma unroll
          for (int pc = 0; pc < 8; ++pc)
            if (pc < npc) tmem_wait_ld16(sv[pc]);
          float mx = -INFINITY;
#pragma unroll
          for (int pc = 0; pc < 8; ++pc)
            if (pc < npc) {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (pc * 16 + j < nv) mx = fmaxf(mx, __uint_as_float(sv[pc][j]));
            }
          mx *= p.scale_log2;
          float alpha = 1.f;
          bool need = false;
          if (i == 0) {
            m_used = mx;
          } else if (mx > m_used + RESCALE_THRESHOLD) {
            need = true;
            alpha = ex2(m_used - mx);
            m_used = mx;
          }
          const bool any_need = __any_sync(0xffffffffu, need);
          float psum = 0.f;
#pragma unroll
          for (int pc = 0; pc < 8; ++pc)
            if (pc < npc) {
              uint32_t pk[8];
#pragma unroll
              for (int jj = 0; jj < 8; ++jj) {
                const int c0 = pc * 16 + 2 * jj;
                float p0 = c0 < nv ? ex2(fmaf(__uint_as_float(sv[pc][2 * jj]), p.scale_log2, -m_used)) : 0.f;
                float p1 = c0 + 1 < nv ? ex2(fmaf(__uint_as_float(sv[pc][2 * jj + 1]), p.scale_log2, -m_used)) : 0.f;
                psum += p0 + p1;
                pk[jj] = pack_bf16(p0, p1);
              }
              tmem_st8(t_s + pc * 8, pk);
            }
          l_sum = l_sum * alpha + psum;
          if (any_need) {
            // O of this tile must be at rest: the previous chunk's P V has to be complete
            if (!wait(bars.pv_done[t], (chunk_cnt[t] + i - 1) & 1)) {
              ok = false;
              break;
            }
            tc_fence_after();
#pragma unroll
            for (int pc = 0; pc < 8; ++pc) {
              uint32_t o[16];
              tmem_ld16(t_o + pc * 16, o);
              tmem_wait_ld16(o);
#pragma unroll
              for (int j = 0; j < 16; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
              tmem_st16(t_o + pc * 16, o);
            }
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(bars.p_ready[t]);
        }
        // ---- output of this range: final rows, or a partial for the combine kernel ----
        if (ok && wait(bars.pv_done[t], (chunk_cnt[t] + nchunks - 1) & 1)) {
          tc_fence_after();
          const int rr = ui.m0 + t * 128 + row;
          const bool valid = rr < ui.rows_q;
          const int n = rr / p.G, j = rr - n * p.G;
          if (whole_unit) {
            const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
            uint4* dst = reinterpret_cast<uint4*>(p.out + ((ui.q_row0 + (valid ? n : 0)) * p.Hq + ui.g * p.G + (valid ? j : 0)) * 128);
#pragma unroll
            for (int pc = 0; pc < 8; ++pc) {
              uint32_t o[16];
              tmem_ld16(t_o + pc * 16, o);
              tmem_wait_ld16(o);
              uint4 a, b;
              a.x = pack_bf16(__uint_as_float(o[0]) * inv, __uint_as_float(o[1]) * inv);
              a.y = pack_bf16(__uint_as_float(o[2]) * inv, __uint_as_float(o[3]) * inv);
              a.z = pack_bf16(__uint_as_float(o[4]) * inv, __uint_as_float(o[5]) * inv);
              a.w = pack_bf16(__uint_as_float(o[6]) * inv, __uint_as_float(o[7]) * inv);
              b.x = pack_bf16(__uint_as_float(o[8]) * inv, __uint_as_float(o[9]) * inv);
              b.y = pack_bf16(__uint_as_float(o[10]) * inv, __uint_as_float(o[11]) * inv);
              b.z = pack_bf16(__uint_as_float(o[12]) * inv, __uint_as_float(o[13]) * inv);
              b.w = pack_bf16(__uint_as_float(o[14]) * inv, __uint_as_float(o[15]) * inv);
              if (valid) {
                dst[pc * 2] = a;
                dst[pc * 2 + 1] = b;
              }
            }
          } else {
            const long long slot = ((long long)blockIdx.x + u) * 2 + t;
            float4* po = reinterpret_cast<float4*>(p.part_o + (slot * 128 + row) * 128);
#pragma unroll
            for (int pc = 0; pc < 8; ++pc) {
              uint32_t o[16];
              tmem_ld16(t_o + pc * 16, o);
              tmem_wait_ld16(o);
              if (valid) {
#pragma unroll
                for (int v4 = 0; v4 < 4; ++v4)
                  po[pc * 4 + v4] = make_float4(__uint_as_float(o[4 * v4]), __uint_as_float(o[4 * v4 + 1]),
                                                __uint_as_float(o[4 * v4 + 2]), __uint_as_float(o[4 * v4 + 3]));
              }
            }
            if (valid) {
              p.part_ml[(slot * 128 + row) * 2] = m_used;
              p.part_ml[(slot * 128 + row) * 2 + 1] = l_sum;
            }
          }
        }
      }
    }
    ring += 2 * nfr;
    chunk_cnt[0] += nchunks;
    if (ui.tiles == 2) chunk_cnt[1] += nchunks;
    pos += nfr;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (*s_abort) break;
  }

  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

// Merge the partials of the units that were cut by a CTA boundary.
// grid = (units, 2 row tiles); 4 warps, a warp per row, float4 per lane.
__global__ void __launch_bounds__(128) combine_tc5_kernel(const TcParams p) {
  const long long u = blockIdx.x;
  const int t = blockIdx.y;
  const long long c_first = (u * p.ncf) / p.per, c_last = ((u + 1) * p.ncf - 1) / p.per;
  if (c_first == c_last) return;  // the unit was produced whole by one CTA
  const UnitInfo ui = decode_unit(p, u);
  if (t >= ui.tiles) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int r = warp; r < 128; r += 4) {
    const int rr = ui.m0 + t * 128 + r;
    if (rr >= ui.rows_q) break;
    float M = -INFINITY;
    for (long long c = c_first; c <= c_last; ++c) M = fmaxf(M, p.part_ml[(((c + u) * 2 + t) * 128 + r) * 2]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    for (long long c = c_first; c <= c_last; ++c) {
      const long long base = ((c + u) * 2 + t) * 128 + r;
      const float m = p.part_ml[base * 2], ls = p.part_ml[base * 2 + 1];
      const float w = ex2(m - M);
      const float4 o = *reinterpret_cast<const float4*>(p.part_o + base * 128 + lane * 4);
      acc.x += w * o.x;
      acc.y += w * o.y;
      acc.z += w * o.z;
      acc.w += w * o.w;
      den += w * ls;
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
    const int n = rr / p.G, j = rr - n * p.G;
    uint2 packed;
    packed.x = pack_bf16(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(p.out + ((ui.q_row0 + n) * p.Hq + ui.g * p.G + j) * 128 + lane * 4) = packed;
  }
}

}  // namespace

cudaError_t rekv_launch_attend_tc5(rekv_ctx* c, const void* q, const QBatch& qb, int ncf, int layer0, int layer1,
                                   void* out, cudaStream_t st, bool timed) {
  const StoreView& s = c->sv;
  TcParams p;
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
  if (p.Npad <= 128) {
    p.NA = p.Npad;
    p.NB = 0;
  } else {
    p.NA = ((p.Npad / 2) + 15) & ~15;
    p.NB = p.Npad - p.NA;
  }
  p.ncf = ncf;
  p.layer0 = layer0;
  p.scale_log2 = 1.4426950408889634f / sqrtf(128.f);
  int MP = 0;
  for (int i = 0; i < qb.nQ; ++i) MP += ((qb.cu[i + 1] - qb.cu[i]) * s.G + 255) / 256;
  p.MP = MP;
  const long long units = (long long)(layer1 - layer0) * s.Hkv * MP;
  p.total = units * ncf;
  const int n_sm = 148;
  long long grid;
  if (units >= 4 * n_sm || (size_t)(n_sm + units) * 2 > c->part_units) {
    grid = units;  // enough units to fill the machine: one whole unit per CTA, no partials
    p.per = ncf;
  } else {
    grid = p.total < n_sm ? p.total : n_sm;
    p.per = (int)((p.total + grid - 1) / grid);
    grid = (p.total + p.per - 1) / p.per;
  }
  const size_t smem = 2 * Q_TILE_BYTES + (size_t)KV_BUFS * 2 * p.Npad * 128 + 8 * (2 * KV_BUFS + 6) + 16 + 1024;
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attend_tc5_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  if (timed) cudaEventRecord(c->ev_t0, st);
  attend_tc5_kernel<<<(unsigned)grid, TC_THREADS, smem, st>>>(p);
  if (timed) {
    cudaEventRecord(c->ev_t1, st);
    c->timing_valid = true;
  }
  c->launches += 1;
  if (p.per != ncf) {
    combine_tc5_kernel<<<dim3((unsigned)units, 2), 128, 0, st>>>(p);
    c->launches += 1;
  }
  return cudaGetLastError();
}
