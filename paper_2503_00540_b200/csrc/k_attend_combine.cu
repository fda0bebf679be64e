// Step 5 (Eq. 3): merge of the partials that the attention kernels leave for units worked on in several parts.
#include "attend_common.cuh"

using namespace rekv_ptx;

namespace rekv_att {

// The unit a block of the merge kernels works on, from blockIdx.x.  When units are not cut (per == ncf) only the units
// with one row tile have partials (their two half-streams): the grid then counts those units only -- blockIdx.x =
// ((layer, kv head) * n_split + rank among the batch's such questions) -- instead of every unit of a large batch, most
// of which would have nothing to do.  Returns -1 if there is none.
__device__ __forceinline__ long long combine_unit(const TcParams& p) {
  if (p.per != p.ncf) return blockIdx.x;
  const int rank = (int)(blockIdx.x % p.n_split);
  const long long lg = blockIdx.x / p.n_split;   // (layer - layer0) * H_kv + kv head
  int mp = 0, seen = 0;
  for (int qi = 0; qi < p.qb.nQ; ++qi) {  // the rank-th question whose last unit has one row tile: that unit
    const int rows = (p.qb.cu[qi + 1] - p.qb.cu[qi]) * p.G;
    const int units_q = (rows + 255) / 256;
    if (((rows - 1) & 255) < 128) {
      if (seen == rank) return lg * p.MP + mp + units_q - 1;
      ++seen;
    }
    mp += units_q;
  }
  return -1;
}

// Merge the partials of the units that were cut by a CTA boundary.
// grid = (units, 2 row tiles, 32 groups of 4 rows); a warp per row, float4 per lane: one short
// dependent chain per warp, enough warps in flight to hide its latency.
__global__ void __launch_bounds__(128) combine_tc5_kernel(const TcParams p) {
  const long long u = combine_unit(p);
  if (u < 0) return;
  const int t = blockIdx.y;
  const long long c_first = (u * p.ncf) / p.per, c_last = ((u + 1) * p.ncf - 1) / p.per;
  const UnitInfo ui = decode_unit(p, u);
  if (c_first == c_last && !ui.split) return;  // the unit was produced whole by one CTA
  if (t >= ui.tiles) return;
  // parts of this (unit, row tile): one per CTA that worked on the unit -- two per CTA, the half-streams, for a
  // unit with one row tile -- each in its partial slot
  const int n_parts = (int)(c_last - c_first + 1) * (ui.split ? 2 : 1);
  auto slot_of = [&](int k) -> long long {
    const long long c = c_first + (ui.split ? k >> 1 : k);
    const long long base = p.per == p.ncf ? (long long)ui.srank : c + u;
    return base * 2 + (ui.split ? (k & 1) : t);
  };
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  grid_dep_wait();
  {
    const int r = blockIdx.z * 4 + warp;
    const int rr = ui.m0 + t * 128 + r;
    if (rr >= ui.rows_q) return;
    const int n = rr / p.G, j = rr - n * p.G;
    const long long out_row = (ui.q_row0 + n) * p.Hq + ui.g * p.G + j;
    // the parts' maxima: a lane per part (independent loads), then the warp's maximum
    float M = p.self_o ? p.self_ml[out_row * 2] : -INFINITY;
    for (int k = lane; k < n_parts; k += 32) M = fmaxf(M, p.part_ml[(slot_of(k) * 128 + r) * 2]);
    for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    if (p.self_o) {  // Eq. 3 in full: the part over the tokens of X is one more partial
      const float w = ex2(p.self_ml[out_row * 2] - M);
      const float4 o = *reinterpret_cast<const float4*>(p.self_o + out_row * 128 + lane * 4);
      acc = make_float4(w * o.x, w * o.y, w * o.z, w * o.w);
      den = w * p.self_ml[out_row * 2 + 1];
    }
    // the numerators, four parts' rows in flight, added in part order
    for (int k0 = 0; k0 < n_parts; k0 += 4) {
      float4 o[4];
      float m[4], ls[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (k0 + i < n_parts) {
          const long long base = slot_of(k0 + i) * 128 + r;
          m[i] = p.part_ml[base * 2];
          ls[i] = p.part_ml[base * 2 + 1];
          o[i] = *reinterpret_cast<const float4*>(p.part_o + base * 128 + lane * 4);
        }
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (k0 + i < n_parts) {
          const float w = ex2(m[i] - M);
          acc.x += w * o[i].x;
          acc.y += w * o[i].y;
          acc.z += w * o[i].z;
          acc.w += w * o[i].w;
          den += w * ls[i];
        }
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
    uint2 packed;
    packed.x = pack_bf16(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(p.out + out_row * 128 + lane * 4) = packed;
  }
}

// The same for units of many parts (a launch of few units, such as one layer, spreads each unit over dozens of CTAs).
// grid = (units, 2 row tiles, 32 groups of 4 rows), 4 warps, float4 of the 128 columns per lane.
__global__ void __launch_bounds__(128) combine_many_kernel(const TcParams p) {
  const long long u = combine_unit(p);
  if (u < 0) return;
  const int t = blockIdx.y;
  const long long c_first = (u * p.ncf) / p.per, c_last = ((u + 1) * p.ncf - 1) / p.per;
  const UnitInfo ui = decode_unit(p, u);
  if (c_first == c_last && !ui.split) return;  // the unit was produced whole by one CTA
  if (t >= ui.tiles) return;
  // parts of this (unit, row tile): one per CTA that worked on the unit -- two per CTA, the half-streams, for a
  // unit with one row tile -- each in its partial slot
  const int n_parts = (int)(c_last - c_first + 1) * (ui.split ? 2 : 1);
  auto slot_of = [&](int k) -> long long {
    const long long c = c_first + (ui.split ? k >> 1 : k);
    const long long base = p.per == p.ncf ? (long long)ui.srank : c + u;
    return base * 2 + (ui.split ? (k & 1) : t);
  };
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // The block joins four rows.  Each warp takes every fourth part of all four rows -- up to six parts of four rows
  // in flight per lane, so that a unit of two dozen parts is one or two rounds of loads deep instead of six -- and
  // keeps a running (max, numerator, sum) per row; the four warps' results meet in shared memory, where warp a
  // finishes row a (the part over the tokens of X joins there).  Fixed order throughout.
  __shared__ float4 s_acc[4][4][32];
  __shared__ float s_m[4][4], s_den[4][4];
  grid_dep_wait();
  const int r0 = blockIdx.z * 4;
  const int rr0 = ui.m0 + t * 128 + r0;
  if (rr0 >= ui.rows_q) return;  // (the whole block)
  {
    float M[4], den[4];
    float4 acc[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      M[a] = -1e30f;  // (not -inf: 2^(m - M) of a part without tokens, m = -inf, is then a plain 0)
      den[a] = 0.f;
      acc[a] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    constexpr int ROUND = 6;
    for (int k0 = warp; k0 < n_parts; k0 += 4 * ROUND) {
      float2 ml[ROUND][4];
      float4 o[ROUND][4];
#pragma unroll
      for (int i = 0; i < ROUND; ++i) {
        const int k = k0 + 4 * i;
        if (k < n_parts) {
          const long long base = slot_of(k) * 128 + r0;
#pragma unroll
          for (int a = 0; a < 4; ++a) {
            ml[i][a] = *reinterpret_cast<const float2*>(p.part_ml + (base + a) * 2);
            o[i][a] = *reinterpret_cast<const float4*>(p.part_o + (base + a) * 128 + lane * 4);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < ROUND; ++i) {
        const int k = k0 + 4 * i;
        if (k < n_parts) {
#pragma unroll
          for (int a = 0; a < 4; ++a) {
            const float mn = fmaxf(M[a], ml[i][a].x);
            const float sc = ex2(M[a] - mn), w = ex2(ml[i][a].x - mn);
            acc[a].x = fmaf(w, o[i][a].x, acc[a].x * sc);
            acc[a].y = fmaf(w, o[i][a].y, acc[a].y * sc);
            acc[a].z = fmaf(w, o[i][a].z, acc[a].z * sc);
            acc[a].w = fmaf(w, o[i][a].w, acc[a].w * sc);
            den[a] = fmaf(w, ml[i][a].y, den[a] * sc);
            M[a] = mn;
          }
        }
      }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      s_acc[warp][a][lane] = acc[a];
      if (lane == 0) {
        s_m[warp][a] = M[a];
        s_den[warp][a] = den[a];
      }
    }
  }
  __syncthreads();
  {
    const int rr = rr0 + warp;  // warp a finishes row a
    if (rr >= ui.rows_q) return;
    const int n = rr / p.G, j = rr - n * p.G;
    const long long out_row = (ui.q_row0 + n) * p.Hq + ui.g * p.G + j;
    float M = p.self_o ? fmaxf(-1e30f, p.self_ml[out_row * 2]) : -1e30f;
#pragma unroll
    for (int w = 0; w < 4; ++w) M = fmaxf(M, s_m[w][warp]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    if (p.self_o) {  // Eq. 3 in full: the part over the tokens of X is one more partial
      const float w = ex2(p.self_ml[out_row * 2] - M);
      const float4 o = *reinterpret_cast<const float4*>(p.self_o + out_row * 128 + lane * 4);
      acc = make_float4(w * o.x, w * o.y, w * o.z, w * o.w);
      den = w * p.self_ml[out_row * 2 + 1];
    }
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float sc = ex2(s_m[w][warp] - M);
      const float4 o = s_acc[w][warp][lane];
      acc.x = fmaf(sc, o.x, acc.x);
      acc.y = fmaf(sc, o.y, acc.y);
      acc.z = fmaf(sc, o.z, acc.z);
      acc.w = fmaf(sc, o.w, acc.w);
      den = fmaf(sc, s_den[w][warp], den);
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
    uint2 packed;
    packed.x = pack_bf16(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(p.out + out_row * 128 + lane * 4) = packed;
  }
}

}  // namespace rekv_att
