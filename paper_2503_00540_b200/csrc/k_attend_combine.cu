// Step 5 (Eq. 3): merge of the partials that the attention kernels leave for units worked on in several parts.
#include "attend_common.cuh"

using namespace rekv_ptx;

namespace rekv_att {

// Merge the partials of the units that were cut by a CTA boundary.
// grid = (units, 2 row tiles, 32 groups of 4 rows); a warp per row, float4 per lane: one short
// dependent chain per warp, enough warps in flight to hide its latency.
__global__ void __launch_bounds__(128) combine_tc5_kernel(const TcParams p) {
  // When units are not cut (per == ncf) only the units with one row tile have partials (their two half-streams): the
  // grid then counts those units only -- blockIdx.x = ((layer, kv head) * n_split + rank among the batch's such
  // questions) -- instead of every unit of a large batch, most of which would have nothing to do.
  long long u = blockIdx.x;
  if (p.per == p.ncf) {
    const int rank = (int)(blockIdx.x % p.n_split);
    const long long lg = blockIdx.x / p.n_split;   // (layer - layer0) * H_kv + kv head
    int mp = 0, seen = 0, found = -1;
    for (int qi = 0; qi < p.qb.nQ; ++qi) {  // the rank-th question whose last unit has one row tile: that unit
      const int rows = (p.qb.cu[qi + 1] - p.qb.cu[qi]) * p.G;
      const int units_q = (rows + 255) / 256;
      if (((rows - 1) & 255) < 128) {
        if (seen == rank) {
          found = mp + units_q - 1;
          break;
        }
        ++seen;
      }
      mp += units_q;
    }
    if (found < 0) return;
    u = lg * p.MP + found;
  }
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

}  // namespace rekv_att
