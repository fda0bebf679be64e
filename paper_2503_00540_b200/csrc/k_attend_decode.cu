#include <algorithm>

#include "attend_common.cuh"

using namespace rekv_ptx;

namespace rekv_att {

// Step 5 (Eq. 3) for few query rows per KV head (decode steps: N_q * G <= 16): the step is bound by reading the
// context, not by the contraction (AI ~ G FLOP/B), so this kernel only has to keep the loads in flight.  Same work
// decomposition as the tensor-core kernel (contiguous ranges of (unit, frame) steps, partials merged by the same kernel),
// but a frame's K and V tiles are double-buffered whole (two frames in flight per SM) and the 16-row
// tile is worked on by eight warps that split the frame's tokens among themselves with mma.sync
// (m16n8k16, ldmatrix straight from the swizzled tiles); their (max, sum, O) are merged through shared
// memory at the end of a range.

// Self-check of an address or index before it is used: a violation is recorded in the status word (read by
// rekv_check_status as error -(1000 + code)) and the access is skipped instead of faulting.
#define DEC_GUARD(cond, code) ((cond) ? true : (atomicExch(p.status, -(1000 + (code))), false))
__global__ void __launch_bounds__(DEC_THREADS, 1) attend_decode_kernel(const TcParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t s_base = smem_u32(smem);
  const uint32_t tile_bytes = 2u * p.Npad * 128u;  // one K (or V) head tile: two 64-dim halves
  const uint32_t half_stride = p.Npad * 128u;
  const uint32_t ring_bytes = max(4u * tile_bytes, DEC_SCRATCH);  // the merge scratch reuses the ring
  const uint32_t bar0 = s_base + ring_bytes;  // full[stage]
  volatile uint32_t* s_abort = reinterpret_cast<volatile uint32_t*>(smem + ring_bytes + 16);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  {  // zero the pad rows [Nf, Npad) of every tile half once; bulk copies never touch them
    const int pad_rows = p.Npad - p.Nf;
    const int n16 = 8 * pad_rows * 8;  // (stage, K/V, half) x rows x 16-byte chunks
    for (int i = tid; i < n16; i += DEC_THREADS) {
      const int c = i & 7, r = (i >> 3) % pad_rows, hh = (i >> 3) / pad_rows;
      *reinterpret_cast<uint4*>(smem + (hh >> 1) * tile_bytes + (hh & 1) * half_stride + (p.Nf + r) * 128 + c * 16) =
          make_uint4(0, 0, 0, 0);
    }
  }
  if (tid == 0) {
    mbar_init(bar0, 1);
    mbar_init(bar0 + 8, 1);
    *s_abort = 0;
    fence_barrier_init();
  }
  fence_proxy_async();
  __syncthreads();
  grid_dep_wait();
  grid_dep_launch();

  const uint32_t half_bytes = (uint32_t)p.Nf * 128u;
  // this warp's tokens of a frame: whole 16-token units, spread as evenly as they go
  const int nu = p.Npad >> 4;
  const int u0 = warp * nu / DEC_WARPS, u1 = (warp + 1) * nu / DEC_WARPS;
  const int t_begin = u0 * 16, n_blk = (u1 - u0) * 2;  // 8-token blocks of this warp (<= 4 for N_f <= 256)
  const int lm = lane >> 3, lr = lane & 7;              // ldmatrix: matrix index and row within it

  long long pos = (long long)blockIdx.x * p.per;
  const long long end = min(pos + (long long)p.per, p.total);
  uint32_t cnt = 0;  // frames consumed so far by this CTA: stage = cnt & 1, phase = (cnt >> 1) & 1
  uint32_t issued = 0;  // thread 0: frames whose copies have been issued (sequence numbers [0, issued))
  const uint32_t wait_limit = p.wait_limit ? p.wait_limit : (1u << 22);
  bool ok = true;

  while (pos < end && ok) {
    const long long u = pos / p.ncf;
    const int f0 = (int)(pos - u * p.ncf);
    const int nfr = (int)min((long long)(p.ncf - f0), end - pos);
    const UnitInfo ui = decode_unit(p, u);
    char* const* pages = p.tbl + ((long long)ui.l * p.qb.nQ + ui.qi) * p.ncf + f0;
    char* const* pages_k = p.tbl_k ? p.tbl_k + ((long long)ui.l * p.qb.nQ + ui.qi) * p.ncf + f0 : nullptr;
    const bool whole_unit = (nfr == p.ncf);
    auto issue = [&](int i) {  // frame i of this range into stage (cnt + i) & 1
      const uint32_t st = (cnt + i) & 1;
      const char* kt = pages[i] + (long long)(ui.g * 2) * p.Nf * 256;
      const char* ks = pages_k ? pages_k[i] + (long long)ui.g * 2 * half_bytes : kt;
      const uint32_t bar = bar0 + 8 * st;
      const uint32_t dst = s_base + st * 2u * tile_bytes;
      issued = cnt + i + 1;
      if (p.skip_copy_entry >= 0 && blockIdx.x == 0 && (int)(cnt + i) == p.skip_copy_entry) return;  // test-only
      if (!DEC_GUARD(pages[i] != nullptr && (reinterpret_cast<uintptr_t>(kt) & 15) == 0 &&
                     (reinterpret_cast<uintptr_t>(ks) & 15) == 0 && (half_bytes & 15) == 0, 1)) return;
      if (!DEC_GUARD(dst + 2u * tile_bytes <= s_base + ring_bytes && (dst & 15) == 0 && (half_stride & 15) == 0, 2)) return;
      mbar_expect_tx(bar, 4u * half_bytes);
      bulk_g2s(dst, ks, half_bytes, bar);
      bulk_g2s(dst + half_stride, ks + half_bytes, half_bytes, bar);
      bulk_g2s(dst + tile_bytes, kt + 2 * half_bytes, half_bytes, bar);
      bulk_g2s(dst + tile_bytes + half_stride, kt + 3 * half_bytes, half_bytes, bar);
    };
    if (tid == 0) {
      issue(0);
      if (nfr > 1) issue(1);
    }
    // Q fragments of the 16-row tile (every warp holds the same rows)
    const int r_lo = lane >> 2, r_hi = r_lo + 8;
    const bool v_lo = r_lo < ui.rows_q, v_hi = r_hi < ui.rows_q;
    auto row_index = [&](int r) {
      const int n = r / p.G, j = r - n * p.G;
      return (ui.q_row0 + n) * p.Hq + ui.g * p.G + j;
    };
    uint32_t qf[8][4];
    {
      const uint32_t* plo = reinterpret_cast<const uint32_t*>(p.q + row_index(v_lo ? r_lo : 0) * 128);
      const uint32_t* phi = reinterpret_cast<const uint32_t*>(p.q + row_index(v_hi ? r_hi : 0) * 128);
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

    for (int i = 0; i < nfr; ++i) {
      const uint32_t st = (cnt + i) & 1;
      bool got = false;
      for (uint32_t it = 0; it < wait_limit; ++it) {
        if (mbar_try_wait(bar0 + 8 * st, ((cnt + i) >> 1) & 1)) {
          got = true;
          break;
        }
        if (*s_abort) break;
        if (it > 2048) __nanosleep(64);
      }
      if (!got) {
        *s_abort = 1;
        ok = false;
      }
      if (ok && n_blk > 0) {
        const uint32_t sK = s_base + st * 2u * tile_bytes, sV = sK + tile_bytes;
        float sacc[4][4];
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) {
          sacc[nb][0] = sacc[nb][1] = sacc[nb][2] = sacc[nb][3] = 0.f;
          if (nb < n_blk) {
            const int tok = t_begin + nb * 8 + lr;
#pragma unroll
            for (int kp = 0; kp < 4; ++kp) {
              const int c = kp * 4 + lm;  // 16-byte chunk (8 dims) of the 128-dim row
              const uint32_t addr = sK + (c >> 3) * half_stride + tok * 128 + (((c & 7) ^ (tok & 7)) << 4);
              uint32_t b0 = 0, b1 = 0, b2 = 0, b3 = 0;
              if (DEC_GUARD(addr + 16 <= s_base + ring_bytes && (addr & 15) == 0, 3)) ldmatrix_x4(b0, b1, b2, b3, addr);
              mma_bf16_16816(sacc[nb], qf[2 * kp], b0, b1);
              mma_bf16_16816(sacc[nb], qf[2 * kp + 1], b2, b3);
            }
          }
        }
        float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
        for (int nb = 0; nb < 4; ++nb)
          if (nb < n_blk) {
            const int col = t_begin + nb * 8 + (lane & 3) * 2;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              float sc = sacc[nb][e] * p.scale_log2;
              if (col + (e & 1) >= p.Nf) sc = -INFINITY;  // the frame's pad tokens
              sacc[nb][e] = sc;
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
        if (__any_sync(0xffffffffu, a_lo != 1.f || a_hi != 1.f)) {
#pragma unroll
          for (int nd = 0; nd < 16; ++nd) {
            oacc[nd][0] *= a_lo;
            oacc[nd][1] *= a_lo;
            oacc[nd][2] *= a_hi;
            oacc[nd][3] *= a_hi;
          }
        }
        uint32_t pf[4][2];
#pragma unroll
        for (int nb = 0; nb < 4; ++nb)
          if (nb < n_blk) {
            const float p0 = ex2(sacc[nb][0] - mn_lo), p1 = ex2(sacc[nb][1] - mn_lo);
            const float p2 = ex2(sacc[nb][2] - mn_hi), p3 = ex2(sacc[nb][3] - mn_hi);
            l_lo += p0 + p1;
            l_hi += p2 + p3;
            pf[nb][0] = pack_bf16(p0, p1);
            pf[nb][1] = pack_bf16(p2, p3);
          }
#pragma unroll
        for (int kb = 0; kb < 2; ++kb)
          if (2 * kb < n_blk) {
            const uint32_t a[4] = {pf[2 * kb][0], pf[2 * kb][1], pf[2 * kb + 1][0], pf[2 * kb + 1][1]};
            const int tok = t_begin + kb * 16 + (lm & 1) * 8 + lr;
#pragma unroll
            for (int dp = 0; dp < 8; ++dp) {
              const int c = dp * 2 + (lm >> 1);
              const uint32_t addr = sV + (c >> 3) * half_stride + tok * 128 + (((c & 7) ^ (tok & 7)) << 4);
              uint32_t b0 = 0, b1 = 0, b2 = 0, b3 = 0;
              if (DEC_GUARD(addr + 16 <= s_base + ring_bytes && (addr & 15) == 0, 4)) ldmatrix_x4_trans(b0, b1, b2, b3, addr);
              mma_bf16_16816(oacc[2 * dp], a, b0, b1);
              mma_bf16_16816(oacc[2 * dp + 1], a, b2, b3);
            }
          }
      }
      __syncthreads();  // every warp is done with this stage
      if (*s_abort) ok = false;
      if (ok && tid == 0 && i + 2 < nfr) issue(i + 2);
    }
    if (!ok) {
      // a copy never completed: record it and give the copies still in flight -- the last two frames issued, one
      // per stage -- a bounded chance to land before the CTA's shared memory is given up
      if (tid == 0) {
        atomicExch(p.status, REKV_ERR_TIMEOUT);
        for (uint32_t e = issued > 2 ? issued - 2 : 0; e < issued; ++e)
          for (uint32_t it = 0; it < wait_limit && !mbar_try_wait(bar0 + 8 * (e & 1), (e >> 1) & 1); ++it)
            __nanosleep(64);
      }
      __syncthreads();
      break;
    }
    cnt += nfr;

    // ---- merge the eight warps' parts through shared memory (no copy is in flight now) ----
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    float* sm_o = reinterpret_cast<float*>(smem);                      // [warp][16 rows][128]
    float* sm_ml = sm_o + DEC_WARPS * 16 * 128;                        // [warp][16 rows][2]
    {
      float* wo = sm_o + warp * 16 * 128;
#pragma unroll
      for (int nd = 0; nd < 16; ++nd) {
        const int d = nd * 8 + (lane & 3) * 2;
        *reinterpret_cast<float2*>(wo + r_lo * 128 + d) = make_float2(oacc[nd][0], oacc[nd][1]);
        *reinterpret_cast<float2*>(wo + r_hi * 128 + d) = make_float2(oacc[nd][2], oacc[nd][3]);
      }
      if ((lane & 3) == 0) {
        float* wm = sm_ml + warp * 32;
        wm[r_lo * 2] = m_lo;
        wm[r_lo * 2 + 1] = l_lo;
        wm[r_hi * 2] = m_hi;
        wm[r_hi * 2 + 1] = l_hi;
      }
    }
    __syncthreads();
    {
      const int r = tid >> 4, d0 = (tid & 15) * 8;  // 16 threads per row, 8 dims each
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, sm_ml[w * 32 + r * 2]);
      float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      float den = 0.f;
#pragma unroll
      for (int w = 0; w < DEC_WARPS; ++w) {
        const float wt = ex2(sm_ml[w * 32 + r * 2] - M);  // a warp without tokens has max -inf, weight 0
        den += wt * sm_ml[w * 32 + r * 2 + 1];
        const float4 x = *reinterpret_cast<const float4*>(sm_o + (w * 16 + r) * 128 + d0);
        const float4 y = *reinterpret_cast<const float4*>(sm_o + (w * 16 + r) * 128 + d0 + 4);
        acc[0] += wt * x.x; acc[1] += wt * x.y; acc[2] += wt * x.z; acc[3] += wt * x.w;
        acc[4] += wt * y.x; acc[5] += wt * y.y; acc[6] += wt * y.z; acc[7] += wt * y.w;
      }
      if (r < ui.rows_q && DEC_GUARD(ui.rows_q <= 16 && ui.qi < p.qb.nQ && ui.g < p.Hkv && ring_bytes >= DEC_SCRATCH, 6)) {
        const long long out_row = row_index(r);
        if (whole_unit) {
          if (p.self_o) {  // Eq. 3 in full: the part over the tokens of X joins here
            const float m_x = p.self_ml[out_row * 2], l_x = p.self_ml[out_row * 2 + 1];
            const float M2 = fmaxf(M, m_x);
            const float w_c = ex2(M - M2), w_x = ex2(m_x - M2);
            const float4 x = *reinterpret_cast<const float4*>(p.self_o + out_row * 128 + d0);
            const float4 y = *reinterpret_cast<const float4*>(p.self_o + out_row * 128 + d0 + 4);
            acc[0] = acc[0] * w_c + x.x * w_x; acc[1] = acc[1] * w_c + x.y * w_x;
            acc[2] = acc[2] * w_c + x.z * w_x; acc[3] = acc[3] * w_c + x.w * w_x;
            acc[4] = acc[4] * w_c + y.x * w_x; acc[5] = acc[5] * w_c + y.y * w_x;
            acc[6] = acc[6] * w_c + y.z * w_x; acc[7] = acc[7] * w_c + y.w * w_x;
            den = den * w_c + l_x * w_x;
          }
          const float inv = den > 0.f ? 1.f / den : 0.f;
          uint4 o;
          o.x = pack_bf16(acc[0] * inv, acc[1] * inv);
          o.y = pack_bf16(acc[2] * inv, acc[3] * inv);
          o.z = pack_bf16(acc[4] * inv, acc[5] * inv);
          o.w = pack_bf16(acc[6] * inv, acc[7] * inv);
          *reinterpret_cast<uint4*>(p.out + out_row * 128 + d0) = o;
        } else if (DEC_GUARD(((long long)blockIdx.x + u) * 2 < 2048, 5)) {
          const long long slot = ((long long)blockIdx.x + u) * 2;
          float* po = p.part_o + (slot * 128 + r) * 128 + d0;
          __stcg(reinterpret_cast<float4*>(po), make_float4(acc[0], acc[1], acc[2], acc[3]));
          __stcg(reinterpret_cast<float4*>(po + 4), make_float4(acc[4], acc[5], acc[6], acc[7]));
          if ((tid & 15) == 0) {
            __stcg(p.part_ml + (slot * 128 + r) * 2, M);
            __stcg(p.part_ml + (slot * 128 + r) * 2 + 1, den);
          }
        }
      }
    }
    if (!whole_unit && p.unit_cnt) {
      // The range covered a part of the unit.  The CTA that finishes a unit's last part merges all of them
      // (no further launch): parts are published with a fence, counted with an atomic, and the counter is
      // left at zero for the next launch.
      volatile int& s_last = *reinterpret_cast<volatile int*>(smem + ring_bytes + 24);  // beside the barriers
      const long long c_first = (u * p.ncf) / p.per, c_last = ((u + 1) * p.ncf - 1) / p.per;
      __threadfence();
      __syncthreads();
      if (tid == 0) {
        const int prev = atomicAdd(p.unit_cnt + u, 1);
        s_last = (prev == (int)(c_last - c_first)) ? 1 : 0;
        if (s_last) p.unit_cnt[u] = 0;
      }
      __syncthreads();
      if (s_last) {
        __threadfence();
        const int r = tid >> 4, d0 = (tid & 15) * 8;
        if (r < ui.rows_q) {
          const long long out_row = row_index(r);
          float M = p.self_o ? p.self_ml[out_row * 2] : -INFINITY;
          for (long long cc = c_first; cc <= c_last; ++cc) M = fmaxf(M, __ldcg(p.part_ml + (((cc + u) * 2) * 128 + r) * 2));
          float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
          float den = 0.f;
          if (p.self_o) {  // Eq. 3 in full: the part over the tokens of X is one more part
            const float wt = ex2(p.self_ml[out_row * 2] - M);
            const float4 x = *reinterpret_cast<const float4*>(p.self_o + out_row * 128 + d0);
            const float4 y = *reinterpret_cast<const float4*>(p.self_o + out_row * 128 + d0 + 4);
            acc[0] = wt * x.x; acc[1] = wt * x.y; acc[2] = wt * x.z; acc[3] = wt * x.w;
            acc[4] = wt * y.x; acc[5] = wt * y.y; acc[6] = wt * y.z; acc[7] = wt * y.w;
            den = wt * p.self_ml[out_row * 2 + 1];
          }
          for (long long c0 = c_first; c0 <= c_last; c0 += 4) {  // four parts in flight, added in part order
            float4 x[4], y[4];
            float pm[4], pl[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
              if (c0 + i <= c_last) {
                const long long base = ((c0 + i + u) * 2) * 128 + r;
                pm[i] = __ldcg(p.part_ml + base * 2);
                pl[i] = __ldcg(p.part_ml + base * 2 + 1);
                x[i] = __ldcg(reinterpret_cast<const float4*>(p.part_o + base * 128 + d0));
                y[i] = __ldcg(reinterpret_cast<const float4*>(p.part_o + base * 128 + d0 + 4));
              }
#pragma unroll
            for (int i = 0; i < 4; ++i)
              if (c0 + i <= c_last) {
                const float wt = ex2(pm[i] - M);
                acc[0] += wt * x[i].x; acc[1] += wt * x[i].y; acc[2] += wt * x[i].z; acc[3] += wt * x[i].w;
                acc[4] += wt * y[i].x; acc[5] += wt * y[i].y; acc[6] += wt * y[i].z; acc[7] += wt * y[i].w;
                den += wt * pl[i];
              }
          }
          const float inv = den > 0.f ? 1.f / den : 0.f;
          uint4 o;
          o.x = pack_bf16(acc[0] * inv, acc[1] * inv);
          o.y = pack_bf16(acc[2] * inv, acc[3] * inv);
          o.z = pack_bf16(acc[4] * inv, acc[5] * inv);
          o.w = pack_bf16(acc[6] * inv, acc[7] * inv);
          *reinterpret_cast<uint4*>(p.out + out_row * 128 + d0) = o;
        }
      }
    }
    __syncthreads();  // the scratch is a K tile again from here on
    if (p.Npad > p.Nf) {  // the merge scratch covered pad rows of the first tiles: zero them again
      const int pad_rows = p.Npad - p.Nf;
      const int n16 = 8 * pad_rows * 8;
      for (int i = tid; i < n16; i += DEC_THREADS) {
        const int c = i & 7, r = (i >> 3) % pad_rows, hh = (i >> 3) / pad_rows;
        *reinterpret_cast<uint4*>(smem + (hh >> 1) * tile_bytes + (hh & 1) * half_stride + (p.Nf + r) * 128 + c * 16) =
            make_uint4(0, 0, 0, 0);
      }
    }
    fence_proxy_async();  // the next range's bulk copies land where these generic-proxy accesses were
    __syncthreads();
    pos += nfr;
  }
}

}  // namespace rekv_att
