// Step 5 (Eq. 3) on the 5th-generation tensor cores: GQA attention of the question tokens over the
// gathered context, read page by page through the context table.
//
// One CTA per SM, persistent over a contiguous range of (unit, context frame) steps ("stream-K"):
// a unit is (layer, kv head, question, pair of 128-row tiles), a row being (question token, query
// head of the KV group).  Eq. 3 without a positional term does not depend on the order or grouping of the
// context tokens, so the frames of a range are taken as ONE token stream and cut into dense chunks of 128
// tokens that run across frame boundaries: every matrix product has the full width, and a 196-token frame
// costs 1.56 chunk phases instead of two.  In the stream a frame takes N_s = N_f rounded up to a multiple
// of 8 rows, so that a token's row in a chunk tile has the swizzle phase (row & 7) it has in its page: a
// chunk tile is then assembled in shared memory by contiguous bulk copies (the tail of one page's tile
// half, the head of the next), with no layout change in HBM.  The N_s - N_f gap rows between two frames
// and the rows after the range's last token are zeroed in shared memory and their logits masked.
// Warp roles:
//   warp 0      assembles K/V chunk tiles in a 5-deep shared-memory ring (bulk copies, one lane)
//   warp 1      tcgen05.mma issue (one lane): S = Q K^T into TMEM, O += P V with P read from TMEM
//               (warps 2, 3 idle: the service warps form one warpgroup and give their registers up)
//   warps 4-7   softmax of row tile 0: one thread per row (= TMEM lane), fp32
//   warps 8-11  softmax of row tile 1 -- the two tiles alternate on the tensor core, so one tile's
//               softmax overlaps the other's matrix products
// After set-up the service warpgroup shrinks to 88 registers per thread and the softmax warpgroups grow to
// 208 (setmaxnreg), so that a softmax thread holds a whole S row chunk (128 values) at once: one TMEM load
// instruction and one wait per chunk, and two TMEM stores for P.  The exponentials take the row maximum of the
// range's first chunk as their reference; later chunks look for no maximum, and only a row sum beyond 2^60 raises the
// reference and rescales O (rare).  Columns without a token are masked in the one 16-column piece that has some,
// behind a warp-uniform switch.
// TMEM (512 columns): O0 [0,128)  O1 [128,256)  S0/P0 [256,384)  S1/P1 [384,512); P (bf16) overwrites
// the front of its S.
// A range that does not cover a whole unit produces a part of it, (max, sum, O) per row.  When units have two or
// three parts the kernel joins them itself: a tile slot that finds every other part of its unit counted finishes the
// unit from its own O in tensor memory; otherwise it writes its part as a partial and counts it, and the slot whose
// count completes a unit lists it for the end of the CTA's range (see "Merge inside the kernel" below; nobody waits
// for anybody).  With more parts per unit the partials are left for the merge kernels.
// A unit with a single row tile (at most 128 rows: short questions, the remainder of long ones) would leave the
// tensor core idle during its softmax; it runs as two half-streams instead -- both tile slots work on the same rows,
// the token chunks of the context dealt to them alternately, each with its own (max, sum, O) -- which are joined
// like the parts of a cut unit.
// Every wait is bounded: on expiry the status word is set and the CTA leaves.
#include <algorithm>
#include <type_traits>

#include "attend_common.cuh"

using namespace rekv_ptx;
using namespace rekv_att;

namespace {

constexpr int TC_THREADS = 384;
constexpr int SM_WARP0 = 4;                            // first softmax warp
constexpr int REGS_SERVICE = 88, REGS_SOFTMAX = 208;   // 128 * service + 256 * softmax <= 384 * 168
constexpr int KV_BUFS = 5;
constexpr int CHUNK = 128;                             // tokens (stream rows) per chunk
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t Q_TILE_BYTES = 128 * 256;  // 128 rows x 128 dims bf16
constexpr uint32_t HALF_BYTES = CHUNK * 128;  // one 64-dim half of a chunk tile
constexpr uint32_t TILE_BYTES = 2 * HALF_BYTES;
constexpr uint32_t STAGE_ROW_F32 = 144, STAGE_ROW_BF16 = 80;  // epilogue staging rows: a quarter row + 16 bytes (no bank conflicts)
constexpr uint32_t STAGE_WARP_BYTES = 32 * STAGE_ROW_F32;
constexpr float RESCALE_SUM_LIMIT = 1.152921504606846976e18f;  // 2^60: a chunk's row sum beyond it raises the reference maximum
constexpr int PEND_MAX = 8;   // units a CTA can have to merge at the end of its range (two cut units x two row tiles)
constexpr uint32_t WAIT_LIMIT = 1u << 22;
// P is cut (not rounded) to bf16: a value with mantissa m in [1, 2) loses u * 2^-7 / m of itself, u uniform in [0, 1).
// The mantissa of 2^x is log-uniform, E[1/m] = 1 / (2 ln 2), so the mean loss is 0.7213 * 2^-8 of the value, and scaling
// by 1 + 0.7213 * 2^-8 beforehand makes the cut value right on average (its spread equals that of rounding to
// nearest).  log2 of that factor, and its inverse for the row sum:
constexpr float TRUNC_GAIN_LOG2 = 0.0040592f;
constexpr float TRUNC_GAIN_INV = 0.99719028f;

// barrier slots after the K/V ring: full[b], empty[b], s_full[t], p_ready[t], pv_done[t]
struct Bars {
  uint32_t base;
  __device__ __forceinline__ uint32_t full(uint32_t b) const { return base + 8 * b; }
  __device__ __forceinline__ uint32_t empty(uint32_t b) const { return base + 8 * (KV_BUFS + b); }
  __device__ __forceinline__ uint32_t s_full(uint32_t t) const { return base + 8 * (2 * KV_BUFS + t); }
  __device__ __forceinline__ uint32_t p_ready(uint32_t t) const { return base + 8 * (2 * KV_BUFS + 2 + t); }
  __device__ __forceinline__ uint32_t pv_done(uint32_t t) const { return base + 8 * (2 * KV_BUFS + 4 + t); }
};

__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// FULL: Eq. 3 in full (rotated K tiles, the part over X joins in the epilogue).  SPLIT: the launch has units with a
// single row tile, which run as two half-streams (compiled out otherwise: the common loop stays as it was).
// EARLYQ: Q does not depend on the kernels just before this launch (the library's own selection kernels, which read Q
// but do not write it): the first segment's Q tiles are loaded before the dependency wait.
template <bool FULL, bool SPLIT, bool EARLYQ>
__global__ void __launch_bounds__(TC_THREADS, 1) attend_tc5_kernel(const __grid_constant__ TcParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t s_base = smem_u32(smem);
  const uint32_t s_q = s_base;                       // two Q row tiles
  const uint32_t s_kv = s_base + 2 * Q_TILE_BYTES;   // ring of KV_BUFS chunk tiles
  const uint32_t s_bar = s_kv + KV_BUFS * TILE_BYTES;
  Bars bars;
  bars.base = s_bar;
  volatile uint32_t* s_tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + (s_bar - s_base) + 8 * (2 * KV_BUFS + 6));
  volatile uint32_t* s_abort = s_tmem_slot + 1;
  volatile uint32_t* s_stop = s_tmem_slot + 2;  // the abort flag as one thread saw it between two segment barriers
  volatile uint32_t* s_pend_n = s_tmem_slot + 3;  // units whose last part this CTA finished: count ...
  volatile uint32_t* s_bad = s_tmem_slot + 4;     // [2] per tile slot: a warp of the slot did not write its partial rows
  volatile uint32_t* s_fast = s_tmem_slot + 6;    // [2] per tile slot: every other part of the unit is in place
  volatile uint32_t* s_pend = s_tmem_slot + 8;    // ... and list [PEND_MAX] of (unit << 2 | row tile << 1 | half-streams)

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- one-time set-up -------------------------------------------------------------------------
  if (tid == 0) {
    for (int i = 0; i < KV_BUFS; ++i) {
      mbar_init(bars.full(i), 2);   // the copies' byte count (with its arrival) and the producer's zeroed rows
      mbar_init(bars.empty(i), 1);
    }
    for (int t = 0; t < 2; ++t) {
      mbar_init(bars.s_full(t), 1);
      mbar_init(bars.p_ready(t), 4);  // one arrival per softmax warp
      mbar_init(bars.pv_done(t), 1);
    }
    *s_abort = 0;
    *s_stop = 0;
    s_bad[0] = s_bad[1] = 0;
    *s_pend_n = 0;
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
  // everything above is independent of earlier kernels; the context table is not, and Q only when the launcher says
  // so (after the library's own selection kernels, which read Q but do not write it, the first segment's Q tiles
  // are loaded while those kernels are still running: the wait then stands after that load in the range loop)
  if constexpr (!EARLYQ) {
    grid_dep_wait();
    grid_dep_launch();
  }
  auto col_o = [](int t) { return (uint32_t)t * 128u; };
  auto col_s = [](int t) { return 256u + (uint32_t)t * 128u; };

  const uint32_t wait_limit = p.wait_limit ? p.wait_limit : WAIT_LIMIT;
  auto wait = [&](uint32_t bar, uint32_t parity) -> bool {
    for (uint32_t it = 0; it < wait_limit; ++it) {
      if (mbar_try_wait(bar, parity)) return true;
      if (*s_abort) return false;
      if (it > 2048) __nanosleep(64);
    }
    *s_abort = 1;
    atomicExch(p.status, REKV_ERR_TIMEOUT);
    return false;
  };

  // Barrier of a range segment for every warp but the copy producer, which runs ahead into the next segment (it is
  // held back by the ring's empty barriers only), so that K/V tiles are already on their way during an epilogue.
  auto seg_sync = [&]() {
    if (warp != 0) asm volatile("bar.sync 1, %0;" ::"n"(TC_THREADS - 32) : "memory");
  };
  // Merge inside the kernel.  After a tile slot's partial rows of a cut unit are written (softmax warps), the parts are
  // published with a fence and counted with an atomic per (unit, row tile); the slot that finishes the unit's last
  // part puts the unit on the CTA's list, and at the end of the CTA's range its softmax warps join the listed units'
  // parts -- in part order, whichever CTA does it -- write the output rows and leave the counters at zero for the
  // next launch.  Nobody waits for anybody.  The barrier is taken by all four warps of the slot whether or not their
  // own partial rows got written (a wait that ran out): a warp that failed marks the slot, which then does not
  // count, and the unit stays unmerged behind the status word that the wait has set.
  auto slot_sync = [&](int t) {  // the four softmax warps of tile slot t
    if (t == 0)
      asm volatile("bar.sync 2, 128;" ::: "memory");
    else
      asm volatile("bar.sync 3, 128;" ::: "memory");
  };
  auto part_range = [&](long long u, long long& c_first, long long& c_last) {
    c_first = (u * p.ncf) / p.per;
    c_last = ((u + 1) * p.ncf - 1) / p.per;
  };
  auto part_slot = [&](const UnitInfo& ui, long long u, long long c_first, bool split, int rt, int k) -> long long {
    const long long c = c_first + (split ? k >> 1 : k);
    const long long base = p.per == p.ncf ? (long long)ui.srank : c + u;
    return base * 2 + (split ? (k & 1) : rt);
  };
  auto count_part = [&](long long u, const UnitInfo& ui, int t, int rt, bool split, bool wrote) {
    if (!wrote) s_bad[t] = 1;
    __threadfence();
    slot_sync(t);
    if ((warp & 3) == 0 && lane == 0) {
      if (!s_bad[t]) {
        long long c_first, c_last;
        part_range(u, c_first, c_last);
        const int n_parts = (int)(c_last - c_first + 1) * (split ? 2 : 1);
        int* cnt = p.unit_cnt + (p.per == p.ncf ? (long long)ui.srank : u) * 2 + (split ? 0 : t);
        if (atomicAdd(cnt, 1) == n_parts - 1) {
          *cnt = 0;
          const uint32_t at = atomicAdd((uint32_t*)s_pend_n, 1u);
          if (at < PEND_MAX)
            s_pend[at] = ((uint32_t)u << 2) | ((uint32_t)rt << 1) | (split ? 1u : 0u);
          else
            atomicExch(p.status, -2033);  // cannot happen: a range cuts two units at most
        }
      }
      s_bad[t] = 0;  // (a warp marks the next segment's failure only after the segment barrier that follows)
    }
  };
  // Both ways of finishing a cut unit do the same arithmetic, so that the output does not depend on which CTA came
  // last: M = the maximum over the parts (the part over X included), weights 2^(m_k - M), numerators and
  // denominator accumulated with fused multiply-adds in part order starting from the part over X, one division.
  //
  // The listed units, by the eight softmax warps: a warp per row, eight rows at a time, a float4 of the 128 columns
  // per lane.
  auto merge_listed = [&]() {
    const uint32_t n_pend = min(*s_pend_n, (uint32_t)PEND_MAX);
    if (n_pend == 0) return;  // (the usual case; the fence below would wait for the output rows just stored)
    __threadfence();
    const int w8 = warp - SM_WARP0;
#pragma unroll 1
    for (uint32_t e = 0; e < n_pend; ++e) {
      const uint32_t code = s_pend[e];
      const long long u = code >> 2;
      const int rt = (code >> 1) & 1;
      const bool split = code & 1u;
      const UnitInfo ui = decode_unit(p, u);
      long long c_first, c_last;
      part_range(u, c_first, c_last);
      const int n_parts = (int)(c_last - c_first + 1) * (split ? 2 : 1);
#pragma unroll 1
      for (int r0 = w8 * 8; r0 < 128; r0 += 64) {
        const int rr0 = ui.m0 + rt * 128 + r0;
        if (rr0 >= ui.rows_q) break;
        float M[8], den[8];
        float4 acc[8];
        long long out_at[8];
#pragma unroll
        for (int a = 0; a < 8; ++a) {
          const int rr = min(rr0 + a, ui.rows_q - 1);
          const int n = rr / p.G, j = rr - n * p.G;
          out_at[a] = ((ui.q_row0 + n) * p.Hq + ui.g * p.G + j) * 128 + lane * 4;
          M[a] = (FULL && p.self_o) ? fmaxf(-1e30f, p.self_ml[(out_at[a] >> 7) * 2]) : -1e30f;
        }
#pragma unroll 1
        for (int k = 0; k < n_parts; ++k) {
          const long long base = part_slot(ui, u, c_first, split, rt, k) * 128 + r0;
#pragma unroll
          for (int a = 0; a < 8; ++a) M[a] = fmaxf(M[a], __ldcg(p.part_ml + (base + a) * 2));
        }
#pragma unroll
        for (int a = 0; a < 8; ++a) {
          den[a] = 0.f;
          acc[a] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (FULL && p.self_o) {
            const long long orow = out_at[a] >> 7;
            const float w = ex2(p.self_ml[orow * 2] - M[a]);
            const float4 o = *reinterpret_cast<const float4*>(p.self_o + out_at[a]);
            den[a] = w * p.self_ml[orow * 2 + 1];
            acc[a] = make_float4(w * o.x, w * o.y, w * o.z, w * o.w);
          }
        }
#pragma unroll 1
        for (int k0 = 0; k0 < n_parts; k0 += 2) {  // sixteen rows in flight
          float4 o[2][8];
          float2 ml[2][8];
#pragma unroll
          for (int i = 0; i < 2; ++i)
            if (k0 + i < n_parts) {
              const long long base = part_slot(ui, u, c_first, split, rt, k0 + i) * 128 + r0;
#pragma unroll
              for (int a = 0; a < 8; ++a) {
                ml[i][a] = __ldcg(reinterpret_cast<const float2*>(p.part_ml + (base + a) * 2));
                o[i][a] = __ldcg(reinterpret_cast<const float4*>(p.part_o + (base + a) * 128 + lane * 4));
              }
            }
#pragma unroll
          for (int i = 0; i < 2; ++i)
            if (k0 + i < n_parts) {
#pragma unroll
              for (int a = 0; a < 8; ++a) {
                const float w = ex2(ml[i][a].x - M[a]);
                den[a] = fmaf(w, ml[i][a].y, den[a]);
                acc[a].x = fmaf(w, o[i][a].x, acc[a].x);
                acc[a].y = fmaf(w, o[i][a].y, acc[a].y);
                acc[a].z = fmaf(w, o[i][a].z, acc[a].z);
                acc[a].w = fmaf(w, o[i][a].w, acc[a].w);
              }
            }
        }
#pragma unroll
        for (int a = 0; a < 8; ++a)
          if (rr0 + a < ui.rows_q) {
            const float inv = den[a] > 0.f ? 1.f / den[a] : 0.f;
            uint2 packed;
            packed.x = pack_bf16(acc[a].x * inv, acc[a].y * inv);
            packed.y = pack_bf16(acc[a].z * inv, acc[a].w * inv);
            *reinterpret_cast<uint2*>(p.out + out_at[a]) = packed;
          }
      }
    }
  };
  // The unit's other parts joined with this tile slot's own part, which is still in tensor memory: one thread per
  // row as in the other epilogues.  The other parts' rows come through the warp's staging rows (contiguous global
  // reads, then each thread takes its row), the result leaves through them as bf16.
  auto finish_from_tmem = [&](long long u, const UnitInfo& ui, int t, int rt, bool split, int row, int rr0, bool valid,
                              int n, int j, float m_own, float l_own, bool own_empty, uint32_t t_o,
                              unsigned char* stage) {
    if (rr0 >= ui.rows_q) return;  // a warp without a valid row (the ragged tile)
    long long c_first, c_last;
    part_range(u, c_first, c_last);
    const int n_parts = (int)(c_last - c_first + 1) * (split ? 2 : 1);
    const int own = (int)(blockIdx.x - c_first) * (split ? 2 : 1) + (split ? t : 0);
    const long long out_row = (ui.q_row0 + (valid ? n : 0)) * p.Hq + ui.g * p.G + (valid ? j : 0);
    // At most three parts reach this path (the launcher sees to it): the (max, sum) of the one or two other parts
    // come in one round of loads.
    const int ka = own == 0 ? 1 : 0, kb = n_parts >= 3 ? (own == 2 ? 1 : 2) : -1;
    const float2 ml_a = __ldcg(reinterpret_cast<const float2*>(p.part_ml + (part_slot(ui, u, c_first, split, rt, ka) * 128 + row) * 2));
    float2 ml_b = make_float2(-INFINITY, 0.f);
    if (kb >= 0)
      ml_b = __ldcg(reinterpret_cast<const float2*>(p.part_ml + (part_slot(ui, u, c_first, split, rt, kb) * 128 + row) * 2));
    float M = fmaxf(fmaxf(-1e30f, m_own), fmaxf(ml_a.x, ml_b.x));
    float den = 0.f, w_x = 0.f;
    const float4* o_x = nullptr;
    if (FULL && p.self_o) {
      const float m_x = p.self_ml[out_row * 2];
      M = fmaxf(M, m_x);
      w_x = ex2(m_x - M);
      den = w_x * p.self_ml[out_row * 2 + 1];
      o_x = reinterpret_cast<const float4*>(p.self_o + out_row * 128);
    }
#pragma unroll
    for (int k = 0; k < 3; ++k)
      if (k < n_parts) {
        const float2 ml = k == own ? make_float2(m_own, l_own) : (k == ka ? ml_a : ml_b);
        den = fmaf(ex2(ml.x - M), ml.y, den);
      }
    const float inv = den > 0.f ? 1.f / den : 0.f;
    // rows this lane stores: r = 8 k + (lane >> 2), 16 bytes (8 bf16) at chunk (lane & 3) of the quarter
    __nv_bfloat16* dst_k[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int r2 = rr0 + 8 * k + (lane >> 2);
      const int n2 = r2 / p.G, j2 = r2 - n2 * p.G;
      dst_k[k] = r2 < ui.rows_q ? p.out + ((ui.q_row0 + n2) * p.Hq + ui.g * p.G + j2) * 128 + (lane & 3) * 8 : nullptr;
    }
    // The other parts' quarter rows are asked for one step ahead: the loads of the next (quarter, part) are in flight
    // while the current one is added up and the quarter's output leaves.
    uint4 x[8];
#define REKV_ASK(QD, K)                                                                                              \
  do {                                                                                                               \
    const float* po_ = p.part_o + ((part_slot(ui, u, c_first, split, rt, (K)) * 128 + ((warp & 3) << 5) + (lane >> 3)) * 128 + \
                                   (lane & 7) * 4) + (QD) * 32;                                                      \
    _Pragma("unroll") for (int kk = 0; kk < 8; ++kk) x[kk] = __ldcg(reinterpret_cast<const uint4*>(po_ + (long long)kk * 4 * 128)); \
  } while (0)
    REKV_ASK(0, ka);
#pragma unroll 1
    for (int qd = 0; qd < 4; ++qd) {
      float acc[32];
#pragma unroll
      for (int v4 = 0; v4 < 8; ++v4) {
        float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
        if (FULL && o_x) y = __ldg(o_x + qd * 8 + v4);
        acc[4 * v4] = w_x * y.x;
        acc[4 * v4 + 1] = w_x * y.y;
        acc[4 * v4 + 2] = w_x * y.z;
        acc[4 * v4 + 3] = w_x * y.w;
      }
#pragma unroll 1
      for (int k = 0; k < n_parts; ++k) {
        if (k == own) {  // (uniform over the slot's warps)
          uint32_t o[2][16];
          tmem_ld16(t_o + qd * 32, o[0]);
          tmem_ld16(t_o + qd * 32 + 16, o[1]);
          tmem_wait_ld16(o[0]);
          tmem_wait_ld16(o[1]);
          const float w = ex2(m_own - M);
#pragma unroll
          for (int e = 0; e < 32; ++e)
            acc[e] = fmaf(w, own_empty ? 0.f : __uint_as_float(o[e >> 4][e & 15]), acc[e]);
        } else {
          const float w = ex2((k == ka ? ml_a.x : ml_b.x) - M);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            *reinterpret_cast<uint4*>(stage + (4 * kk + (lane >> 3)) * STAGE_ROW_F32 + (lane & 7) * 16) = x[kk];
          __syncwarp();
          // the next step that reads another part: this quarter's second other part, else the next quarter's first
          if (k == ka && kb >= 0) {
            REKV_ASK(qd, kb);
          } else if (qd < 3) {
            REKV_ASK(qd + 1, ka);
          }
#pragma unroll
          for (int v4 = 0; v4 < 8; ++v4) {
            const float4 y = *reinterpret_cast<const float4*>(stage + lane * STAGE_ROW_F32 + v4 * 16);
            acc[4 * v4] = fmaf(w, y.x, acc[4 * v4]);
            acc[4 * v4 + 1] = fmaf(w, y.y, acc[4 * v4 + 1]);
            acc[4 * v4 + 2] = fmaf(w, y.z, acc[4 * v4 + 2]);
            acc[4 * v4 + 3] = fmaf(w, y.w, acc[4 * v4 + 3]);
          }
          __syncwarp();
        }
      }
#undef REKV_ASK
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint4 a, b;
        const float* c = acc + 16 * h;
        a.x = pack_bf16(c[0] * inv, c[1] * inv);
        a.y = pack_bf16(c[2] * inv, c[3] * inv);
        a.z = pack_bf16(c[4] * inv, c[5] * inv);
        a.w = pack_bf16(c[6] * inv, c[7] * inv);
        b.x = pack_bf16(c[8] * inv, c[9] * inv);
        b.y = pack_bf16(c[10] * inv, c[11] * inv);
        b.z = pack_bf16(c[12] * inv, c[13] * inv);
        b.w = pack_bf16(c[14] * inv, c[15] * inv);
        *reinterpret_cast<uint4*>(stage + lane * STAGE_ROW_BF16 + h * 32) = a;
        *reinterpret_cast<uint4*>(stage + lane * STAGE_ROW_BF16 + h * 32 + 16) = b;
      }
      __syncwarp();
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint4 x = *reinterpret_cast<const uint4*>(stage + (8 * k + (lane >> 2)) * STAGE_ROW_BF16 + (lane & 3) * 16);
        if (dst_k[k]) *reinterpret_cast<uint4*>(dst_k[k] + qd * 32) = x;
      }
      __syncwarp();
    }
  };
  const uint32_t page_half_bytes = (uint32_t)p.Nf * 128u;   // one 64-dim half of a head tile in a page
  const uint32_t idesc_pv = idesc_bf16(128, 128, 1);

  // The roles run the same range loop with the role as a compile-time constant, so that each side of the
  // register reallocation below is compiled against its own register budget.
  auto run = [&](auto role) {
  constexpr bool SOFTMAX = decltype(role)::value;
  long long pos = (long long)blockIdx.x * p.per;
  const long long end = min(pos + (long long)p.per, p.total);
  uint32_t ring = 0;    // chunk tiles moved so far (K and V of a chunk are consecutive ring entries)
  uint32_t ring_issued = 0;  // copy producer: ring entries whose copies have been issued
  uint32_t chunk_cnt[2] = {0u, 0u};  // token chunks processed so far, per row tile (barrier phases)

  while (pos < end) {
    const long long u = pos / p.ncf;
    const int f0 = (int)(pos - u * p.ncf);
    const int nfr = (int)min((long long)(p.ncf - f0), end - pos);
    const UnitInfo ui = decode_unit(p, u);
    // the segment's token stream: frame i at rows [i N_s, i N_s + N_f); the last frame's gap rows are cut off
    const int Lrows = (nfr - 1) * p.Ns + p.Nf;
    const int nchunks = (Lrows + CHUNK - 1) / CHUNK;
    const bool split = SPLIT && ui.split != 0;
    const int vtiles = split ? 2 : ui.tiles;  // tile slots in use
    // chunks per tile slot and a slot's j-th chunk among the segment's: every chunk for both tiles, or alternately
    const int nch0 = split ? (nchunks + 1) >> 1 : nchunks, nch1 = split ? nchunks >> 1 : nchunks;
    auto chunk_of = [&](int T, int j) { return split ? 2 * j + T : j; };
    auto chunk_n = [&](int I) { return (min(CHUNK, Lrows - I * CHUNK) + 15) & ~15; };  // columns of chunk I's products
    char* const* pages = p.tbl + ((long long)ui.l * p.qb.nQ + ui.qi) * p.ncf + f0;
    char* const* pages_k = (FULL && p.tbl_k) ? p.tbl_k + ((long long)ui.l * p.qb.nQ + ui.qi) * p.ncf + f0 : nullptr;
    const bool whole_unit = (nfr == p.ncf) && !split;

    // ---- Q row tiles -> shared memory in the swizzled K-major operand layout -------------------
    if (warp >= SM_WARP0) {
      const int t = (warp - SM_WARP0) >> 2;
      const int row = ((warp & 3) << 5) | lane;
      if (t < vtiles) {
        const int rr = ui.m0 + (split ? 0 : t) * 128 + row;
        const bool valid = rr < ui.rows_q;
        const int n = rr / p.G, j = rr - n * p.G;
        const uint4* src =
            reinterpret_cast<const uint4*>(p.q + ((ui.q_row0 + (valid ? n : 0)) * p.Hq + ui.g * p.G + (valid ? j : 0)) * 128);
        unsigned char* dst = smem + t * Q_TILE_BYTES + row * 128;
        uint4 x[16];
#pragma unroll
        // (before the dependency wait the rows are read past L1: nothing has invalidated it since an earlier launch
        // may have read other contents at the same addresses)
        for (int c = 0; c < 16; ++c) x[c] = valid ? (EARLYQ ? __ldcg(src + c) : __ldg(src + c)) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int c = 0; c < 16; ++c)
          *reinterpret_cast<uint4*>(dst + (c >> 3) * (Q_TILE_BYTES / 2) + (((c & 7) ^ (row & 7)) << 4)) = x[c];
      }
      fence_proxy_async();
    }
    if constexpr (EARLYQ) {
      if (pos == (long long)blockIdx.x * p.per) {  // first segment: only now the earlier kernels' results
        grid_dep_wait();
        grid_dep_launch();
      }
    }
    seg_sync();

    if constexpr (!SOFTMAX) {
    if (warp == 0) {
      // ================= copy producer =================
      // the whole warp walks the ring (uniform control flow).  Per chunk tile: the rows no page covers (gap rows
      // between frames, the rows after the stream's end up to the products' width) are zeroed by all lanes, then one
      // elected lane issues the copies -- per frame that overlaps the chunk and per 64-dim half one contiguous piece.
      const long long head_off = (long long)(ui.g * 2) * p.Nf * 256;   // this KV head's K tile inside a page
      bool stop = false;
      for (int I = 0; I < nchunks && !stop; ++I) {
        const int row0 = I * CHUNK;
        const int nrows = min(CHUNK, Lrows - row0);     // stream rows of this chunk
        const int N = (nrows + 15) & ~15;
        const int fi0 = row0 / p.Ns, fi1 = (row0 + nrows - 1) / p.Ns;
        const int pos0 = row0 - fi0 * p.Ns;             // the chunk's first row inside frame fi0
        uint32_t bytes = 0;
        for (int fi = fi0; fi <= fi1; ++fi) {
          const int ta = max(0, row0 - fi * p.Ns), tb = min(p.Nf, row0 + nrows - fi * p.Ns);
          if (tb > ta) bytes += 2u * (uint32_t)(tb - ta) * 128u;
        }
#pragma unroll
        for (int kv = 0; kv < 2; ++kv) {
          const uint32_t r = ring + 2 * I + kv;
          const uint32_t b = r % KV_BUFS, use = r / KV_BUFS;
          if (use > 0 && !wait(bars.empty(b), (use - 1) & 1)) {
            stop = true;
            break;
          }
          const uint32_t dst = s_kv + b * TILE_BYTES;
          // copies first: nothing stands between the slot becoming free and its next tile being on its way
          const bool skip = p.skip_copy_entry >= 0 && blockIdx.x == 0 && (int)r == p.skip_copy_entry;  // test-only
          if (elect_one() && !skip) {
            mbar_expect_tx(bars.full(b), bytes);
            for (int fi = fi0; fi <= fi1; ++fi) {
              const int ta = max(0, row0 - fi * p.Ns), tb = min(p.Nf, row0 + nrows - fi * p.Ns);
              if (tb <= ta) continue;
              const char* src = pages[fi] + head_off + (long long)kv * 2 * page_half_bytes;
              if (FULL && kv == 0 && pages_k) src = pages_k[fi] + (long long)ui.g * 2 * page_half_bytes;  // rotated K tiles
              const uint32_t d = dst + (uint32_t)(fi * p.Ns + ta - row0) * 128u;
              const uint32_t nb = (uint32_t)(tb - ta) * 128u;
              // (checks build) a piece must lie inside its ring tile half and start on 16 bytes at both ends; a piece
              // that does not is left out, and the wait for the tile then runs out and reports it
              if (!REKV_CHECK(pages[fi] != nullptr && (reinterpret_cast<uintptr_t>(src) & 15) == 0 && d >= dst &&
                                  d + nb <= dst + HALF_BYTES && fi * p.Ns + ta - row0 >= 0,
                              p.status, 31))
                continue;
              bulk_g2s(d, src + (long long)ta * 128, nb, bars.full(b));
              bulk_g2s(d + HALF_BYTES, src + page_half_bytes + (long long)ta * 128, nb, bars.full(b));
            }
          }
          {  // then the rows without a token (the copies do not touch them); the tile's second arrival follows them
            int x = pos0 + lane;
            // (no such row in a chunk that lies inside one frame's tokens and is full)
            const bool all_covered = nrows == N && pos0 + nrows <= p.Nf;
            for (int rr = all_covered ? N : lane; rr < N; rr += 32, x += 32) {
              if (p.Ns >= CHUNK) {
                if (x >= p.Ns) x -= p.Ns;
              } else {
                x %= p.Ns;
              }
              if (rr >= nrows || x >= p.Nf) {
                unsigned char* row_ptr = smem + (dst - s_base) + rr * 128;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                  *reinterpret_cast<uint4*>(row_ptr + c * 16) = make_uint4(0, 0, 0, 0);
                  *reinterpret_cast<uint4*>(row_ptr + HALF_BYTES + c * 16) = make_uint4(0, 0, 0, 0);
                }
              }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0 && !skip) mbar_arrive(bars.full(b));
          }
          ring_issued = r + 1;
          __syncwarp();
        }
        if (*s_abort) stop = true;
      }
    } else if (warp == 1) {
      // ================= MMA issuer =================
      // Descriptors are built once; per instruction only the 14-bit start-address field advances.
      {
        const uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);  // SBO = 1024 B, version, SWIZZLE_128B
        const uint32_t lbo_v = ((HALF_BYTES >> 4) & 0x3FFFu) << 16;       // pitch of V's two 64-dim blocks
        const uint32_t lbo_k = 1u << 16;                                  // unused for K-major operands
        const uint32_t half16 = HALF_BYTES >> 4;
        const int tiles = vtiles;
        bool ok = true;
#define REKV_DESC(lo) (((uint64_t)desc_hi << 32) | (uint64_t)(lo))
#define REKV_ISSUE_S(T, I)                                                                                    \
  do {                                                                                                        \
    const uint32_t r_ = ring + 2 * (I), b_ = r_ % KV_BUFS;                                                    \
    const uint32_t N_ = (uint32_t)chunk_n(I);                                                                 \
    if ((T) == 0 || split) ok = wait(bars.full(b_), (r_ / KV_BUFS) & 1);                                      \
    if (ok) {                                                                                                 \
      tc_fence_after();                                                                                       \
      const uint32_t k_lo = ((s_kv + b_ * TILE_BYTES) >> 4) | lbo_k;                                          \
      const uint32_t q_lo = ((s_q + (T) * Q_TILE_BYTES) >> 4) | lbo_k;                                        \
      const uint32_t idesc_ = idesc_bf16(128, N_, 0);                                                         \
      const uint32_t d_ = tmem + col_s(T);                                                                    \
      if (elect_one()) {                                                                                      \
      _Pragma("unroll") for (int kk = 0; kk < 4; ++kk)                                                        \
          mma_ss(d_, REKV_DESC(q_lo + 2 * kk), REKV_DESC(k_lo + 2 * kk), idesc_, kk > 0);                     \
      _Pragma("unroll") for (int kk = 0; kk < 4; ++kk)                                                        \
          mma_ss(d_, REKV_DESC(q_lo + (Q_TILE_BYTES / 32) + 2 * kk), REKV_DESC(k_lo + half16 + 2 * kk), idesc_, 1); \
      tc_commit(bars.s_full(T));                                                                              \
      if ((T) == tiles - 1 || split) tc_commit(bars.empty(b_)); /* K tile done */                             \
      }                                                                                                       \
      __syncwarp();                                                                                           \
    }                                                                                                         \
  } while (0)
#define REKV_ISSUE_PV(T, I, J)                                                                                \
  do {                                                                                                        \
    const uint32_t r_ = ring + 2 * (I) + 1, b_ = r_ % KV_BUFS;                                                \
    const uint32_t nk_ = (uint32_t)chunk_n(I) >> 4;                                                           \
    if ((T) == 0 || split) ok = wait(bars.full(b_), (r_ / KV_BUFS) & 1);                                      \
    if (ok) ok = wait(bars.p_ready(T), (chunk_cnt[T] + (J)) & 1);                                             \
    if (ok) {                                                                                                 \
      tc_fence_after();                                                                                       \
      const uint32_t v_lo = ((s_kv + b_ * TILE_BYTES) >> 4) | lbo_v;                                          \
      const uint32_t d_ = tmem + col_o(T), a_ = tmem + col_s(T);                                              \
      if (elect_one()) {                                                                                      \
      _Pragma("unroll") for (int kk = 0; kk < 8; ++kk)                                                        \
          if (kk < (int)nk_) mma_ts(d_, a_ + 8 * kk, REKV_DESC(v_lo + 128 * kk), idesc_pv, ((J) > 0) | (kk > 0)); \
      tc_commit(bars.pv_done(T));                                                                             \
      if ((T) == tiles - 1 || split) tc_commit(bars.empty(b_)); /* V tile done */                             \
      }                                                                                                       \
      __syncwarp();                                                                                           \
    }                                                                                                         \
  } while (0)
        REKV_ISSUE_S(0, 0);
        if (tiles == 2 && ok && chunk_of(1, 0) < nchunks) REKV_ISSUE_S(1, chunk_of(1, 0));
        for (int j = 0; j < nch0 && ok; ++j) {
          REKV_ISSUE_PV(0, chunk_of(0, j), j);
          if (chunk_of(0, j + 1) < nchunks && ok) REKV_ISSUE_S(0, chunk_of(0, j + 1));
          if (tiles == 2 && ok && chunk_of(1, j) < nchunks) {
            REKV_ISSUE_PV(1, chunk_of(1, j), j);
            if (chunk_of(1, j + 1) < nchunks && ok) REKV_ISSUE_S(1, chunk_of(1, j + 1));
          }
        }
#undef REKV_ISSUE_S
#undef REKV_ISSUE_PV
#undef REKV_DESC
      }
      __syncwarp();
    }
    } else {
      // ================= softmax + output, one thread per row =================
      const int t = (warp - SM_WARP0) >> 2;
      if (t < vtiles) {
        const int rt = split ? 0 : t;              // the row tile this slot works on
        const int nch = t ? nch1 : nch0;           // its chunks in this segment
        const uint32_t lane_base = (uint32_t)((warp & 3) << 5) << 16;
        const int row = ((warp & 3) << 5) | lane;
        const uint32_t t_s = tmem + lane_base + col_s(t);
        const uint32_t t_o = tmem + lane_base + col_o(t);
        float m_used = -INFINITY, l_sum = 0.f;
        bool ok = true;
        // a warp whose 32 rows all lie beyond the unit's rows (the ragged second tile) only keeps the barriers moving
        const bool warp_idle = ui.m0 + rt * 128 + ((warp & 3) << 5) >= ui.rows_q;
        for (int i = 0; i < nch && ok; ++i) {  // i counts this slot's chunks
          // ---- the chunk's shape, worked out while its S is still being computed ----
          const int I = chunk_of(t, i);
          const int row0 = I * CHUNK;
          const int nrows = min(CHUNK, Lrows - row0);
          // columns without a token, a bit per column (warp-uniform): a lane looks at columns lane, lane + 32, ...
          unsigned long long mw_lo, mw_hi;
          {
            const int pos0 = row0 % p.Ns;
            uint32_t mw[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int col = lane + 32 * k;
              int x = pos0 + col;
              if (p.Ns >= CHUNK) {
                if (x >= p.Ns) x -= p.Ns;
              } else {
                x %= p.Ns;
              }
              mw[k] = __ballot_sync(0xffffffffu, col >= nrows || x >= p.Nf);
            }
            mw_lo = (unsigned long long)mw[0] | ((unsigned long long)mw[1] << 32);
            mw_hi = (unsigned long long)mw[2] | ((unsigned long long)mw[3] << 32);
          }
          // -1: nothing to mask; 0..7: the only piece with masked columns, and its bits; 8: several pieces
          int mask_pc = -1;
          uint32_t mask_bits = 0;
#pragma unroll
          for (int pc = 0; pc < 8; ++pc) {
            const uint32_t m16 = (uint32_t)(((pc & 4) ? mw_hi : mw_lo) >> ((pc & 3) * 16)) & 0xFFFFu;
            if (m16) {
              mask_pc = mask_pc < 0 ? pc : 8;
              mask_bits = m16;
            }
          }
          if (!wait(bars.s_full(t), (chunk_cnt[t] + i) & 1)) {
            ok = false;
            break;
          }
          tc_fence_after();
          if (warp_idle) {  // no valid row in this warp's 32 lanes: their P and O rows are never read back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bars.p_ready(t));
            continue;
          }
          // The whole S row chunk comes into registers with ONE TMEM load instruction (a warp's tcgen05.ld/st
          // instructions run one after the other at about 90 cycles each, whatever their width), so there is one
          // wait, one row maximum and one rescaling decision per chunk.  Columns without a token -- a frame
          // boundary's gap, the stream's end, the columns beyond the products' width, which hold stale values -- are
          // masked piece by piece behind a warp-uniform test, so that only the piece that has some pays for it.
          // Lazy rescaling: the maximum in use is raised only when this chunk exceeds it by more than the threshold
          // (always on the first chunk); O and the running sum then shrink by 2^(old - new).
          const float NEG_INF = -INFINITY;
          uint32_t sv[128];
          tmem_ld128(t_s, sv);
          tmem_wait_ld128(sv);
          if (mask_pc >= 0) {
            auto mask16 = [&](uint32_t* v, uint32_t m16) {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if ((m16 >> j) & 1u) v[j] = __float_as_uint(NEG_INF);
            };
            switch (mask_pc) {  // the one piece that has masked columns (warp-uniform)
              case 0: mask16(sv, mask_bits); break;
              case 1: mask16(sv + 16, mask_bits); break;
              case 2: mask16(sv + 32, mask_bits); break;
              case 3: mask16(sv + 48, mask_bits); break;
              case 4: mask16(sv + 64, mask_bits); break;
              case 5: mask16(sv + 80, mask_bits); break;
              case 6: mask16(sv + 96, mask_bits); break;
              case 7: mask16(sv + 112, mask_bits); break;
              default:  // several pieces (N_f < 128, or the stream's last chunk): every piece tested
#pragma unroll
                for (int pc = 0; pc < 8; ++pc) {
                  const uint32_t m16 = (uint32_t)(((pc & 4) ? mw_hi : mw_lo) >> ((pc & 3) * 16)) & 0xFFFFu;
                  if (m16) mask16(sv + 16 * pc, m16);
                }
                break;
            }
          }
          auto row_max = [&]() -> float {  // of the chunk's logits, in log2 units
            float gmx[8];
#pragma unroll
            for (int a8 = 0; a8 < 8; ++a8)
              gmx[a8] = max3(__uint_as_float(sv[a8]), __uint_as_float(sv[8 + a8]), __uint_as_float(sv[16 + a8]));
#pragma unroll
            for (int c = 24; c + 16 <= 128; c += 16)
#pragma unroll
              for (int a8 = 0; a8 < 8; ++a8)
                gmx[a8] = max3(gmx[a8], __uint_as_float(sv[c + a8]), __uint_as_float(sv[c + 8 + a8]));
#pragma unroll
            for (int a8 = 0; a8 < 8; ++a8) gmx[a8] = fmaxf(gmx[a8], __uint_as_float(sv[120 + a8]));
            return max3(max3(gmx[0], gmx[1], gmx[2]), max3(gmx[3], gmx[4], gmx[5]), fmaxf(gmx[6], gmx[7])) * p.scale_log2;
          };
          // P = 2^(S*scale - m) as bf16 pairs over the front of S (two stores of 32 columns); returns the row sum.
          // The conversion instruction shares the transcendental unit with ex2 (a quarter-rate pipe: 8 cycles per
          // ex2 and 4 per packed pair and warp), which made that pipe the busiest part of the SM; so P is cut to
          // bf16 by taking the upper halves (one byte permute per pair) of 2^(x - m) * (1 + TRUNC_GAIN), the factor
          // that makes the cut value equal to 2^(x - m) on average over the mantissa -- folded into the exponent,
          // and taken out of the row sum once at the end of the range.  All 128 columns are done whatever the
          // chunk's width (masked columns give exactly 0): one straight run of code lets the compiler keep the
          // transcendental unit fed.
          auto exp_pass = [&]() -> float {
            const float neg_m = TRUNC_GAIN_LOG2 - m_used;
            float ps0 = 0.f, ps1 = 0.f, ps2 = 0.f, ps3 = 0.f;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
              uint32_t pk[32];
#pragma unroll
              for (int jj = 0; jj < 32; jj += 2) {
                const uint32_t* v = sv + 64 * hf;
                const float p0 = ex2(fmaf(__uint_as_float(v[2 * jj]), p.scale_log2, neg_m));
                const float p1 = ex2(fmaf(__uint_as_float(v[2 * jj + 1]), p.scale_log2, neg_m));
                const float p2 = ex2(fmaf(__uint_as_float(v[2 * jj + 2]), p.scale_log2, neg_m));
                const float p3 = ex2(fmaf(__uint_as_float(v[2 * jj + 3]), p.scale_log2, neg_m));
                ps0 += p0;
                ps1 += p1;
                ps2 += p2;
                ps3 += p3;
                pk[jj] = __byte_perm(__float_as_uint(p0), __float_as_uint(p1), 0x7632);
                pk[jj + 1] = __byte_perm(__float_as_uint(p2), __float_as_uint(p3), 0x7632);
              }
              tmem_st32(t_s + 32 * hf, pk);
            }
            return (ps0 + ps1) + (ps2 + ps3);
          };
          // The reference value m of the exponentials is the row maximum of the range's FIRST chunk.  Later chunks
          // do not look for their maximum at all (128 min/max instructions per row cost about 400 cycles a chunk):
          // a softmax does not depend on m, which only has to keep 2^(x - m) inside the fp32 range, and values far
          // above 1 lose nothing in fp32 sums or in bf16's 8 exponent bits.  So the exponentials are taken with the m
          // in use, and only if a row's sum leaves [0, 2^60) -- a logit more than 60 octaves above m, or an overflow
          // -- does the warp find the true maximum, shrink O and the running sum by 2^(old - new), and repeat the
          // pass from the registers (the P stores of the first pass are simply overwritten).
          if (i == 0) m_used = row_max();
          float cs = exp_pass();
          const bool need = !(cs < RESCALE_SUM_LIMIT);
          if (__any_sync(0xffffffffu, need)) {
            const float gm = row_max();
            const float alpha = need ? ex2(m_used - gm) : 1.f;
            if (need) m_used = gm;
            l_sum *= alpha;
            if (i > 0) {  // O holds earlier chunks; their P V is complete (this chunk's S came after it)
#pragma unroll 1
              for (int pc = 0; pc < 8; ++pc) {
                uint32_t o[16];
                tmem_ld16(t_o + pc * 16, o);
                tmem_wait_ld16(o);
#pragma unroll
                for (int j = 0; j < 16; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
                tmem_st16(t_o + pc * 16, o);
              }
            }
            cs = exp_pass();
          }
          l_sum += cs;
          tmem_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bars.p_ready(t));
        }
        l_sum *= TRUNC_GAIN_INV;  // the row sum was taken over the scaled values
        // ---- output of this range: final rows, or a partial for the combine kernel ----
        // A cut unit whose other parts are all in place is finished here, from this slot's O in tensor memory (the
        // usual case for the CTA that holds a unit's head: the later CTAs worked on its tail first): no partial of
        // its own is written or read back.  Otherwise the slot writes its partial and counts it.
        const bool cut = !whole_unit && p.unit_cnt != nullptr;
        bool fast = false;
        if (cut) {
          if ((warp & 3) == 0 && lane == 0) {
            long long c_first, c_last;
            part_range(u, c_first, c_last);
            const int n_parts = (int)(c_last - c_first + 1) * (split ? 2 : 1);
            int* cnt = p.unit_cnt + (p.per == p.ncf ? (long long)ui.srank : u) * 2 + (split ? 0 : t);
            s_fast[t] = atomicAdd(cnt, 0) == n_parts - 1;
          }
          slot_sync(t);
          fast = s_fast[t] != 0;
          if (fast) __threadfence();
        }
        bool wrote = false;  // this thread's rows are in place (partial or final)
        if (ok && (nch == 0 || wait(bars.pv_done(t), (chunk_cnt[t] + nch - 1) & 1))) {
          tc_fence_after();
          const int rr = ui.m0 + rt * 128 + row;
          const bool valid = rr < ui.rows_q;
          const int n = rr / p.G, j = rr - n * p.G;
          // Rows leave through this warp's staging rows in the tile's Q region (no product reads Q any more), a
          // quarter of the 128 columns at a time, so that the global stores are contiguous per row instead of one
          // 16-byte piece per lane in 32 different rows.
          unsigned char* stage = smem + t * Q_TILE_BYTES + (warp & 3) * STAGE_WARP_BYTES;
          const int rr0 = ui.m0 + rt * 128 + ((warp & 3) << 5);  // first row of this warp
          if (whole_unit) {
            float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
            const long long out_row = (ui.q_row0 + (valid ? n : 0)) * p.Hq + ui.g * p.G + (valid ? j : 0);
            // Eq. 3 in full: the part over the tokens of X joins here, O = (O_c w_c + O_x w_x) / (l_c w_c + l_x w_x)
            float w_x = 0.f;
            const float4* o_x = nullptr;
            if (FULL && p.self_o) {
              const float m_x = p.self_ml[out_row * 2], l_x = p.self_ml[out_row * 2 + 1];
              const float M = fmaxf(m_used, m_x);
              const float w_c = ex2(m_used - M);
              w_x = ex2(m_x - M);
              const float den = l_sum * w_c + l_x * w_x;
              inv = den > 0.f ? w_c / den : 0.f;
              w_x = den > 0.f ? w_x / den : 0.f;
              o_x = reinterpret_cast<const float4*>(p.self_o + out_row * 128);
            }
            // rows this lane stores: r = 8 k + (lane >> 2), 16 bytes (8 bf16) at chunk (lane & 3) of the quarter
            __nv_bfloat16* dst_k[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int r2 = rr0 + 8 * k + (lane >> 2);
              const int n2 = r2 / p.G, j2 = r2 - n2 * p.G;
              dst_k[k] = r2 < ui.rows_q ? p.out + ((ui.q_row0 + n2) * p.Hq + ui.g * p.G + j2) * 128 + (lane & 3) * 8 : nullptr;
            }
#pragma unroll 1
            for (int qd = 0; qd < 4; ++qd) {
              uint32_t o[2][16];
              tmem_ld16(t_o + qd * 32, o[0]);
              tmem_ld16(t_o + qd * 32 + 16, o[1]);
              tmem_wait_ld16(o[0]);
              tmem_wait_ld16(o[1]);
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                if (FULL && o_x) {
#pragma unroll
                  for (int v4 = 0; v4 < 4; ++v4) {
                    const float4 x = __ldg(o_x + qd * 8 + h * 4 + v4);
                    o[h][4 * v4] = __float_as_uint(__uint_as_float(o[h][4 * v4]) * inv + x.x * w_x);
                    o[h][4 * v4 + 1] = __float_as_uint(__uint_as_float(o[h][4 * v4 + 1]) * inv + x.y * w_x);
                    o[h][4 * v4 + 2] = __float_as_uint(__uint_as_float(o[h][4 * v4 + 2]) * inv + x.z * w_x);
                    o[h][4 * v4 + 3] = __float_as_uint(__uint_as_float(o[h][4 * v4 + 3]) * inv + x.w * w_x);
                  }
                } else {
#pragma unroll
                  for (int e = 0; e < 16; ++e) o[h][e] = __float_as_uint(__uint_as_float(o[h][e]) * inv);
                }
                uint4 a, b;
                a.x = pack_bf16(__uint_as_float(o[h][0]), __uint_as_float(o[h][1]));
                a.y = pack_bf16(__uint_as_float(o[h][2]), __uint_as_float(o[h][3]));
                a.z = pack_bf16(__uint_as_float(o[h][4]), __uint_as_float(o[h][5]));
                a.w = pack_bf16(__uint_as_float(o[h][6]), __uint_as_float(o[h][7]));
                b.x = pack_bf16(__uint_as_float(o[h][8]), __uint_as_float(o[h][9]));
                b.y = pack_bf16(__uint_as_float(o[h][10]), __uint_as_float(o[h][11]));
                b.z = pack_bf16(__uint_as_float(o[h][12]), __uint_as_float(o[h][13]));
                b.w = pack_bf16(__uint_as_float(o[h][14]), __uint_as_float(o[h][15]));
                *reinterpret_cast<uint4*>(stage + lane * STAGE_ROW_BF16 + h * 32) = a;
                *reinterpret_cast<uint4*>(stage + lane * STAGE_ROW_BF16 + h * 32 + 16) = b;
              }
              __syncwarp();
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const uint4 x = *reinterpret_cast<const uint4*>(stage + (8 * k + (lane >> 2)) * STAGE_ROW_BF16 + (lane & 3) * 16);
                if (dst_k[k]) *reinterpret_cast<uint4*>(dst_k[k] + qd * 32) = x;
              }
              __syncwarp();
            }
          } else if (fast) {
            finish_from_tmem(u, ui, t, rt, split, row, rr0, valid, n, j, m_used, l_sum, nch == 0, t_o, stage);
            wrote = true;
          } else {
            const long long slot_raw = (p.per == p.ncf ? (long long)ui.srank : (long long)blockIdx.x + u) * 2 + t;
            const bool slot_ok = REKV_CHECK(slot_raw >= 0 && slot_raw < p.part_slots, p.status, 32);  // (checks build)
            const long long slot = slot_ok ? slot_raw : 0;
            // rows this lane stores: r = 4 k + (lane >> 3), 16 bytes (4 floats) at chunk (lane & 7) of the quarter
            float* po = p.part_o + ((slot * 128 + ((warp & 3) << 5) + (lane >> 3)) * 128 + (lane & 7) * 4);
            const int nrows_w = slot_ok ? ui.rows_q - rr0 : 0;  // valid rows of this warp (may exceed 32)
#pragma unroll 1
            for (int qd = 0; qd < 4; ++qd) {
              uint32_t o[2][16];
              tmem_ld16(t_o + qd * 32, o[0]);
              tmem_ld16(t_o + qd * 32 + 16, o[1]);
              tmem_wait_ld16(o[0]);
              tmem_wait_ld16(o[1]);
              if (nch == 0) {  // a half-stream without a chunk in this segment: the neutral partial (-inf, 0, 0)
#pragma unroll
                for (int e = 0; e < 16; ++e) o[0][e] = o[1][e] = 0u;
              }
#pragma unroll
              for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int v4 = 0; v4 < 4; ++v4)
                  *reinterpret_cast<uint4*>(stage + lane * STAGE_ROW_F32 + h * 64 + v4 * 16) =
                      make_uint4(o[h][4 * v4], o[h][4 * v4 + 1], o[h][4 * v4 + 2], o[h][4 * v4 + 3]);
              __syncwarp();
#pragma unroll
              for (int k = 0; k < 8; ++k) {
                const uint4 x = *reinterpret_cast<const uint4*>(stage + (4 * k + (lane >> 3)) * STAGE_ROW_F32 + (lane & 7) * 16);
                if (4 * k + (lane >> 3) < nrows_w) *reinterpret_cast<uint4*>(po + (long long)k * 4 * 128 + qd * 32) = x;
              }
              __syncwarp();
            }
            if (valid && slot_ok) {
              p.part_ml[(slot * 128 + row) * 2] = m_used;
              p.part_ml[(slot * 128 + row) * 2 + 1] = l_sum;
            }
            wrote = slot_ok;
          }
        }
        if (cut) {
          if (!fast) {
            count_part(u, ui, t, rt, split, wrote);
          } else if ((warp & 3) == 0 && lane == 0) {  // every other part had been counted: nobody else touches it
            p.unit_cnt[(p.per == p.ncf ? (long long)ui.srank : u) * 2 + (split ? 0 : t)] = 0;
          }
        }
      }
    }
    ring += 2 * nchunks;
    chunk_cnt[0] += nch0;
    if (vtiles == 2) chunk_cnt[1] += nch1;
    pos += nfr;
    tc_fence_before();
    seg_sync();
    tc_fence_after();
    // The copy producer is outside the segment barriers and may raise the abort flag at any moment; the other warps
    // must all leave together (one that left alone would never reach the next segment barrier), so they act on one
    // thread's reading of the flag, taken between two barriers.
    if (warp == 0) {
      if (*s_abort) break;
    } else {
      if (warp == 1 && lane == 0 && *s_abort) *s_stop = 1;
      seg_sync();
      if (*s_stop) break;
    }
  }
  if constexpr (SOFTMAX) {
    if (p.unit_cnt && !*s_stop) merge_listed();
  }
  if constexpr (!SOFTMAX) {
    // A CTA that gives up must not return while copies into its shared memory are still on their way: the producer
    // waits (bounded) for the tiles it has issued and nobody consumed -- at most the ring's depth.
    if (warp == 0 && *s_abort) {
      const uint32_t issued = ring_issued;
      for (uint32_t r = issued > KV_BUFS ? issued - KV_BUFS : 0; r < issued; ++r)
        for (uint32_t it = 0; it < wait_limit && !mbar_try_wait(bars.full(r % KV_BUFS), (r / KV_BUFS) & 1); ++it)
          __nanosleep(64);
    }
  }

  };
  if (warp < SM_WARP0) {
    reg_dealloc<REGS_SERVICE>();
    run(std::false_type{});
  } else {
    reg_alloc<REGS_SOFTMAX>();
    run(std::true_type{});
  }

  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

}  // namespace

cudaError_t rekv_launch_attend_tc5(rekv_ctx* c, const void* q, const QBatch& qb, int ncf, int layer0, int layer1,
                                   void* out, cudaStream_t st, bool timed, const AttendFullArgs* full) {
  const StoreView& s = c->sv;
  TcParams p;
  p.tbl_k = full ? full->tbl_k : nullptr;
  p.self_o = full ? full->self_o : nullptr;
  p.self_ml = full ? full->self_ml : nullptr;
  p.q = (const __nv_bfloat16*)q;
  p.out = (__nv_bfloat16*)out;
  p.tbl = c->ctx_tbl;
  p.part_o = c->part_o;
  p.part_ml = c->part_ml;
  p.unit_cnt = c->unit_cnt;
  p.status = c->status;
  p.qb = qb;
  p.Hq = s.Hq;
  p.Hkv = s.Hkv;
  p.G = s.G;
  p.Nf = s.Nf;
  p.Npad = (s.Nf + 15) & ~15;
  p.Ns = (s.Nf + 7) & ~7;
  p.wait_limit = c->test_wait_limit;
  p.skip_copy_entry = c->test_skip_copy_entry;
  p.part_slots = (long long)c->part_units;
  p.ncf = ncf;
  p.layer0 = layer0;
  p.n_split = 0;
  p.scale_log2 = 1.4426950408889634f / sqrtf(128.f);
  int MP = 0;
  for (int i = 0; i < qb.nQ; ++i) MP += ((qb.cu[i + 1] - qb.cu[i]) * s.G + 255) / 256;
  p.MP = MP;
  const long long units = (long long)(layer1 - layer0) * s.Hkv * MP;
  p.total = units * ncf;
  const int n_sm = rekv_sm_count();
  long long grid;
  if (units >= 4 * n_sm || (size_t)(n_sm + units) * 2 > c->part_units) {
    grid = units;  // enough units to fill the machine: one whole unit per CTA, no partials
    p.per = ncf;
  } else {
    grid = p.total < n_sm ? p.total : n_sm;
    p.per = (int)((p.total + grid - 1) / grid);
    // a launch of few units (one layer): at least three frames per CTA -- fewer, longer ranges amortise a range's fixed
    // cost and leave fewer partials (one layer of config 2: 37 us with two or three frames per CTA, 49 with one, 40
    // with four)
    if (p.per < 3) p.per = ncf < 3 ? ncf : 3;
    grid = (p.total + p.per - 1) / p.per;
  }
  // decode-shaped batches (at most 16 query rows per KV head in every question) take the kernel that is built
  // around the loads; it needs two whole frames of one KV head in shared memory
  bool few_rows = true;
  for (int i = 0; i < qb.nQ; ++i) few_rows = few_rows && (qb.cu[i + 1] - qb.cu[i]) * s.G <= 16;
  const size_t smem_dec = std::max((size_t)4 * 2 * p.Npad * 128, (size_t)DEC_SCRATCH) + 64 + 1024;
  if (few_rows && smem_dec <= 227 * 1024 && (size_t)units <= c->part_units) {
    static PerDeviceOnce dec_attr;
    cudaError_t e = dec_attr.run([] {
      return cudaFuncSetAttribute(attend_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    });
    if (e != cudaSuccess) return e;
    // A unit cut into a few parts is merged by the CTA that finishes its last part (no further launch); when a
    // launch has few units and therefore many parts per unit (one layer at a time), the merge kernel's
    // parallelism is worth its launch.
    if (p.per < 4 && p.per != ncf) {  // a small launch (one layer): four frames per CTA amortise its fixed cost
      p.per = ncf < 4 ? ncf : 4;
      grid = (p.total + p.per - 1) / p.per;
    }
    if ((ncf + p.per - 1) / p.per + 1 > 4) p.unit_cnt = nullptr;
    if (timed) cudaEventRecord(c->ev_t0, st);
    cudaError_t e1 = rekv_launch_pdl(attend_decode_kernel, dim3((unsigned)grid), dim3(DEC_THREADS), smem_dec, st, p);
    if (e1 != cudaSuccess) return e1;
    if (timed) {
      cudaEventRecord(c->ev_t1, st);
      c->timing_valid = true;
      c->merge_timed = false;
    }
    c->launches += 1;
    if (p.per != ncf && !p.unit_cnt) {
      const bool many = (ncf + p.per - 1) / p.per + 1 > 8;  // parts per unit
      cudaError_t e2 = rekv_launch_pdl(many ? combine_many_kernel : combine_tc5_kernel, dim3((unsigned)units, 2, 32), dim3(128), 0, st, p);
      if (e2 != cudaSuccess) return e2;
      c->launches += 1;
      if (timed) {
        cudaEventRecord(c->ev_t2, st);
        c->merge_timed = true;
      }
    }
    return cudaGetLastError();
  }
  // units with a single row tile run as two half-streams whose partials the merge kernel joins; when units are
  // not cut, those partials need two slots per such unit
  {
    int n_split = 0;
    for (int i = 0; i < qb.nQ; ++i) n_split += (((qb.cu[i + 1] - qb.cu[i]) * s.G - 1) & 255) < 128;
    if (p.per == ncf && (size_t)(layer1 - layer0) * s.Hkv * n_split * 2 > c->part_units) n_split = 0;
    p.n_split = n_split;
  }
  const size_t smem = 2 * Q_TILE_BYTES + (size_t)KV_BUFS * TILE_BYTES + 8 * (2 * KV_BUFS + 6) + 64 + 1024;
  static_assert(2 * Q_TILE_BYTES + KV_BUFS * TILE_BYTES + 8 * (2 * KV_BUFS + 6) + 64 + 1024 <= 227 * 1024,
                "shared-memory plan of the attention kernel");
  static PerDeviceOnce attr;
  cudaError_t ea = attr.run([] {
    const void* kernels[] = {(const void*)attend_tc5_kernel<false, false, false>, (const void*)attend_tc5_kernel<true, false, false>,
                             (const void*)attend_tc5_kernel<false, true, false>,  (const void*)attend_tc5_kernel<true, true, false>,
                             (const void*)attend_tc5_kernel<false, false, true>,  (const void*)attend_tc5_kernel<false, true, true>};
    for (const void* k : kernels) {
      cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
      if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
  });
  if (ea != cudaSuccess) return ea;
  // A unit cut into two or three parts is finished inside the kernel by the CTA that completes its last part; with more
  // parts per unit (fewer units than SMs: 8 to 16 layers of a single question lose 2 to 13 us that way, one layer more)
  // the merge kernel's parallelism is worth its launch.
  {
    const int ctas_per_unit = p.per == ncf ? 1 : (ncf + p.per - 1) / p.per + 1;
    // (cut units that also run as two half-streams have four to six parts: 10-token question 209 against 220 us)
    if (ctas_per_unit * (p.n_split > 0 ? 2 : 1) > 3) p.unit_cnt = nullptr;
  }
  if (timed) cudaEventRecord(c->ev_t0, st);
  const bool early_q = c->q_early_ok && !full;
  auto kernel = full ? (p.n_split > 0 ? attend_tc5_kernel<true, true, false> : attend_tc5_kernel<true, false, false>)
                : early_q ? (p.n_split > 0 ? attend_tc5_kernel<false, true, true> : attend_tc5_kernel<false, false, true>)
                          : (p.n_split > 0 ? attend_tc5_kernel<false, true, false> : attend_tc5_kernel<false, false, false>);
  cudaError_t e1 = rekv_launch_pdl(kernel, dim3((unsigned)grid), dim3(TC_THREADS), smem, st, p);
  if (e1 != cudaSuccess) return e1;
  if (timed) {
    cudaEventRecord(c->ev_t1, st);
    c->timing_valid = true;
    c->merge_timed = false;
  }
  c->launches += 1;
  if ((p.per != ncf || p.n_split > 0) && !p.unit_cnt) {
    // units cut at CTA boundaries: a block group per unit; whole units: only those with half-stream partials
    const long long merge_units = p.per != ncf ? units : (long long)(layer1 - layer0) * s.Hkv * p.n_split;
    // (units with half-streams have one row tile)
    const bool many = p.per != ncf && ((ncf + p.per - 1) / p.per + 1) * (p.n_split > 0 ? 2 : 1) > 8;  // parts per unit
    cudaError_t e2 = rekv_launch_pdl(many ? combine_many_kernel : combine_tc5_kernel,
                                     dim3((unsigned)merge_units, p.per != ncf ? 2 : 1, 32), dim3(128), 0, st, p);
    if (e2 != cudaSuccess) return e2;
    c->launches += 1;
    if (timed) {
      cudaEventRecord(c->ev_t2, st);
      c->merge_timed = true;
    }
  }
  return cudaGetLastError();
}
