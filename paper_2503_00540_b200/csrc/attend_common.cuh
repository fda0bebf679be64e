// Shared by the attention kernels of step 5 (Eq. 3): the launch parameters, the decoding of a unit index and the
// kernels' declarations.  A unit is (layer, kv head, question, pair of 128-row tiles); a launch covers
// units * ncf (unit, context frame) steps, cut into contiguous ranges of `per` steps per CTA.
#pragma once

#include "ptx_helpers.cuh"
#include "rekv_internal.cuh"

namespace rekv_att {

struct TcParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  char* const* tbl;
  // Eq. 3 in full (FULL instantiation and the merge kernel only; null otherwise)
  char* const* tbl_k;      // per context slot: rotated copy of the page's K tiles, or null = K from the page
  const float* self_o;     // per output row: sum of p*v over the tokens of X the row sees, relative to self_ml[0]
  const float* self_ml;    // per output row: (max, sum) of that part, log2 domain
  float* part_o;
  float* part_ml;
  int* unit_cnt;     // per unit: parts finished so far (decode kernel: the last part merges; self-resetting)
  int* status;
  QBatch qb;
  int Hq, Hkv, G, Nf, Npad, ncf, MP, layer0;
  int Ns;           // tensor-core kernel: rows a frame takes in the token stream, N_f rounded up to a multiple of 8
  // test-only knobs (0 = off): iteration limit of the bounded waits, and the ring entry whose copy the
  // producer of CTA 0 leaves out so that a wait runs out with nothing in flight
  unsigned wait_limit;
  int skip_copy_entry;
  long long part_slots;   // capacity of part_o / part_ml in 128-row partial slots (checks build)
  int per;          // (unit, frame) steps per CTA
  // A unit with one row tile has no second tile to overlap with; it is run as two half-streams on the two tile
  // slots instead -- the same rows, the frame's token chunks dealt alternately -- whose (max, sum, O) partials the
  // merge kernel joins.  n_split = questions whose last unit is such a unit (0 = off).
  int n_split;
  long long total;  // units * ncf
  float scale_log2;
};

struct UnitInfo {
  int l, g, qi, m0, rows_q, tiles;
  int split;   // one row tile, run as two half-streams
  int srank;   // its rank among the launch's split units (partial slots when units are not cut)
  long long q_row0;
};

__device__ __forceinline__ UnitInfo decode_unit(const TcParams& p, long long u) {
  UnitInfo ui;
  int mpg = (int)(u % p.MP);
  long long r = u / p.MP;
  ui.g = (int)(r % p.Hkv);
  ui.l = p.layer0 + (int)(r / p.Hkv);
  int qi = 0, mp = mpg, before = 0;  // before = earlier questions whose last unit has one row tile
  for (; qi < p.qb.nQ - 1; ++qi) {
    const int rows = (p.qb.cu[qi + 1] - p.qb.cu[qi]) * p.G;
    int t = (rows + 255) / 256;
    if (mp < t) break;
    mp -= t;
    before += ((rows - 1) & 255) < 128;
  }
  ui.qi = qi;
  ui.rows_q = (p.qb.cu[qi + 1] - p.qb.cu[qi]) * p.G;
  ui.m0 = mp * 256;
  ui.tiles = (ui.rows_q - ui.m0 > 128) ? 2 : 1;
  ui.split = p.n_split > 0 && ui.tiles == 1;
  ui.srank = ((ui.l - p.layer0) * p.Hkv + ui.g) * p.n_split + before;
  ui.q_row0 = (long long)ui.l * p.qb.sumNq + p.qb.cu[qi];
  return ui;
}

// k_attend_decode.cu: the load-bound kernel for questions of at most 16 rows per KV head
constexpr int DEC_THREADS = 256;
constexpr int DEC_WARPS = 8;
constexpr uint32_t DEC_SCRATCH = DEC_WARPS * 16 * (128 + 2) * 4;  // the warps' (O, max, sum) at the end of a range
__global__ void attend_decode_kernel(const TcParams p);
// k_attend_combine.cu: joins the (max, sum, O) partials of a unit's parts
__global__ void combine_tc5_kernel(const TcParams p);
__global__ void combine_many_kernel(const TcParams p);  // units of many parts (launches of few units)

}  // namespace rekv_att
