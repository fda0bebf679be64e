// Internal declarations shared by the librekv translation units: the context, the store's
// address arithmetic and the kernel launchers.  Nothing here is part of the public ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "rekv.h"

#define REKV_MAX_QUESTIONS 64
#define REKV_HEAD_DIM 128

// ---------------------------------------------------------------------------------------------
// Store layout
//
// One page = one (frame, layer): for every KV head a K tile followed by a V tile.
// A tile holds the head's N_f tokens x 128 dims as two 64-dim halves, each half a dense
// [N_f rows][128 bytes] block whose 16-byte chunks are XOR-swizzled with (row & 7) -- the 128-byte
// shared-memory swizzle of the tensor-core operand layouts.  A tile half can therefore be moved
// into shared memory with one contiguous bulk copy and used by MMA instructions as it lands.
//   page_bytes = H_kv * 2 * N_f * 256
//   tile(h, kv) at (h*2 + kv) * N_f*256;  half hh at + hh * N_f*128
//   element (row, dim): + row*128 + (((dim%64)/8) ^ (row&7))*16 + (dim%8)*2
// Pages are frame-major: page(frame, layer) = base + (slot(frame)*L + layer) * page_bytes, so one
// appended frame is one contiguous range (one D2H copy to the host tier).
// FP8 host tier (REKV_FLAG_HOST_FP8): a host page holds, for the same (head, K/V) tiles, rows of 128 E4M3
// codes in natural dim order -- tile(h, kv) at (h*2 + kv) * N_f*128, row r at + r*128 -- followed by one
// float scale per row, scale[(h*2 + kv)*N_f + r], at H_kv*2*N_f*128; padded to a multiple of 16 bytes.
// ---------------------------------------------------------------------------------------------
struct StoreView {
  char* hbm;                   // HBM tier (all frames, or a ring of `tail` frames when offloaded)
  char* const* host_arenas;    // device array of pinned-host arena base pointers (offloaded only)
  char* staging;               // HBM staging pages for host-tier gathers (offloaded only)
  float* reps;                 // [L][max_frames][D'] fp32
  long long page_bytes;
  long long host_page_bytes;   // bytes of a page in the host tier (= page_bytes, or the FP8 form)
  char* q8_ring;               // FP8 host tier: the quantised form of the ring's frames, source of the write-through
  int host_fp8;                // the host tier holds FP8 E4M3 codes + one float scale per page row
  int L, Hq, Hkv, G, Nf, Dp;   // Dp = Hkv * 128
  int max_frames, tail, frames_per_arena;
};

__host__ __device__ inline long long rekv_tile_bytes(int Nf) { return (long long)Nf * 256; }

__host__ __device__ inline long long rekv_hbm_page_offset(const StoreView& s, int frame, int layer) {
  int slot = s.tail > 0 ? frame % s.tail : frame;
  return ((long long)slot * s.L + layer) * s.page_bytes;
}

// Context geometry of a question.  With block retrieval (b > 1, Eq. 2 paragraph) only complete blocks of the
// candidate frames [0, n_visible - W) can be retrieved; every frame after the last complete block is in the
// context: the recent window plus the frames that do not fill a block yet.  b = 1 gives the plain rule.
struct CtxGeom {
  int n_items;   // retrieval candidates: frames (b = 1) or complete blocks
  int k_items;   // items actually retrieved
  int k_eff;     // frames actually retrieved = k_items * b
  int w_eff;     // trailing frames that are always in the context
  int ncf;       // context frames = k_eff + w_eff
};
inline CtxGeom rekv_geom(int n_visible, int window, int b, int top_k) {
  CtxGeom g;
  int n_cand = n_visible - window;
  if (n_cand < 0) n_cand = 0;
  g.n_items = n_cand / b;
  g.k_items = top_k / b < g.n_items ? top_k / b : g.n_items;
  g.k_eff = g.k_items * b;
  g.w_eff = n_visible - g.n_items * b;
  g.ncf = g.k_eff + g.w_eff;
  return g;
}

// Batch of questions, passed to kernels by value (no device-side table to keep alive).
struct QBatch {
  int nQ;
  int sumNq;
  int cu[REKV_MAX_QUESTIONS + 1];  // prefix sums of question lengths
};

struct rekv_ctx {
  rekv_config cfg;
  StoreView sv;
  int device;
  int frames;                       // appended so far
  std::string err;
  int64_t launches;

  // host tier
  std::vector<char*> host_arenas;   // pinned
  char** d_host_arenas;             // device copy of the pointer table
  cudaStream_t side;                // D2H write-through and host-tier gathers
  std::vector<cudaEvent_t> slot_events;   // per ring slot: its D2H write-through finished
  std::vector<char> slot_event_valid;
  cudaEvent_t ev_main;              // caller stream -> side stream fence
  cudaEvent_t ev_side;              // side stream -> caller stream fence
  std::vector<cudaEvent_t> layer_events;  // per layer: its host-tier gather finished
  bool d2h_pending;
  cudaEvent_t ring_reader_ev;       // offloaded: the last gather on the side stream, which reads ring pages; the next
                                    // append (it recycles a ring slot on the caller's stream) waits for it once
  // REKV_FLAG_TIMING: event pairs around the stages of the last question; rekv_stats reads the pairs that have
  // completed (cudaEventQuery) and never waits.  ev_t0/ev_t1 around the attention kernel, ev_t2 after its merge kernel;
  // ev_r0/ev_r1 around steps 2-3; ev_p0/ev_p1 (on the side stream) around the host-tier pulls of a gather.
  cudaEvent_t ev_t0, ev_t1, ev_t2, ev_r0, ev_r1, ev_p0, ev_p1;
  bool timing_valid, merge_timed, retrieve_timed, pull_timed;
  unsigned long long* h_link_bytes; // pinned host mirror of link_bytes, refreshed (asynchronously) after each gather

  // scratch (device)
  float* qa;                        // [L][max_questions][Dp] fp32 question vectors
  float* qnorm;                     // [L][max_questions][H_kv] partial sums of squares of the question vector
  float* scores;                    // [L][max_questions][max_frames]
  char** ctx_tbl;                   // [L][max_questions][max_topk + W] page pointers
  float* part_o;                    // split-KV partial outputs
  float* part_ml;                   // split-KV partial (max, sum)
  size_t part_units;                // capacity in (unit) entries of 128 rows
  int* unit_cnt;                    // [part_units] parts finished per unit (zero between launches)
  int* status;                      // device status word
  unsigned long long* link_bytes;   // device counter: bytes pulled over the host link
  int32_t* idx_own;                 // [L][max_questions][max_topk]: selections of the layer-sequential calls

  // external retrieval (allocated when ext_embed_dim > 0)
  float* ext_emb;                   // [max_frames][ext_embed_dim] frame embeddings
  int ext_frames;                   // embeddings are set for frames [0, ext_frames)

  // Eq. 3 in full (allocated when max_self_tokens > 0)
  float* self_o;                    // [L][max_q_tokens][H_q][128]
  float* self_ml;                   // [L][max_q_tokens][H_q][2]
  __nv_bfloat16* q_rot;             // [L][max_q_tokens][H_q][128] rotated queries (rope_theta > 0)
  float2* rope_tab;                 // [rope_positions][64] (cos, sin)
  int rope_positions;
  char* k_rot;                      // [L][max_questions][ctx frames][H_kv] rotated K tiles
  char** tbl_k;                     // [L][max_questions][ctx frames]
  int ctx_frames_max;

  // test-only knobs of the bounded device-side waits (rekv_test_set_wait_limit); 0 / -1 = off
  unsigned test_wait_limit;
  int test_skip_copy_entry;
  bool self_forked = false;         // Eq. 3 in full: the part over X is on the internal stream, ev_side marks its end
  bool q_early_ok = false;          // the attention launch that follows is chained to the library's own selection kernels (which only read Q)

  // state of the last gather.  The context table has one geometry (questions x context frames) for all layers; a
  // layer's context is valid while the table still has the geometry it was built with (layer_ctx_valid).
  std::vector<char> layer_ctx_valid;
  bool gathered;
  bool gather_layerwise;            // layer events are pending (offloaded context)
  int g_nQ, g_ncf, g_keff, g_nvis, g_topk;
};

#define REKV_FAIL(ctx, code, ...)                         \
  do {                                                    \
    char _b[512];                                         \
    snprintf(_b, sizeof(_b), __VA_ARGS__);                \
    rekv_set_error((ctx), _b);                            \
    return (code);                                        \
  } while (0)

#define REKV_CUDA(ctx, call)                                                                   \
  do {                                                                                         \
    cudaError_t _e = (call);                                                                   \
    if (_e != cudaSuccess)                                                                     \
      REKV_FAIL(ctx, REKV_ERR_CUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(_e),    \
                __FILE__, __LINE__);                                                           \
  } while (0)

void rekv_set_error(rekv_ctx* ctx, const char* msg);

// Checks build (-DREKV_CHECKS): the stand-in for a memory checker on machines where none can run.  Index and address
// computations of the kernels are tested before use; a violation is recorded in the context's status word as
// -(2000 + site) -- rekv_check_status then fails with that code -- and the access is skipped.  Nothing traps or faults.
// In the shipped build the tests compile to nothing.
#ifdef REKV_CHECKS
#define REKV_CHECK(cond, status, site) ((cond) ? true : ((status) ? (atomicExch((status), -(2000 + (site))), false) : false))
#else
#define REKV_CHECK(cond, status, site) (true)
#endif

// Launch state that belongs to one device: a function attribute (the dynamic shared-memory limit) is set on the
// function of the CURRENT device only, so "already set" is kept per device ordinal, and the SM count is asked of
// each device once.  A context created on a second device of the same process gets its own settings.
constexpr int REKV_MAX_DEVICES = 64;
struct PerDeviceOnce {
  bool done[REKV_MAX_DEVICES] = {};
  // runs set() unless it has succeeded before on the current device
  template <typename F>
  cudaError_t run(F&& set) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const bool known = dev >= 0 && dev < REKV_MAX_DEVICES;
    if (known && done[dev]) return cudaSuccess;
    e = set();
    if (e == cudaSuccess && known) done[dev] = true;
    return e;
  }
};
inline int rekv_sm_count() {  // of the current device
  static int sms[REKV_MAX_DEVICES] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 1;
  const bool known = dev >= 0 && dev < REKV_MAX_DEVICES;
  if (known && sms[dev] > 0) return sms[dev];
  int n = 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 1;
  if (known) sms[dev] = n;
  return n;
}

// Launch with programmatic stream serialization: the kernel may begin (its prologue up to
// grid_dep_wait()) while the previous kernel of the stream is still draining.
template <typename... KArgs, typename... Args>
inline cudaError_t rekv_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                   Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Extra inputs of the attention kernel for Eq. 3 in full.
struct AttendFullArgs {
  char* const* tbl_k;    // rotated K tiles per context slot (null without rotary embedding)
  const float* self_o;   // [L][sum_Nq][H_q][128] partial numerators over the tokens of X
  const float* self_ml;  // [L][sum_Nq][H_q][2] their (max, sum), log2 domain
};

// ---- kernel launchers (each returns the cudaError_t of its launches) -----------------------
// k_append.cu
cudaError_t rekv_launch_append(rekv_ctx* c, const void* k, const void* v, int frame, cudaStream_t st);
cudaError_t rekv_launch_unswizzle_page(rekv_ctx* c, const char* page, void* k_out, void* v_out, cudaStream_t st);
// k_retrieve.cu
cudaError_t rekv_launch_retrieve(rekv_ctx* c, const void* q, const QBatch& qb, int top_k, const CtxGeom& geom,
                                 int n_visible, int layer0, int layer1, int32_t* idx_out, float* scores, cudaStream_t st,
                                 bool write_table = false);
cudaError_t rekv_launch_retrieve_external(rekv_ctx* c, const float* q_emb, int nQ, int top_k, const CtxGeom& geom,
                                          int n_visible, float tau, int32_t* idx_out, float* scores, cudaStream_t st);
// k_gather.cu
cudaError_t rekv_launch_quantize_frame(rekv_ctx* c, int frame, cudaStream_t st);
cudaError_t rekv_launch_dequant_page(rekv_ctx* c, const char* host_page, char* dst_page, cudaStream_t st);
cudaError_t rekv_launch_page_table(rekv_ctx* c, const int32_t* idx, int nQ, int top_k, const CtxGeom& geom,
                                   int n_visible, int layer0, int layer1, int frames_now, cudaStream_t st);
cudaError_t rekv_launch_materialize(rekv_ctx* c, int nQ, int ncf, void* k_ctx, void* v_ctx, cudaStream_t st);
// k_attend_tc5.cu
cudaError_t rekv_launch_attend_tc5(rekv_ctx* c, const void* q, const QBatch& qb, int ncf, int layer0, int layer1,
                                   void* out, cudaStream_t st, bool timed, const AttendFullArgs* full = nullptr);
// k_attend_full.cu: the pieces of Eq. 3 in full around the attention kernel
cudaError_t rekv_launch_rope_table(rekv_ctx* c, cudaStream_t st);
cudaError_t rekv_launch_attend_full_self(rekv_ctx* c, const void* q, const void* k_self, const void* v_self,
                                         const QBatch& qb, const QBatch& sb, int ncf, cudaStream_t st, int layer0,
                                         int layer1, bool early);
cudaError_t rekv_launch_attend_full_ctx(rekv_ctx* c, const QBatch& qb, int ncf, cudaStream_t st, int layer0,
                                        int layer1);
cudaError_t rekv_launch_self_finalize(rekv_ctx* c, const QBatch& qb, void* out, cudaStream_t st, int layer0,
                                      int layer1);
