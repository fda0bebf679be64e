// The C ABI of librekv: context life cycle, argument checks, stream/event plumbing.
// Every step of the path runs in the kernels of the k_*.cu files; this file only launches them.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>

#include "rekv_internal.cuh"

static thread_local std::string g_create_error;

void rekv_set_error(rekv_ctx* ctx, const char* msg) {
  if (ctx)
    ctx->err = msg;
  else
    g_create_error = msg;
}

namespace {

struct DeviceGuard {
  int prev = -1;
  explicit DeviceGuard(int dev) {
    cudaGetDevice(&prev);
    if (prev != dev) cudaSetDevice(dev);
  }
  ~DeviceGuard() {
    int cur = -1;
    cudaGetDevice(&cur);
    if (prev >= 0 && cur != prev) cudaSetDevice(prev);
  }
};

constexpr long long ARENA_BYTES = 4ll << 30;

int build_qbatch(rekv_ctx* c, const int32_t* cu_q, int nQ, QBatch* qb) {
  if (!cu_q) REKV_FAIL(c, REKV_ERR_ARG, "cu_q is null");
  if (nQ < 1 || nQ > c->cfg.max_questions) REKV_FAIL(c, REKV_ERR_ARG, "nQ=%d outside [1, %d]", nQ, c->cfg.max_questions);
  if (cu_q[0] != 0) REKV_FAIL(c, REKV_ERR_ARG, "cu_q[0] must be 0");
  qb->nQ = nQ;
  for (int i = 0; i < nQ; ++i) {
    if (cu_q[i + 1] <= cu_q[i]) REKV_FAIL(c, REKV_ERR_ARG, "question %d has no tokens", i);
    qb->cu[i] = cu_q[i];
  }
  qb->cu[nQ] = cu_q[nQ];
  qb->sumNq = cu_q[nQ];
  if (qb->sumNq > c->cfg.max_q_tokens)
    REKV_FAIL(c, REKV_ERR_ARG, "sum of question lengths %d exceeds max_q_tokens %d", qb->sumNq, c->cfg.max_q_tokens);
  return 0;
}

void free_ctx(rekv_ctx* c) {
  if (!c) return;
  cudaDeviceSynchronize();
  cudaFree(c->sv.hbm);
  cudaFree(c->sv.staging);
  cudaFree(c->sv.q8_ring);
  cudaFree(c->sv.reps);
  cudaFree(c->d_host_arenas);
  cudaFree(c->qa);
  cudaFree(c->qnorm);
  cudaFree(c->scores);
  cudaFree(c->ctx_tbl);
  cudaFree(c->part_o);
  cudaFree(c->part_ml);
  cudaFree(c->unit_cnt);
  cudaFree(c->status);
  cudaFree(c->idx_own);
  cudaFree(c->ext_emb);
  cudaFree(c->self_o);
  cudaFree(c->self_ml);
  cudaFree(c->q_rot);
  cudaFree(c->rope_tab);
  cudaFree(c->k_rot);
  cudaFree(c->tbl_k);
  cudaFree(c->link_bytes);
  for (char* a : c->host_arenas) cudaFreeHost(a);
  for (cudaEvent_t e : c->slot_events) cudaEventDestroy(e);
  for (cudaEvent_t e : c->layer_events) cudaEventDestroy(e);
  if (c->ev_main) cudaEventDestroy(c->ev_main);
  if (c->ev_side) cudaEventDestroy(c->ev_side);
  for (cudaEvent_t e : {c->ev_t0, c->ev_t1, c->ev_t2, c->ev_r0, c->ev_r1, c->ev_p0, c->ev_p1})
    if (e) cudaEventDestroy(e);
  if (c->h_link_bytes) cudaFreeHost(c->h_link_bytes);
  if (c->side) cudaStreamDestroy(c->side);
  delete c;
}

// The kernels index q, out and idx with the absolute layer; a per-layer buffer is passed moved back
// by `layer` layers (only the addresses inside the caller's buffer are ever formed by the kernels).
template <typename T>
T* layer_view(T* base, int layer, long long bytes_per_layer) {
  return reinterpret_cast<T*>(reinterpret_cast<intptr_t>(base) - (intptr_t)layer * bytes_per_layer);
}

int attend_one_layer(rekv_ctx* c, int layer, const void* q, const QBatch& qb, void* out, cudaStream_t st) {
  const StoreView& s = c->sv;
  const long long row_bytes = (long long)s.Hq * REKV_HEAD_DIM * 2;
  if (c->g_ncf == 0) {
    REKV_CUDA(c, cudaMemsetAsync(out, 0, (size_t)(qb.sumNq * row_bytes), st));
    return REKV_OK;
  }
  REKV_CUDA(c, rekv_launch_attend_tc5(c, layer_view(q, layer, qb.sumNq * row_bytes), qb, c->g_ncf, layer, layer + 1,
                      layer_view(out, layer, qb.sumNq * row_bytes), st, false, nullptr));
  if (s.tail > 0) {
    // later appends (ring slots) and gathers (staging) on the side stream must not overtake this read
    REKV_CUDA(c, cudaEventRecord(c->ev_side, st));
    REKV_CUDA(c, cudaStreamWaitEvent(c->side, c->ev_side, 0));
  }
  return REKV_OK;
}
}  // namespace

extern "C" {

int rekv_create(const rekv_config* cfg, rekv_ctx** out) {
  if (!cfg || !out) REKV_FAIL(nullptr, REKV_ERR_ARG, "null config or output pointer");
  *out = nullptr;
  if (cfg->head_dim != REKV_HEAD_DIM) REKV_FAIL(nullptr, REKV_ERR_ARG, "head_dim must be 128, got %d", cfg->head_dim);
  if (cfg->n_layers < 1 || cfg->n_layers > 1023) REKV_FAIL(nullptr, REKV_ERR_ARG, "n_layers=%d out of range", cfg->n_layers);
  if (cfg->n_kv_heads < 1 || cfg->n_kv_heads > 8 || cfg->n_q_heads < cfg->n_kv_heads ||
      cfg->n_q_heads % cfg->n_kv_heads)
    REKV_FAIL(nullptr, REKV_ERR_ARG, "unsupported head counts: %d query / %d kv (kv <= 8, query a multiple of kv)",
              cfg->n_q_heads, cfg->n_kv_heads);
  if (cfg->tokens_per_frame < 1 || cfg->tokens_per_frame > 1024)
    REKV_FAIL(nullptr, REKV_ERR_ARG, "tokens_per_frame=%d outside [1, 1024]", cfg->tokens_per_frame);
  if (cfg->max_frames < 1) REKV_FAIL(nullptr, REKV_ERR_ARG, "max_frames must be positive");
  if (cfg->block_frames < 1 || cfg->block_frames > 64)
    REKV_FAIL(nullptr, REKV_ERR_ARG, "block_frames=%d outside [1, 64]", cfg->block_frames);
  if (cfg->max_topk % cfg->block_frames)
    REKV_FAIL(nullptr, REKV_ERR_ARG, "max_topk=%d must be a multiple of block_frames=%d", cfg->max_topk, cfg->block_frames);
  if (cfg->window_frames < 0) REKV_FAIL(nullptr, REKV_ERR_ARG, "window_frames must be >= 0");
  if (cfg->hbm_tail_frames < 0 ||
      (cfg->hbm_tail_frames > 0 && cfg->window_frames + cfg->block_frames - 1 > cfg->hbm_tail_frames))
    REKV_FAIL(nullptr, REKV_ERR_ARG, "window_frames=%d must fit in hbm_tail_frames=%d", cfg->window_frames,
              cfg->hbm_tail_frames);
  if (cfg->max_questions < 1 || cfg->max_questions > REKV_MAX_QUESTIONS)
    REKV_FAIL(nullptr, REKV_ERR_ARG, "max_questions=%d outside [1, %d]", cfg->max_questions, REKV_MAX_QUESTIONS);
  if (cfg->max_q_tokens < 1 || cfg->max_topk < 0) REKV_FAIL(nullptr, REKV_ERR_ARG, "max_q_tokens / max_topk out of range");
  if (cfg->max_self_tokens < 0 || !(cfg->rope_theta >= 0.f) || (cfg->rope_theta > 0.f && cfg->rope_theta < 1.f))
    REKV_FAIL(nullptr, REKV_ERR_ARG, "max_self_tokens must be >= 0 and rope_theta 0 or >= 1");
  if (cfg->ext_embed_dim < 0 || cfg->ext_embed_dim > 2048 || cfg->ext_embed_dim % 4)
    REKV_FAIL(nullptr, REKV_ERR_ARG, "ext_embed_dim=%d must be a multiple of 4 in [0, 2048]", cfg->ext_embed_dim);

  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev == 0) {
    cudaGetLastError();
    REKV_FAIL(nullptr, REKV_ERR_CUDA, "no CUDA device: librekv has no CPU path");
  }
  if (cfg->device < 0 || cfg->device >= n_dev) REKV_FAIL(nullptr, REKV_ERR_ARG, "device %d not present", cfg->device);
  DeviceGuard guard(cfg->device);

  rekv_ctx* c = new (std::nothrow) rekv_ctx();
  if (!c) REKV_FAIL(nullptr, REKV_ERR_ALLOC, "out of host memory");
  c->cfg = *cfg;
  c->device = cfg->device;
  c->frames = 0;
  c->launches = 0;
  c->d_host_arenas = nullptr;
  c->side = nullptr;
  c->ev_main = c->ev_side = nullptr;
  c->ev_t0 = c->ev_t1 = c->ev_t2 = c->ev_r0 = c->ev_r1 = c->ev_p0 = c->ev_p1 = nullptr;
  c->timing_valid = c->merge_timed = c->retrieve_timed = c->pull_timed = false;
  c->h_link_bytes = nullptr;
  c->d2h_pending = false;
  c->ring_reader_ev = nullptr;
  c->layer_ctx_valid.assign(cfg->n_layers, 0);
  c->gathered = false;
  c->gather_layerwise = false;
  memset(&c->sv, 0, sizeof(c->sv));
  c->qa = c->qnorm = c->scores = c->part_o = c->part_ml = nullptr;
  c->unit_cnt = nullptr;
  c->ctx_tbl = nullptr;
  c->status = nullptr;
  c->link_bytes = nullptr;
  c->idx_own = nullptr;
  c->self_o = c->self_ml = nullptr;
  c->ext_emb = nullptr;
  c->ext_frames = 0;
  c->q_rot = nullptr;
  c->rope_tab = nullptr;
  c->k_rot = nullptr;
  c->tbl_k = nullptr;
  c->rope_positions = 0;
  c->test_wait_limit = 0;
  c->test_skip_copy_entry = -1;

  StoreView& s = c->sv;
  s.L = cfg->n_layers;
  s.Hq = cfg->n_q_heads;
  s.Hkv = cfg->n_kv_heads;
  s.G = s.Hq / s.Hkv;
  s.Nf = cfg->tokens_per_frame;
  s.Dp = s.Hkv * REKV_HEAD_DIM;
  s.max_frames = cfg->max_frames;
  s.tail = cfg->hbm_tail_frames;
  s.page_bytes = (long long)s.Hkv * 2 * s.Nf * 256;
  s.host_fp8 = (s.tail > 0 && (cfg->flags & REKV_FLAG_HOST_FP8)) ? 1 : 0;
  // FP8 host tier: 128 codes + one float scale per page row, padded to a multiple of 16 bytes
  s.host_page_bytes = s.host_fp8 ? (((long long)s.Hkv * 2 * s.Nf * (128 + 4) + 15) & ~15ll) : s.page_bytes;
  const long long frame_bytes = s.page_bytes * s.L;
  const long long host_frame_bytes = s.host_page_bytes * s.L;
  s.frames_per_arena = (int)(ARENA_BYTES / host_frame_bytes);
  if (s.frames_per_arena < 1) s.frames_per_arena = 1;

#define CREATE_CUDA(call, what)                                                                              \
  do {                                                                                                       \
    cudaError_t _e = (call);                                                                                 \
    if (_e != cudaSuccess) {                                                                                 \
      char _b[256];                                                                                          \
      snprintf(_b, sizeof(_b), "%s: %s", what, cudaGetErrorString(_e));                                      \
      cudaGetLastError();                                                                                    \
      free_ctx(c);                                                                                           \
      rekv_set_error(nullptr, _b);                                                                           \
      return _e == cudaErrorMemoryAllocation ? REKV_ERR_ALLOC : REKV_ERR_CUDA;                               \
    }                                                                                                        \
  } while (0)

  const long long hbm_frames = s.tail > 0 ? s.tail : s.max_frames;
  CREATE_CUDA(cudaMalloc(&s.hbm, (size_t)(hbm_frames * frame_bytes)), "allocating the HBM frame store");
  CREATE_CUDA(cudaMalloc(&s.reps, (size_t)s.L * s.max_frames * s.Dp * sizeof(float)), "allocating the representative table");
  const int ctx_frames_max = cfg->max_topk + cfg->window_frames + cfg->block_frames - 1;
  const int maxQ = cfg->max_questions;
  CREATE_CUDA(cudaMalloc(&c->qa, (size_t)s.L * maxQ * s.Dp * sizeof(float)), "allocating question vectors");
  CREATE_CUDA(cudaMalloc(&c->qnorm, (size_t)s.L * maxQ * s.Hkv * sizeof(float)), "allocating question norms");
  CREATE_CUDA(cudaMalloc(&c->scores, (size_t)s.L * maxQ * s.max_frames * sizeof(float)), "allocating the score buffer");
  CREATE_CUDA(cudaMalloc(&c->ctx_tbl, (size_t)s.L * maxQ * (ctx_frames_max + 1) * sizeof(char*)), "allocating the context table");
  // 2048 slots cover every launch whose units are cut at CTA boundaries; launches of many whole units park two
  // half-stream partials per unit with a single row tile (at most one per layer, KV head and question), up to a cap
  c->part_units = std::min<size_t>(8192, std::max<size_t>(2048, (size_t)2 * s.L * s.Hkv * maxQ + 16));
  CREATE_CUDA(cudaMalloc(&c->part_o, c->part_units * 128 * 128 * sizeof(float)), "allocating split-KV partials");
  CREATE_CUDA(cudaMalloc(&c->part_ml, c->part_units * 128 * 2 * sizeof(float)), "allocating split-KV partials");
  CREATE_CUDA(cudaMalloc(&c->unit_cnt, c->part_units * sizeof(int)), "allocating split-KV counters");
  CREATE_CUDA(cudaMemset(c->unit_cnt, 0, c->part_units * sizeof(int)), "clearing split-KV counters");
  CREATE_CUDA(cudaMalloc(&c->status, sizeof(int)), "allocating the status word");
  CREATE_CUDA(cudaMemset(c->status, 0, sizeof(int)), "clearing the status word");
  CREATE_CUDA(cudaMalloc(&c->idx_own, (size_t)s.L * maxQ * (c->cfg.max_topk > 0 ? c->cfg.max_topk : 1) * sizeof(int32_t)),
              "allocating the selection buffer");
  c->ctx_frames_max = ctx_frames_max;
  if (c->cfg.ext_embed_dim > 0)
    CREATE_CUDA(cudaMalloc(&c->ext_emb, (size_t)s.max_frames * c->cfg.ext_embed_dim * sizeof(float)),
                "allocating the embedding table");
  if (c->cfg.max_self_tokens > 0) {  // workspaces of rekv_attend_full
    const size_t rows = (size_t)s.L * c->cfg.max_q_tokens * s.Hq;
    CREATE_CUDA(cudaMalloc(&c->self_o, rows * 128 * sizeof(float)), "allocating the self-attention partials");
    CREATE_CUDA(cudaMalloc(&c->self_ml, rows * 2 * sizeof(float)), "allocating the self-attention partials");
    if (c->cfg.rope_theta > 0.f) {
      const bool static_ctx = (cfg->flags & REKV_FLAG_ROPE_STATIC) != 0;
      c->rope_positions = (static_ctx ? 1 : ctx_frames_max * s.Nf) + c->cfg.max_self_tokens;
      CREATE_CUDA(cudaMalloc(&c->q_rot, rows * 128 * sizeof(__nv_bfloat16)), "allocating rotated queries");
      CREATE_CUDA(cudaMalloc(&c->rope_tab, (size_t)c->rope_positions * 64 * sizeof(float2)), "allocating the rotary table");
      if (!static_ctx) {
        CREATE_CUDA(cudaMalloc(&c->k_rot, (size_t)s.L * maxQ * ctx_frames_max * (s.page_bytes / 2)),
                    "allocating rotated key tiles");
        CREATE_CUDA(cudaMalloc(&c->tbl_k, (size_t)s.L * maxQ * (ctx_frames_max + 1) * sizeof(char*)),
                    "allocating the rotated-key table");
      }
      CREATE_CUDA(rekv_launch_rope_table(c, 0), "building the rotary table");
      CREATE_CUDA(cudaDeviceSynchronize(), "building the rotary table");
    }
  }
  CREATE_CUDA(cudaMalloc(&c->link_bytes, sizeof(unsigned long long)), "allocating counters");
  CREATE_CUDA(cudaMemset(c->link_bytes, 0, sizeof(unsigned long long)), "clearing counters");
  CREATE_CUDA(cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking), "creating the side stream");
  CREATE_CUDA(cudaEventCreateWithFlags(&c->ev_main, cudaEventDisableTiming), "creating events");
  CREATE_CUDA(cudaEventCreateWithFlags(&c->ev_side, cudaEventDisableTiming), "creating events");
  for (cudaEvent_t* e : {&c->ev_t0, &c->ev_t1, &c->ev_t2, &c->ev_r0, &c->ev_r1, &c->ev_p0, &c->ev_p1})
    CREATE_CUDA(cudaEventCreate(e), "creating events");
  CREATE_CUDA(cudaHostAlloc((void**)&c->h_link_bytes, sizeof(unsigned long long), cudaHostAllocDefault), "allocating counters");
  *c->h_link_bytes = 0;

  if (s.tail > 0) {
    // pinned-host tier: arenas of whole frames, allocated up front so that append never blocks
    const int n_arenas = (s.max_frames + s.frames_per_arena - 1) / s.frames_per_arena;
    for (int a = 0; a < n_arenas; ++a) {
      int fr = s.max_frames - a * s.frames_per_arena;
      if (fr > s.frames_per_arena) fr = s.frames_per_arena;
      char* p = nullptr;
      cudaError_t e = cudaHostAlloc((void**)&p, (size_t)fr * host_frame_bytes, cudaHostAllocDefault);
      if (e != cudaSuccess) {
        cudaGetLastError();
        char b[256];
        snprintf(b, sizeof(b), "pinning host arena %d of %d (%lld bytes): %s", a, n_arenas, fr * host_frame_bytes,
                 cudaGetErrorString(e));
        free_ctx(c);
        rekv_set_error(nullptr, b);
        return REKV_ERR_ALLOC;
      }
      c->host_arenas.push_back(p);
    }
    CREATE_CUDA(cudaMalloc(&c->d_host_arenas, n_arenas * sizeof(char*)), "allocating the arena table");
    CREATE_CUDA(cudaMemcpy(c->d_host_arenas, c->host_arenas.data(), n_arenas * sizeof(char*), cudaMemcpyHostToDevice),
                "uploading the arena table");
    s.host_arenas = c->d_host_arenas;
    CREATE_CUDA(cudaMalloc(&s.staging, (size_t)s.L * maxQ * ctx_frames_max * s.page_bytes), "allocating gather staging");
    if (s.host_fp8)
      CREATE_CUDA(cudaMalloc(&s.q8_ring, (size_t)s.tail * host_frame_bytes), "allocating the quantised write-through ring");
    c->slot_events.resize(s.tail);
    c->slot_event_valid.assign(s.tail, 0);
    for (int i = 0; i < s.tail; ++i)
      CREATE_CUDA(cudaEventCreateWithFlags(&c->slot_events[i], cudaEventDisableTiming), "creating events");
    c->layer_events.resize(s.L);
    for (int i = 0; i < s.L; ++i)
      CREATE_CUDA(cudaEventCreateWithFlags(&c->layer_events[i], cudaEventDisableTiming), "creating events");
  }
#undef CREATE_CUDA
  *out = c;
  return REKV_OK;
}

int rekv_destroy(rekv_ctx* ctx) {
  if (!ctx) return REKV_ERR_ARG;
  DeviceGuard guard(ctx->device);
  free_ctx(ctx);
  return REKV_OK;
}

int rekv_append_frame(rekv_ctx* c, const void* k, const void* v, void* stream) {
  if (!c) return REKV_ERR_ARG;
  if (!k || !v) REKV_FAIL(c, REKV_ERR_ARG, "null K or V");
  if (c->frames >= c->cfg.max_frames) REKV_FAIL(c, REKV_ERR_FULL, "store is full (%d frames)", c->cfg.max_frames);
  DeviceGuard guard(c->device);
  cudaStream_t st = (cudaStream_t)stream;
  const int f = c->frames;
  const StoreView& s = c->sv;
  if (s.tail > 0) {
    // the ring slot is reused: its previous occupant's write-through must have left HBM
    const int slot = f % s.tail;
    if (c->slot_event_valid[slot]) REKV_CUDA(c, cudaStreamWaitEvent(st, c->slot_events[slot], 0));
    // ... and a gather that is still copying ring pages into its context (side stream) must have read them
    if (c->ring_reader_ev) {
      REKV_CUDA(c, cudaStreamWaitEvent(st, c->ring_reader_ev, 0));
      c->ring_reader_ev = nullptr;
    }
  }
  REKV_CUDA(c, rekv_launch_append(c, k, v, f, st));
  if (s.tail > 0) {
    const int slot = f % s.tail;
    const long long host_frame_bytes = s.host_page_bytes * s.L;
    char* dst = c->host_arenas[f / s.frames_per_arena] + (long long)(f % s.frames_per_arena) * host_frame_bytes;
    const char* src = s.hbm + rekv_hbm_page_offset(s, f, 0);
    if (s.host_fp8) {  // the frame's FP8 form is made on the caller's stream and written through instead
      REKV_CUDA(c, rekv_launch_quantize_frame(c, f, st));
      src = s.q8_ring + (long long)slot * host_frame_bytes;
    }
    REKV_CUDA(c, cudaEventRecord(c->ev_main, st));
    REKV_CUDA(c, cudaStreamWaitEvent(c->side, c->ev_main, 0));
    REKV_CUDA(c, cudaMemcpyAsync(dst, src, (size_t)host_frame_bytes, cudaMemcpyDeviceToHost, c->side));
    REKV_CUDA(c, cudaEventRecord(c->slot_events[slot], c->side));
    c->slot_event_valid[slot] = 1;
    c->d2h_pending = true;
  }
  c->frames = f + 1;
  return f;
}

int rekv_retrieve(rekv_ctx* c, const void* q, const int32_t* cu_q, int nQ, int top_k, int n_visible, int32_t* idx_out,
                  float* scores_out, void* stream) {
  if (!c) return REKV_ERR_ARG;
  if (!q) REKV_FAIL(c, REKV_ERR_ARG, "null q");
  if (top_k < 0 || top_k > c->cfg.max_topk) REKV_FAIL(c, REKV_ERR_ARG, "top_k=%d outside [0, %d]", top_k, c->cfg.max_topk);
  if (top_k > 0 && !idx_out) REKV_FAIL(c, REKV_ERR_ARG, "null idx_out");
  if (n_visible < 0 || n_visible > c->frames)
    REKV_FAIL(c, REKV_ERR_ARG, "n_visible=%d outside [0, %d]", n_visible, c->frames);
  if (n_visible == 0) REKV_FAIL(c, REKV_ERR_EMPTY, "no visible frame");
  QBatch qb;
  int rc = build_qbatch(c, cu_q, nQ, &qb);
  if (rc) return rc;
  if (top_k % c->cfg.block_frames)
    REKV_FAIL(c, REKV_ERR_ARG, "top_k=%d must be a multiple of block_frames=%d", top_k, c->cfg.block_frames);
  DeviceGuard guard(c->device);
  const CtxGeom geom = rekv_geom(n_visible, c->cfg.window_frames, c->cfg.block_frames, top_k);
  const bool timed = (c->cfg.flags & REKV_FLAG_TIMING) != 0;
  if (timed) REKV_CUDA(c, cudaEventRecord(c->ev_r0, (cudaStream_t)stream));
  REKV_CUDA(c, rekv_launch_retrieve(c, q, qb, top_k, geom, n_visible, 0, c->sv.L, idx_out, scores_out ? scores_out : c->scores,
                                    (cudaStream_t)stream));
  if (timed) REKV_CUDA(c, cudaEventRecord(c->ev_r1, (cudaStream_t)stream));
  c->retrieve_timed = timed;
  return geom.k_eff;
}

int rekv_gather(rekv_ctx* c, const int32_t* idx, int nQ, int top_k, int n_visible, void* k_ctx, void* v_ctx,
                void* stream) {
  if (!c) return REKV_ERR_ARG;
  if (nQ < 1 || nQ > c->cfg.max_questions) REKV_FAIL(c, REKV_ERR_ARG, "nQ=%d outside [1, %d]", nQ, c->cfg.max_questions);
  if (top_k < 0 || top_k > c->cfg.max_topk) REKV_FAIL(c, REKV_ERR_ARG, "top_k=%d outside [0, %d]", top_k, c->cfg.max_topk);
  if (n_visible < 0 || n_visible > c->frames)
    REKV_FAIL(c, REKV_ERR_ARG, "n_visible=%d outside [0, %d]", n_visible, c->frames);
  if (n_visible == 0) REKV_FAIL(c, REKV_ERR_EMPTY, "no visible frame");
  if ((k_ctx == nullptr) != (v_ctx == nullptr)) REKV_FAIL(c, REKV_ERR_ARG, "k_ctx and v_ctx must both be given or both be null");
  if (top_k % c->cfg.block_frames)
    REKV_FAIL(c, REKV_ERR_ARG, "top_k=%d must be a multiple of block_frames=%d", top_k, c->cfg.block_frames);
  const CtxGeom geom = rekv_geom(n_visible, c->cfg.window_frames, c->cfg.block_frames, top_k);
  const int k_eff = geom.k_eff, ncf = geom.ncf;
  if (k_eff > 0 && !idx) REKV_FAIL(c, REKV_ERR_ARG, "null idx");
  DeviceGuard guard(c->device);
  cudaStream_t st = (cudaStream_t)stream;
  const StoreView& s = c->sv;
  if (s.tail == 0) {
    REKV_CUDA(c, rekv_launch_page_table(c, idx, nQ, top_k, geom, n_visible, 0, s.L, c->frames, st));
    c->gather_layerwise = false;
    c->pull_timed = false;
    *c->h_link_bytes = 0;
  } else {
    // host tier: the pulls run layer by layer on the side stream (behind every write-through that is
    // still in flight there); attention of layer l only waits for layer l's event
    REKV_CUDA(c, cudaMemsetAsync(c->link_bytes, 0, sizeof(unsigned long long), st));
    REKV_CUDA(c, cudaEventRecord(c->ev_main, st));
    REKV_CUDA(c, cudaStreamWaitEvent(c->side, c->ev_main, 0));
    const bool timed = (c->cfg.flags & REKV_FLAG_TIMING) != 0;
    if (timed) REKV_CUDA(c, cudaEventRecord(c->ev_p0, c->side));
    for (int l = 0; l < s.L; ++l) {
      REKV_CUDA(c, rekv_launch_page_table(c, idx, nQ, top_k, geom, n_visible, l, l + 1, c->frames, c->side));
      REKV_CUDA(c, cudaEventRecord(c->layer_events[l], c->side));
    }
    if (timed) REKV_CUDA(c, cudaEventRecord(c->ev_p1, c->side));
    c->pull_timed = timed;
    // the bytes that crossed the link, mirrored to pinned host memory behind the pulls (rekv_stats reads the mirror)
    REKV_CUDA(c, cudaMemcpyAsync(c->h_link_bytes, c->link_bytes, sizeof(unsigned long long), cudaMemcpyDeviceToHost, c->side));
    c->ring_reader_ev = c->layer_events[s.L - 1];
    c->gather_layerwise = true;
  }
  c->gathered = true;
  c->layer_ctx_valid.assign(s.L, 1);
  c->g_nQ = nQ;
  c->g_ncf = ncf;
  c->g_keff = k_eff;
  c->g_nvis = n_visible;
  c->g_topk = top_k;
  if (k_ctx) {
    if (c->gather_layerwise) REKV_CUDA(c, cudaStreamWaitEvent(st, c->layer_events[s.L - 1], 0));
    REKV_CUDA(c, rekv_launch_materialize(c, nQ, ncf, k_ctx, v_ctx, st));
  }
  return ncf;
}

int rekv_attend(rekv_ctx* c, const void* q, const int32_t* cu_q, int nQ, void* out, void* stream) {
  if (!c) return REKV_ERR_ARG;
  if (!q || !out) REKV_FAIL(c, REKV_ERR_ARG, "null q or out");
  if (!c->gathered) REKV_FAIL(c, REKV_ERR_STATE, "rekv_attend needs a preceding rekv_gather");
  for (int l = 0; l < c->sv.L; ++l)
    if (!c->layer_ctx_valid[l])
      REKV_FAIL(c, REKV_ERR_STATE, "layer %d has no context with the geometry of the latest gather", l);
  if (nQ != c->g_nQ) REKV_FAIL(c, REKV_ERR_STATE, "nQ=%d differs from the gathered batch (%d)", nQ, c->g_nQ);
  QBatch qb;
  int rc = build_qbatch(c, cu_q, nQ, &qb);
  if (rc) return rc;
  DeviceGuard guard(c->device);
  cudaStream_t st = (cudaStream_t)stream;
  const StoreView& s = c->sv;
  if (c->g_ncf == 0) {  // no context at all (W == 0 and nothing retrieved): the output is defined as zero
    REKV_CUDA(c, cudaMemsetAsync(out, 0, (size_t)s.L * qb.sumNq * s.Hq * REKV_HEAD_DIM * 2, st));
    return REKV_OK;
  }
  auto launch = rekv_launch_attend_tc5;
  if (!c->gather_layerwise) {
    REKV_CUDA(c, launch(c, q, qb, c->g_ncf, 0, s.L, out, st, (c->cfg.flags & REKV_FLAG_TIMING) != 0, nullptr));
  } else {
    for (int l = 0; l < s.L; ++l) {
      REKV_CUDA(c, cudaStreamWaitEvent(st, c->layer_events[l], 0));
      REKV_CUDA(c, launch(c, q, qb, c->g_ncf, l, l + 1, out, st, false, nullptr));
    }
    // later appends (ring slots) and gathers (staging) on the side stream must not overtake this read
    REKV_CUDA(c, cudaEventRecord(c->ev_side, st));
    REKV_CUDA(c, cudaStreamWaitEvent(c->side, c->ev_side, 0));
  }
  return REKV_OK;
}

int rekv_question(rekv_ctx* c, const void* q, const int32_t* cu_q, int nQ, int top_k, int n_visible, int32_t* idx_out,
                  void* out, void* stream) {
  if (!c) return REKV_ERR_ARG;
  if (!q || !out) REKV_FAIL(c, REKV_ERR_ARG, "null q or out");
  int32_t* idx = idx_out ? idx_out : c->idx_own;
  const StoreView& s = c->sv;
  if (s.tail > 0 || top_k == 0) {  // offloaded cache (or nothing to select): the three calls as they are
    int rc = rekv_retrieve(c, q, cu_q, nQ, top_k, n_visible, idx, nullptr, stream);
    if (rc < 0) return rc;
    const int ncf = rekv_gather(c, idx, nQ, top_k, n_visible, nullptr, nullptr, stream);
    if (ncf < 0) return ncf;
    rc = rekv_attend(c, q, cu_q, nQ, out, stream);
    return rc < 0 ? rc : ncf;
  }
  if (top_k < 0 || top_k > c->cfg.max_topk) REKV_FAIL(c, REKV_ERR_ARG, "top_k=%d outside [0, %d]", top_k, c->cfg.max_topk);
  if (n_visible < 0 || n_visible > c->frames)
    REKV_FAIL(c, REKV_ERR_ARG, "n_visible=%d outside [0, %d]", n_visible, c->frames);
  if (n_visible == 0) REKV_FAIL(c, REKV_ERR_EMPTY, "no visible frame");
  if (top_k % c->cfg.block_frames)
    REKV_FAIL(c, REKV_ERR_ARG, "top_k=%d must be a multiple of block_frames=%d", top_k, c->cfg.block_frames);
  QBatch qb;
  int rc = build_qbatch(c, cu_q, nQ, &qb);
  if (rc) return rc;
  DeviceGuard guard(c->device);
  cudaStream_t st = (cudaStream_t)stream;
  const CtxGeom geom = rekv_geom(n_visible, c->cfg.window_frames, c->cfg.block_frames, top_k);
  const bool timed = (c->cfg.flags & REKV_FLAG_TIMING) != 0;
  if (timed) REKV_CUDA(c, cudaEventRecord(c->ev_r0, st));
  REKV_CUDA(c, rekv_launch_retrieve(c, q, qb, top_k, geom, n_visible, 0, s.L, idx, c->scores, st, true));
  if (timed) REKV_CUDA(c, cudaEventRecord(c->ev_r1, st));
  c->retrieve_timed = timed;
  c->pull_timed = false;
  c->gathered = true;
  c->layer_ctx_valid.assign(s.L, 1);
  c->gather_layerwise = false;
  c->g_nQ = nQ;
  c->g_ncf = geom.ncf;
  c->g_keff = geom.k_eff;
  c->g_nvis = n_visible;
  c->g_topk = top_k;
  rc = rekv_attend(c, q, cu_q, nQ, out, stream);
  return rc < 0 ? rc : geom.ncf;
}

namespace {
int attend_full_range(rekv_ctx* c, int layer0, int layer1, const void* q, const void* k_self, const void* v_self,
                      const QBatch& qb, const QBatch& sb, void* out, cudaStream_t st, bool self_done);
int build_self_batch(rekv_ctx* c, const QBatch& qb, const int32_t* cu_self, int nQ, QBatch* sb);
}  // namespace

// steps 2-5 of one layer; with k_self != null step 5 is Eq. 3 in full (the questions' own K/V after the context)
static int question_layer_impl(rekv_ctx* c, int layer, const void* q, const void* k_self, const void* v_self,
                               const int32_t* cu_q, const int32_t* cu_self, int nQ, int top_k, int n_visible,
                               int32_t* idx_out, void* out, void* stream) {
  if (!c) return REKV_ERR_ARG;
  if (!q || !out) REKV_FAIL(c, REKV_ERR_ARG, "null q or out");
  if (layer < 0 || layer >= c->sv.L) REKV_FAIL(c, REKV_ERR_ARG, "layer=%d outside [0, %d)", layer, c->sv.L);
  if (top_k < 0 || top_k > c->cfg.max_topk) REKV_FAIL(c, REKV_ERR_ARG, "top_k=%d outside [0, %d]", top_k, c->cfg.max_topk);
  if (n_visible < 0 || n_visible > c->frames)
    REKV_FAIL(c, REKV_ERR_ARG, "n_visible=%d outside [0, %d]", n_visible, c->frames);
  if (n_visible == 0) REKV_FAIL(c, REKV_ERR_EMPTY, "no visible frame");
  if (top_k % c->cfg.block_frames)
    REKV_FAIL(c, REKV_ERR_ARG, "top_k=%d must be a multiple of block_frames=%d", top_k, c->cfg.block_frames);
  QBatch qb, sb;
  int rc = build_qbatch(c, cu_q, nQ, &qb);
  if (rc) return rc;
  if (k_self) {
    rc = build_self_batch(c, qb, cu_self, nQ, &sb);
    if (rc) return rc;
  }
  DeviceGuard guard(c->device);
  cudaStream_t st = (cudaStream_t)stream;
  const StoreView& s = c->sv;
  const CtxGeom geom = rekv_geom(n_visible, c->cfg.window_frames, c->cfg.block_frames, top_k);
  const long long row_bytes = (long long)s.Hq * REKV_HEAD_DIM * 2;
  // the selection goes to the caller's buffer if there is one, else to the context's own
  int32_t* idx = idx_out ? layer_view(idx_out, layer, (long long)nQ * top_k * 4) : c->idx_own;
  // Eq. 3 in full on an HBM-resident cache: the part over X needs nothing of the retrieval, so it starts on the internal
  // stream now and runs beside the layer's retrieval kernels (it joins before the attention kernel)
  const bool self_early = k_self != nullptr && s.tail == 0 && geom.ncf > 0;
  if (self_early) {
    const long long kv_layer = (long long)sb.sumNq * s.Hkv * REKV_HEAD_DIM * 2;
    REKV_CUDA(c, rekv_launch_attend_full_self(c, layer_view(q, layer, qb.sumNq * row_bytes),
                                              layer_view(k_self, layer, kv_layer), layer_view(v_self, layer, kv_layer),
                                              qb, sb, geom.ncf, st, layer, layer + 1, true));
  }
  // cache all in HBM: the selection kernel writes the layer's context table itself (top_k > 0 launches it)
  const bool fused_table = s.tail == 0 && top_k > 0;
  REKV_CUDA(c, rekv_launch_retrieve(c, layer_view(q, layer, qb.sumNq * row_bytes), qb, top_k, geom, n_visible, layer,
                                    layer + 1, idx, c->scores, st, fused_table));
  if (fused_table) {
  } else if (s.tail == 0) {
    REKV_CUDA(c, rekv_launch_page_table(c, idx, nQ, top_k, geom, n_visible, layer, layer + 1, c->frames, st));
  } else {
    REKV_CUDA(c, cudaEventRecord(c->ev_main, st));
    REKV_CUDA(c, cudaStreamWaitEvent(c->side, c->ev_main, 0));
    REKV_CUDA(c, rekv_launch_page_table(c, idx, nQ, top_k, geom, n_visible, layer, layer + 1, c->frames, c->side));
    REKV_CUDA(c, cudaEventRecord(c->layer_events[layer], c->side));
    c->ring_reader_ev = c->layer_events[layer];
    REKV_CUDA(c, cudaStreamWaitEvent(st, c->layer_events[layer], 0));
  }
  // the table's row pitch follows (nQ, context frames): a layer call with another geometry re-lays it out, and the
  // contexts the other layers built under the old one are gone
  if (!c->gathered || c->g_nQ != nQ || c->g_ncf != geom.ncf) c->layer_ctx_valid.assign(s.L, 0);
  c->layer_ctx_valid[layer] = 1;
  c->gathered = true;
  c->gather_layerwise = s.tail > 0;
  c->g_nQ = nQ;
  c->g_ncf = geom.ncf;
  c->g_keff = geom.k_eff;
  c->g_nvis = n_visible;
  c->g_topk = top_k;
  if (k_self) {
    const long long kv_layer = (long long)sb.sumNq * s.Hkv * REKV_HEAD_DIM * 2;
    rc = attend_full_range(c, layer, layer + 1, layer_view(q, layer, qb.sumNq * row_bytes),
                           layer_view(k_self, layer, kv_layer), layer_view(v_self, layer, kv_layer), qb, sb,
                           layer_view(out, layer, qb.sumNq * row_bytes), st, self_early);
    return rc ? rc : geom.ncf;
  }
  c->q_early_ok = fused_table;  // the selection kernel, which only reads Q, is directly before the attention
  rc = attend_one_layer(c, layer, q, qb, out, st);
  c->q_early_ok = false;
  return rc ? rc : geom.ncf;
}

int rekv_question_layer(rekv_ctx* c, int layer, const void* q, const int32_t* cu_q, int nQ, int top_k, int n_visible,
                        int32_t* idx_out, void* out, void* stream) {
  return question_layer_impl(c, layer, q, nullptr, nullptr, cu_q, nullptr, nQ, top_k, n_visible, idx_out, out, stream);
}

int rekv_question_layer_full(rekv_ctx* c, int layer, const void* q, const void* k_self, const void* v_self,
                             const int32_t* cu_q, const int32_t* cu_self, int nQ, int top_k, int n_visible,
                             int32_t* idx_out, void* out, void* stream) {
  if (!c) return REKV_ERR_ARG;
  if (!k_self || !v_self) REKV_FAIL(c, REKV_ERR_ARG, "null k_self or v_self");
  if (c->cfg.max_self_tokens <= 0) REKV_FAIL(c, REKV_ERR_STATE, "the context was created with max_self_tokens == 0");
  return question_layer_impl(c, layer, q, k_self, v_self, cu_q, cu_self, nQ, top_k, n_visible, idx_out, out, stream);
}

int rekv_attend_layer(rekv_ctx* c, int layer, const void* q, const int32_t* cu_q, int nQ, void* out, void* stream) {
  if (!c) return REKV_ERR_ARG;
  if (!q || !out) REKV_FAIL(c, REKV_ERR_ARG, "null q or out");
  if (layer < 0 || layer >= c->sv.L) REKV_FAIL(c, REKV_ERR_ARG, "layer=%d outside [0, %d)", layer, c->sv.L);
  if (!c->gathered || !c->layer_ctx_valid[layer])
    REKV_FAIL(c, REKV_ERR_STATE, "rekv_attend_layer needs a preceding gather of the layer (with the geometry of the "
                                 "latest gather: a layer call with other question or frame counts re-lays the table out)");
  if (nQ != c->g_nQ) REKV_FAIL(c, REKV_ERR_STATE, "nQ=%d differs from the gathered batch (%d)", nQ, c->g_nQ);
  QBatch qb;
  int rc = build_qbatch(c, cu_q, nQ, &qb);
  if (rc) return rc;
  DeviceGuard guard(c->device);
  cudaStream_t st = (cudaStream_t)stream;
  if (c->gather_layerwise) REKV_CUDA(c, cudaStreamWaitEvent(st, c->layer_events[layer], 0));
  return attend_one_layer(c, layer, q, qb, out, st);
}

int rekv_set_frame_embedding(rekv_ctx* c, int frame, const float* emb, void* stream) {
  if (!c) return REKV_ERR_ARG;
  if (c->cfg.ext_embed_dim <= 0) REKV_FAIL(c, REKV_ERR_STATE, "the context was created with ext_embed_dim == 0");
  if (!emb) REKV_FAIL(c, REKV_ERR_ARG, "null embedding");
  if (frame < 0 || frame >= c->frames) REKV_FAIL(c, REKV_ERR_ARG, "frame=%d outside [0, %d)", frame, c->frames);
  DeviceGuard guard(c->device);
  const size_t bytes = (size_t)c->cfg.ext_embed_dim * sizeof(float);
  REKV_CUDA(c, cudaMemcpyAsync(c->ext_emb + (size_t)frame * c->cfg.ext_embed_dim, emb, bytes, cudaMemcpyDeviceToDevice,
                               (cudaStream_t)stream));
  if (frame == c->ext_frames) c->ext_frames = frame + 1;  // embeddings are expected in frame order
  return REKV_OK;
}

int rekv_retrieve_external(rekv_ctx* c, const float* q_emb, int nQ, int top_k, int n_visible, float tau,
                           int32_t* idx_out, float* scores_out, void* stream) {
  if (!c) return REKV_ERR_ARG;
  if (c->cfg.ext_embed_dim <= 0) REKV_FAIL(c, REKV_ERR_STATE, "the context was created with ext_embed_dim == 0");
  if (!q_emb) REKV_FAIL(c, REKV_ERR_ARG, "null q_emb");
  if (nQ < 1 || nQ > c->cfg.max_questions) REKV_FAIL(c, REKV_ERR_ARG, "nQ=%d outside [1, %d]", nQ, c->cfg.max_questions);
  if (top_k < 0 || top_k > c->cfg.max_topk) REKV_FAIL(c, REKV_ERR_ARG, "top_k=%d outside [0, %d]", top_k, c->cfg.max_topk);
  if (top_k > 0 && !idx_out) REKV_FAIL(c, REKV_ERR_ARG, "null idx_out");
  if (!(tau > 0.f)) REKV_FAIL(c, REKV_ERR_ARG, "tau must be positive");
  if (n_visible < 0 || n_visible > c->frames)
    REKV_FAIL(c, REKV_ERR_ARG, "n_visible=%d outside [0, %d]", n_visible, c->frames);
  if (n_visible == 0) REKV_FAIL(c, REKV_ERR_EMPTY, "no visible frame");
  if (n_visible > c->ext_frames)
    REKV_FAIL(c, REKV_ERR_STATE, "embeddings are set for %d frames, %d are visible", c->ext_frames, n_visible);
  if (top_k % c->cfg.block_frames)
    REKV_FAIL(c, REKV_ERR_ARG, "top_k=%d must be a multiple of block_frames=%d", top_k, c->cfg.block_frames);
  DeviceGuard guard(c->device);
  const CtxGeom geom = rekv_geom(n_visible, c->cfg.window_frames, c->cfg.block_frames, top_k);
  REKV_CUDA(c, rekv_launch_retrieve_external(c, q_emb, nQ, top_k, geom, n_visible, tau, idx_out,
                                             scores_out ? scores_out : c->scores, (cudaStream_t)stream));
  return geom.k_eff;
}

namespace {

// the batch's own K/V lengths, checked against the query lengths and the context's capacity
int build_self_batch(rekv_ctx* c, const QBatch& qb, const int32_t* cu_self, int nQ, QBatch* sb) {
  if (!cu_self || cu_self[0] != 0) REKV_FAIL(c, REKV_ERR_ARG, "cu_self must start at 0");
  sb->nQ = nQ;
  for (int i = 0; i <= nQ; ++i) sb->cu[i] = cu_self[i];
  sb->sumNq = cu_self[nQ];
  for (int i = 0; i < nQ; ++i)
    if (sb->cu[i + 1] - sb->cu[i] < qb.cu[i + 1] - qb.cu[i])
      REKV_FAIL(c, REKV_ERR_ARG, "question %d: %d tokens of its own K/V for %d query rows", i, sb->cu[i + 1] - sb->cu[i],
                qb.cu[i + 1] - qb.cu[i]);
  if (sb->sumNq > c->cfg.max_self_tokens)
    REKV_FAIL(c, REKV_ERR_ARG, "%d tokens of own K/V exceed max_self_tokens=%d", sb->sumNq, c->cfg.max_self_tokens);
  return REKV_OK;
}

// Eq. 3 in full for layers [layer0, layer1).  q, k_self, v_self and out are indexed with the absolute layer: a caller
// that holds one layer's rows passes pointers moved back by layer0 layers (layer_view).
int attend_full_range(rekv_ctx* c, int layer0, int layer1, const void* q, const void* k_self, const void* v_self,
                      const QBatch& qb, const QBatch& sb, void* out, cudaStream_t st, bool self_done) {
  // an offloaded context: the range's pages must have arrived before the keys are rotated
  if (c->gather_layerwise) REKV_CUDA(c, cudaStreamWaitEvent(st, c->layer_events[layer1 - 1], 0));
  if (!self_done)
    REKV_CUDA(c, rekv_launch_attend_full_self(c, q, k_self, v_self, qb, sb, c->g_ncf, st, layer0, layer1, false));
  REKV_CUDA(c, rekv_launch_attend_full_ctx(c, qb, c->g_ncf, st, layer0, layer1));
  const bool rope = c->cfg.rope_theta > 0.f && !(c->cfg.flags & REKV_FLAG_ROPE_STATIC);  // rotated copies of the context's keys
  const bool rope_q = c->cfg.rope_theta > 0.f;
  if (c->g_ncf == 0) {
    REKV_CUDA(c, rekv_launch_self_finalize(c, qb, out, st, layer0, layer1));
  } else {
    AttendFullArgs fa;
    fa.tbl_k = rope ? c->tbl_k : nullptr;
    fa.self_o = c->self_o;
    fa.self_ml = c->self_ml;
    REKV_CUDA(c, rekv_launch_attend_tc5(c, rope_q ? (const void*)c->q_rot : q, qb, c->g_ncf, layer0, layer1, out, st,
                                        (c->cfg.flags & REKV_FLAG_TIMING) != 0 && layer1 - layer0 == c->sv.L, &fa));
  }
  if (c->gather_layerwise || (c->sv.tail > 0 && layer1 - layer0 < c->sv.L)) {
    // later appends (ring slots) and gathers (staging) on the side stream must not overtake this read
    REKV_CUDA(c, cudaEventRecord(c->ev_side, st));
    REKV_CUDA(c, cudaStreamWaitEvent(c->side, c->ev_side, 0));
  }
  return REKV_OK;
}

}  // namespace

int rekv_attend_full(rekv_ctx* c, const void* q, const void* k_self, const void* v_self, const int32_t* cu_q,
                     const int32_t* cu_self, int nQ, void* out, void* stream) {
  if (!c) return REKV_ERR_ARG;
  if (!q || !k_self || !v_self || !out) REKV_FAIL(c, REKV_ERR_ARG, "null q, k_self, v_self or out");
  if (c->cfg.max_self_tokens <= 0) REKV_FAIL(c, REKV_ERR_STATE, "the context was created with max_self_tokens == 0");
  if (!c->gathered) REKV_FAIL(c, REKV_ERR_STATE, "rekv_attend_full needs a preceding rekv_gather");
  for (int l = 0; l < c->sv.L; ++l)
    if (!c->layer_ctx_valid[l])
      REKV_FAIL(c, REKV_ERR_STATE, "layer %d has no context with the geometry of the latest gather", l);
  if (nQ != c->g_nQ) REKV_FAIL(c, REKV_ERR_STATE, "nQ=%d differs from the gathered batch (%d)", nQ, c->g_nQ);
  QBatch qb, sb;
  int rc = build_qbatch(c, cu_q, nQ, &qb);
  if (rc) return rc;
  rc = build_self_batch(c, qb, cu_self, nQ, &sb);
  if (rc) return rc;
  DeviceGuard guard(c->device);
  return attend_full_range(c, 0, c->sv.L, q, k_self, v_self, qb, sb, out, (cudaStream_t)stream, false);
}

int rekv_attend_full_layer(rekv_ctx* c, int layer, const void* q, const void* k_self, const void* v_self,
                           const int32_t* cu_q, const int32_t* cu_self, int nQ, void* out, void* stream) {
  if (!c) return REKV_ERR_ARG;
  if (!q || !k_self || !v_self || !out) REKV_FAIL(c, REKV_ERR_ARG, "null q, k_self, v_self or out");
  if (layer < 0 || layer >= c->sv.L) REKV_FAIL(c, REKV_ERR_ARG, "layer=%d outside [0, %d)", layer, c->sv.L);
  if (c->cfg.max_self_tokens <= 0) REKV_FAIL(c, REKV_ERR_STATE, "the context was created with max_self_tokens == 0");
  if (!c->gathered || !c->layer_ctx_valid[layer])
    REKV_FAIL(c, REKV_ERR_STATE, "rekv_attend_full_layer needs a preceding gather of the layer (with the geometry of "
                                 "the latest gather)");
  if (nQ != c->g_nQ) REKV_FAIL(c, REKV_ERR_STATE, "nQ=%d differs from the gathered batch (%d)", nQ, c->g_nQ);
  QBatch qb, sb;
  int rc = build_qbatch(c, cu_q, nQ, &qb);
  if (rc) return rc;
  rc = build_self_batch(c, qb, cu_self, nQ, &sb);
  if (rc) return rc;
  DeviceGuard guard(c->device);
  const StoreView& s = c->sv;
  const long long q_layer = (long long)qb.sumNq * s.Hq * REKV_HEAD_DIM * 2;
  const long long kv_layer = (long long)sb.sumNq * s.Hkv * REKV_HEAD_DIM * 2;
  return attend_full_range(c, layer, layer + 1, layer_view(q, layer, q_layer), layer_view(k_self, layer, kv_layer),
                           layer_view(v_self, layer, kv_layer), qb, sb, layer_view(out, layer, q_layer),
                           (cudaStream_t)stream, false);
}

int rekv_geometry(rekv_ctx* c, int n_visible, int top_k, int32_t* n_scored, int32_t* k_eff, int32_t* w_eff) {
  if (!c) return REKV_ERR_ARG;
  if (n_visible < 0 || top_k < 0) REKV_FAIL(c, REKV_ERR_ARG, "n_visible and top_k must be >= 0");
  if (top_k % c->cfg.block_frames)
    REKV_FAIL(c, REKV_ERR_ARG, "top_k=%d must be a multiple of block_frames=%d", top_k, c->cfg.block_frames);
  const CtxGeom g = rekv_geom(n_visible, c->cfg.window_frames, c->cfg.block_frames, top_k);
  if (n_scored) *n_scored = c->cfg.block_frames == 1 ? n_visible : g.n_items;
  if (k_eff) *k_eff = g.k_eff;
  if (w_eff) *w_eff = g.w_eff;
  return REKV_OK;
}

int rekv_stats(rekv_ctx* c, rekv_stats_t* out) {
  if (!c || !out) return REKV_ERR_ARG;
  DeviceGuard guard(c->device);
  const StoreView& s = c->sv;
  memset(out, 0, sizeof(*out));
  out->frames = c->frames;
  out->page_bytes = s.page_bytes;
  const long long frame_bytes = s.page_bytes * s.L;
  const long long resident = s.tail > 0 ? (c->frames < s.tail ? c->frames : s.tail) : c->frames;
  out->kv_bytes_hbm = resident * frame_bytes;
  out->kv_bytes_host = s.tail > 0 ? (long long)c->frames * s.host_page_bytes * s.L : 0;
  out->kv_bytes_logical = 2ll * s.L * c->frames * s.Nf * s.Hkv * REKV_HEAD_DIM * 2;
  out->rep_bytes = (long long)s.L * c->frames * s.Dp * (long long)sizeof(float);
  // nothing here waits for the device: counters and timings are those of the work that has completed
  out->last_link_bytes = (int64_t)*c->h_link_bytes;
  auto elapsed_us = [](cudaEvent_t a, cudaEvent_t b) -> double {
    float ms = 0.f;
    if (cudaEventQuery(b) != cudaSuccess || cudaEventElapsedTime(&ms, a, b) != cudaSuccess) {
      cudaGetLastError();
      return 0.0;
    }
    return 1e3 * ms;
  };
  if (c->timing_valid) out->last_attend_kernel_us = elapsed_us(c->ev_t0, c->ev_t1);
  if (c->timing_valid && c->merge_timed) out->last_merge_us = elapsed_us(c->ev_t1, c->ev_t2);
  if (c->retrieve_timed) out->last_retrieve_us = elapsed_us(c->ev_r0, c->ev_r1);
  if (c->pull_timed) out->last_pull_us = elapsed_us(c->ev_p0, c->ev_p1);
  out->last_k_eff = c->gathered ? c->g_keff : 0;
  out->last_ctx_frames = c->gathered ? c->g_ncf : 0;
  return REKV_OK;
}

int rekv_set_timing(rekv_ctx* c, int enable) {
  if (!c) return REKV_ERR_ARG;
  if (enable) {
    c->cfg.flags |= REKV_FLAG_TIMING;
  } else {
    c->cfg.flags &= ~(uint32_t)REKV_FLAG_TIMING;
    c->timing_valid = c->merge_timed = c->retrieve_timed = c->pull_timed = false;
  }
  return REKV_OK;
}

int rekv_test_set_wait_limit(rekv_ctx* c, unsigned iterations, int skip_copy_entry) {
  if (!c) return REKV_ERR_ARG;
  c->test_wait_limit = iterations;
  c->test_skip_copy_entry = skip_copy_entry;
  return REKV_OK;
}

int rekv_check_status(rekv_ctx* c, void* stream) {
  if (!c) return REKV_ERR_ARG;
  DeviceGuard guard(c->device);
  REKV_CUDA(c, cudaStreamSynchronize((cudaStream_t)stream));
  if (c->side) REKV_CUDA(c, cudaStreamSynchronize(c->side));
  int st = 0;
  REKV_CUDA(c, cudaMemcpy(&st, c->status, sizeof(int), cudaMemcpyDeviceToHost));
  if (st != 0) {
    REKV_CUDA(c, cudaMemset(c->status, 0, sizeof(int)));
    REKV_CUDA(c, cudaMemset(c->unit_cnt, 0, c->part_units * sizeof(int)));  // a kernel that gave up may have left counts
    if (st == REKV_ERR_TIMEOUT) REKV_FAIL(c, REKV_ERR_TIMEOUT, "a device-side wait expired");
    REKV_FAIL(c, st, "a kernel reported error %d (an index outside the visible frames?)", st);
  }
  return REKV_OK;
}

const char* rekv_last_error(rekv_ctx* c) { return c ? c->err.c_str() : g_create_error.c_str(); }

int rekv_get_reps(rekv_ctx* c, int layer, int n_frames, float* dev_out, void* stream) {
  if (!c || !dev_out) return REKV_ERR_ARG;
  if (layer < 0 || layer >= c->sv.L || n_frames < 0 || n_frames > c->frames)
    REKV_FAIL(c, REKV_ERR_ARG, "layer %d / n_frames %d out of range", layer, n_frames);
  DeviceGuard guard(c->device);
  const StoreView& s = c->sv;
  REKV_CUDA(c, cudaMemcpyAsync(dev_out, s.reps + (long long)layer * s.max_frames * s.Dp,
                               (size_t)n_frames * s.Dp * sizeof(float), cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return REKV_OK;
}

int rekv_get_page(rekv_ctx* c, int frame, int layer, void* k_out, void* v_out, void* stream) {
  if (!c || !k_out || !v_out) return REKV_ERR_ARG;
  if (layer < 0 || layer >= c->sv.L || frame < 0 || frame >= c->frames)
    REKV_FAIL(c, REKV_ERR_ARG, "frame %d / layer %d out of range", frame, layer);
  DeviceGuard guard(c->device);
  const StoreView& s = c->sv;
  cudaStream_t st = (cudaStream_t)stream;
  const char* page;
  if (s.tail == 0 || frame >= c->frames - s.tail) {
    page = s.hbm + rekv_hbm_page_offset(s, frame, layer);
  } else {
    // host-only page: read it zero-copy once its write-through has landed
    REKV_CUDA(c, cudaStreamSynchronize(c->side));
    page = c->host_arenas[frame / s.frames_per_arena] +
           ((long long)(frame % s.frames_per_arena) * s.L + layer) * s.host_page_bytes;
    if (s.host_fp8) {  // back to bf16 in the first staging page (nothing else is in flight: test helper)
      REKV_CUDA(c, cudaStreamSynchronize(st));
      REKV_CUDA(c, rekv_launch_dequant_page(c, page, s.staging, st));
      page = s.staging;
      c->gathered = false;  // the staging page belonged to the last gather's context
    }
  }
  REKV_CUDA(c, rekv_launch_unswizzle_page(c, page, k_out, v_out, st));
  return REKV_OK;
}

int64_t rekv_launch_count(rekv_ctx* c) { return c ? c->launches : 0; }

}  // extern "C"
