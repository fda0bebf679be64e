/*
 * librekv -- in-context video KV-cache retrieval hot path for one B200 (sm_100a).
 *
 * A video stream's per-layer K/V is appended frame by frame; a question is answered from
 * the query-relevant frames only.  The library covers the five steps of the paper's
 * internal retrieval (Section "ReKV"):
 *
 *   1. frame representative = mean of the frame's N_f key vectors, heads concatenated
 *      ("Internal Video KV-Cache Retrieval": v = 1/N_f * sum_j k_j)       rekv_append_frame
 *   2. question vector = mean of the question's N_q query vectors; cosine similarity with
 *      tau = 1 (Eq. 2), independently in every layer                        rekv_retrieve
 *   3. the r most similar frames are kept (Eq. 2 paragraph)                rekv_retrieve
 *   4. the retrieved K/V, R, are brought onto the GPU as the context        rekv_gather
 *   5. O = Attn(Q, R_k, R_v)  (Eq. 3), GQA, over retrieved frames plus a recent window
 *                                                                           rekv_attend
 *
 * Conventions
 *   - C ABI, plain pointers.  "device" pointers are CUDA device addresses on the context's
 *     device; "host" pointers are ordinary host memory.  bf16 tensors are passed as void*.
 *   - Every call returns 0 (or a non-negative value where stated) on success and a negative
 *     REKV_ERR_* code on failure; it never aborts.  rekv_last_error() gives the message.
 *   - The caller owns every input and output buffer; the context owns the store, the
 *     representative table and all scratch memory.
 *   - Work is enqueued on the caller's CUDA stream (`stream`, a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and the call returns without synchronising.
 *     Internal side streams are fenced to the caller's stream with events.
 *   - A context is not thread-safe.  Append and question calls may be interleaved freely
 *     from one thread; a question sees exactly the frames [0, n_visible).
 *   - The library has no CPU fallback: without a CUDA device rekv_create fails.
 */
#ifndef REKV_H_
#define REKV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rekv_ctx rekv_ctx;

enum {
  REKV_OK = 0,
  REKV_ERR_ARG = -1,     /* bad argument (null pointer, size out of range, unsupported shape) */
  REKV_ERR_FULL = -2,    /* append past max_frames */
  REKV_ERR_EMPTY = -3,   /* question with n_visible == 0 */
  REKV_ERR_ALLOC = -4,   /* device or pinned-host allocation failed */
  REKV_ERR_CUDA = -5,    /* a CUDA call or launch failed */
  REKV_ERR_TIMEOUT = -6, /* a bounded device-side wait expired (read from the status word) */
  REKV_ERR_STATE = -7    /* call order violated (attend without a preceding gather, ...) */
};

/* rekv_config.flags */
enum {
  REKV_FLAG_TIMING = 1u << 2,                   /* bracket the attention kernel with CUDA events on the caller's
                                                  stream; rekv_stats then reports its duration */
  REKV_FLAG_ROPE_STATIC = 1u << 4,              /* rekv_attend_full with rope_theta > 0: the static position variant of
                                                  the "Positional Encoding" paragraph -- every context token gets the
                                                  same position (0) and token s of X position 1 + s -- instead of
                                                  consecutive positions.  The stored keys are then used as they are
                                                  (no rotated copies of the context), only the queries and X rotate */
  REKV_FLAG_HOST_FP8 = 1u << 3                  /* offloaded contexts only: the pinned-host tier holds each page row
                                                  (128 dims of one token of one KV head) as 128 FP8 E4M3 codes and
                                                  one float scale = amax / 448; pages pulled from it come back as
                                                  bf16(code * scale).  Halves the bytes that cross the host link and
                                                  the host memory; frames still in the HBM tail stay exact.  (The
                                                  paper names quantisation as future work; not part of its method.) */
};

typedef struct {
  int32_t n_layers;          /* L */
  int32_t n_q_heads;         /* H_q; must be a multiple of n_kv_heads */
  int32_t n_kv_heads;        /* H_kv */
  int32_t head_dim;          /* D; must be 128 */
  int32_t tokens_per_frame;  /* N_f, fixed per context (the paper's M); 1..1024.  The attention kernel streams the
                                context in 128-token chunks whatever N_f is; the load-bound decode kernel needs two
                                whole frames of a KV head in shared memory and hands frames of more than 224 tokens
                                to the tensor-core kernel */
  int32_t max_frames;        /* stream capacity; an append past it returns REKV_ERR_FULL */
  int32_t hbm_tail_frames;   /* 0: the whole cache lives in HBM.  n > 0: every page lives in pinned host
                                memory and only the most recent n frames are also kept in HBM */
  int32_t window_frames;     /* W: the last W visible frames are always part of a question's context and
                                are not retrieval candidates; W <= hbm_tail_frames when offloaded */
  int32_t block_frames;      /* frames per retrieval block (the paper's b), 1..64; max_topk and top_k must be
                                multiples of it */
  int32_t max_q_tokens;      /* upper bound on the sum of question lengths in one batch */
  int32_t max_topk;          /* upper bound on top_k */
  int32_t max_questions;     /* upper bound on questions per batch (<= 64) */
  int32_t device;            /* CUDA device ordinal */
  uint32_t flags;
  int32_t max_self_tokens;   /* rekv_attend_full: upper bound on the summed lengths of the questions' own
                                K/V (question plus generated tokens) in one batch; 0 = that call is not used
                                and its workspaces are not allocated */
  float rope_theta;          /* rekv_attend_full: base of the rotary position embedding (1e6 for the paper's
                                Qwen2-based models); 0 = no positional term */
  int32_t ext_embed_dim;     /* external retrieval: dimension of the frame / question embeddings of a CLIP-like
                                encoder (1152 for the paper's SigLIP-SO400M); a multiple of 4, <= 2048; 0 = the
                                embedding table is not allocated */
} rekv_config;

typedef struct {
  int64_t frames;            /* frames appended so far */
  int64_t kv_bytes_hbm;      /* bytes of K/V pages currently resident in HBM */
  int64_t kv_bytes_host;     /* bytes of K/V pages held in pinned host memory */
  int64_t kv_bytes_logical;  /* 2 * L * frames * N_f * H_kv * D * 2: the appendix's cache-size expression */
  int64_t rep_bytes;         /* bytes of the representative table in use */
  int64_t page_bytes;        /* bytes of one (layer, frame) page: K and V, all KV heads */
  int64_t last_link_bytes;   /* bytes the last rekv_gather pulled from pinned host memory */
  int32_t last_k_eff;        /* frames actually retrieved per (layer, question) by the last question */
  int32_t last_ctx_frames;   /* k_eff + window frames of the last gather */
  double last_attend_kernel_us; /* device time of the last attention kernel launch (REKV_FLAG_TIMING, HBM
                                   tier): it includes the joining of units cut between CTAs when the kernel does
                                   that itself (two or three parts per unit), not a merge kernel that followed
                                   (last_merge_us); 0 when not measured */
  double last_retrieve_us;      /* REKV_FLAG_TIMING: steps 2-3 of the last question (question vectors, scores,
                                   selection) on the caller's stream; 0 when not measured or not finished yet */
  double last_pull_us;          /* REKV_FLAG_TIMING, offloaded contexts: the last gather's pulls over the host
                                   link, all layers, on the internal stream; 0 when not measured or not finished */
  double last_merge_us;         /* REKV_FLAG_TIMING: the merge kernel that followed the last attention kernel
                                   (units cut into more than three parts); 0 when none ran or not measured */
} rekv_stats_t;

/* Creates a context on cfg->device: allocates the frame store (HBM tier, and the pinned-host tier
 * when hbm_tail_frames > 0), the fp32 representative table [L][max_frames][H_kv*D] and scratch
 * sized from the max_* fields.  *out receives the context.  Fails with REKV_ERR_ARG on an
 * unsupported shape and REKV_ERR_ALLOC / REKV_ERR_CUDA when memory or a device is missing. */
int rekv_create(const rekv_config* cfg, rekv_ctx** out);

/* Frees everything the context owns.  Synchronises the device first. */
int rekv_destroy(rekv_ctx* ctx);

/* Step 1 (+ paging).  k, v: device bf16 [L][N_f][H_kv][D], token-major as a decoder emits them.
 * Stores the frame's K/V as page (frame, layer) and the frame representative
 * rep[layer][frame][h*D+d] = 1/N_f * sum_t k[layer][t][h][d] (fp32).  On an offloaded context the
 * page is also written through to pinned host memory on an internal stream.
 * Returns the new frame's index (>= 0), REKV_ERR_FULL when the store is full. */
int rekv_append_frame(rekv_ctx* ctx, const void* k, const void* v, void* stream);

/* Steps 2-3 for a batch of nQ independent questions, in every layer.
 *   q         device bf16, packed [L][sum_Nq][H_q][D]; question i owns rows cu_q[i] .. cu_q[i+1]
 *   cu_q      HOST int32[nQ+1], prefix sums of the question lengths, cu_q[0] == 0
 *   top_k     frames to retrieve per (layer, question) (the paper's r), 0..max_topk
 *   n_visible frames the questions may see: frames [0, n_visible) (question time stamp)
 *   idx_out   device int32 [L][nQ][top_k]: the selected frames in ascending frame order, padded
 *             with -1 past k_eff = min(top_k, max(n_visible - W, 0))
 *   scores_out (nullable) device fp32 [L][nQ][n_visible]: cosine similarity of every visible frame
 * The question vector averages the question's tokens and the G = H_q/H_kv query heads of each KV
 * group; score = <q, rep> / (max(|q|,1e-8) * max(|rep|,1e-8)).  Candidates are frames
 * [0, n_visible - W); ties go to the lower frame index; NaN ranks below every number.
 * Block retrieval (block_frames = b > 1, Eq. 2 paragraph): the candidates are the complete blocks of b
 * consecutive frames inside [0, n_visible - W); a block's vector is the mean of its frames'
 * representatives; top_k / b blocks are kept and written to idx_out as their frames; scores_out is then
 * [L][nQ][n_blocks].  Every frame after the last complete block (the window plus the frames that do not
 * fill a block yet, W_eff = n_visible - b*n_blocks of them) is always part of the context.
 * Returns k_eff (frames). */
int rekv_retrieve(rekv_ctx* ctx, const void* q, const int32_t* cu_q, int nQ, int top_k, int n_visible,
                  int32_t* idx_out, float* scores_out, void* stream);

/* Step 4.  idx: device int32 [L][nQ][top_k] as written by rekv_retrieve, or the caller's own list
 * with the same shape: its first k_eff = min(top_k, max(n_visible - W, 0)) entries per (layer,
 * question) must be frames in [0, n_visible) (an entry outside that range is reported by
 * rekv_check_status as REKV_ERR_ARG).  Builds the context of every (layer, question):
 * the selected frames in list order, then frames max(n_visible - W, 0) .. n_visible-1.  Pages that
 * live only in pinned host memory are pulled over the host link into an HBM staging area (on an
 * internal stream, layer by layer); on an offloaded context the frames still in the HBM tail are
 * copied there too, so the context keeps its bytes when later appends recycle the tail's slots
 * (an append enqueued after the gather waits for those copies).  rekv_attend reads this context.
 *   k_ctx, v_ctx (nullable, both or neither): device bf16 [L][nQ][H_kv][(k_eff+W')*N_f][D] with
 *   W' = min(W, n_visible); when given, the context is also written out contiguously, token rows
 *   in context order -- a bit-exact copy of the stored K/V.
 * Returns the number of context frames per (layer, question). */
int rekv_gather(rekv_ctx* ctx, const int32_t* idx, int nQ, int top_k, int n_visible, void* k_ctx, void* v_ctx,
                void* stream);

/* Step 5 (Eq. 3).  q, cu_q, nQ as in rekv_retrieve and consistent with the preceding rekv_gather.
 * out: device bf16 [L][sum_Nq][H_q][D].  For every layer, question token n and query head h:
 * out = softmax(q . K_ctx^T / sqrt(D)) V_ctx over the gathered context of KV head floor(h/G);
 * no mask (every context token precedes the question); bf16 operands, fp32 accumulation and softmax.
 * Returns 0, or REKV_ERR_STATE without a preceding gather.
 * rekv_retrieve, rekv_gather (page-list mode) and rekv_attend allocate nothing and do not synchronise the host:
 * on a context whose cache is all in HBM the three calls may be captured into one CUDA graph. */
int rekv_attend(rekv_ctx* ctx, const void* q, const int32_t* cu_q, int nQ, void* out, void* stream);

/* Eq. 3 in full: O = Attn(W_Q X, [R_k, W_K X], [R_v, W_V X]).  The context of the preceding rekv_gather
 * is followed by the K/V of X itself -- the question's tokens and the tokens generated so far -- which a
 * query row sees causally.
 *   q         device bf16 [L][sum_Nq][H_q][D]: the rows of X being computed
 *   k_self, v_self   device bf16 [L][sum_Ns][H_kv][D]: K/V of all of X, token-major, questions packed back
 *             to back (not stored by the library)
 *   cu_q, cu_self    HOST int32 [nQ+1] prefix sums of N_q and N_s per question, 1 <= N_q <= N_s:
 *             query row n of a question is token N_s - N_q + n of its X and sees all of R and the tokens
 *             0 .. N_s - N_q + n of X.  N_s == N_q: the question itself; N_q == 1: one decode step
 *   out       device bf16 [L][sum_Nq][H_q][D]
 * With rope_theta > 0 the rotary embedding (pairs i, i + D/2; angle = position * theta^(-2i/D)) is applied
 * to q and to every key, the retrieved tokens taken as consecutive tokens ("Positional Encoding"
 * paragraph): context token j (context order: retrieved frames ascending, then the trailing frames) has
 * position j, token s of X has position n_ctx + s.  q, k_self and the stored keys are given UN-rotated;
 * rotated vectors are rounded to bf16.  The rotated copies of the context's keys are written to a
 * workspace first (one extra pass over the context's K).
 * Needs max_self_tokens > 0 at creation.  Returns 0 or an error code (REKV_ERR_STATE without a gather). */
int rekv_attend_full(rekv_ctx* ctx, const void* q, const void* k_self, const void* v_self, const int32_t* cu_q,
                     const int32_t* cu_self, int nQ, void* out, void* stream);

/* External retrieval (Eq. 2 with its temperature; the paper's baseline retriever).  The embeddings come from
 * a CLIP-like encoder outside this library.  rekv_set_frame_embedding stores the embedding of an appended
 * frame (device fp32 [ext_embed_dim], copied).  rekv_retrieve_external scores every visible frame -- or
 * every complete block of block_frames frames, whose vector is the mean of its frames' embeddings --
 *   Sim(v, q) = <v, q> / (tau |v| |q|)        (norms clamped at 1e-8)
 * against each of nQ question embeddings (q_emb: device fp32 [nQ][ext_embed_dim]) and selects as
 * rekv_retrieve does (candidates exclude the window, ties to the lower index, ascending output).  One
 * selection serves all layers: idx_out, device int32 [L][nQ][top_k], receives it in every layer's block, so
 * that rekv_gather takes it unchanged.  scores_out (nullable): device fp32 [nQ][n_scored], n_scored as in
 * rekv_retrieve.  Needs ext_embed_dim > 0 and embeddings for all of [0, n_visible).  tau > 0.
 * Returns k_eff or a negative error code. */
int rekv_set_frame_embedding(rekv_ctx* ctx, int frame, const float* emb, void* stream);
int rekv_retrieve_external(rekv_ctx* ctx, const float* q_emb, int nQ, int top_k, int n_visible, float tau,
                           int32_t* idx_out, float* scores_out, void* stream);

/* Steps 2-5 in one call, for all layers: what rekv_retrieve, rekv_gather (page-list mode) and rekv_attend do
 * in sequence on the library's own selection, with the same results.  idx_out (nullable): device int32
 * [L][nQ][top_k].  On a cache that is all in HBM the selection kernel writes the context table itself (one
 * launch fewer).  Returns the number of context frames, or a negative error code. */
int rekv_question(rekv_ctx* ctx, const void* q, const int32_t* cu_q, int nQ, int top_k, int n_visible, int32_t* idx_out,
                  void* out, void* stream);

/* Layer-sequential form of steps 2-5.  A decoder produces layer l+1's queries only from layer l's
 * output, and the paper retrieves independently in every layer, so a model integrates the path one
 * layer at a time: this call enqueues retrieve -> gather -> attend of ONE layer on `stream`.
 *   layer     0 .. n_layers-1
 *   q         device bf16 [sum_Nq][H_q][D]: that layer's query rows, questions packed back to back
 *   cu_q, nQ, top_k, n_visible   as in rekv_retrieve
 *   idx_out   device int32 [nQ][top_k] (nullable): the layer's selection, ascending, -1 past k_eff
 *   out       device bf16 [sum_Nq][H_q][D]
 * Same arithmetic, kernels and results as the all-layer calls restricted to that layer.  Nothing is
 * allocated and the host is not synchronised; on a context whose cache is all in HBM the call may be
 * captured into a CUDA graph (one graph per layer, replayed while the stored frames, n_visible and the
 * buffers stay the same); an offloaded context uses the internal side stream and must not be captured.
 * The context built for the layer stays valid for rekv_attend_layer until the next gather of that layer, or
 * until a gather of ANY layer with another number of questions or context frames (top_k, n_visible): all
 * layers share one context table, whose layout follows those counts; rekv_attend_layer, rekv_attend and
 * rekv_attend_full then return REKV_ERR_STATE for the layers that were not gathered again.
 * Returns the number of context frames, or a negative error code. */
int rekv_question_layer(rekv_ctx* ctx, int layer, const void* q, const int32_t* cu_q, int nQ, int top_k, int n_visible,
                        int32_t* idx_out, void* out, void* stream);

/* Step 5 of one layer over the context that layer's last rekv_question_layer (or rekv_gather) built:
 * the decode steps that follow a question reuse its retrieved context with new query rows.
 * q, out: device bf16 [sum_Nq][H_q][D]; nQ must equal the gathered batch.  Returns 0 or an error code. */
int rekv_attend_layer(rekv_ctx* ctx, int layer, const void* q, const int32_t* cu_q, int nQ, void* out, void* stream);

/* The two layer calls with Eq. 3 in full -- what a decoder layer calls with the Q, K, V it has just made of X:
 * rekv_question_layer_full = steps 2-4 of the layer as in rekv_question_layer, then step 5 over [R, X] as in
 * rekv_attend_full; rekv_attend_full_layer = that step 5 alone over the layer's existing context (decode steps).
 *   q               device bf16 [sum_Nq][H_q][D] of this layer
 *   k_self, v_self  device bf16 [sum_Ns][H_kv][D] of this layer; cu_q, cu_self as in rekv_attend_full
 *   idx_out, out    as in rekv_question_layer
 * Positions under rope_theta > 0, the static variant, the validity of a layer's context and the error codes are those
 * of rekv_attend_full and rekv_question_layer.  Needs max_self_tokens > 0 at creation.  Returns the number of context
 * frames (rekv_question_layer_full) or 0 (rekv_attend_full_layer), or an error code. */
int rekv_question_layer_full(rekv_ctx* ctx, int layer, const void* q, const void* k_self, const void* v_self,
                             const int32_t* cu_q, const int32_t* cu_self, int nQ, int top_k, int n_visible,
                             int32_t* idx_out, void* out, void* stream);
int rekv_attend_full_layer(rekv_ctx* ctx, int layer, const void* q, const void* k_self, const void* v_self,
                           const int32_t* cu_q, const int32_t* cu_self, int nQ, void* out, void* stream);

/* Disk tier.  rekv_save synchronises the device and writes the context's stream state -- configuration, frame
 * count, representatives, frame embeddings, every page (host tier as it is held, plus the exact frames of the HBM
 * tail) -- to `path`.  rekv_load creates a context on `device` from such a file, ready for further appends and
 * questions: the stream can be encoded by one process and questioned by others.  Both return 0 or an error code
 * (rekv_last_error(NULL) after a failed load). */
int rekv_save(rekv_ctx* ctx, const char* path);
int rekv_load(const char* path, int device, rekv_ctx** out);

/* Output geometry of a question that sees n_visible frames and asks for top_k: how the library sizes what
 * rekv_retrieve and rekv_gather write (readings of the Eq. 2 paragraph: the last W visible frames are never
 * candidates; with block retrieval only complete blocks are).  Host-side only, no device work.
 *   n_scored   items scored per (layer, question): candidate blocks when block_frames > 1, else -- the score
 *              array then covers every visible frame -- n_visible
 *   k_eff      frames actually retrieved, min(top_k, candidates) rounded to whole blocks
 *   w_eff      trailing frames that are always in the context; context frames = k_eff + w_eff
 * Any of the three output pointers may be NULL.  Returns 0, or REKV_ERR_ARG on a negative argument or a
 * top_k that is not a multiple of block_frames. */
int rekv_geometry(rekv_ctx* ctx, int n_visible, int top_k, int32_t* n_scored, int32_t* k_eff, int32_t* w_eff);

/* Fills *out with store accounting and the last call's counters.  Never waits for the device: the byte counter
 * of the host link and the stage timings describe work that has COMPLETED (synchronise the stream first for the
 * figures of the call just enqueued); a stage whose events have not completed yet reads 0. */
int rekv_stats(rekv_ctx* ctx, rekv_stats_t* out);

/* Switches REKV_FLAG_TIMING on (enable != 0) or off for the calls that follow.  The two event records around
 * the attention kernel stand between it and its neighbours in the stream, so a timed question is a few
 * microseconds slower than an untimed one (its kernels no longer overlap each other's prologues): measure the
 * kernel with the flag on and the question with it off.  Host-side only; returns REKV_OK. */
int rekv_set_timing(rekv_ctx* ctx, int enable);

/* Reads (and clears) the device status word after synchronising `stream`: 0, or REKV_ERR_TIMEOUT
 * if a bounded device-side wait gave up since the last check. */
int rekv_check_status(rekv_ctx* ctx, void* stream);

/* TEST-ONLY.  The kernels' device-side waits (on a copy, a matrix product, another warp) are bounded: when a
 * wait runs out of iterations the kernel writes REKV_ERR_TIMEOUT to the status word, releases what it holds
 * and returns, and the context stays usable.  This call makes that path reachable without a fault:
 *   iterations       limit of every bounded wait of the attention kernels launched from now on (0 = the
 *                    built-in limit, about a third of a second)
 *   skip_copy_entry  >= 0: the copy producer of the attention kernel's first CTA leaves out the K/V tile copy
 *                    with this sequence number, so that the wait for it expires with nothing in flight; -1 = off
 * The affected launches produce no valid output; rekv_check_status then returns REKV_ERR_TIMEOUT once.
 * Host-side only; returns REKV_OK. */
int rekv_test_set_wait_limit(rekv_ctx* ctx, unsigned iterations, int skip_copy_entry);

/* Message of the last failure on this context (or of the last failed rekv_create when ctx is NULL).
 * The pointer stays valid until the next failing call. */
const char* rekv_last_error(rekv_ctx* ctx);

/* Test helpers.  rekv_get_reps copies the representatives of frames [0, n_frames) of one layer to
 * dev_out, device fp32 [n_frames][H_kv*D].  rekv_get_page copies one stored (frame, layer) page back
 * in plain layout: k_out, v_out device bf16 [H_kv][N_f][D] (from HBM if resident, else from host). */
int rekv_get_reps(rekv_ctx* ctx, int layer, int n_frames, float* dev_out, void* stream);
int rekv_get_page(rekv_ctx* ctx, int frame, int layer, void* k_out, void* v_out, void* stream);

/* Scoring without allocation (the paper has no counterpart; this entry point exists for hosts that
 * cannot let a library allocate device memory -- a serving engine that owns the whole GPU through its
 * own pool, or a latency-critical thread that must not meet cudaMalloc's device synchronisation).
 * Computes, for one layer, the cosine score of every frame representative against each of nQ question
 * vectors, exactly as rekv_retrieve does (question vector = mean over the question's tokens and over
 * the G query heads of each KV group; norms clamped at 1e-8), without a context and without calling
 * cudaMalloc, cudaFree or any allocating routine: its intermediate lives in a 66 048-byte array that
 * is part of the library image (held by every GPU that loads the library until the process exits).
 *   q          device bf16 [sum_Nq][H_q][128], the layer's query rows, questions packed back to back
 *   cu_q       HOST int32[nQ+1] prefix sums of the question lengths; 1 <= nQ <= 16
 *   reps       device fp32 [n_frames][H_kv*128] frame representatives (e.g. from rekv_get_reps)
 *   scores_out device fp32 [nQ][n_frames]
 * Limits: head_dim == 128, H_kv <= 8 (H_kv*128 <= 1024), nQ <= 16; anything larger is rejected with
 * REKV_ERR_ARG and a message (rekv_last_error(NULL)).  Runs on the CURRENT device, on `stream`.
 * The first call on a device resolves the array's device address (cudaGetSymbolAddress); make that
 * first call outside any stream capture.  All calls on a device share the array: each call rewrites
 * it completely and leaves its contents behind, and calls whose kernels overlap on the GPU race. */
int rekv_score_frames_static(const void* q, const int32_t* cu_q, int nQ, int n_q_heads, int n_kv_heads, int head_dim,
                             const float* reps, int n_frames, float* scores_out, void* stream);

/* Number of kernels this library has launched on the context since creation (for launch counting). */
int64_t rekv_launch_count(rekv_ctx* ctx);

#ifdef __cplusplus
}
#endif

#endif /* REKV_H_ */
