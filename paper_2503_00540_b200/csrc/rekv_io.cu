// Disk tier: a context's stream state written to and read back from a file, so that a stream encoded by
// one process can be questioned by another (the paper keeps the KV-cache in RAM or on disk and separates
// video encoding from question answering across processes and GPUs).
//
// File layout (little endian, no padding between sections):
//   char[8]      "REKVCTX1"
//   rekv_config  the creating configuration (the `device` field is replaced at load time)
//   int32        frames appended, int32 frames with an external embedding
//   float        representatives: for every layer, frames x (H_kv*128)
//   float        external embeddings: ext_frames x ext_embed_dim (absent without an embedding table)
//   bytes        pages, frame-major -- a cache all in HBM: frames x L x page_bytes;
//                an offloaded cache: the host tier's frames x L x host_page_bytes (FP8 form if the context
//                uses it), then the frames still in the HBM tail, exact: min(frames, tail) x L x page_bytes
#include <cstdio>
#include <vector>

#include "rekv_internal.cuh"

namespace {

struct File {
  FILE* f = nullptr;
  ~File() {
    if (f) fclose(f);
  }
};

// device <-> file through a bounded pinned bounce buffer
bool dev_to_file(FILE* f, const char* dev, size_t bytes, char* bounce, size_t bounce_bytes) {
  for (size_t off = 0; off < bytes; off += bounce_bytes) {
    const size_t n = bytes - off < bounce_bytes ? bytes - off : bounce_bytes;
    if (cudaMemcpy(bounce, dev + off, n, cudaMemcpyDeviceToHost) != cudaSuccess) return false;
    if (fwrite(bounce, 1, n, f) != n) return false;
  }
  return true;
}
bool file_to_dev(FILE* f, char* dev, size_t bytes, char* bounce, size_t bounce_bytes) {
  for (size_t off = 0; off < bytes; off += bounce_bytes) {
    const size_t n = bytes - off < bounce_bytes ? bytes - off : bounce_bytes;
    if (fread(bounce, 1, n, f) != n) return false;
    if (cudaMemcpy(dev + off, bounce, n, cudaMemcpyHostToDevice) != cudaSuccess) return false;
  }
  return true;
}

constexpr char MAGIC[8] = {'R', 'E', 'K', 'V', 'C', 'T', 'X', '1'};
constexpr size_t BOUNCE = 64u << 20;

}  // namespace

extern "C" {

int rekv_save(rekv_ctx* c, const char* path) {
  if (!c) return REKV_ERR_ARG;
  if (!path) REKV_FAIL(c, REKV_ERR_ARG, "null path");
  cudaSetDevice(c->device);
  REKV_CUDA(c, cudaDeviceSynchronize());  // appends and write-throughs in flight are part of the state
  const StoreView& s = c->sv;
  File file;
  file.f = fopen(path, "wb");
  if (!file.f) REKV_FAIL(c, REKV_ERR_ARG, "cannot open %s for writing", path);
  std::vector<char> bounce_v;
  char* bounce = nullptr;
  REKV_CUDA(c, cudaHostAlloc((void**)&bounce, BOUNCE, cudaHostAllocDefault));
  bool ok = fwrite(MAGIC, 1, 8, file.f) == 8 && fwrite(&c->cfg, sizeof(rekv_config), 1, file.f) == 1;
  const int32_t counts[2] = {c->frames, c->ext_frames};
  ok = ok && fwrite(counts, sizeof(int32_t), 2, file.f) == 2;
  for (int l = 0; ok && l < s.L; ++l)
    ok = dev_to_file(file.f, (const char*)(s.reps + (size_t)l * s.max_frames * s.Dp), (size_t)c->frames * s.Dp * sizeof(float),
                     bounce, BOUNCE);
  if (ok && c->cfg.ext_embed_dim > 0)
    ok = dev_to_file(file.f, (const char*)c->ext_emb, (size_t)c->ext_frames * c->cfg.ext_embed_dim * sizeof(float), bounce,
                     BOUNCE);
  const size_t frame_bytes = (size_t)s.page_bytes * s.L, host_frame_bytes = (size_t)s.host_page_bytes * s.L;
  if (s.tail == 0) {
    if (ok) ok = dev_to_file(file.f, s.hbm, (size_t)c->frames * frame_bytes, bounce, BOUNCE);
  } else {
    for (int f = 0; ok && f < c->frames; ++f) {
      const char* src = c->host_arenas[f / s.frames_per_arena] + (size_t)(f % s.frames_per_arena) * host_frame_bytes;
      ok = fwrite(src, 1, host_frame_bytes, file.f) == host_frame_bytes;
    }
    const int n_tail = c->frames < s.tail ? c->frames : s.tail;
    for (int f = c->frames - n_tail; ok && f < c->frames; ++f)
      ok = dev_to_file(file.f, s.hbm + rekv_hbm_page_offset(s, f, 0), frame_bytes, bounce, BOUNCE);
  }
  cudaFreeHost(bounce);
  if (!ok) REKV_FAIL(c, REKV_ERR_CUDA, "writing %s failed", path);
  return REKV_OK;
}

int rekv_load(const char* path, int device, rekv_ctx** out) {
  if (!path || !out) REKV_FAIL(nullptr, REKV_ERR_ARG, "null path or output pointer");
  *out = nullptr;
  File file;
  file.f = fopen(path, "rb");
  if (!file.f) REKV_FAIL(nullptr, REKV_ERR_ARG, "cannot open %s", path);
  char magic[8];
  rekv_config cfg;
  int32_t counts[2];
  if (fread(magic, 1, 8, file.f) != 8 || memcmp(magic, MAGIC, 8) != 0 || fread(&cfg, sizeof(cfg), 1, file.f) != 1 ||
      fread(counts, sizeof(int32_t), 2, file.f) != 2)
    REKV_FAIL(nullptr, REKV_ERR_ARG, "%s is not a saved context", path);
  cfg.device = device;
  if (counts[0] < 0 || counts[0] > cfg.max_frames || counts[1] < 0 || counts[1] > counts[0])
    REKV_FAIL(nullptr, REKV_ERR_ARG, "%s: frame counts out of range", path);
  rekv_ctx* c = nullptr;
  const int rc = rekv_create(&cfg, &c);
  if (rc != REKV_OK) return rc;
  const StoreView& s = c->sv;
  char* bounce = nullptr;
  bool ok = cudaHostAlloc((void**)&bounce, BOUNCE, cudaHostAllocDefault) == cudaSuccess;
  const int frames = counts[0];
  for (int l = 0; ok && l < s.L; ++l)
    ok = file_to_dev(file.f, (char*)(s.reps + (size_t)l * s.max_frames * s.Dp), (size_t)frames * s.Dp * sizeof(float), bounce,
                     BOUNCE);
  if (ok && cfg.ext_embed_dim > 0)
    ok = file_to_dev(file.f, (char*)c->ext_emb, (size_t)counts[1] * cfg.ext_embed_dim * sizeof(float), bounce, BOUNCE);
  const size_t frame_bytes = (size_t)s.page_bytes * s.L, host_frame_bytes = (size_t)s.host_page_bytes * s.L;
  if (s.tail == 0) {
    if (ok) ok = file_to_dev(file.f, s.hbm, (size_t)frames * frame_bytes, bounce, BOUNCE);
  } else {
    for (int f = 0; ok && f < frames; ++f) {
      char* dst = c->host_arenas[f / s.frames_per_arena] + (size_t)(f % s.frames_per_arena) * host_frame_bytes;
      ok = fread(dst, 1, host_frame_bytes, file.f) == host_frame_bytes;
    }
    const int n_tail = frames < s.tail ? frames : s.tail;
    for (int f = frames - n_tail; ok && f < frames; ++f)
      ok = file_to_dev(file.f, s.hbm + rekv_hbm_page_offset(s, f, 0), frame_bytes, bounce, BOUNCE);
  }
  if (bounce) cudaFreeHost(bounce);
  if (!ok) {
    rekv_destroy(c);
    REKV_FAIL(nullptr, REKV_ERR_CUDA, "reading %s failed (truncated file or a CUDA error)", path);
  }
  c->frames = frames;
  c->ext_frames = counts[1];
  *out = c;
  return REKV_OK;
}

}  // extern "C"
