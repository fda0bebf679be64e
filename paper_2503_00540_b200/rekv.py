"""Python binding of librekv: argument marshalling only.

Every step of the path (pooling, scoring, selection, gather, attention) runs in the CUDA
kernels behind the C ABI declared in include/rekv.h; this module converts torch tensors to
raw pointers, passes torch's current stream, and turns negative return codes into exceptions.
There is no CPU fallback: loading fails loudly if the shared library is missing or cannot be
built, and creating a context fails without a CUDA device.
"""
import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Sequence, Tuple

import torch

from . import _build

OK, ERR_ARG, ERR_FULL, ERR_EMPTY, ERR_ALLOC, ERR_CUDA, ERR_TIMEOUT, ERR_STATE = 0, -1, -2, -3, -4, -5, -6, -7
FLAG_TIMING = 1 << 2
FLAG_HOST_FP8 = 1 << 3
FLAG_ROPE_STATIC = 1 << 4


class RekvError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"librekv error {code}: {msg}")
        self.code = code


class rekv_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "n_layers", "n_q_heads", "n_kv_heads", "head_dim", "tokens_per_frame", "max_frames", "hbm_tail_frames",
        "window_frames", "block_frames", "max_q_tokens", "max_topk", "max_questions", "device")] + [
            ("flags", ctypes.c_uint32), ("max_self_tokens", ctypes.c_int32), ("rope_theta", ctypes.c_float),
            ("ext_embed_dim", ctypes.c_int32)]


class rekv_stats_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in (
        "frames", "kv_bytes_hbm", "kv_bytes_host", "kv_bytes_logical", "rep_bytes", "page_bytes",
        "last_link_bytes")] + [("last_k_eff", ctypes.c_int32), ("last_ctx_frames", ctypes.c_int32),
                                       ("last_attend_kernel_us", ctypes.c_double), ("last_retrieve_us", ctypes.c_double),
                                       ("last_pull_us", ctypes.c_double), ("last_merge_us", ctypes.c_double)]


EXPORTS = ("rekv_create", "rekv_destroy", "rekv_append_frame", "rekv_retrieve", "rekv_gather", "rekv_attend",
           "rekv_stats", "rekv_check_status", "rekv_last_error", "rekv_get_reps", "rekv_get_page",
           "rekv_launch_count", "rekv_score_frames_static", "rekv_question_layer", "rekv_attend_layer", "rekv_attend_full",
           "rekv_question_layer_full", "rekv_attend_full_layer",
           "rekv_set_frame_embedding", "rekv_retrieve_external", "rekv_question",
           "rekv_save", "rekv_load", "rekv_set_timing", "rekv_geometry",
           "rekv_test_set_wait_limit")

_lib = None


def lib() -> ctypes.CDLL:
    """Loads (building in-tree if stale) librekv.so.  Raises if that is impossible."""
    global _lib
    if _lib is None:
        # REKV_CHECKS=1 in the environment selects the self-checking build of the same sources (test runs only)
        # REKV_SANITIZE=1 selects the build whose host code runs under AddressSanitizer/UBSan (the process must have
        # the sanitizer runtime preloaded)
        path = _build.build_librekv(checks=os.environ.get("REKV_CHECKS", "") == "1",
                                    sanitize=os.environ.get("REKV_SANITIZE", "") == "1")
        L = ctypes.CDLL(path)
        vp, i32, ip = ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_int32)
        L.rekv_create.argtypes = [ctypes.POINTER(rekv_config), ctypes.POINTER(vp)]
        L.rekv_destroy.argtypes = [vp]
        L.rekv_append_frame.argtypes = [vp, vp, vp, vp]
        L.rekv_retrieve.argtypes = [vp, vp, ip, i32, i32, i32, vp, vp, vp]
        L.rekv_gather.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
        L.rekv_attend.argtypes = [vp, vp, ip, i32, vp, vp]
        L.rekv_question_layer.argtypes = [vp, i32, vp, ip, i32, i32, i32, vp, vp, vp]
        L.rekv_question.argtypes = [vp, vp, ip, i32, i32, i32, vp, vp, vp]
        L.rekv_save.argtypes = [vp, ctypes.c_char_p]
        L.rekv_load.argtypes = [ctypes.c_char_p, i32, ctypes.POINTER(vp)]
        L.rekv_attend_layer.argtypes = [vp, i32, vp, ip, i32, vp, vp]
        L.rekv_attend_full.argtypes = [vp, vp, vp, vp, ip, ip, i32, vp, vp]
        L.rekv_question_layer_full.argtypes = [vp, i32, vp, vp, vp, ip, ip, i32, i32, i32, vp, vp, vp]
        L.rekv_attend_full_layer.argtypes = [vp, i32, vp, vp, vp, ip, ip, i32, vp, vp]
        L.rekv_set_frame_embedding.argtypes = [vp, i32, vp, vp]
        L.rekv_retrieve_external.argtypes = [vp, vp, i32, i32, i32, ctypes.c_float, vp, vp, vp]
        L.rekv_stats.argtypes = [vp, ctypes.POINTER(rekv_stats_t)]
        L.rekv_check_status.argtypes = [vp, vp]
        L.rekv_set_timing.argtypes = [vp, i32]
        L.rekv_test_set_wait_limit.argtypes = [vp, ctypes.c_uint, i32]
        L.rekv_geometry.argtypes = [vp, i32, i32, ip, ip, ip]
        L.rekv_last_error.argtypes = [vp]
        L.rekv_last_error.restype = ctypes.c_char_p
        L.rekv_get_reps.argtypes = [vp, i32, i32, vp, vp]
        L.rekv_get_page.argtypes = [vp, i32, i32, vp, vp, vp]
        L.rekv_score_frames_static.argtypes = [vp, ip, i32, i32, i32, i32, vp, i32, vp, vp]
        L.rekv_launch_count.argtypes = [vp]
        L.rekv_launch_count.restype = ctypes.c_int64
        for name in EXPORTS:
            if name not in ("rekv_last_error", "rekv_launch_count"):
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _cu_array(cu_q: Sequence[int]):
    return (ctypes.c_int32 * len(cu_q))(*cu_q)


def _ptr(t: Optional[torch.Tensor], dtype=None, cuda: bool = True):
    if t is None:
        return None
    if cuda and not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return t.data_ptr()


class ReKV:
    """One retrieval context (one video stream) on one GPU.  Methods mirror the C entry points."""

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, tokens_per_frame: int,
                 max_frames: int, window_frames: int, hbm_tail_frames: int = 0, max_q_tokens: int = 64,
                 max_topk: int = 64, max_questions: int = 1, device: int = 0, flags: int = 0,
                 block_frames: int = 1, max_self_tokens: int = 0, rope_theta: float = 0.0, ext_embed_dim: int = 0):
        self.cfg = rekv_config(n_layers, n_q_heads, n_kv_heads, head_dim, tokens_per_frame, max_frames,
                               hbm_tail_frames, window_frames, block_frames, max_q_tokens, max_topk, max_questions,
                               device, flags, max_self_tokens, rope_theta, ext_embed_dim)
        self._h = ctypes.c_void_p()
        rc = lib().rekv_create(ctypes.byref(self.cfg), ctypes.byref(self._h))
        if rc != 0:
            raise RekvError(rc, (lib().rekv_last_error(None) or b"").decode())
        self.device = torch.device("cuda", device)
        self.L, self.Hq, self.Hkv, self.D, self.Nf, self.W = (n_layers, n_q_heads, n_kv_heads, head_dim,
                                                              tokens_per_frame, window_frames)
        self.b = block_frames

    def save(self, path: str) -> None:
        """Writes the stream state (representatives, embeddings, every page) to a file."""
        self._check(lib().rekv_save(self._h, path.encode()))

    @classmethod
    def load(cls, path: str, device: int = 0) -> "ReKV":
        """A context created from a file written by save(), ready for further appends and questions."""
        h = ctypes.c_void_p()
        rc = lib().rekv_load(path.encode(), device, ctypes.byref(h))
        if rc != 0:
            raise RekvError(rc, (lib().rekv_last_error(None) or b"").decode())
        self = cls.__new__(cls)
        self._h = h
        self.device = torch.device("cuda", device)
        cfg = rekv_config.from_buffer_copy(open(path, "rb").read(8 + ctypes.sizeof(rekv_config))[8:])
        cfg.device = device
        self.cfg = cfg
        self.L, self.Hq, self.Hkv, self.D, self.Nf, self.W = (cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                                                              cfg.tokens_per_frame, cfg.window_frames)
        self.b = cfg.block_frames
        return self

    def geometry(self, n_visible: int, top_k: int) -> Tuple[int, int, int]:
        """(items scored per question, frames retrieved, trailing frames always in the context) as
        rekv_geometry reports them: the sizes of what retrieve and gather write."""
        n, k, w = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        self._check(lib().rekv_geometry(self._h, n_visible, top_k, ctypes.byref(n), ctypes.byref(k), ctypes.byref(w)))
        return n.value, k.value, w.value

    # ------------------------------------------------------------------ plumbing
    def _check(self, rc: int) -> int:
        if rc < 0:
            raise RekvError(rc, (lib().rekv_last_error(self._h) or b"").decode())
        return rc

    def _stream(self) -> int:
        return torch.cuda.current_stream(self.device).cuda_stream

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().rekv_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ the five calls
    def append_frame(self, k: torch.Tensor, v: torch.Tensor) -> int:
        """k, v: bf16 [L][N_f][H_kv][D] on the context's device.  Returns the frame index."""
        shape = (self.L, self.Nf, self.Hkv, self.D)
        if tuple(k.shape) != shape or tuple(v.shape) != shape:
            raise ValueError(f"expected K/V of shape {shape}")
        return self._check(lib().rekv_append_frame(self._h, _ptr(k, torch.bfloat16), _ptr(v, torch.bfloat16),
                                                   self._stream()))

    def retrieve(self, q: torch.Tensor, cu_q: Sequence[int], top_k: int, n_visible: int,
                 want_scores: bool = False) -> Tuple[torch.Tensor, int, Optional[torch.Tensor]]:
        """q: bf16 [L][sum_Nq][H_q][D].  Returns (idx int32 [L][nQ][top_k], k_eff, scores or None)."""
        nQ = len(cu_q) - 1
        if tuple(q.shape) != (self.L, cu_q[-1], self.Hq, self.D):
            raise ValueError("q must be [L][sum_Nq][H_q][D]")
        idx = torch.empty((self.L, nQ, max(top_k, 0)), dtype=torch.int32, device=self.device)
        n_scored = self.geometry(n_visible, top_k)[0]
        scores = (torch.empty((self.L, nQ, n_scored), dtype=torch.float32, device=self.device)
                  if want_scores and n_visible > 0 else None)
        k_eff = self._check(lib().rekv_retrieve(self._h, _ptr(q, torch.bfloat16), _cu_array(cu_q), nQ, top_k,
                                                n_visible, _ptr(idx), _ptr(scores), self._stream()))
        return idx, k_eff, scores

    def gather(self, idx: torch.Tensor, nQ: int, top_k: int, n_visible: int,
               materialize: bool = False) -> Tuple[int, Optional[torch.Tensor], Optional[torch.Tensor]]:
        """idx: int32 [L][nQ][top_k].  Returns (context frames, k_ctx, v_ctx); the last two are bf16
        [L][nQ][H_kv][n_ctx][D] when materialize is set, else None."""
        if tuple(idx.shape) != (self.L, nQ, top_k):
            raise ValueError("idx must be [L][nQ][top_k]")
        k_ctx = v_ctx = None
        if materialize:
            _, k_eff, w_eff = self.geometry(n_visible, top_k)
            n_ctx = (k_eff + w_eff) * self.Nf
            shape = (self.L, nQ, self.Hkv, n_ctx, self.D)
            k_ctx = torch.empty(shape, dtype=torch.bfloat16, device=self.device)
            v_ctx = torch.empty(shape, dtype=torch.bfloat16, device=self.device)
        ncf = self._check(lib().rekv_gather(self._h, _ptr(idx, torch.int32), nQ, top_k, n_visible, _ptr(k_ctx),
                                            _ptr(v_ctx), self._stream()))
        return ncf, k_ctx, v_ctx

    def attend(self, q: torch.Tensor, cu_q: Sequence[int], out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """q: bf16 [L][sum_Nq][H_q][D] -> bf16 of the same shape."""
        if out is None:
            out = torch.empty_like(q)
        self._check(lib().rekv_attend(self._h, _ptr(q, torch.bfloat16), _cu_array(cu_q), len(cu_q) - 1,
                                      _ptr(out, torch.bfloat16), self._stream()))
        return out

    def question(self, q: torch.Tensor, cu_q: Sequence[int], top_k: int, n_visible: int,
                 out: Optional[torch.Tensor] = None, idx: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Steps 2-5 for a batch of questions: rekv_question on the library's own selection, or gather + attend on
        a selection the caller passes."""
        nQ = len(cu_q) - 1
        if idx is None:
            if tuple(q.shape) != (self.L, cu_q[-1], self.Hq, self.D):
                raise ValueError("q must be [L][sum_Nq][H_q][D]")
            if out is None:
                out = torch.empty_like(q)
            self._check(lib().rekv_question(self._h, _ptr(q, torch.bfloat16), _cu_array(cu_q), nQ, top_k, n_visible,
                                            None, _ptr(out, torch.bfloat16), self._stream()))
            return out
        self.gather(idx, nQ, top_k, n_visible)
        return self.attend(q, cu_q, out)

    def set_frame_embedding(self, frame: int, emb: torch.Tensor) -> None:
        """emb: float32 [ext_embed_dim], the external encoder's embedding of an appended frame."""
        self._check(lib().rekv_set_frame_embedding(self._h, frame, _ptr(emb, torch.float32), self._stream()))

    def retrieve_external(self, q_emb: torch.Tensor, top_k: int, n_visible: int, tau: float,
                          want_scores: bool = False) -> Tuple[torch.Tensor, int, Optional[torch.Tensor]]:
        """q_emb: float32 [nQ][ext_embed_dim].  Returns (idx int32 [L][nQ][top_k], the same selection in every
        layer; k_eff; scores float32 [nQ][n_scored] or None)."""
        nQ = q_emb.shape[0]
        idx = torch.empty((self.L, nQ, max(top_k, 0)), dtype=torch.int32, device=self.device)
        n_scored = self.geometry(n_visible, top_k)[0]
        scores = (torch.empty((nQ, n_scored), dtype=torch.float32, device=self.device)
                  if want_scores and n_visible > 0 else None)
        k_eff = self._check(lib().rekv_retrieve_external(self._h, _ptr(q_emb, torch.float32), nQ, top_k, n_visible,
                                                         tau, _ptr(idx), _ptr(scores), self._stream()))
        return idx, k_eff, scores

    def attend_full(self, q: torch.Tensor, k_self: torch.Tensor, v_self: torch.Tensor, cu_q: Sequence[int],
                    cu_self: Sequence[int], out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Eq. 3 in full over the gathered context followed by the questions' own K/V (causal).
        q: bf16 [L][sum_Nq][H_q][D]; k_self, v_self: bf16 [L][sum_Ns][H_kv][D] -> bf16 like q."""
        if tuple(q.shape) != (self.L, cu_q[-1], self.Hq, self.D):
            raise ValueError("q must be [L][sum_Nq][H_q][D]")
        if tuple(k_self.shape) != (self.L, cu_self[-1], self.Hkv, self.D) or k_self.shape != v_self.shape:
            raise ValueError("k_self and v_self must be [L][sum_Ns][H_kv][D]")
        if out is None:
            out = torch.empty_like(q)
        self._check(lib().rekv_attend_full(self._h, _ptr(q, torch.bfloat16), _ptr(k_self, torch.bfloat16),
                                           _ptr(v_self, torch.bfloat16), _cu_array(cu_q), _cu_array(cu_self),
                                           len(cu_q) - 1, _ptr(out, torch.bfloat16), self._stream()))
        return out

    def question_layer(self, layer: int, q: torch.Tensor, cu_q: Sequence[int], top_k: int, n_visible: int,
                       out: Optional[torch.Tensor] = None, idx: Optional[torch.Tensor] = None) -> torch.Tensor:
        """retrieve -> gather -> attend of one layer.  q: bf16 [sum_Nq][H_q][D] of that layer -> same shape.
        idx (optional, int32 [nQ][top_k]) receives the layer's selection."""
        nQ = len(cu_q) - 1
        if tuple(q.shape) != (cu_q[-1], self.Hq, self.D):
            raise ValueError("q must be [sum_Nq][H_q][D]")
        if idx is not None and tuple(idx.shape) != (nQ, top_k):
            raise ValueError("idx must be [nQ][top_k]")
        if out is None:
            out = torch.empty_like(q)
        self._check(lib().rekv_question_layer(self._h, layer, _ptr(q, torch.bfloat16), _cu_array(cu_q), nQ, top_k,
                                              n_visible, _ptr(idx, torch.int32), _ptr(out, torch.bfloat16),
                                              self._stream()))
        return out

    def question_layer_full(self, layer: int, q: torch.Tensor, k_self: torch.Tensor, v_self: torch.Tensor,
                            cu_q: Sequence[int], cu_self: Sequence[int], top_k: int, n_visible: int,
                            out: Optional[torch.Tensor] = None, idx: Optional[torch.Tensor] = None) -> torch.Tensor:
        """retrieve -> gather of one layer, then Eq. 3 in full over [R, X].  q: bf16 [sum_Nq][H_q][D];
        k_self, v_self: bf16 [sum_Ns][H_kv][D], all of this layer -> bf16 like q."""
        nQ = len(cu_q) - 1
        self._check_layer_full_shapes(q, k_self, v_self, cu_q, cu_self)
        if idx is not None and tuple(idx.shape) != (nQ, top_k):
            raise ValueError("idx must be [nQ][top_k]")
        if out is None:
            out = torch.empty_like(q)
        self._check(lib().rekv_question_layer_full(self._h, layer, _ptr(q, torch.bfloat16), _ptr(k_self, torch.bfloat16),
                                                   _ptr(v_self, torch.bfloat16), _cu_array(cu_q), _cu_array(cu_self),
                                                   nQ, top_k, n_visible, _ptr(idx, torch.int32),
                                                   _ptr(out, torch.bfloat16), self._stream()))
        return out

    def attend_full_layer(self, layer: int, q: torch.Tensor, k_self: torch.Tensor, v_self: torch.Tensor,
                          cu_q: Sequence[int], cu_self: Sequence[int],
                          out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Eq. 3 in full of one layer over the context its last question_layer(_full) (or gather) built."""
        self._check_layer_full_shapes(q, k_self, v_self, cu_q, cu_self)
        if out is None:
            out = torch.empty_like(q)
        self._check(lib().rekv_attend_full_layer(self._h, layer, _ptr(q, torch.bfloat16), _ptr(k_self, torch.bfloat16),
                                                 _ptr(v_self, torch.bfloat16), _cu_array(cu_q), _cu_array(cu_self),
                                                 len(cu_q) - 1, _ptr(out, torch.bfloat16), self._stream()))
        return out

    def _check_layer_full_shapes(self, q, k_self, v_self, cu_q, cu_self):
        if tuple(q.shape) != (cu_q[-1], self.Hq, self.D):
            raise ValueError("q must be [sum_Nq][H_q][D]")
        if tuple(k_self.shape) != (cu_self[-1], self.Hkv, self.D) or k_self.shape != v_self.shape:
            raise ValueError("k_self and v_self must be [sum_Ns][H_kv][D]")

    def attend_layer(self, layer: int, q: torch.Tensor, cu_q: Sequence[int],
                     out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Attention of one layer over the context its last question_layer (or gather) built."""
        if tuple(q.shape) != (cu_q[-1], self.Hq, self.D):
            raise ValueError("q must be [sum_Nq][H_q][D]")
        if out is None:
            out = torch.empty_like(q)
        self._check(lib().rekv_attend_layer(self._h, layer, _ptr(q, torch.bfloat16), _cu_array(cu_q), len(cu_q) - 1,
                                            _ptr(out, torch.bfloat16), self._stream()))
        return out

    # ------------------------------------------------------------------ accounting and test helpers
    def stats(self) -> rekv_stats_t:
        st = rekv_stats_t()
        self._check(lib().rekv_stats(self._h, ctypes.byref(st)))
        return st

    def check_status(self) -> None:
        self._check(lib().rekv_check_status(self._h, self._stream()))

    def set_timing(self, enable: bool) -> None:
        """Event records around the attention kernel on or off for the calls that follow (see rekv_set_timing)."""
        self._check(lib().rekv_set_timing(self._h, 1 if enable else 0))

    def test_set_wait_limit(self, iterations: int, skip_copy_entry: int = -1) -> None:
        """Test-only: shortens the kernels' bounded waits and makes one tile copy go missing (rekv_test_set_wait_limit)."""
        self._check(lib().rekv_test_set_wait_limit(self._h, iterations, skip_copy_entry))

    def launch_count(self) -> int:
        return int(lib().rekv_launch_count(self._h))

    def get_reps(self, layer: int, n_frames: int) -> torch.Tensor:
        out = torch.empty((n_frames, self.Hkv * self.D), dtype=torch.float32, device=self.device)
        self._check(lib().rekv_get_reps(self._h, layer, n_frames, _ptr(out), self._stream()))
        return out

    def get_page(self, frame: int, layer: int) -> Tuple[torch.Tensor, torch.Tensor]:
        k = torch.empty((self.Hkv, self.Nf, self.D), dtype=torch.bfloat16, device=self.device)
        v = torch.empty_like(k)
        self._check(lib().rekv_get_page(self._h, frame, layer, _ptr(k), _ptr(v), self._stream()))
        return k, v


def score_frames_static(q: torch.Tensor, cu_q: Sequence[int], n_kv_heads: int, reps: torch.Tensor,
                        out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Allocation-free scoring of one layer (see rekv_score_frames_static in include/rekv.h).

    q: bf16 [sum_Nq][H_q][128]; reps: fp32 [n_frames][H_kv*128]; returns fp32 [nQ][n_frames].  The output
    tensor is the caller's (pass `out` to keep this call itself free of allocations)."""
    nQ = len(cu_q) - 1
    if out is None:
        out = torch.empty((nQ, reps.shape[0]), dtype=torch.float32, device=q.device)
    with torch.cuda.device(q.device):
        rc = lib().rekv_score_frames_static(_ptr(q, torch.bfloat16), _cu_array(cu_q), nQ, q.shape[1], n_kv_heads,
                                            q.shape[2], _ptr(reps, torch.float32), reps.shape[0],
                                            _ptr(out, torch.float32), torch.cuda.current_stream(q.device).cuda_stream)
    if rc < 0:
        raise RekvError(rc, (lib().rekv_last_error(None) or b"").decode())
    return out
