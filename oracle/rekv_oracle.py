"""ctypes binding of the C++ oracle plus a small driver that walks the five steps.

TEST INFRASTRUCTURE ONLY (see rekv_oracle.cpp).  All tensors are CPU torch tensors;
bf16 data is passed as raw 16-bit words.  Nothing here is imported by the CUDA package.
"""
import ctypes
import math
from typing import List, Optional, Sequence, Tuple

import torch

from . import build as _build

_lib = ctypes.CDLL(_build.build())

_u16p = ctypes.c_void_p
_lib.oracle_pool_frame.argtypes = [_u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
_lib.oracle_pool_frame.restype = None
_lib.oracle_question_vector.argtypes = [_u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                        ctypes.c_void_p]
_lib.oracle_question_vector.restype = None
_lib.oracle_score.argtypes = [_u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                              ctypes.c_int, ctypes.c_void_p]
_lib.oracle_score.restype = None
_lib.oracle_score_blocks.argtypes = [_u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                     ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
_lib.oracle_score_blocks.restype = None
_lib.oracle_select.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                               ctypes.POINTER(ctypes.c_double)]
_lib.oracle_select.restype = ctypes.c_int
_lib.oracle_gather.argtypes = [_u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_int,
                               ctypes.c_int, ctypes.c_int, _u16p]
_lib.oracle_gather.restype = ctypes.c_int
_lib.oracle_attend.argtypes = [_u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, _u16p, _u16p,
                               ctypes.c_long, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
_lib.oracle_attend.restype = None
_lib.oracle_score_external.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_double, ctypes.c_void_p]
_lib.oracle_score_external.restype = None
_lib.oracle_e4m3_encode.argtypes = [ctypes.c_float]
_lib.oracle_e4m3_encode.restype = ctypes.c_uint8
_lib.oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
_lib.oracle_e4m3_decode.restype = ctypes.c_double
_lib.oracle_fp8_roundtrip.argtypes = [_u16p, ctypes.c_long, ctypes.c_int, _u16p, ctypes.c_void_p]
_lib.oracle_fp8_roundtrip.restype = None
_lib.oracle_rope.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_long, ctypes.c_double, ctypes.c_void_p]
_lib.oracle_rope.restype = None
_lib.oracle_attend_full.argtypes = [_u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, _u16p, _u16p,
                                    ctypes.c_long, _u16p, _u16p, ctypes.c_int, ctypes.c_double, ctypes.c_int, ctypes.c_void_p,
                                    ctypes.c_void_p]
_lib.oracle_attend_full.restype = None
_lib.oracle_kv_cache_bytes.argtypes = [ctypes.c_int, ctypes.c_long, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_int]
_lib.oracle_kv_cache_bytes.restype = ctypes.c_double


def _chk(t: torch.Tensor, dtype) -> torch.Tensor:
    assert t.device.type == "cpu" and t.dtype == dtype and t.is_contiguous(), (t.device, t.dtype)
    return t


def pool_frame(k: torch.Tensor) -> torch.Tensor:
    """k: bf16 [N_f][H_kv][D] (one layer of one frame) -> float32 [H_kv*D]."""
    _chk(k, torch.bfloat16)
    n_tokens, n_kv, d = k.shape
    rep = torch.empty(n_kv * d, dtype=torch.float32)
    _lib.oracle_pool_frame(k.data_ptr(), n_tokens, n_kv, d, rep.data_ptr())
    return rep


def question_vector(q: torch.Tensor, n_kv_heads: int) -> torch.Tensor:
    """q: bf16 [N_q][H_q][D] -> float64 [H_kv*D]."""
    _chk(q, torch.bfloat16)
    n_q, n_qh, d = q.shape
    qa = torch.empty(n_kv_heads * d, dtype=torch.float64)
    _lib.oracle_question_vector(q.data_ptr(), n_q, n_qh, n_kv_heads, d, qa.data_ptr())
    return qa


def score(q: torch.Tensor, reps: torch.Tensor, n_kv_heads: int) -> torch.Tensor:
    """q: bf16 [N_q][H_q][D]; reps: float32 [T][H_kv*D] -> float32 [T]."""
    _chk(q, torch.bfloat16)
    _chk(reps, torch.float32)
    n_q, n_qh, d = q.shape
    n_frames = reps.shape[0]
    assert reps.shape[1] == n_kv_heads * d
    out = torch.empty(n_frames, dtype=torch.float32)
    _lib.oracle_score(q.data_ptr(), n_q, n_qh, n_kv_heads, d, reps.data_ptr(), n_frames, out.data_ptr())
    return out


def score_blocks(q: torch.Tensor, reps: torch.Tensor, n_kv_heads: int, n_blocks: int, b: int) -> torch.Tensor:
    """Cosine score of each complete block of b frames (block vector = mean of its frame vectors) -> float32 [n_blocks]."""
    _chk(q, torch.bfloat16)
    _chk(reps, torch.float32)
    n_q, n_qh, d = q.shape
    assert reps.shape[0] >= n_blocks * b and reps.shape[1] == n_kv_heads * d
    out = torch.empty(n_blocks, dtype=torch.float32)
    _lib.oracle_score_blocks(q.data_ptr(), n_q, n_qh, n_kv_heads, d, reps.data_ptr(), n_blocks, b, out.data_ptr())
    return out


def score_external(q_emb: torch.Tensor, embs: torch.Tensor, tau: float, n_items: int = None, b: int = 1) -> torch.Tensor:
    """Eq. 2 with its temperature on external embeddings.  q_emb: float32 [E]; embs: float32 [T][E];
    n_items frames (b == 1) or complete blocks of b frames -> float32 [n_items]."""
    _chk(q_emb, torch.float32)
    _chk(embs, torch.float32)
    n_items = embs.shape[0] // b if n_items is None else n_items
    assert embs.shape[1] == q_emb.shape[0] and embs.shape[0] >= n_items * b
    out = torch.empty(n_items, dtype=torch.float32)
    _lib.oracle_score_external(q_emb.data_ptr(), embs.data_ptr(), q_emb.shape[0], n_items, b, tau, out.data_ptr())
    return out


def retrieve_external(q_emb: torch.Tensor, embs: torch.Tensor, tau: float, top_k: int, n_visible: int, window: int,
                      b: int = 1):
    """External retrieval of one question: one selection for all layers.
    -> (scores float32, idx int32 [top_k] ascending frames padded with -1, k_eff, gap)."""
    if b == 1:
        s = score_external(q_emb, embs[:n_visible].contiguous(), tau)
        i, k_eff, g = select(s, n_visible, window, top_k)
        return s, i, k_eff, g
    n_blocks, k_blocks, _ = block_geometry(n_visible, window, b, top_k)
    s = score_external(q_emb, embs[:n_visible].contiguous(), tau, n_blocks, b)
    bi, kb, g = select(s, n_blocks, 0, top_k // b)
    assert kb == k_blocks
    i = torch.full((top_k,), -1, dtype=torch.int32)
    for j in range(kb):
        for f in range(b):
            i[j * b + f] = int(bi[j]) * b + f
    return s, i, kb * b, g


def block_geometry(n_visible: int, window: int, b: int, top_k: int):
    """Block retrieval geometry: only complete blocks of the candidate frames [0, n_visible - window) can be
    retrieved; every frame after the last complete block is part of the context (the window plus the frames
    that do not fill a block yet).  -> (n_blocks, k_blocks, window_eff)."""
    n_cand = max(n_visible - window, 0)
    n_blocks = n_cand // b
    k_blocks = min(top_k // b, n_blocks)
    return n_blocks, k_blocks, n_visible - n_blocks * b


def select(scores: torch.Tensor, n_visible: int, window: int, k: int) -> Tuple[torch.Tensor, int, float]:
    """-> (idx int32 [k] ascending, padded with -1; k_eff; gap between last kept and best rejected)."""
    _chk(scores, torch.float32)
    assert scores.numel() >= max(n_visible - window, 0)
    idx = torch.empty(max(k, 0), dtype=torch.int32)
    gap = ctypes.c_double(0.0)
    k_eff = _lib.oracle_select(scores.data_ptr(), n_visible, window, k, idx.data_ptr(), ctypes.byref(gap))
    return idx, k_eff, gap.value


def gather(cache: torch.Tensor, idx: torch.Tensor, k_eff: int, n_visible: int, window: int) -> torch.Tensor:
    """cache: bf16 [T][N_f][H_kv][D] (one layer, K or V) -> bf16 [H_kv][n_ctx][D]."""
    _chk(cache, torch.bfloat16)
    _chk(idx, torch.int32)
    _, n_tokens, n_kv, d = cache.shape
    n_frames_ctx = k_eff + (n_visible - max(n_visible - window, 0))
    ctx = torch.empty(n_kv, n_frames_ctx * n_tokens, d, dtype=torch.bfloat16)
    got = _lib.oracle_gather(cache.data_ptr(), n_tokens, n_kv, d, idx.data_ptr(), k_eff, n_visible, window,
                             ctx.data_ptr())
    assert got == n_frames_ctx
    return ctx


def attend(q: torch.Tensor, k_ctx: torch.Tensor, v_ctx: torch.Tensor, want_probs: bool = False):
    """q: bf16 [N_q][H_q][D]; k_ctx, v_ctx: bf16 [H_kv][n_ctx][D].
    -> (out float32 [N_q][H_q][D], out bf16 same shape, probs float64 [N_q][H_q][n_ctx] or None)."""
    _chk(q, torch.bfloat16)
    _chk(k_ctx, torch.bfloat16)
    _chk(v_ctx, torch.bfloat16)
    n_q, n_qh, d = q.shape
    n_kv, n_ctx, _ = k_ctx.shape
    out = torch.empty(n_q, n_qh, d, dtype=torch.float32)
    out_b = torch.empty(n_q, n_qh, d, dtype=torch.bfloat16)
    probs = torch.empty(n_q, n_qh, n_ctx, dtype=torch.float64) if want_probs else None
    _lib.oracle_attend(q.data_ptr(), n_q, n_qh, n_kv, d, k_ctx.data_ptr(), v_ctx.data_ptr(), n_ctx, out.data_ptr(),
                       out_b.data_ptr(), probs.data_ptr() if want_probs else None)
    return out, out_b, probs


def e4m3_encode(x: float) -> int:
    return int(_lib.oracle_e4m3_encode(x))


def e4m3_decode(code: int) -> float:
    return float(_lib.oracle_e4m3_decode(code))


def fp8_roundtrip(x: torch.Tensor, want_scales: bool = False):
    """x: bf16 [..., 128]: every row through the quantised host tier (E4M3 codes + one float scale) and back."""
    _chk(x, torch.bfloat16)
    d = x.shape[-1]
    rows = x.numel() // d
    out = torch.empty_like(x)
    scales = torch.empty(rows, dtype=torch.float32) if want_scales else None
    _lib.oracle_fp8_roundtrip(x.data_ptr(), rows, d, out.data_ptr(), scales.data_ptr() if want_scales else None)
    return (out, scales) if want_scales else out


def rope(x: torch.Tensor, pos: int, theta: float) -> torch.Tensor:
    """Rotary embedding of one float64 vector [D] at position pos (pairs i, i + D/2)."""
    _chk(x, torch.float64)
    out = torch.empty_like(x)
    _lib.oracle_rope(x.data_ptr(), x.shape[0], pos, theta, out.data_ptr())
    return out


def attend_full(q: torch.Tensor, k_ctx: torch.Tensor, v_ctx: torch.Tensor, k_self: torch.Tensor, v_self: torch.Tensor,
                rope_theta: float = 0.0, static_ctx: bool = False):
    """The whole of Eq. 3.  q: bf16 [N_q][H_q][D]; k_ctx, v_ctx: bf16 [H_kv][n_ctx][D] (n_ctx may be 0);
    k_self, v_self: bf16 [N_self][H_kv][D], N_self >= N_q.  -> (out float32, out bf16) [N_q][H_q][D].
    static_ctx: the static position variant (every context token at position 0, token s of X at 1 + s)."""
    for t in (q, k_ctx, v_ctx, k_self, v_self):
        _chk(t, torch.bfloat16)
    n_q, n_qh, d = q.shape
    n_kv, n_ctx, _ = k_ctx.shape
    n_self = k_self.shape[0]
    assert n_self >= n_q and k_self.shape == v_self.shape == (n_self, n_kv, d)
    out = torch.empty(n_q, n_qh, d, dtype=torch.float32)
    out_b = torch.empty(n_q, n_qh, d, dtype=torch.bfloat16)
    _lib.oracle_attend_full(q.data_ptr(), n_q, n_qh, n_kv, d, k_ctx.data_ptr(), v_ctx.data_ptr(), n_ctx,
                            k_self.data_ptr(), v_self.data_ptr(), n_self, rope_theta, 1 if static_ctx else 0, out.data_ptr(),
                            out_b.data_ptr())
    return out, out_b


def kv_cache_bytes(n_layers: int, n_frames: int, tokens_per_frame: int, n_kv_heads: int, head_dim: int,
                   bytes_per_element: int = 2) -> float:
    return _lib.oracle_kv_cache_bytes(n_layers, n_frames, tokens_per_frame, n_kv_heads, head_dim, bytes_per_element)


class OracleCache:
    """Holds a (small) stream's K/V token-major and walks the five steps per layer and question.

    k_frames / v_frames: bf16 [T][L][N_f][H_kv][D] -- frame f as the decoder emitted it.
    """

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, tokens_per_frame: int,
                 window: int, block: int = 1):
        self.L, self.Hq, self.Hkv, self.D, self.Nf, self.W = (n_layers, n_q_heads, n_kv_heads, head_dim,
                                                              tokens_per_frame, window)
        self.b = block
        self.k_frames: List[torch.Tensor] = []
        self.v_frames: List[torch.Tensor] = []
        self.reps: List[torch.Tensor] = []  # per frame: float32 [L][D']

    def append(self, k: torch.Tensor, v: torch.Tensor) -> int:
        """k, v: bf16 [L][N_f][H_kv][D]."""
        assert tuple(k.shape) == (self.L, self.Nf, self.Hkv, self.D)
        self.k_frames.append(k.contiguous())
        self.v_frames.append(v.contiguous())
        self.reps.append(torch.stack([pool_frame(k[l].contiguous()) for l in range(self.L)]))
        return len(self.k_frames) - 1

    def rep_table(self, layer: int, n_visible: Optional[int] = None) -> torch.Tensor:
        n = len(self.reps) if n_visible is None else n_visible
        return torch.stack([self.reps[f][layer] for f in range(n)]).contiguous()

    def retrieve(self, q: torch.Tensor, top_k: int, n_visible: int):
        """q: bf16 [L][N_q][H_q][D] (one question) ->
        (scores float32 [L][n_visible], idx int32 [L][top_k], k_eff, gaps [L])."""
        scores, idxs, gaps = [], [], []
        k_eff = 0
        for l in range(self.L):
            if self.b == 1:
                s = score(q[l].contiguous(), self.rep_table(l, n_visible), self.Hkv)
                i, k_eff, g = select(s, n_visible, self.W, top_k)
            else:
                # block retrieval: score complete blocks, keep top_k/b of them, expand to their frames
                n_blocks, k_blocks, _ = block_geometry(n_visible, self.W, self.b, top_k)
                s = score_blocks(q[l].contiguous(), self.rep_table(l, n_visible), self.Hkv, n_blocks, self.b)
                bi, kb, g = select(s, n_blocks, 0, top_k // self.b)
                assert kb == k_blocks
                k_eff = kb * self.b
                i = torch.full((top_k,), -1, dtype=torch.int32)
                for j in range(kb):
                    for f in range(self.b):
                        i[j * self.b + f] = int(bi[j]) * self.b + f
            scores.append(s)
            idxs.append(i)
            gaps.append(g)
        return torch.stack(scores), torch.stack(idxs), k_eff, gaps

    def window_eff(self, n_visible: int, top_k: int) -> int:
        if self.b == 1:
            return min(self.W, n_visible)
        return block_geometry(n_visible, self.W, self.b, top_k)[2]

    def layer_cache(self, layer: int, which: str) -> torch.Tensor:
        src = self.k_frames if which == "k" else self.v_frames
        return torch.stack([f[layer] for f in src]).contiguous()

    def gather(self, idx: torch.Tensor, k_eff: int, n_visible: int):
        """idx: int32 [L][top_k] -> (k_ctx, v_ctx) bf16 [L][H_kv][n_ctx][D]."""
        ks, vs = [], []
        w_eff = self.window_eff(n_visible, idx.shape[-1])
        for l in range(self.L):
            ks.append(gather(self.layer_cache(l, "k"), idx[l].contiguous(), k_eff, n_visible, w_eff))
            vs.append(gather(self.layer_cache(l, "v"), idx[l].contiguous(), k_eff, n_visible, w_eff))
        return torch.stack(ks), torch.stack(vs)

    def attend(self, q: torch.Tensor, k_ctx: torch.Tensor, v_ctx: torch.Tensor):
        """-> (out float32, out bf16) [L][N_q][H_q][D]."""
        of, ob = [], []
        for l in range(self.L):
            o, b, _ = attend(q[l].contiguous(), k_ctx[l].contiguous(), v_ctx[l].contiguous())
            of.append(o)
            ob.append(b)
        return torch.stack(of), torch.stack(ob)

    def question(self, q: torch.Tensor, top_k: int, n_visible: int):
        scores, idx, k_eff, gaps = self.retrieve(q, top_k, n_visible)
        k_ctx, v_ctx = self.gather(idx, k_eff, n_visible)
        out_f, out_b = self.attend(q, k_ctx, v_ctx)
        return dict(scores=scores, idx=idx, k_eff=k_eff, gaps=gaps, k_ctx=k_ctx, v_ctx=v_ctx, out=out_f,
                    out_bf16=out_b)
