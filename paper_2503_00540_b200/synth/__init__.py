"""Seeded synthetic inputs (K/V frames, question queries) for tests and benchmarks.

Thin ctypes binding of the host and device fillers; every element is a pure function of
(seed, tensor, layer, frame, token, head, dim), so the host and device versions agree bit
for bit and no cache ever has to be shipped between them.  No method arithmetic here.
"""
import ctypes
from typing import List

import torch

from .. import _build

K, V, Q = 1, 2, 5
_cpu = None
_cuda = None


def _cpu_lib():
    global _cpu
    if _cpu is None:
        _build.build_synth()
        _cpu = ctypes.CDLL(_build.LIBSYNTH_CPU)
        _cpu.rekv_synth_fill_frame_cpu.argtypes = [ctypes.c_uint64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                                   ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                                   ctypes.c_float, ctypes.c_void_p]
        _cpu.rekv_synth_fill_frame_cpu.restype = None
        _cpu.rekv_synth_fill_q_cpu.argtypes = [ctypes.c_uint64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                               ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
        _cpu.rekv_synth_fill_q_cpu.restype = None
        _cpu.rekv_synth_mix64_c.argtypes = [ctypes.c_uint64]
        _cpu.rekv_synth_mix64_c.restype = ctypes.c_uint64
    return _cpu


def _cuda_lib():
    global _cuda
    if _cuda is None:
        _build.build_synth()
        _cuda = ctypes.CDLL(_build.LIBSYNTH_CUDA)
        _cuda.rekv_synth_fill_frame_cuda.argtypes = [ctypes.c_uint64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                                     ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                                     ctypes.c_float, ctypes.c_void_p, ctypes.c_void_p]
        _cuda.rekv_synth_fill_frame_cuda.restype = ctypes.c_int
        _cuda.rekv_synth_fill_q_cuda.argtypes = [ctypes.c_uint64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                                 ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                                 ctypes.c_void_p]
        _cuda.rekv_synth_fill_q_cuda.restype = ctypes.c_int
    return _cuda


def _stream_ptr(device) -> int:
    return torch.cuda.current_stream(device).cuda_stream


def frame(seed: int, which: int, f: int, n_layers: int, n_tokens: int, n_kv_heads: int, head_dim: int,
          off_scale: float = 0.5, device="cpu", layer0: int = 0, out: torch.Tensor = None) -> torch.Tensor:
    """One frame's K (which=K) or V (which=V): bf16 [n_layers][n_tokens][n_kv_heads][head_dim]."""
    device = torch.device(device)
    shape = (n_layers, n_tokens, n_kv_heads, head_dim)
    if out is None:
        out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    assert out.is_contiguous() and out.numel() == n_layers * n_tokens * n_kv_heads * head_dim
    if device.type == "cpu":
        _cpu_lib().rekv_synth_fill_frame_cpu(seed, which, f, layer0, n_layers, n_tokens, n_kv_heads, head_dim,
                                             off_scale, out.data_ptr())
    else:
        with torch.cuda.device(device):
            rc = _cuda_lib().rekv_synth_fill_frame_cuda(seed, which, f, layer0, n_layers, n_tokens, n_kv_heads,
                                                        head_dim, off_scale, out.data_ptr(), _stream_ptr(device))
        if rc != 0:
            raise RuntimeError(f"synthetic frame fill failed: cudaError {rc}")
    return out


def question(seed: int, qid: int, n_layers: int, n_tokens: int, n_q_heads: int, head_dim: int, device="cpu",
             layer0: int = 0) -> torch.Tensor:
    """One question's queries: bf16 [n_layers][n_tokens][n_q_heads][head_dim]."""
    device = torch.device(device)
    out = torch.empty((n_layers, n_tokens, n_q_heads, head_dim), dtype=torch.bfloat16, device=device)
    if device.type == "cpu":
        _cpu_lib().rekv_synth_fill_q_cpu(seed, qid, layer0, n_layers, n_tokens, n_q_heads, head_dim, out.data_ptr())
    else:
        with torch.cuda.device(device):
            rc = _cuda_lib().rekv_synth_fill_q_cuda(seed, qid, layer0, n_layers, n_tokens, n_q_heads, head_dim,
                                                    out.data_ptr(), _stream_ptr(device))
        if rc != 0:
            raise RuntimeError(f"synthetic question fill failed: cudaError {rc}")
    return out


def question_lengths(seed: int, n_questions: int, lo: int, hi: int) -> List[int]:
    """Seeded question lengths, uniform on [lo, hi]."""
    lib = _cpu_lib()
    return [lo + int(lib.rekv_synth_mix64_c((seed << 20) ^ (0xA11CE + i)) % (hi - lo + 1))
            for i in range(n_questions)]
