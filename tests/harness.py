"""Shared pieces of the parity tests: build the same seeded stream for the CUDA library and for the
CPU oracle, and the comparison rules (tolerances are the ones the tests state and the design derives)."""
from dataclasses import dataclass
from typing import List

import torch

from oracle import rekv_oracle as orc
from paper_2503_00540_b200 import synth
from paper_2503_00540_b200.rekv import ReKV

REL_TOL = 1e-4           # representatives and scores, fp32
ATT_MAX_ABS = 2e-2       # attention output, bf16 vs the oracle's float
ATT_MEAN_ABS = 2e-3
TIE_GAP = 1e-4           # below this gap between the k-th and (k+1)-th score several selections are correct


@dataclass
class Shape:
    L: int
    Hq: int
    Hkv: int
    Nf: int
    T: int
    W: int
    k: int
    seed: int = 2503
    off_scale: float = 0.5
    D: int = 128
    tail: int = 0
    b: int = 1


TINY = Shape(L=1, Hq=8, Hkv=2, Nf=16, T=64, W=4, k=8, off_scale=0.0)


def build_gpu(s: Shape, max_questions: int = 1, max_q_tokens: int = 64, max_frames: int = None, flags: int = 0,
              n_frames: int = None, **extra) -> ReKV:
    r = ReKV(s.L, s.Hq, s.Hkv, s.D, s.Nf, max_frames or s.T, s.W, hbm_tail_frames=s.tail, max_q_tokens=max_q_tokens,
             max_topk=max(s.k, s.b), max_questions=max_questions, flags=flags, block_frames=s.b, **extra)
    for f in range(s.T if n_frames is None else n_frames):
        k = synth.frame(s.seed, synth.K, f, s.L, s.Nf, s.Hkv, s.D, s.off_scale, device="cuda")
        v = synth.frame(s.seed, synth.V, f, s.L, s.Nf, s.Hkv, s.D, s.off_scale, device="cuda")
        assert r.append_frame(k, v) == f
    return r


def build_oracle(s: Shape, n_frames: int = None) -> orc.OracleCache:
    c = orc.OracleCache(s.L, s.Hq, s.Hkv, s.D, s.Nf, s.W, block=s.b)
    for f in range(s.T if n_frames is None else n_frames):
        c.append(synth.frame(s.seed, synth.K, f, s.L, s.Nf, s.Hkv, s.D, s.off_scale),
                 synth.frame(s.seed, synth.V, f, s.L, s.Nf, s.Hkv, s.D, s.off_scale))
    return c


def self_kv(s: Shape, lengths: List[int], device="cpu", first_id: int = 0):
    """Seeded K/V of the questions' own tokens, packed [L][sum][H_kv][D], and their prefix sums."""
    ks = [synth.frame(s.seed, synth.K, 1_000_000 + first_id + i, s.L, n, s.Hkv, s.D, 0.0, device=device)
          for i, n in enumerate(lengths)]
    vs = [synth.frame(s.seed, synth.V, 1_000_000 + first_id + i, s.L, n, s.Hkv, s.D, 0.0, device=device)
          for i, n in enumerate(lengths)]
    cu = [0]
    for n in lengths:
        cu.append(cu[-1] + n)
    return torch.cat(ks, dim=1).contiguous(), torch.cat(vs, dim=1).contiguous(), cu


def questions(s: Shape, lengths: List[int], device="cpu", first_id: int = 0):
    """Packed q [L][sum][Hq][D] and cu_q for seeded questions of the given lengths."""
    qs = [synth.question(s.seed, first_id + i, s.L, n, s.Hq, s.D, device=device) for i, n in enumerate(lengths)]
    cu = [0]
    for n in lengths:
        cu.append(cu[-1] + n)
    return torch.cat(qs, dim=1).contiguous(), cu


def assert_close_rel(got: torch.Tensor, ref: torch.Tensor, what: str):
    """Row-wise: ||got-ref||_2 <= 1e-4 ||ref||_2, and element-wise |got-ref| <= 1e-4 max(|ref|, rms(ref))."""
    got = got.double().cpu().reshape(-1, got.shape[-1])
    ref = ref.double().cpu().reshape(-1, ref.shape[-1])
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    num = (got - ref).norm(dim=1)
    den = ref.norm(dim=1).clamp_min(1e-30)
    assert (num <= REL_TOL * den).all(), f"{what}: row-wise rel err {(num / den).max().item():.3e}"
    rms = ref.pow(2).mean(dim=1, keepdim=True).sqrt()
    bound = REL_TOL * torch.maximum(ref.abs(), rms)
    assert ((got - ref).abs() <= bound).all(), f"{what}: element-wise err {((got - ref).abs() / bound).max().item():.3e} x bound"


def assert_indices(gpu_idx: torch.Tensor, ref_idx: torch.Tensor, ref_scores: torch.Tensor, gap: float, k_eff: int,
                   what: str):
    """Bit-exact, except inside a near-tie (oracle gap < 1e-4): then the sets may differ only on frames whose
    oracle score is within 1e-4 of the k-th best, and the list must still be valid (ascending, distinct)."""
    g = gpu_idx.cpu().tolist()
    r = ref_idx.tolist()
    assert g[k_eff:] == [-1] * (len(g) - k_eff), what
    if g == r:
        return
    assert gap < TIE_GAP, f"{what}: selection differs although the oracle's gap is {gap:.3e}"
    gs, rs = g[:k_eff], r[:k_eff]
    assert gs == sorted(set(gs)), f"{what}: not ascending/distinct"
    kth = min(ref_scores[i].item() for i in rs)
    for f in set(gs) ^ set(rs):
        assert abs(ref_scores[f].item() - kth) < TIE_GAP, f"{what}: frame {f} is not inside the near-tie"


def assert_attention(got_bf16: torch.Tensor, ref_f32: torch.Tensor, what: str):
    d = (got_bf16.float().cpu() - ref_f32).abs()
    rel = (got_bf16.float().cpu() - ref_f32).norm() / ref_f32.norm().clamp_min(1e-30)
    assert d.max().item() <= ATT_MAX_ABS, f"{what}: max abs err {d.max().item():.3e} (normwise rel {rel:.3e})"
    assert d.mean().item() <= ATT_MEAN_ABS, f"{what}: mean abs err {d.mean().item():.3e} (normwise rel {rel:.3e})"
    assert rel.item() <= 2e-2, f"{what}: normwise rel err {rel.item():.3e}"
    return d.max().item(), d.mean().item(), rel.item()
