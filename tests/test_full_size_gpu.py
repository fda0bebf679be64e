"""Parity at the full workload sizes, in the launch configuration the benchmark times.

The caches are far too large for the oracle to walk whole, so it checks sampled layers: for each
sampled layer the oracle pools every frame (regenerated from the seeded generator), scores and
selects, regenerates only the frames it selected, gathers them and attends.  The CUDA library runs
the whole workload (all layers) through the C ABI; the sampled layers are compared element by
element with the same rules as the small cases.
"""
import gc

import pytest
import torch

from oracle import rekv_oracle as orc
from paper_2503_00540_b200 import rekv, synth
from tests import harness as H

pytestmark = pytest.mark.gpu


def _host_gb_available() -> float:
    for line in open("/proc/meminfo"):
        if line.startswith("MemAvailable"):
            return int(line.split()[1]) / 1e6
    return 0.0


def _fill(g: rekv.ReKV, s: H.Shape, n_frames: int):
    k = torch.empty((s.L, s.Nf, s.Hkv, s.D), dtype=torch.bfloat16, device="cuda")
    v = torch.empty_like(k)
    for f in range(n_frames):
        synth.frame(s.seed, synth.K, f, s.L, s.Nf, s.Hkv, s.D, s.off_scale, device="cuda", out=k)
        synth.frame(s.seed, synth.V, f, s.L, s.Nf, s.Hkv, s.D, s.off_scale, device="cuda", out=v)
        assert g.append_frame(k, v) == f


def _oracle_layer(s: H.Shape, layer: int, n_frames: int) -> torch.Tensor:
    """Representatives of one layer for frames [0, n_frames), by the oracle, from regenerated keys."""
    reps = torch.empty(n_frames, s.Hkv * s.D, dtype=torch.float32)
    for f in range(n_frames):
        reps[f] = orc.pool_frame(synth.frame(s.seed, synth.K, f, 1, s.Nf, s.Hkv, s.D, s.off_scale, layer0=layer)[0])
    return reps


def _sampled_parity(g: rekv.ReKV, s: H.Shape, lengths, layers, n_visible, first_qid=0, widened=False):
    nQ = len(lengths)
    q_gpu, cu = H.questions(s, lengths, device="cuda", first_id=first_qid)
    q_cpu = q_gpu.cpu()
    idx, k_eff, scores = g.retrieve(q_gpu, cu, s.k, n_visible, want_scores=True)
    assert k_eff == min(s.k, n_visible - s.W)
    idx_mix = idx.clone()
    ref = {}
    for l in layers:
        reps = _oracle_layer(s, l, n_visible)
        H.assert_close_rel(g.get_reps(l, n_visible), reps, f"reps layer {l}")
        for i in range(nQ):
            ql = q_cpu[l, cu[i]:cu[i + 1]].contiguous()
            sc = orc.score(ql, reps, s.Hkv)
            sel, ke, gap = orc.select(sc, n_visible, s.W, s.k)
            H.assert_close_rel(scores[l, i][None], sc[None], f"scores l{l} q{i}")
            H.assert_indices(idx[l, i], sel, sc, gap, k_eff, f"idx l{l} q{i}")
            idx_mix[l, i] = sel.cuda()
            ref[(l, i)] = sel
    # steps 4-5 on the oracle's selection in the sampled layers (the library's own elsewhere)
    ncf, k_ctx, v_ctx = g.gather(idx_mix, nQ, s.k, n_visible, materialize=True)
    out = g.attend(q_gpu, cu)
    g.check_status()
    worst = (0.0, 0.0, 0.0)
    for l in layers:
        for i in range(nQ):
            frames = ref[(l, i)][:k_eff].tolist() + list(range(n_visible - min(s.W, n_visible), n_visible))
            ck = torch.stack([synth.frame(s.seed, synth.K, f, 1, s.Nf, s.Hkv, s.D, s.off_scale, layer0=l)[0] for f in frames])
            cv = torch.stack([synth.frame(s.seed, synth.V, f, 1, s.Nf, s.Hkv, s.D, s.off_scale, layer0=l)[0] for f in frames])
            sub = torch.arange(k_eff, dtype=torch.int32)
            kc = orc.gather(ck.contiguous(), sub, k_eff, len(frames), min(s.W, n_visible))
            vc = orc.gather(cv.contiguous(), sub, k_eff, len(frames), min(s.W, n_visible))
            assert torch.equal(k_ctx[l, i].cpu(), kc), f"gathered K differs: layer {l} question {i}"
            assert torch.equal(v_ctx[l, i].cpu(), vc), f"gathered V differs: layer {l} question {i}"
            o, _, _ = orc.attend(q_cpu[l, cu[i]:cu[i + 1]].contiguous(), kc, vc)
            r = H.assert_attention(out[l, cu[i]:cu[i + 1]], o, f"attention l{l} q{i}")
            worst = tuple(max(a, b) for a, b in zip(worst, r))
    del k_ctx, v_ctx
    if widened:
        worst_full = _widened_rows(g, s, lengths, layers, n_visible, q_gpu, cu, idx, idx_mix, ref, k_eff, out)
        return worst, worst_full
    return worst


def _widened_rows(g, s, lengths, layers, n_visible, q_gpu, cu, idx, idx_mix, ref, k_eff, out_plain):
    """The rows built beyond the five steps, at the same full size: the layer-sequential calls against the
    all-layer result, and Eq. 3 in full (own K/V, rotary embedding at consecutive positions) against the oracle
    in the sampled layers, on the oracle's selection."""
    nQ = len(lengths)
    q_cpu = q_gpu.cpu()
    # layer-sequential calls use the library's own selection: same indices, same attention where it is the oracle's
    for l in layers:
        idx_l = torch.empty((nQ, s.k), dtype=torch.int32, device="cuda")
        out_l = g.question_layer(l, q_gpu[l], cu, s.k, n_visible, idx=idx_l)
        assert torch.equal(idx_l, idx[l])
        if torch.equal(idx[l], idx_mix[l]):
            d = (out_l.float() - out_plain[l].float()).abs()
            assert d.max().item() <= 4e-3, f"layer call differs from the all-layer call in layer {l}: {d.max().item()}"
    g.check_status()
    # Eq. 3 in full
    ks, vs, cus = H.self_kv(s, lengths, device="cuda")
    g.gather(idx_mix, nQ, s.k, n_visible)
    out = g.attend_full(q_gpu, ks, vs, cu, cus)
    g.check_status()
    theta = float(g.cfg.rope_theta)
    worst = (0.0, 0.0, 0.0)
    for l in layers:
        for i in range(nQ):
            frames = ref[(l, i)][:k_eff].tolist() + list(range(n_visible - min(s.W, n_visible), n_visible))
            ck = torch.stack([synth.frame(s.seed, synth.K, f, 1, s.Nf, s.Hkv, s.D, s.off_scale, layer0=l)[0] for f in frames])
            cv = torch.stack([synth.frame(s.seed, synth.V, f, 1, s.Nf, s.Hkv, s.D, s.off_scale, layer0=l)[0] for f in frames])
            sub = torch.arange(k_eff, dtype=torch.int32)
            kc = orc.gather(ck.contiguous(), sub, k_eff, len(frames), min(s.W, n_visible))
            vc = orc.gather(cv.contiguous(), sub, k_eff, len(frames), min(s.W, n_visible))
            o, _ = orc.attend_full(q_cpu[l, cu[i]:cu[i + 1]].contiguous(), kc, vc, ks[l, cus[i]:cus[i + 1]].cpu().contiguous(),
                                   vs[l, cus[i]:cus[i + 1]].cpu().contiguous(), theta)
            r = H.assert_attention(out[l, cu[i]:cu[i + 1]], o, f"Eq. 3 in full l{l} q{i}")
            worst = tuple(max(a, b) for a, b in zip(worst, r))
    return worst


def test_config2_7b_hbm_resident_1800_frames():
    """28 layers, 28/4 heads, 1800 x 196-token frames (20.2 GB in HBM), question 32, window 8, top-k 64."""
    s = H.Shape(L=28, Hq=28, Hkv=4, Nf=196, T=1800, W=8, k=64, seed=2503)
    g = rekv.ReKV(s.L, s.Hq, s.Hkv, s.D, s.Nf, s.T, s.W, max_q_tokens=32, max_topk=64, flags=rekv.FLAG_TIMING,
                  max_self_tokens=32, rope_theta=1e6)
    _fill(g, s, s.T)
    st = g.stats()
    assert st.kv_bytes_hbm == st.kv_bytes_logical == orc.kv_cache_bytes(28, 1800, 196, 4, 128)
    assert round(st.kv_bytes_logical / 2**30, 1) == 18.8  # the appendix's worked value
    worst, worst_full = _sampled_parity(g, s, [32], layers=[0, 13, 27], n_visible=s.T, widened=True)
    print("config 2 attention max/mean/rel:", worst, "Eq. 3 in full with rotary embedding:", worst_full)
    g.close()


def test_config4_streaming_append_with_batched_questions():
    """Frames appended into a 7B-shape stream that grows to its 1800 frames, interleaved with batches of 16
    questions of 24..64 tokens, each with its own top-32 retrieval; questions see exactly the frames appended so
    far.  1780 frames are there when the checked part starts; two rounds of ten appends and a batch follow (the
    shape of the paper's streaming speed run: questions scattered through a one-hour stream at 0.5 fps)."""
    s = H.Shape(L=28, Hq=28, Hkv=4, Nf=196, T=1800, W=8, k=32, seed=540)
    lengths = synth.question_lengths(s.seed, 16, 24, 64)
    g = rekv.ReKV(s.L, s.Hq, s.Hkv, s.D, s.Nf, s.T, s.W, max_q_tokens=sum(lengths), max_topk=32, max_questions=16)
    first = s.T - 20
    _fill(g, s, first)
    k = torch.empty((s.L, s.Nf, s.Hkv, s.D), dtype=torch.bfloat16, device="cuda")
    v = torch.empty_like(k)
    reps_seen = {}   # the oracle's representatives grow with the stream: frames pooled once per layer
    for batch in range(2):
        for f in range(first + 10 * batch, first + 10 + 10 * batch):
            synth.frame(s.seed, synth.K, f, s.L, s.Nf, s.Hkv, s.D, s.off_scale, device="cuda", out=k)
            synth.frame(s.seed, synth.V, f, s.L, s.Nf, s.Hkv, s.D, s.off_scale, device="cuda", out=v)
            assert g.append_frame(k, v) == f
        n_vis = first + 10 + 10 * batch
        sub = [0, 5, 15] if batch == 0 else [3, 9]
        # the oracle checks a subset of the 16 questions in two layers; the library runs all 16
        q_gpu, cu = H.questions(s, lengths, device="cuda", first_id=100 * batch)
        out_all = g.question(q_gpu, cu, s.k, n_vis)
        g.check_status()
        idx, k_eff, scores = g.retrieve(q_gpu, cu, s.k, n_vis, want_scores=True)
        assert k_eff == s.k
        q_cpu = q_gpu.cpu()
        for l in (1, 20):
            old = reps_seen.get(l)
            n_old = 0 if old is None else old.shape[0]
            new = torch.stack([orc.pool_frame(synth.frame(s.seed, synth.K, f, 1, s.Nf, s.Hkv, s.D, s.off_scale, layer0=l)[0])
                               for f in range(n_old, n_vis)])
            reps = new if old is None else torch.cat([old, new])
            reps_seen[l] = reps
            H.assert_close_rel(g.get_reps(l, n_vis), reps, f"reps batch {batch} layer {l}")
            for i in sub:
                ql = q_cpu[l, cu[i]:cu[i + 1]].contiguous()
                sc = orc.score(ql, reps, s.Hkv)
                sel, ke, gap = orc.select(sc, n_vis, s.W, s.k)
                H.assert_close_rel(scores[l, i][None], sc[None], f"scores l{l} q{i}")
                H.assert_indices(idx[l, i], sel, sc, gap, k_eff, f"idx l{l} q{i}")
                if torch.equal(idx[l, i].cpu(), sel):
                    frames = sel[:k_eff].tolist() + list(range(n_vis - s.W, n_vis))
                    ck = torch.stack([synth.frame(s.seed, synth.K, f, 1, s.Nf, s.Hkv, s.D, s.off_scale, layer0=l)[0] for f in frames])
                    cv = torch.stack([synth.frame(s.seed, synth.V, f, 1, s.Nf, s.Hkv, s.D, s.off_scale, layer0=l)[0] for f in frames])
                    subi = torch.arange(k_eff, dtype=torch.int32)
                    kc = orc.gather(ck.contiguous(), subi, k_eff, len(frames), s.W)
                    vc = orc.gather(cv.contiguous(), subi, k_eff, len(frames), s.W)
                    o, _, _ = orc.attend(ql, kc, vc)
                    H.assert_attention(out_all[l, cu[i]:cu[i + 1]], o, f"attention batch {batch} l{l} q{i}")
    assert g.stats().frames == s.T
    g.close()


def _offloaded(s: H.Shape, q_tokens: int, layers, need_gb: float):
    if _host_gb_available() < need_gb + 40:
        pytest.skip(f"needs {need_gb:.0f} GB of pinned host memory plus headroom")
    g = rekv.ReKV(s.L, s.Hq, s.Hkv, s.D, s.Nf, s.T, s.W, hbm_tail_frames=s.tail, max_q_tokens=q_tokens, max_topk=s.k)
    _fill(g, s, s.T)
    st = g.stats()
    assert st.kv_bytes_host == st.kv_bytes_logical == orc.kv_cache_bytes(s.L, s.T, s.Nf, s.Hkv, s.D)
    assert st.kv_bytes_hbm == st.kv_bytes_logical * s.tail // s.T
    worst = _sampled_parity(g, s, [q_tokens], layers=layers, n_visible=s.T)
    g.check_status()
    st = g.stats()
    # every selected frame outside the HBM tail crossed the host link exactly once
    assert 0 < st.last_link_bytes <= s.L * s.k * st.page_bytes
    g.close()
    del g
    gc.collect()
    return worst


def test_config3_7b_offloaded_10800_frames():
    """3-hour stream at 1 fps: 10800 frames (121 GB) in pinned host memory, last 64 frames in HBM."""
    s = H.Shape(L=28, Hq=28, Hkv=4, Nf=196, T=10800, W=8, k=64, tail=64, seed=7)
    print("config 3 attention max/mean/rel:", _offloaded(s, 32, layers=[2, 26], need_gb=121.4))


def test_config5_72b_offloaded_1800_frames():
    """72B shape: 80 layers, 64/8 heads, 1800 frames (116 GB) in pinned host memory, last 32 frames in HBM."""
    s = H.Shape(L=80, Hq=64, Hkv=8, Nf=196, T=1800, W=8, k=32, tail=32, seed=2503)
    print("config 5 attention max/mean/rel:", _offloaded(s, 64, layers=[0, 79], need_gb=115.6))
