"""Disk tier: a context written to a file and read back (possibly by another process) answers questions with the
same bits, keeps its accounting, and takes further frames."""
import pytest
import torch

from paper_2503_00540_b200 import rekv, synth
from tests import harness as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape,flags,extra", [
    (H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=30, W=4, k=6), 0, {}),
    (H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=30, W=4, k=6, tail=8, seed=540), 0, {}),
    (H.Shape(L=1, Hq=4, Hkv=1, Nf=37, T=20, W=2, k=5, tail=4, seed=7), rekv.FLAG_HOST_FP8, {}),
    (H.Shape(L=2, Hq=8, Hkv=2, Nf=16, T=40, W=4, k=8, b=2), 0, dict(ext_embed_dim=64)),
])
def test_save_then_load_gives_the_same_context(tmp_path, shape, flags, extra):
    s = shape
    g = H.build_gpu(s, max_questions=2, max_q_tokens=48, max_frames=s.T + 2, flags=flags, **extra)
    if extra:
        emb = torch.randn(s.T, 64, generator=torch.Generator().manual_seed(1)).cuda()
        for f in range(s.T):
            g.set_frame_embedding(f, emb[f])
    q, cu = H.questions(s, [16, 32], device="cuda")
    before = g.question(q, cu, s.k, s.T).clone()
    path = str(tmp_path / "ctx.rekv")
    g.save(path)
    h = rekv.ReKV.load(path)
    st_g, st_h = g.stats(), h.stats()
    for field in ("frames", "kv_bytes_hbm", "kv_bytes_host", "kv_bytes_logical", "rep_bytes", "page_bytes"):
        assert getattr(st_g, field) == getattr(st_h, field), field
    for l in range(s.L):
        assert torch.equal(g.get_reps(l, s.T), h.get_reps(l, s.T))
        for f in (0, s.T // 2, s.T - 1):
            (k1, v1), (k2, v2) = g.get_page(f, l), h.get_page(f, l)
            assert torch.equal(k1, k2) and torch.equal(v1, v2)
    after = h.question(q, cu, s.k, s.T)
    h.check_status()
    assert torch.equal(after, before)
    if extra:
        qe = torch.randn(2, 64, generator=torch.Generator().manual_seed(2)).cuda()
        i1, k1, s1 = g.retrieve_external(qe, s.k, s.T, 0.5, want_scores=True)
        i2, k2, s2 = h.retrieve_external(qe, s.k, s.T, 0.5, want_scores=True)
        assert k1 == k2 and torch.equal(i1, i2) and torch.equal(s1, s2)
    # both take the next frame and still agree
    kf = synth.frame(s.seed, synth.K, s.T, s.L, s.Nf, s.Hkv, s.D, s.off_scale, device="cuda")
    vf = synth.frame(s.seed, synth.V, s.T, s.L, s.Nf, s.Hkv, s.D, s.off_scale, device="cuda")
    assert g.append_frame(kf, vf) == s.T and h.append_frame(kf, vf) == s.T
    assert torch.equal(g.question(q, cu, s.k, s.T + 1), h.question(q, cu, s.k, s.T + 1))
    g.check_status()
    h.check_status()
    g.close()
    h.close()


def test_load_rejects_what_is_not_a_saved_context(tmp_path):
    p = tmp_path / "junk.bin"
    p.write_bytes(b"not a context" * 10)
    with pytest.raises(rekv.RekvError) as e:
        rekv.ReKV.load(str(p))
    assert e.value.code == rekv.ERR_ARG
    with pytest.raises(rekv.RekvError):
        rekv.ReKV.load(str(tmp_path / "missing.rekv"))
    # a truncated file
    s = H.TINY
    g = H.build_gpu(s)
    full = tmp_path / "full.rekv"
    g.save(str(full))
    g.close()
    cut = tmp_path / "cut.rekv"
    cut.write_bytes(full.read_bytes()[: full.stat().st_size // 2])
    with pytest.raises(rekv.RekvError):
        rekv.ReKV.load(str(cut))
