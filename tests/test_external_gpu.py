"""External retrieval (Eq. 2 with its temperature, CLIP-like frame embeddings) on the GPU against the CPU oracle."""
import pytest
import torch

from oracle import rekv_oracle as orc
from paper_2503_00540_b200 import rekv
from tests import harness as H

pytestmark = pytest.mark.gpu


def _embeddings(seed, T, E, nQ):
    """Seeded stand-ins for a CLIP-like encoder's outputs: unit-scale vectors with a shared component (as real
    embeddings have), so that scores are not centred on zero."""
    g = torch.Generator().manual_seed(seed)
    common = torch.randn(E, generator=g)
    embs = (torch.randn(T, E, generator=g) + 0.7 * common).contiguous()
    q = (torch.randn(nQ, E, generator=g) + 0.7 * common).contiguous()
    return embs, q


def _run(s: H.Shape, E, nQ, tau, n_visible=None):
    n_visible = s.T if n_visible is None else n_visible
    g = H.build_gpu(s, max_questions=nQ, max_q_tokens=16 * nQ, ext_embed_dim=E)
    embs, q = _embeddings(s.seed, s.T, E, nQ)
    embs_gpu = embs.cuda()
    for f in range(s.T):
        g.set_frame_embedding(f, embs_gpu[f])
    idx, k_eff, scores = g.retrieve_external(q.cuda(), s.k, n_visible, tau, want_scores=True)
    g.check_status()
    for i in range(nQ):
        rs, ri, rk, gap = orc.retrieve_external(q[i].contiguous(), embs, tau, s.k, n_visible, s.W, s.b)
        assert k_eff == rk
        H.assert_close_rel(scores[i][None], rs[None], f"external scores q{i}")
        for l in range(s.L):  # one selection, present in every layer's block
            H.assert_indices(idx[l, i], ri, rs, gap, k_eff, f"external idx l{l} q{i}")
        assert all(torch.equal(idx[l, i], idx[0, i]) for l in range(s.L))
    # the selection drives the rest of the path unchanged
    ql, cu = H.questions(s, [16] * nQ, device="cuda")
    ncf, _, _ = g.gather(idx, nQ, s.k, n_visible)
    assert ncf == k_eff + (g.geometry(n_visible, s.k)[2])
    out = g.attend(ql, cu)
    g.check_status()
    assert torch.isfinite(out.float()).all()
    g.close()


@pytest.mark.parametrize("tau", [1.0, 0.07])
def test_siglip_sized_embeddings(tau):
    _run(H.Shape(L=3, Hq=8, Hkv=2, Nf=16, T=300, W=8, k=16), 1152, 3, tau)


def test_many_questions_span_several_shared_memory_groups():
    _run(H.Shape(L=2, Hq=8, Hkv=2, Nf=16, T=130, W=4, k=8, seed=540), 1152, 40, 0.5)


def test_small_and_large_dims_and_questions_in_the_past():
    _run(H.Shape(L=1, Hq=8, Hkv=2, Nf=16, T=70, W=4, k=8, seed=7), 4, 2, 1.0)
    _run(H.Shape(L=2, Hq=8, Hkv=2, Nf=16, T=70, W=4, k=8, seed=7), 2048, 2, 2.0, n_visible=33)
    _run(H.Shape(L=2, Hq=8, Hkv=2, Nf=16, T=10, W=4, k=8, seed=7), 512, 1, 1.0, n_visible=3)   # window only


@pytest.mark.parametrize("b", [2, 4])
def test_block_level_external_retrieval(b):
    _run(H.Shape(L=2, Hq=8, Hkv=2, Nf=16, T=90, W=4, k=16, b=b, seed=540), 1152, 2, 0.1)


def test_errors():
    s = H.TINY
    g0 = H.build_gpu(s)  # no embedding table
    e = torch.zeros(64, device="cuda")
    with pytest.raises(rekv.RekvError) as err:
        g0.set_frame_embedding(0, e)
    assert err.value.code == rekv.ERR_STATE
    g0.close()
    g = H.build_gpu(s, ext_embed_dim=64)
    q = torch.ones(1, 64, device="cuda")
    with pytest.raises(rekv.RekvError) as err:  # embeddings missing for the visible frames
        g.retrieve_external(q, s.k, s.T, 1.0)
    assert err.value.code == rekv.ERR_STATE
    with pytest.raises(rekv.RekvError) as err:
        g.set_frame_embedding(s.T, e)
    assert err.value.code == rekv.ERR_ARG
    for f in range(s.T):
        g.set_frame_embedding(f, e)
    with pytest.raises(rekv.RekvError) as err:
        g.retrieve_external(q, s.k, s.T, 0.0)
    assert err.value.code == rekv.ERR_ARG
    idx, k_eff, _ = g.retrieve_external(q, s.k, s.T, 1.0)  # all scores equal (zero vectors): lowest indices win
    assert idx[0, 0].tolist() == list(range(s.k)) and k_eff == s.k
    g.close()
