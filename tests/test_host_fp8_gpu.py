"""Quantised host tier (REKV_FLAG_HOST_FP8): pages that cross the host link come back as the oracle's
FP8 round trip of the original rows, bit for bit; frames still in the HBM tail stay exact; attention over the
mixed context agrees with the oracle on the same context and stays inside the tolerance against the exact one."""
import pytest
import torch

from oracle import rekv_oracle as orc
from paper_2503_00540_b200 import rekv, synth
from tests import harness as H

pytestmark = pytest.mark.gpu


def _roundtrip_ctx(o, s, idx, k_eff, n_visible, n_frames_now):
    """The oracle's context with every frame that is no longer in the HBM tail passed through the FP8 round trip."""
    k_ctx, v_ctx = o.gather(idx, k_eff, n_visible)      # [L][H_kv][n_ctx][D], exact
    frames = [int(f) for f in idx[0][:k_eff]]           # (checked per layer below)
    out_k, out_v = k_ctx.clone(), v_ctx.clone()
    w_eff = o.window_eff(n_visible, idx.shape[-1])
    for l in range(s.L):
        fl = [int(f) for f in idx[l][:k_eff]] + list(range(n_visible - w_eff, n_visible))
        for j, f in enumerate(fl):
            if f < n_frames_now - s.tail:                # host-only: quantised
                sl = slice(j * s.Nf, (j + 1) * s.Nf)
                out_k[l][:, sl] = orc.fp8_roundtrip(k_ctx[l][:, sl].contiguous())
                out_v[l][:, sl] = orc.fp8_roundtrip(v_ctx[l][:, sl].contiguous())
    return k_ctx, v_ctx, out_k, out_v


@pytest.mark.parametrize("shape,lengths", [
    (H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=40, W=4, k=8, tail=8), [16, 32]),
    (H.Shape(L=1, Hq=4, Hkv=1, Nf=37, T=20, W=2, k=5, tail=4, seed=7), [9]),      # page padding, odd N_f
    (H.Shape(L=1, Hq=64, Hkv=8, Nf=196, T=16, W=4, k=6, tail=6, seed=540), [1]),  # decode-shaped question
])
def test_fp8_host_tier(shape, lengths):
    s = shape
    nQ = len(lengths)
    g = H.build_gpu(s, max_questions=nQ, max_q_tokens=sum(lengths), flags=rekv.FLAG_HOST_FP8)
    o = H.build_oracle(s)
    st = g.stats()
    host_page = (s.Hkv * 2 * s.Nf * 132 + 15) // 16 * 16
    assert st.kv_bytes_host == s.T * s.L * host_page and st.kv_bytes_host < 0.53 * st.kv_bytes_logical
    # stored pages: host-only frames are the round trip of the original, tail frames the original
    for f in (0, s.T - s.tail - 1, s.T - s.tail, s.T - 1):
        for l in range(s.L):
            k, v = g.get_page(f, l)
            ko, vo = o.k_frames[f][l].permute(1, 0, 2).contiguous(), o.v_frames[f][l].permute(1, 0, 2).contiguous()
            if f < s.T - s.tail:
                ko, vo = orc.fp8_roundtrip(ko), orc.fp8_roundtrip(vo)
            assert torch.equal(k.cpu(), ko) and torch.equal(v.cpu(), vo), f"page of frame {f} layer {l}"
    q, cu = H.questions(s, lengths, device="cuda")
    q_cpu = q.cpu()
    refs = [o.question(q_cpu[:, cu[i]:cu[i + 1]].contiguous(), s.k, s.T) for i in range(nQ)]
    idx = torch.stack([r["idx"] for r in refs], dim=1).contiguous().cuda()  # retrieval is unaffected (fp32 representatives)
    idx_gpu, _, _ = g.retrieve(q, cu, s.k, s.T)
    for i in range(nQ):
        for l in range(s.L):
            H.assert_indices(idx_gpu[l, i], refs[i]["idx"][l], refs[i]["scores"][l], refs[i]["gaps"][l], refs[i]["k_eff"],
                             f"idx l{l} q{i}")
    ncf, k_ctx, v_ctx = g.gather(idx, nQ, s.k, s.T, materialize=True)
    out = g.attend(q, cu)
    g.check_status()
    pulled = 0
    for i in range(nQ):
        ke, ve, kq, vq = _roundtrip_ctx(o, s, refs[i]["idx"], refs[i]["k_eff"], s.T, s.T)
        assert torch.equal(k_ctx[:, i].cpu(), kq) and torch.equal(v_ctx[:, i].cpu(), vq), f"context of question {i}"
        of, _ = o.attend(q_cpu[:, cu[i]:cu[i + 1]].contiguous(), kq, vq)
        H.assert_attention(out[:, cu[i]:cu[i + 1]], of, f"attention on the quantised context, question {i}")
        # and against the exact cache: the rounding noise of E4M3 rows averages out over the context, so the
        # standard tolerance holds for contexts of the configurations' size (thousands of tokens); a context of a
        # few hundred tokens only gets a normwise bound
        if ncf * s.Nf >= 2000:
            H.assert_attention(out[:, cu[i]:cu[i + 1]], refs[i]["out"], f"attention against the exact cache, question {i}")
        else:
            d = out[:, cu[i]:cu[i + 1]].float().cpu() - refs[i]["out"]
            assert (d.norm() / refs[i]["out"].norm()).item() <= 5e-2
        pulled += sum(1 for l in range(s.L) for f in refs[i]["idx"][l][:refs[i]["k_eff"]] if int(f) < s.T - s.tail)
    g.check_status()  # the counter's host mirror is refreshed behind the pulls, on the library's own stream
    assert g.stats().last_link_bytes == pulled * host_page
    g.close()


def test_flag_without_a_host_tier_changes_nothing():
    s = H.Shape(L=1, Hq=8, Hkv=2, Nf=16, T=12, W=2, k=4)
    g = H.build_gpu(s, flags=rekv.FLAG_HOST_FP8)
    st = g.stats()
    assert st.kv_bytes_host == 0 and st.kv_bytes_hbm == st.kv_bytes_logical
    k, v = g.get_page(3, 0)
    assert torch.equal(k.cpu(), synth.frame(s.seed, synth.K, 3, 1, s.Nf, s.Hkv, s.D, s.off_scale)[0].permute(1, 0, 2))
    g.close()
