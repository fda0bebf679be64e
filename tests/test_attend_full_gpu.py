"""Eq. 3 in full on the GPU (the questions' own K/V after the retrieved context, causal; rotary embedding with
the retrieved tokens at consecutive positions) against the CPU oracle, through the C ABI."""
import pytest
import torch

from oracle import rekv_oracle as orc
from paper_2503_00540_b200 import rekv
from tests import harness as H

pytestmark = pytest.mark.gpu

THETAS = [pytest.param(0.0, id="no_rope"), pytest.param(1e6, id="rope_1e6")]


def _run(s: H.Shape, nq_lengths, ns_lengths, theta, n_visible=None, top_k=None, static_ctx=False):
    n_visible = s.T if n_visible is None else n_visible
    top_k = s.k if top_k is None else top_k
    nQ = len(nq_lengths)
    g = H.build_gpu(s, max_questions=nQ, max_q_tokens=sum(nq_lengths), max_self_tokens=sum(ns_lengths),
                    rope_theta=theta, flags=rekv.FLAG_ROPE_STATIC if static_ctx else 0)
    o = H.build_oracle(s)
    q, cu = H.questions(s, nq_lengths, device="cuda")
    ks, vs, cus = H.self_kv(s, ns_lengths, device="cuda")
    q_cpu, ks_cpu, vs_cpu = q.cpu(), ks.cpu(), vs.cpu()
    # the context is the oracle's selection (inside a near-tie several selections are correct)
    refs = [o.question(q_cpu[:, cu[i]:cu[i + 1]].contiguous(), top_k, n_visible) for i in range(nQ)]
    idx = torch.stack([r["idx"] for r in refs], dim=1).contiguous().cuda()
    g.gather(idx, nQ, top_k, n_visible)
    out = g.attend_full(q, ks, vs, cu, cus)
    g.check_status()
    worst = 0.0
    for i in range(nQ):
        for l in range(s.L):
            ref, _ = orc.attend_full(q_cpu[l, cu[i]:cu[i + 1]].contiguous(), refs[i]["k_ctx"][l].contiguous(),
                                     refs[i]["v_ctx"][l].contiguous(), ks_cpu[l, cus[i]:cus[i + 1]].contiguous(),
                                     vs_cpu[l, cus[i]:cus[i + 1]].contiguous(), theta, static_ctx=static_ctx)
            H.assert_attention(out[l:l + 1, cu[i]:cu[i + 1]], ref[None], f"Eq. 3 in full, layer {l} question {i}")
            worst = max(worst, (out[l, cu[i]:cu[i + 1]].float().cpu() - ref).abs().max().item())
    # the plain call must differ (the self part matters) unless nothing of X is visible -- never the case
    plain = g.attend(q, cu)
    assert not torch.equal(plain, out)
    g.close()
    return worst


@pytest.mark.parametrize("theta", THETAS)
def test_tiny(theta):
    _run(H.TINY, [16], [16], theta)


@pytest.mark.parametrize("theta", THETAS)
def test_7b_shape_question_prefill(theta):
    """224 query rows per KV head (two row tiles), 196-token frames, units cut by CTA boundaries and whole."""
    _run(H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=40, W=8, k=12), [32], [32], theta)


@pytest.mark.parametrize("theta", THETAS)
def test_batch_of_mixed_lengths_with_generated_tokens(theta):
    """N_s > N_q: some tokens of X (earlier question tokens, generated tokens) precede the query rows."""
    s = H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=30, W=4, k=6, seed=540)
    _run(s, [24, 64, 1, 5], [24, 80, 37, 9], theta)


@pytest.mark.parametrize("theta", THETAS)
def test_decode_step_with_a_long_own_history(theta):
    """One query row per question, 150 tokens of own K/V (three 64-token tiles in the self kernel)."""
    s = H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=24, W=4, k=8, seed=7)
    _run(s, [1, 1], [150, 65], theta)


@pytest.mark.parametrize("theta", THETAS)
def test_72b_head_shape(theta):
    _run(H.Shape(L=1, Hq=64, Hkv=8, Nf=196, T=20, W=4, k=6, seed=7), [48], [48], theta)


@pytest.mark.parametrize("theta", THETAS)
def test_units_cut_in_two_or_three_are_finished_in_the_kernel_with_the_part_over_x(theta):
    """80 units of two row tiles over 146 CTAs: every unit is cut into two or three parts, which the CTA that completes
    the last one joins -- together with the part over X, the first part in the fixed order."""
    s = H.Shape(L=10, Hq=16, Hkv=8, Nf=100, T=28, W=4, k=16, seed=2503)
    _run(s, [80], [96], theta)


@pytest.mark.parametrize("theta", THETAS)
def test_many_units_take_the_whole_unit_path(theta):
    """Enough (layer, head, question) units that every unit is produced whole by one CTA."""
    s = H.Shape(L=8, Hq=16, Hkv=8, Nf=64, T=12, W=2, k=4)
    _run(s, [8] * 12, [8] * 12, theta)


@pytest.mark.parametrize("theta", THETAS)
def test_many_short_questions_half_streams(theta):
    """640 uncut units of one row tile each: two half-streams per unit, joined with the part over X by the merge
    kernel."""
    s = H.Shape(L=4, Hq=16, Hkv=8, Nf=33, T=12, W=2, k=4, seed=540)
    nq = [9 + (7 * i) % 32 for i in range(20)]
    _run(s, nq, [n + (i % 3) for i, n in enumerate(nq)], theta)


@pytest.mark.parametrize("theta", THETAS)
def test_host_tier(theta):
    s = H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=40, W=4, k=8, tail=8)
    _run(s, [16, 32], [16, 40], theta)


def test_no_context_is_causal_self_attention():
    """top_k = 0 and W = 0: nothing retrieved, the result is the causal attention of X over itself."""
    s = H.Shape(L=2, Hq=8, Hkv=2, Nf=16, T=8, W=0, k=0)
    for theta in (0.0, 1e4):
        g = H.build_gpu(s, max_questions=2, max_q_tokens=40, max_self_tokens=40, rope_theta=theta)
        q, cu = H.questions(s, [16, 24], device="cuda")
        ks, vs, cus = H.self_kv(s, [16, 24], device="cuda")
        idx = torch.empty((s.L, 2, 0), dtype=torch.int32, device="cuda")
        assert g.gather(idx, 2, 0, s.T)[0] == 0
        out = g.attend_full(q, ks, vs, cu, cus)
        g.check_status()
        empty = torch.empty(s.Hkv, 0, s.D, dtype=torch.bfloat16)
        for i in range(2):
            for l in range(s.L):
                ref, _ = orc.attend_full(q[l, cu[i]:cu[i + 1]].cpu().contiguous(), empty, empty,
                                         ks[l, cus[i]:cus[i + 1]].cpu().contiguous(),
                                         vs[l, cus[i]:cus[i + 1]].cpu().contiguous(), theta)
                H.assert_attention(out[l:l + 1, cu[i]:cu[i + 1]], ref[None], f"self only, layer {l} question {i}")
        g.close()


def test_argument_and_state_errors():
    s = H.TINY
    q, cu = H.questions(s, [16], device="cuda")
    ks, vs, cus = H.self_kv(s, [16], device="cuda")
    g0 = H.build_gpu(s, max_questions=1, max_q_tokens=16)  # created without the workspaces
    idx, _, _ = g0.retrieve(q, cu, s.k, s.T)
    g0.gather(idx, 1, s.k, s.T)
    with pytest.raises(rekv.RekvError) as e:
        g0.attend_full(q, ks, vs, cu, cus)
    assert e.value.code == rekv.ERR_STATE
    g0.close()
    g = H.build_gpu(s, max_questions=1, max_q_tokens=16, max_self_tokens=16)
    with pytest.raises(rekv.RekvError) as e:  # no gather yet
        g.attend_full(q, ks, vs, cu, cus)
    assert e.value.code == rekv.ERR_STATE
    g.gather(idx, 1, s.k, s.T)
    with pytest.raises(rekv.RekvError) as e:  # fewer own tokens than query rows
        g.attend_full(q, ks[:, :8].contiguous(), vs[:, :8].contiguous(), cu, [0, 8])
    assert e.value.code == rekv.ERR_ARG
    ks2, vs2, cus2 = H.self_kv(s, [20], device="cuda")
    with pytest.raises(rekv.RekvError) as e:  # more own tokens than the workspaces hold
        g.attend_full(q, ks2, vs2, cu, cus2)
    assert e.value.code == rekv.ERR_ARG
    g.close()


@pytest.mark.parametrize("theta", THETAS)
def test_stream_encoding_step_is_the_same_computation(theta):
    """Eq. 1 (sliding-window encoding): O = Attn(W_Q X, [L_k, W_K X], [L_v, W_V X]) with L the local window of the
    stored K/V and X the incoming chunk.  With nothing retrieved (top_k = 0) the context of rekv_gather is exactly
    the last W frames, so the encode step of a new frame is rekv_gather + rekv_attend_full on the frame's own
    Q/K/V, followed by rekv_append_frame."""
    s = H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=12, W=3, k=0, seed=540)
    g = H.build_gpu(s, max_questions=1, max_q_tokens=s.Nf, max_self_tokens=s.Nf, rope_theta=theta, max_frames=s.T + 1)
    o = H.build_oracle(s)
    # the chunk X: one new frame's tokens (queries, keys, values as the decoder layer makes them)
    q, cu = H.questions(s, [s.Nf], device="cuda", first_id=77)
    kx, vx, cux = H.self_kv(s, [s.Nf], device="cuda", first_id=77)
    idx = torch.empty((s.L, 1, 0), dtype=torch.int32, device="cuda")
    assert g.gather(idx, 1, 0, s.T)[0] == s.W
    out = g.attend_full(q, kx, vx, cu, cux)
    g.check_status()
    assert g.append_frame(kx, vx) == s.T  # the chunk's K/V join the store (same [L][N_f][H_kv][D] layout)
    k_win, v_win = o.gather(torch.empty((s.L, 0), dtype=torch.int32), 0, s.T)
    for l in range(s.L):
        ref, _ = orc.attend_full(q[l].cpu().contiguous(), k_win[l].contiguous(), v_win[l].contiguous(),
                                 kx[l].cpu().contiguous(), vx[l].cpu().contiguous(), theta)
        H.assert_attention(out[l:l + 1], ref[None], f"encode step, layer {l}")
    g.close()


def test_static_position_variant():
    """REKV_FLAG_ROPE_STATIC: every context token at one position (the paragraph's static variant), X after it;
    prefill over two row tiles with cut units, a mixed batch with generated tokens, and decode steps."""
    _run(H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=40, W=8, k=12), [32], [32], 1e6, static_ctx=True)
    _run(H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=30, W=4, k=6, seed=540), [24, 64, 1, 5], [24, 80, 37, 9], 1e6, static_ctx=True)
    _run(H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=24, W=4, k=8, seed=7), [1, 1], [150, 65], 1e6, static_ctx=True)


@pytest.mark.parametrize("theta", THETAS)
@pytest.mark.parametrize("tail,k", [(0, 8), (8, 8), (0, 26)])
def test_layer_calls_of_eq3_in_full(theta, tail, k):
    """What a decoder layer calls with the Q, K, V it has just made of X: rekv_question_layer_full per layer (steps 2-5
    with Eq. 3 in full), then decode steps through rekv_attend_full_layer over the layer's context -- against the
    oracle per layer, and against the all-layer calls on the same selection."""
    # (k = 26: 30 context frames, ten or eleven partials per unit of a one-layer launch -- the merge kernel for units of
    # many parts takes the part over X in)
    s = H.Shape(L=3, Hq=28, Hkv=4, Nf=196, T=40, W=4, k=k, seed=540, tail=tail)
    nq, ns = [24, 33], [24, 40]
    g = H.build_gpu(s, max_questions=2, max_q_tokens=sum(nq), max_self_tokens=sum(ns) + 2, rope_theta=theta)
    o = H.build_oracle(s)
    q, cu = H.questions(s, nq, device="cuda")
    ks, vs, cus = H.self_kv(s, ns, device="cuda")
    out = torch.empty_like(q)
    idx = torch.zeros((s.L, 2, s.k), dtype=torch.int32, device="cuda")
    for l in range(s.L):
        g.question_layer_full(l, q[l], ks[l], vs[l], cu, cus, s.k, s.T, out=out[l], idx=idx[l])
    g.check_status()
    q_cpu, ks_cpu, vs_cpu = q.cpu(), ks.cpu(), vs.cpu()
    refs = [o.question(q_cpu[:, cu[i]:cu[i + 1]].contiguous(), s.k, s.T) for i in range(2)]
    for i in range(2):
        for l in range(s.L):
            if not torch.equal(idx[l, i].cpu(), refs[i]["idx"][l]):
                continue  # (a near-tie: another selection is as correct; the all-layer comparison below still holds)
            ref, _ = orc.attend_full(q_cpu[l, cu[i]:cu[i + 1]].contiguous(), refs[i]["k_ctx"][l].contiguous(),
                                     refs[i]["v_ctx"][l].contiguous(), ks_cpu[l, cus[i]:cus[i + 1]].contiguous(),
                                     vs_cpu[l, cus[i]:cus[i + 1]].contiguous(), theta)
            H.assert_attention(out[l:l + 1, cu[i]:cu[i + 1]], ref[None], f"layer call of Eq. 3 in full, layer {l} question {i}")
    # decode steps: one more token of X per question, over the same contexts, layer by layer
    qd, cud = H.questions(s, [1, 1], device="cuda", first_id=11)
    ks2, vs2, cus2 = H.self_kv(s, [ns[0] + 1, ns[1] + 1], device="cuda")
    outd = torch.empty_like(qd)
    for l in range(s.L):
        g.attend_full_layer(l, qd[l], ks2[l], vs2[l], cud, cus2, out=outd[l])
    g.check_status()
    # the all-layer calls on the same selection give the same rows (other launch shapes: close, not bit-equal)
    g.gather(idx, 2, s.k, s.T)
    all_prefill = g.attend_full(q, ks, vs, cu, cus)
    all_decode = g.attend_full(qd, ks2, vs2, cud, cus2)
    g.check_status()
    for a, b, what in ((out, all_prefill, "prefill"), (outd, all_decode, "decode")):
        d = (a.float() - b.float()).abs()
        assert d.max().item() <= 4e-3 and d.mean().item() <= 2e-4, f"layer calls vs all-layer calls, {what}: {d.max().item()}"
    g.close()


@pytest.mark.parametrize("theta", THETAS)
def test_layer_calls_of_eq3_in_full_replayed_from_a_cuda_graph(theta):
    """A decoder captured whole: the layers' rekv_question_layer_full calls as nodes of one graph (the part over X forks
    to the library's internal stream and joins again inside the capture).  The replay gives the eager calls' bits,
    also after the buffers were given another question."""
    s = H.Shape(L=3, Hq=28, Hkv=4, Nf=196, T=40, W=4, k=8, seed=7)
    g = H.build_gpu(s, max_questions=1, max_q_tokens=32, max_self_tokens=32, rope_theta=theta)
    q, cu = H.questions(s, [32], device="cuda")
    ks, vs, cus = H.self_kv(s, [32], device="cuda")
    q2, _ = H.questions(s, [32], device="cuda", first_id=5)
    ks2, vs2, _ = H.self_kv(s, [32], device="cuda", first_id=5)

    def eager(qq, kk, vv):
        o = torch.empty_like(qq)
        for l in range(s.L):
            g.question_layer_full(l, qq[l], kk[l], vv[l], cu, cus, s.k, s.T, out=o[l])
        return o

    ref1, ref2 = eager(q, ks, vs), eager(q2, ks2, vs2)
    qb, kb, vb, out = q.clone(), ks.clone(), vs.clone(), torch.zeros_like(q)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=side):
            for l in range(s.L):
                g.question_layer_full(l, qb[l], kb[l], vb[l], cu, cus, s.k, s.T, out=out[l])
    torch.cuda.current_stream().wait_stream(side)
    gr.replay()
    torch.cuda.synchronize()
    g.check_status()
    assert torch.equal(out, ref1)
    qb.copy_(q2)
    kb.copy_(ks2)
    vb.copy_(vs2)
    gr.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, ref2)
    g.close()
