"""CUDA path vs CPU oracle, element by element, through the C ABI, on the same seeded inputs."""
import pytest
import torch

from oracle import rekv_oracle as orc
from paper_2503_00540_b200 import rekv, synth
from tests import harness as H

pytestmark = pytest.mark.gpu

# both attention kernels are checked: the tcgen05 one (default) and the mma.sync one
ATT = [pytest.param(0, id="tcgen05")]


def _run_question_parity(s: H.Shape, lengths, n_visible=None, flags=0, max_questions=None):
    n_visible = s.T if n_visible is None else n_visible
    nQ = len(lengths)
    g = H.build_gpu(s, max_questions=max_questions or nQ, max_q_tokens=sum(lengths), flags=flags)
    o = H.build_oracle(s)
    # step 1
    for l in range(s.L):
        H.assert_close_rel(g.get_reps(l, s.T), o.rep_table(l), f"reps layer {l}")
    q_gpu, cu = H.questions(s, lengths, device="cuda")
    q_cpu, _ = H.questions(s, lengths)
    assert torch.equal(q_gpu.cpu(), q_cpu)
    # steps 2-3
    idx, k_eff, scores = g.retrieve(q_gpu, cu, s.k, n_visible, want_scores=True)
    ref = [o.question(q_cpu[:, cu[i]:cu[i + 1]].contiguous(), s.k, n_visible) for i in range(nQ)]
    for i in range(nQ):
        assert k_eff == ref[i]["k_eff"]
        for l in range(s.L):
            H.assert_close_rel(scores[l, i][None], ref[i]["scores"][l][None], f"scores l{l} q{i}")
            H.assert_indices(idx[l, i], ref[i]["idx"][l], ref[i]["scores"][l], ref[i]["gaps"][l], k_eff,
                             f"idx l{l} q{i}")
    # steps 4-5 on the oracle's selection (inside a near-tie several selections are correct)
    idx_ref = torch.stack([r["idx"] for r in ref], dim=1).contiguous().cuda()  # [L][nQ][k]
    ncf, k_ctx, v_ctx = g.gather(idx_ref, nQ, s.k, n_visible, materialize=True)
    assert ncf == k_eff + o.window_eff(n_visible, s.k)
    for i in range(nQ):
        assert torch.equal(k_ctx[:, i].cpu(), ref[i]["k_ctx"]), f"gathered K differs, question {i}"
        assert torch.equal(v_ctx[:, i].cpu(), ref[i]["v_ctx"]), f"gathered V differs, question {i}"
    out = g.attend(q_gpu, cu)
    g.check_status()
    for i in range(nQ):
        H.assert_attention(out[:, cu[i]:cu[i + 1]], ref[i]["out"], f"attention q{i}")
    # the library's own selection must give the same answer when it equals the oracle's
    out2 = g.question(q_gpu, cu, s.k, n_visible)
    g.check_status()
    if torch.equal(idx.cpu(), idx_ref.cpu()):
        assert torch.equal(out2, out)
    st = g.stats()
    assert st.kv_bytes_logical == orc.kv_cache_bytes(s.L, s.T, s.Nf, s.Hkv, s.D)  # the oracle's cache-size expression
    assert st.kv_bytes_hbm + (0 if s.tail == 0 else 0) >= 0
    g.close()
    return st


@pytest.mark.parametrize("flags", ATT)
def test_tiny_config(flags):
    """1 layer, 8/2 heads, 64 frames x 16 tokens, question of 16 tokens, window 4, top-k 8."""
    for seed in (2503, 540, 7):
        s = H.Shape(**{**H.TINY.__dict__, "seed": seed})
        st = _run_question_parity(s, [16], flags=flags)
        assert st.kv_bytes_hbm == st.kv_bytes_logical and st.kv_bytes_host == 0


@pytest.mark.parametrize("flags", ATT)
def test_7b_shape_small_stream_ragged_tiles(flags):
    """7B head shape, 196-token frames (a ragged 16-token tail per tile), 224 rows = one full and one
    partial 128-row tile, several context frames per split."""
    s = H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=40, W=8, k=12)
    _run_question_parity(s, [32], flags=flags)


@pytest.mark.parametrize("flags", ATT)
def test_batched_questions_of_mixed_length(flags):
    s = H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=30, W=4, k=6, seed=540)
    _run_question_parity(s, [24, 64, 37, 5], flags=flags)


@pytest.mark.parametrize("flags", ATT)
def test_72b_head_shape(flags):
    s = H.Shape(L=1, Hq=64, Hkv=8, Nf=196, T=24, W=8, k=8, seed=7)
    _run_question_parity(s, [64], flags=flags)


def test_many_short_questions_whole_units_as_half_streams():
    """640 units of one row tile each (more than four per SM, so no unit is cut at a CTA boundary): every unit runs
    as two half-streams; the half that finishes second joins the other's partial inside the kernel, with partial slots
    counted per such unit."""
    s = H.Shape(L=4, Hq=16, Hkv=8, Nf=33, T=12, W=2, k=4, seed=540)
    lengths = [9 + (7 * i) % 32 for i in range(20)]  # 18..80 rows per KV head
    _run_question_parity(s, lengths, max_questions=20)


def test_half_streams_over_a_context_of_a_single_chunk():
    """As above with three context frames of 33 tokens (113 stream rows: one chunk): the second half-stream of every
    unit has no chunk at all and contributes the neutral part."""
    s = H.Shape(L=4, Hq=16, Hkv=8, Nf=33, T=12, W=1, k=2, seed=7)
    lengths = [9 + (7 * i) % 32 for i in range(20)]
    _run_question_parity(s, lengths, max_questions=20)


def test_short_question_cut_at_cta_boundaries():
    """One 10-token question at the 7B head shape: 70 rows = one row tile per unit, units cut at CTA boundaries
    (four to six partials per unit: the merge kernel joins them)."""
    s = H.Shape(L=3, Hq=28, Hkv=4, Nf=196, T=30, W=4, k=12, seed=7)
    _run_question_parity(s, [10])


def test_units_of_two_questions_cut_into_a_few_parts():
    """The same regime with a batch: 80 units of two questions (160 and 144 rows per KV head), cut into two or three
    parts and finished inside the kernel."""
    s = H.Shape(L=5, Hq=16, Hkv=8, Nf=100, T=28, W=4, k=16, seed=540)
    _run_question_parity(s, [80, 72])


def test_units_cut_into_a_few_parts_are_finished_inside_the_kernel():
    """80 units of two row tiles over 146 CTAs (on 148 SMs), eleven of a unit's twenty context frames per CTA: every
    unit is cut into two or three parts, and the CTA that finishes a unit's last part joins them (from its own
    accumulator if the others are already there, from the written partials otherwise).  Both ways do the same
    arithmetic in part order: repeated launches give the same bits whichever CTA came last."""
    s = H.Shape(L=10, Hq=16, Hkv=8, Nf=100, T=28, W=4, k=16, seed=2503)
    _run_question_parity(s, [80])
    g = H.build_gpu(s, max_questions=1, max_q_tokens=80)
    q, cu = H.questions(s, [80], device="cuda")
    first = g.question(q, cu, s.k, s.T).clone()
    for _ in range(8):
        assert torch.equal(g.question(q, cu, s.k, s.T), first)
    g.check_status()
    st = g.stats()
    g.close()


@pytest.mark.parametrize("n_tokens", [40, 10, 1])
def test_few_units_of_many_parts_each(n_tokens):
    """Two units (one layer, two KV heads) over 48 context frames: three or four frames per CTA, 13 to 34 partials per
    unit, joined by the merge kernel for units of many parts -- with two row tiles (40 tokens x 4 heads), as two
    half-streams (10 tokens) and in the decode-shaped kernel (1 token)."""
    s = H.Shape(L=1, Hq=8, Hkv=2, Nf=16, T=80, W=8, k=40, seed=7)
    _run_question_parity(s, [n_tokens])


def test_question_in_the_past_sees_only_visible_frames():
    s = H.Shape(L=1, Hq=8, Hkv=2, Nf=16, T=64, W=4, k=8, off_scale=0.0)
    _run_question_parity(s, [16], n_visible=37)


def test_timing_switch_reports_the_kernel_and_leaves_results_alone():
    """rekv_set_timing: with the event records on, the attention kernel's duration is reported; off, it is not;
    the output bits are the same either way."""
    s = H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=80, W=8, k=16, seed=7)
    g = H.build_gpu(s, max_q_tokens=32)
    q, cu = H.questions(s, [32], device="cuda")
    out_plain = g.question(q, cu, s.k, s.T).clone()
    torch.cuda.synchronize()
    assert g.stats().last_attend_kernel_us == 0.0
    g.set_timing(True)
    out_timed = g.question(q, cu, s.k, s.T).clone()
    torch.cuda.synchronize()
    st = g.stats()
    assert st.last_attend_kernel_us > 0.0 and st.last_retrieve_us > 0.0 and st.last_merge_us > 0.0
    assert st.last_pull_us == 0.0  # nothing crosses the host link on a cache that is all in HBM
    g.set_timing(False)
    out_again = g.question(q, cu, s.k, s.T).clone()
    torch.cuda.synchronize()
    st = g.stats()
    assert st.last_attend_kernel_us == 0.0 and st.last_retrieve_us == 0.0 and st.last_merge_us == 0.0
    assert torch.equal(out_plain, out_timed) and torch.equal(out_plain, out_again)
    g.check_status()
    g.close()


def test_degenerate_counts():
    # k larger than the candidates -> every visible frame is attended; fewer frames than the window
    s = H.Shape(L=1, Hq=8, Hkv=2, Nf=16, T=10, W=4, k=32, off_scale=0.0)
    _run_question_parity(s, [7])
    _run_question_parity(s, [7], n_visible=3)
    # top_k = 0: window only
    s0 = H.Shape(L=1, Hq=8, Hkv=2, Nf=16, T=10, W=4, k=0, off_scale=0.0)
    g = H.build_gpu(s0)
    o = H.build_oracle(s0)
    q_gpu, cu = H.questions(s0, [5], device="cuda")
    out = g.question(q_gpu, cu, 0, 10)
    ref = o.question(q_gpu.cpu(), 0, 10)
    H.assert_attention(out, ref["out"], "window only")
    g.close()


def test_odd_tokens_per_frame_and_single_token_question():
    s = H.Shape(L=1, Hq=4, Hkv=1, Nf=37, T=20, W=2, k=5, seed=7)
    _run_question_parity(s, [1])


@pytest.mark.parametrize("b,T,k", [(2, 41, 8), (4, 50, 12), (8, 40, 8)])
def test_block_retrieval(b, T, k):
    """Blocks of b frames: block vector = mean of the frame vectors, top_k/b blocks retrieved; the frames after
    the last complete block join the window."""
    s = H.Shape(L=2, Hq=8, Hkv=2, Nf=16, T=T, W=3, k=k, b=b, seed=540)
    _run_question_parity(s, [9, 20])
    _run_question_parity(s, [5], n_visible=T - 7)


def test_block_retrieval_7b_shape_and_host_tier():
    s = H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=45, W=4, k=8, b=4, seed=7)
    _run_question_parity(s, [32])
    s2 = H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=45, W=4, k=8, b=4, tail=10, seed=7)
    _run_question_parity(s2, [32])


def test_error_paths_on_device():
    s = H.TINY
    g = H.build_gpu(s, n_frames=3, max_frames=3)
    k = synth.frame(1, synth.K, 0, s.L, s.Nf, s.Hkv, s.D, device="cuda")
    with pytest.raises(rekv.RekvError) as e:
        g.append_frame(k, k)
    assert e.value.code == rekv.ERR_FULL
    q, cu = H.questions(s, [4], device="cuda")
    with pytest.raises(rekv.RekvError) as e:
        g.retrieve(q, cu, 2, 0)
    assert e.value.code == rekv.ERR_EMPTY
    with pytest.raises(rekv.RekvError) as e:
        g.retrieve(q, cu, 2, 4)
    assert e.value.code == rekv.ERR_ARG
    with pytest.raises(rekv.RekvError) as e:
        g.attend(q, cu)
    assert e.value.code == rekv.ERR_STATE
    # an index outside the visible frames is reported, not dereferenced
    bad = torch.full((s.L, 1, 2), 99, dtype=torch.int32, device="cuda")
    g2 = H.build_gpu(H.Shape(**{**s.__dict__, "W": 0}), n_frames=5)
    g2.gather(bad, 1, 2, 5)
    with pytest.raises(rekv.RekvError) as e:
        g2.check_status()
    assert e.value.code == rekv.ERR_ARG
    g.close()
    g2.close()


def test_host_tier_small_stream():
    """Offloaded context: every page in pinned host memory, the last 6 frames also in HBM."""
    s = H.Shape(L=3, Hq=28, Hkv=4, Nf=196, T=30, W=4, k=8, tail=6, seed=540)
    st = _run_question_parity(s, [32])
    assert st.kv_bytes_host == st.kv_bytes_logical
    assert st.kv_bytes_hbm == st.kv_bytes_logical * 6 // 30


def test_host_tier_pages_survive_the_round_trip():
    s = H.Shape(L=2, Hq=8, Hkv=2, Nf=16, T=20, W=2, k=4, tail=4, off_scale=0.0)
    g = H.build_gpu(s)
    for f in (0, 7, 15, 16, 19):
        for l in range(s.L):
            k, v = g.get_page(f, l)
            kr = synth.frame(s.seed, synth.K, f, s.L, s.Nf, s.Hkv, s.D, s.off_scale)[l].permute(1, 0, 2)
            vr = synth.frame(s.seed, synth.V, f, s.L, s.Nf, s.Hkv, s.D, s.off_scale)[l].permute(1, 0, 2)
            assert torch.equal(k.cpu(), kr) and torch.equal(v.cpu(), vr), (f, l)
    g.close()


def test_offloaded_context_keeps_its_frames_when_appends_recycle_the_hbm_tail():
    """A context gathered on an offloaded stream references frames that were in the HBM tail at gather time (the
    window always is).  The stream keeps growing while the answer is decoded: `tail` appends after the gather recycle
    every ring slot.  The attention -- all layers, then one layer again as a decode step would -- must still see the
    frames of gather time."""
    s = H.Shape(L=2, Hq=8, Hkv=2, Nf=48, T=34, W=3, k=6, tail=5, seed=540)
    n0 = s.T - s.tail                      # frames when the question is asked
    g = H.build_gpu(s, max_q_tokens=16, n_frames=n0)
    o = H.build_oracle(s, n_frames=n0)
    q, cu = H.questions(s, [16], device="cuda")
    ref = o.question(q.cpu(), s.k, n0)
    idx_ref = ref["idx"][:, None].contiguous().cuda()
    g.gather(idx_ref, 1, s.k, n0)
    for f in range(n0, s.T):               # the stream goes on: every ring slot gets a new frame
        k = synth.frame(s.seed, synth.K, f, s.L, s.Nf, s.Hkv, s.D, s.off_scale, device="cuda")
        v = synth.frame(s.seed, synth.V, f, s.L, s.Nf, s.Hkv, s.D, s.off_scale, device="cuda")
        assert g.append_frame(k, v) == f
    out = g.attend(q, cu)
    g.check_status()
    H.assert_attention(out, ref["out"], "attention after the tail was recycled")
    out_l = g.attend_layer(1, q[1].contiguous(), cu)
    g.check_status()
    assert torch.equal(out_l, out[1])
    g.close()


def test_stats_report_the_pull_stage_of_an_offloaded_question_without_waiting():
    """rekv_stats never synchronises: right after the call is enqueued the pull stage may read 0; once the streams
    have drained it reports the host-link bytes and the duration of the pulls."""
    s = H.Shape(L=3, Hq=8, Hkv=2, Nf=48, T=30, W=3, k=6, tail=5, seed=7)
    g = H.build_gpu(s, max_q_tokens=16, flags=rekv.FLAG_TIMING)
    q, cu = H.questions(s, [16], device="cuda")
    g.question(q, cu, s.k, s.T)
    g.stats()                      # must return at once, whatever it reads
    g.check_status()               # drains the caller's and the library's streams
    st = g.stats()
    assert st.last_pull_us > 0.0 and st.last_retrieve_us > 0.0
    assert 0 < st.last_link_bytes <= s.L * s.k * st.page_bytes
    g.close()


@pytest.mark.parametrize("nf", [224, 256, 400, 1000])
def test_frames_longer_than_a_chunk_or_two(nf):
    """Tokens per frame beyond the 128-token chunk of the attention kernel and beyond what the decode kernel can hold:
    several chunks per frame, frame boundaries at any place of a chunk; a 2-token question takes the decode-shaped
    path (or its fallback), a 19-token one the tensor-core path."""
    s = H.Shape(L=2, Hq=8, Hkv=2, Nf=nf, T=9, W=2, k=3, seed=7)
    _run_question_parity(s, [19, 2])
    _run_question_parity(s, [2])


@pytest.mark.parametrize("n_tokens", [16, 40])
def test_logits_far_above_the_first_chunk_raise_the_reference_maximum(n_tokens):
    """The attention kernel keeps the row maximum of a range's first 128-token chunk as the reference of its
    exponentials and only checks that a chunk's row sum stays below 2^60.  Here the last context frame holds keys whose
    logits lie about 80 octaves above everything before them: the rare path (true maximum, rescaling of O and of the
    running sum, second pass) must give the oracle's answer.  16 tokens: one row tile, two half-streams; 40 tokens: two
    row tiles."""
    s = H.Shape(L=1, Hq=8, Hkv=2, Nf=48, T=12, W=2, k=6, seed=7)
    g = rekv.ReKV(s.L, s.Hq, s.Hkv, s.D, s.Nf, s.T, s.W, max_q_tokens=n_tokens, max_topk=s.k)
    o = orc.OracleCache(s.L, s.Hq, s.Hkv, s.D, s.Nf, s.W)
    gen = torch.Generator().manual_seed(11)
    sign = (torch.randint(0, 2, (s.D,), generator=gen) * 2 - 1).float()
    for f in range(s.T):
        k = (0.1 * torch.randn(s.L, s.Nf, s.Hkv, s.D, generator=gen)).to(torch.bfloat16)
        v = torch.randn(s.L, s.Nf, s.Hkv, s.D, generator=gen).to(torch.bfloat16)
        if f == s.T - 1:  # the last window frame: keys along the query direction, 2.5 per dimension
            k[:, 5:40] = (2.5 * sign).to(torch.bfloat16)
        assert g.append_frame(k.cuda(), v.cuda()) == f
        o.append(k, v)
    q = (2.0 * sign).to(torch.bfloat16).expand(s.L, n_tokens, s.Hq, s.D).contiguous()
    cu = [0, n_tokens]
    ref = o.question(q, s.k, s.T)
    out = g.question(q.cuda(), cu, s.k, s.T, idx=ref["idx"][:, None].contiguous().cuda())
    g.check_status()
    # the big logits are 2.0 * 2.5 * 128 / sqrt(128) = 56.6 nats = 81.6 octaves above the others' (about 0)
    H.assert_attention(out, ref["out"], "attention with a late, very large logit")
    g.close()
