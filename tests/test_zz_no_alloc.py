"""The allocation-free scoring entry point against the regular one.

rekv_score_frames_static serves callers that may not allocate device memory (a host that owns the GPU
through its own pool, or a thread that cannot afford cudaMalloc's device synchronisation): its scratch
is a fixed array inside the library.  It must give the scores rekv_retrieve gives -- and the CPU
oracle's Eq. 2 scores on the same inputs -- on every call: the array keeps the previous call's
contents, so two calls in a row with different questions are checked.  This file is named to be
collected last.
"""
import pytest
import torch

from oracle import rekv_oracle as orc
from paper_2503_00540_b200 import rekv
from tests import harness as H

pytestmark = pytest.mark.gpu


def test_static_scratch_scores_match_retrieve_on_two_calls_in_a_row():
    s = H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=150, W=8, k=16, seed=540)
    g = H.build_gpu(s, max_questions=3, max_q_tokens=128)
    o = H.build_oracle(s)
    for call, lengths in enumerate(([32], [24, 64, 7])):
        q, cu = H.questions(s, lengths, device="cuda", first_id=10 * call)
        _, _, want = g.retrieve(q, cu, s.k, s.T, want_scores=True)  # [L][nQ][T]
        for l in range(s.L):
            reps = g.get_reps(l, s.T)
            out = torch.full((len(lengths), s.T), float("nan"), dtype=torch.float32, device="cuda")
            got = rekv.score_frames_static(q[l].contiguous(), cu, s.Hkv, reps, out=out)
            torch.cuda.synchronize()
            for i in range(len(lengths)):
                H.assert_close_rel(got[i][None], want[l, i][None], f"call {call} layer {l} question {i}")
                ref = orc.score(q[l, cu[i]:cu[i + 1]].cpu().contiguous(), o.rep_table(l), s.Hkv)
                H.assert_close_rel(got[i][None], ref[None], f"against the oracle: call {call} layer {l} question {i}")
    g.close()


def test_static_scratch_rejects_sizes_beyond_its_maximum():
    q = torch.zeros((17, 8, 128), dtype=torch.bfloat16, device="cuda")
    reps = torch.zeros((4, 256), dtype=torch.float32, device="cuda")
    with pytest.raises(rekv.RekvError) as e:
        rekv.score_frames_static(q, list(range(18)), 2, reps)  # 17 questions > 16
    assert e.value.code == rekv.ERR_ARG and "16 questions" in str(e.value)
    q9 = torch.zeros((1, 18, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rekv.RekvError) as e:
        rekv.score_frames_static(q9, [0, 1], 9, torch.zeros((4, 9 * 128), dtype=torch.float32, device="cuda"))
    assert e.value.code == rekv.ERR_ARG
