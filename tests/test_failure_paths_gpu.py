"""The device-side failure path: a bounded wait that runs out.

Every wait inside the attention kernels (on a tile copy, a matrix product, another warp) has an iteration limit;
when it is reached the kernel writes REKV_ERR_TIMEOUT to the status word, waits (again bounded) for its own copies
in flight, releases tensor memory and returns, so the context stays usable.  The test-only call
rekv_test_set_wait_limit shortens the limit and makes the copy producer of one CTA leave out one tile copy, so
that the wait for that tile expires with nothing in flight -- no fault, no trap, no endless loop.  Checked: the
call returns, rekv_check_status reports REKV_ERR_TIMEOUT exactly once, and the next question on the same context
matches the oracle.
"""
import pytest
import torch

from paper_2503_00540_b200 import rekv
from tests import harness as H

pytestmark = pytest.mark.gpu


def _expire_then_recover(s: H.Shape, lengths, skip_entry: int):
    g = H.build_gpu(s, max_questions=len(lengths), max_q_tokens=sum(lengths))
    o = H.build_oracle(s)
    q, cu = H.questions(s, lengths, device="cuda")
    # 1. a healthy question first: the kernels' function attributes and the context are set up
    out0 = g.question(q, cu, s.k, s.T)
    g.check_status()
    # 2. the wait runs out
    g.test_set_wait_limit(20000, skip_entry)
    g.question(q, cu, s.k, s.T)
    with pytest.raises(rekv.RekvError) as e:
        g.check_status()
    assert e.value.code == rekv.ERR_TIMEOUT and "wait expired" in str(e.value)
    g.check_status()  # the status word was cleared by the read
    # 3. the same context answers the next question correctly
    g.test_set_wait_limit(0, -1)
    out1 = g.question(q, cu, s.k, s.T)
    g.check_status()
    assert torch.equal(out0, out1)
    for i in range(len(lengths)):
        ref = o.question(q[:, cu[i]:cu[i + 1]].cpu().contiguous(), s.k, s.T)
        H.assert_attention(out1[:, cu[i]:cu[i + 1]], ref["out"], f"after the expired wait, question {i}")
    g.close()


@pytest.mark.parametrize("skip_entry", [0, 1, 3])
def test_tensor_core_kernel_gives_up_when_a_tile_never_arrives(skip_entry):
    """64 query rows per KV head: the tcgen05 kernel.  Entry 0 is a K tile (the S product waits for it), entry 1 a V
    tile (the P V product waits), entry 3 the second chunk's V tile of the first CTA's range (320 (unit, frame) steps
    over 148 CTAs: three 48-token frames = two chunks per CTA)."""
    s = H.Shape(L=4, Hq=8, Hkv=2, Nf=48, T=60, W=4, k=36, seed=7)
    _expire_then_recover(s, [16], skip_entry)


def test_a_cta_that_gives_up_leaves_its_units_unfinished_and_their_counters_are_cleared():
    """80 units of two row tiles, each cut into two or three parts that the attention kernel joins itself by counting
    the parts per unit.  The first CTA gives up on its first K tile: its parts are never counted, the units it shares
    stay unfinished behind the status word, and reading the status clears the counters -- the next question would
    otherwise join the wrong parts."""
    s = H.Shape(L=10, Hq=16, Hkv=8, Nf=100, T=28, W=4, k=16, seed=2503)
    _expire_then_recover(s, [80], 0)


def test_decode_kernel_gives_up_when_a_frame_never_arrives():
    """One query token (4 rows per KV head): the load-bound decode kernel."""
    s = H.Shape(L=4, Hq=8, Hkv=2, Nf=48, T=60, W=4, k=36, seed=7)
    _expire_then_recover(s, [1], 0)
