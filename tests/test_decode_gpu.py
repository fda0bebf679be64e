"""Decode-shaped questions (at most 16 query rows per KV head) take the load-bound attention kernel: the same
parity checks as the other shapes, on the shapes that reach its branches."""
import pytest
import torch

from tests import harness as H
from tests.test_parity_gpu import _run_question_parity

pytestmark = pytest.mark.gpu


def test_one_token_question_7b_shape():
    """7 rows per KV head, 196-token frames, ranges cut by CTA boundaries (partials merged)."""
    _run_question_parity(H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=40, W=8, k=12), [1])


def test_two_tokens_and_batches_of_decode_steps():
    _run_question_parity(H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=30, W=4, k=6, seed=540), [2])
    _run_question_parity(H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=30, W=4, k=6, seed=7), [1, 2, 1])


def test_72b_head_shape_sixteen_rows():
    _run_question_parity(H.Shape(L=1, Hq=64, Hkv=8, Nf=196, T=20, W=4, k=6, seed=7), [2])


def test_short_and_odd_frames():
    """16-token frames (one warp has all the tokens), 100-token frames (ragged last unit), 208-token frames
    (the largest the library takes)."""
    _run_question_parity(H.TINY, [1])
    _run_question_parity(H.Shape(L=2, Hq=8, Hkv=2, Nf=100, T=20, W=3, k=5, seed=540), [2])
    _run_question_parity(H.Shape(L=1, Hq=8, Hkv=2, Nf=208, T=12, W=2, k=4, seed=7), [1])
    _run_question_parity(H.Shape(L=1, Hq=8, Hkv=2, Nf=208, T=12, W=2, k=4, seed=7), [30])  # and the tcgen05 kernel


def test_many_units_are_produced_whole():
    """More units than four times the SM count: every unit is one CTA's, no partials."""
    _run_question_parity(H.Shape(L=20, Hq=16, Hkv=8, Nf=32, T=10, W=2, k=4), [1] * 4, max_questions=4)


def test_host_tier_and_a_question_in_the_past():
    _run_question_parity(H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=40, W=4, k=8, tail=8), [1, 1])
    _run_question_parity(H.Shape(L=2, Hq=28, Hkv=4, Nf=196, T=40, W=8, k=12), [1], n_visible=21)
