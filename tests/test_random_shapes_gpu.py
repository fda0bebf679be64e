"""Seeded random small configurations through the full parity check (steps 1-5 against the oracle): head counts,
tokens per frame on both sides of every chunk and piece boundary of the attention kernels, window and top-k
counts including zero, question batches of mixed lengths, questions in the past."""
import random

import pytest

from tests import harness as H
from tests.test_parity_gpu import _run_question_parity

pytestmark = pytest.mark.gpu

NF = [1, 3, 15, 16, 17, 31, 33, 48, 64, 80, 81, 96, 100, 112, 127, 128, 129, 144, 160, 176, 196, 200, 208]
NQ_TOKENS = [1, 2, 3, 5, 16, 17, 19, 32, 37, 40, 64, 70]


@pytest.mark.parametrize("seed", [2503, 540, 7])
def test_random_small_configurations(seed):
    rng = random.Random(seed)
    for _ in range(40):
        hkv = rng.choice([1, 2, 4, 8])
        g = rng.choice([1, 2, 4, 7, 8])
        t = rng.randint(2, 40)
        lengths = [rng.choice(NQ_TOKENS) for _ in range(rng.choice([1, 1, 2, 3]))]
        s = H.Shape(L=rng.choice([1, 2, 3]), Hq=hkv * g, Hkv=hkv, Nf=rng.choice(NF), T=t, W=rng.randint(0, 6),
                    k=rng.randint(0, 12), seed=rng.randint(1, 10**6), off_scale=rng.choice([0.0, 0.5]))
        _run_question_parity(s, lengths, n_visible=rng.randint(max(1, t // 2), t))
