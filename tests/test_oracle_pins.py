"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle's own code.

Each oracle function is checked against closed forms, brute force, invariants or a library
routine, chosen so that a dropped term, a wrong sign/index or a transposed operand fails.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import rekv_oracle as orc
from paper_2503_00540_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16(x):
    return torch.as_tensor(x, dtype=torch.float32).to(torch.bfloat16).contiguous()


# ----------------------------------------------------------------------------- cache size (appendix formula)
def test_kv_cache_size_matches_printed_values():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "kv_cache_size.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 2
    for name, L, T, M, H, D, b, printed in rows:
        got = orc.kv_cache_bytes(int(L), int(T), int(M), int(H), int(D), int(b))
        assert round(got / 2**30, 1) == float(printed), (name, got / 2**30)
    # term-by-term: doubling any factor doubles the size
    base = orc.kv_cache_bytes(28, 1800, 196, 4, 128, 2)
    assert base == 2 * 28 * 1800 * 196 * 4 * 128 * 2
    assert orc.kv_cache_bytes(56, 1800, 196, 4, 128, 2) == 2 * base


# ----------------------------------------------------------------------------- step 1: frame representative
def test_pool_constant_frame_is_that_constant():
    k = bf16(torch.full((16, 2, 128), 0.375))
    assert torch.equal(orc.pool_frame(k), torch.full((256,), 0.375))


def test_pool_ramp_is_midpoint_and_heads_concatenate_in_order():
    n_tok, H, D = 9, 2, 4
    k = torch.zeros(n_tok, H, D)
    for t in range(n_tok):
        for h in range(H):
            for d in range(D):
                k[t, h, d] = t * (h + 1) + d  # exact in bf16 (small integers)
    rep = orc.pool_frame(bf16(k))
    want = torch.tensor([[4.0 * (h + 1) + d for d in range(D)] for h in range(H)]).reshape(-1)
    assert torch.equal(rep, want)


def test_pool_brute_force_double_loop():
    k = synth.frame(2503, synth.K, 5, 1, 16, 2, 128)[0]
    rep = orc.pool_frame(k)
    kd = k.double().numpy()
    want = np.zeros(256)
    for h in range(2):
        for d in range(128):
            acc = 0.0
            for t in range(16):
                acc += kd[t, h, d]
            want[h * 128 + d] = acc / 16
    np.testing.assert_allclose(rep.numpy(), want.astype(np.float32), rtol=0, atol=0)


# ----------------------------------------------------------------------------- step 2: question vector + cosine
def test_question_vector_brute_force_gqa_grouping():
    q = synth.question(7, 0, 1, 5, 8, 128)[0]  # [5][8][128], G = 4 with 2 kv heads
    qa = orc.question_vector(q, 2).numpy()
    qd = q.double().numpy()
    for g in range(2):
        for d in (0, 17, 127):
            want = np.mean([qd[n, h, d] for n in range(5) for h in range(4 * g, 4 * g + 4)])
            assert abs(qa[g * 128 + d] - want) < 1e-15


def _q_from_vector(vec, n_q, Hq, Hkv, D):
    """A question whose every token/head in group g equals vec[g] (so its question vector is vec)."""
    G = Hq // Hkv
    q = torch.zeros(n_q, Hq, D)
    for h in range(Hq):
        q[:, h, :] = vec[h // G]
    return bf16(q)


def test_score_closed_forms_parallel_antiparallel_orthogonal():
    Hq, Hkv, D = 8, 2, 128
    torch.manual_seed(0)
    r = bf16(torch.randn(Hkv, D)).float()
    reps = torch.stack([r.reshape(-1), -r.reshape(-1), torch.zeros(Hkv * D), 3.0 * r.reshape(-1)]).contiguous()
    # an orthogonal vector: swap pairs with a sign flip
    orth = r.reshape(-1).clone().reshape(-1, 2).flip(1)
    orth[:, 0] = -orth[:, 0]
    reps[2] = orth.reshape(-1)
    q = _q_from_vector(r, 3, Hq, Hkv, D)
    s = orc.score(q, reps, Hkv)
    assert abs(s[0].item() - 1.0) < 1e-6
    assert abs(s[1].item() + 1.0) < 1e-6
    assert abs(s[2].item()) < 1e-6
    assert abs(s[3].item() - 1.0) < 1e-6  # scale invariance in the frame vector


def test_score_scale_invariance_in_question_and_zero_norm_clamp():
    Hq, Hkv, D = 8, 2, 128
    q = synth.question(3, 1, 1, 6, Hq, D)[0]
    reps = torch.randn(10, Hkv * D, generator=torch.Generator().manual_seed(1))
    reps[4] = 0.0
    s1 = orc.score(q, reps, Hkv)
    s2 = orc.score(bf16(q.float() * 4.0), reps, Hkv)  # *4 is exact in bf16
    assert torch.equal(s1, s2)
    assert s1[4].item() == 0.0 and torch.isfinite(s1).all()


def test_score_matches_library_cosine_and_repeat_k_reading_ranks_equal():
    Hq, Hkv, D, T = 8, 2, 128, 40
    G = Hq // Hkv
    q = synth.question(11, 2, 1, 7, Hq, D)[0]
    reps = torch.stack([orc.pool_frame(synth.frame(11, synth.K, f, 1, 16, Hkv, D)[0]) for f in range(T)])
    s = orc.score(q, reps, Hkv)
    # library routine on independently pooled vectors
    qbar = q.double().mean(0)  # [Hq][D]
    qa = qbar.reshape(Hkv, G, D).mean(1).reshape(-1)
    lib = torch.nn.functional.cosine_similarity(qa[None, :], reps.double(), dim=1)
    assert torch.allclose(s.double(), lib, atol=1e-7, rtol=0)
    # the other natural GQA reading: concatenate all H_q query heads, repeat each key head G times
    q_cat = qbar.reshape(-1)
    reps_rep = reps.double().reshape(T, Hkv, 1, D).expand(T, Hkv, G, D).reshape(T, -1)
    alt = torch.nn.functional.cosine_similarity(q_cat[None, :], reps_rep, dim=1)
    assert torch.equal(torch.argsort(alt, descending=True, stable=True), torch.argsort(lib, descending=True, stable=True))


def test_block_scores_are_cosine_with_the_mean_of_the_frame_vectors():
    Hq, Hkv, D, T, b = 8, 2, 128, 23, 4
    q = synth.question(11, 3, 1, 6, Hq, D)[0]
    reps = torch.stack([orc.pool_frame(synth.frame(11, synth.K, f, 1, 16, Hkv, D)[0]) for f in range(T)])
    n_blocks = T // b
    s = orc.score_blocks(q, reps, Hkv, n_blocks, b)
    qa = orc.question_vector(q, Hkv)
    blocks = reps[:n_blocks * b].double().reshape(n_blocks, b, -1).mean(1)
    lib = torch.nn.functional.cosine_similarity(qa[None, :], blocks, dim=1)
    assert torch.allclose(s.double(), lib, atol=1e-7, rtol=0)
    # b = 1 is the frame rule; identical frames inside a block give that frame's score
    assert torch.equal(orc.score_blocks(q, reps, Hkv, T, 1), orc.score(q, reps, Hkv))
    same = reps[:1].expand(b, -1).contiguous()
    assert abs(orc.score_blocks(q, same, Hkv, 1, b)[0].item() - orc.score(q, reps[:1].contiguous(), Hkv)[0].item()) < 1e-7


def test_block_geometry_and_selection():
    # 23 visible frames, window 3, blocks of 4: candidates [0,20) -> 5 complete blocks, no leftover
    assert orc.block_geometry(23, 3, 4, 8) == (5, 2, 3)
    # 26 visible: candidates [0,23) -> 5 blocks, frames 20..25 (window 3 + 3 that fill no block) always in context
    assert orc.block_geometry(26, 3, 4, 8) == (5, 2, 6)
    assert orc.block_geometry(5, 3, 4, 8) == (0, 0, 5)
    L, Hq, Hkv, D, Nf, T = 1, 8, 2, 128, 16, 26
    cache = orc.OracleCache(L, Hq, Hkv, D, Nf, window=3, block=4)
    for f in range(T):
        cache.append(synth.frame(2503, synth.K, f, L, Nf, Hkv, D), synth.frame(2503, synth.V, f, L, Nf, Hkv, D))
    q = synth.question(2503, 1, L, 8, Hq, D)
    res = cache.question(q, top_k=8, n_visible=T)
    idx = res["idx"][0].tolist()
    assert res["k_eff"] == 8 and idx == sorted(idx)
    assert all(idx[j * 4 + f] == idx[j * 4] + f and idx[j * 4] % 4 == 0 for j in range(2) for f in range(4))
    best = torch.argsort(res["scores"][0], descending=True, stable=True)[:2].sort().values.tolist()
    assert [idx[0] // 4, idx[4] // 4] == best
    assert res["k_ctx"].shape[2] == (8 + 6) * Nf  # retrieved frames + the six trailing frames


# ----------------------------------------------------------------------------- step 3: selection
def _brute_select(scores, n_vis, W, k):
    cand = list(range(max(n_vis - W, 0)))
    key = lambda f: (-(scores[f] if not math.isnan(scores[f]) else -math.inf), f)
    order = sorted(cand, key=key)
    return sorted(order[:min(k, len(cand))])


def test_select_brute_force_and_nestedness():
    g = torch.Generator().manual_seed(5)
    for trial in range(20):
        T = int(torch.randint(1, 64, (1,), generator=g))
        W = int(torch.randint(0, 6, (1,), generator=g))
        s = torch.randn(T, generator=g)
        prev = set()
        for k in range(0, T + 2):
            idx, k_eff, gap = orc.select(s, T, W, k)
            want = _brute_select(s.tolist(), T, W, k)
            assert k_eff == len(want)
            assert idx[:k_eff].tolist() == want
            assert (idx[k_eff:] == -1).all()
            assert prev <= set(want)
            prev = set(want)
            assert gap >= 0


def test_select_ties_go_to_lowest_index_and_nan_ranks_last():
    s = torch.tensor([0.5, 0.7, 0.5, 0.7, 0.5, float("nan"), 0.1])
    idx, k_eff, gap = orc.select(s, 7, 0, 3)
    assert idx.tolist() == [0, 1, 3] and k_eff == 3 and gap == 0.0
    idx, k_eff, _ = orc.select(s, 7, 0, 6)
    assert idx.tolist() == [0, 1, 2, 3, 4, 6]
    idx, k_eff, _ = orc.select(s, 7, 0, 7)
    assert idx.tolist() == [0, 1, 2, 3, 4, 5, 6]


def test_select_window_excluded_and_degenerate_counts():
    s = torch.tensor([0.1, 0.9, 0.2, 0.95, 0.99])
    idx, k_eff, _ = orc.select(s, 5, 2, 2)  # frames 3, 4 are the window
    assert idx.tolist() == [1, 2] and k_eff == 2
    idx, k_eff, gap = orc.select(s, 5, 2, 8)
    assert idx.tolist() == [0, 1, 2, -1, -1, -1, -1, -1] and k_eff == 3 and gap == math.inf
    idx, k_eff, _ = orc.select(s, 2, 4, 3)  # fewer visible frames than the window
    assert k_eff == 0 and idx.tolist() == [-1, -1, -1]
    idx, k_eff, _ = orc.select(s, 4, 2, 2)  # n_visible cuts the stream
    assert idx.tolist() == [0, 1]


def test_select_permutation_invariance():
    g = torch.Generator().manual_seed(9)
    s = torch.randn(50, generator=g)
    perm = torch.randperm(50, generator=g)
    idx, k_eff, _ = orc.select(s, 50, 0, 12)
    idx_p, k_eff_p, _ = orc.select(s[perm].contiguous(), 50, 0, 12)
    # position j of the permuted array holds original frame perm[j]
    assert sorted(perm[idx_p[:k_eff_p].long()].tolist()) == idx[:k_eff].tolist()


def test_planted_needle_frame_is_retrieved():
    """Adding a multiple of one frame's representative to every question token makes that frame win."""
    L, Hq, Hkv, D, Nf, T = 1, 8, 2, 128, 16, 64
    G = Hq // Hkv
    cache = orc.OracleCache(L, Hq, Hkv, D, Nf, window=4)
    for f in range(T):
        cache.append(synth.frame(2503, synth.K, f, L, Nf, Hkv, D), synth.frame(2503, synth.V, f, L, Nf, Hkv, D))
    target = 23
    q = synth.question(2503, 0, L, 16, Hq, D).float()
    rep = cache.reps[target][0].reshape(Hkv, D)
    for h in range(Hq):
        q[0, :, h, :] += 8.0 * rep[h // G]
    scores, idx, k_eff, _ = cache.retrieve(bf16(q), 1, T)
    assert k_eff == 1 and idx[0, 0].item() == target


# ----------------------------------------------------------------------------- step 4: gather
def test_gather_is_a_pure_copy_in_temporal_order():
    L, Hkv, D, Nf, T, W = 1, 2, 128, 16, 20, 3
    cacheK = torch.stack([synth.frame(1, synth.K, f, L, Nf, Hkv, D)[0] for f in range(T)]).contiguous()
    idx = torch.tensor([2, 7, 11, -1], dtype=torch.int32)
    ctx = orc.gather(cacheK, idx, 3, 18, W)  # n_visible = 18 -> window frames 15, 16, 17
    frames = [2, 7, 11, 15, 16, 17]
    assert ctx.shape == (Hkv, len(frames) * Nf, D)
    for h in range(Hkv):
        for j, f in enumerate(frames):
            assert torch.equal(ctx[h, j * Nf:(j + 1) * Nf], cacheK[f, :, h, :])


# ----------------------------------------------------------------------------- step 5: attention (Eq. 3)
def _rand_ctx(seed, Hkv, n_ctx, D):
    g = torch.Generator().manual_seed(seed)
    return bf16(torch.randn(Hkv, n_ctx, D, generator=g)), bf16(torch.randn(Hkv, n_ctx, D, generator=g))


def test_attend_softmax_rows_sum_to_one_and_ones_value_gives_ones():
    q = synth.question(1, 0, 1, 4, 8, 128)[0]
    k, _ = _rand_ctx(0, 2, 37, 128)
    v = bf16(torch.ones(2, 37, 128))
    out, out_b, probs = orc.attend(q, k, v, want_probs=True)
    assert torch.allclose(probs.sum(-1), torch.ones(4, 8, dtype=torch.float64), atol=1e-14)
    assert (probs >= 0).all()
    assert torch.allclose(out, torch.ones_like(out), atol=1e-6)


def test_attend_single_token_returns_its_value_and_equal_keys_give_mean_value():
    q = synth.question(1, 1, 1, 3, 8, 128)[0]
    k, v = _rand_ctx(1, 2, 1, 128)
    out, _, _ = orc.attend(q, k, v)
    for h in range(8):
        assert torch.equal(out[:, h, :], v[h // 4, 0].float().expand(3, 128))
    k2 = bf16(torch.randn(2, 1, 128, generator=torch.Generator().manual_seed(3))).expand(2, 9, 128).contiguous()
    _, v2 = _rand_ctx(2, 2, 9, 128)
    out2, _, _ = orc.attend(q, k2, v2)
    for h in range(8):
        want = v2[h // 4].double().mean(0).float()
        assert torch.allclose(out2[0, h], want, atol=1e-6)


def test_attend_matches_library_sdpa_with_gqa_head_repeat():
    Hq, Hkv, D, n_ctx, n_q = 8, 2, 128, 83, 5
    q = synth.question(4, 2, 1, n_q, Hq, D)[0]
    k, v = _rand_ctx(4, Hkv, n_ctx, D)
    out, out_b, _ = orc.attend(q, k, v)
    qd = q.double().permute(1, 0, 2)[None]  # [1][Hq][n_q][D]
    kd = k.double().repeat_interleave(Hq // Hkv, dim=0)[None]
    vd = v.double().repeat_interleave(Hq // Hkv, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(qd, kd, vd)[0].permute(1, 0, 2)
    assert torch.allclose(out.double(), ref, atol=2e-7, rtol=0)
    assert torch.equal(out_b, out.to(torch.bfloat16))


def test_full_retrieval_equals_full_attention_over_all_visible_frames():
    """k >= number of candidates: the retrieved context is every visible frame, so the whole
    five-step path must equal plain attention over the visible stream."""
    L, Hq, Hkv, D, Nf, T, W = 1, 8, 2, 128, 16, 24, 4
    cache = orc.OracleCache(L, Hq, Hkv, D, Nf, window=W)
    for f in range(T):
        cache.append(synth.frame(540, synth.K, f, L, Nf, Hkv, D), synth.frame(540, synth.V, f, L, Nf, Hkv, D))
    q = synth.question(540, 0, L, 6, Hq, D)
    n_vis = 21
    res = cache.question(q, top_k=64, n_visible=n_vis)
    assert res["k_eff"] == n_vis - W
    assert res["idx"][0, :n_vis - W].tolist() == list(range(n_vis - W))
    k_all = cache.layer_cache(0, "k")[:n_vis].permute(2, 0, 1, 3).reshape(Hkv, n_vis * Nf, D)
    v_all = cache.layer_cache(0, "v")[:n_vis].permute(2, 0, 1, 3).reshape(Hkv, n_vis * Nf, D)
    assert torch.equal(res["k_ctx"][0], k_all) and torch.equal(res["v_ctx"][0], v_all)
    qd = q[0].double().permute(1, 0, 2)[None]
    kd = k_all.double().repeat_interleave(Hq // Hkv, dim=0)[None]
    vd = v_all.double().repeat_interleave(Hq // Hkv, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(qd, kd, vd)[0].permute(1, 0, 2)
    assert torch.allclose(res["out"][0].double(), ref, atol=2e-7, rtol=0)


def test_attention_is_invariant_to_context_order():
    q = synth.question(8, 0, 1, 2, 8, 128)[0]
    k, v = _rand_ctx(8, 2, 40, 128)
    perm = torch.randperm(40, generator=torch.Generator().manual_seed(0))
    a, _, _ = orc.attend(q, k, v)
    b, _, _ = orc.attend(q, k[:, perm].contiguous(), v[:, perm].contiguous())
    assert torch.allclose(a, b, atol=1e-6)


# ----------------------------------------------------------------------------- external retrieval (Eq. 2 with tau)
def test_external_scores_closed_forms_and_library_cosine():
    g = torch.Generator().manual_seed(9)
    E, T = 1152, 40
    embs = torch.randn(T, E, generator=g)
    q = torch.randn(E, generator=g)
    embs[3] = 2.5 * q          # parallel -> 1 / tau
    embs[4] = -0.5 * q         # antiparallel -> -1 / tau
    embs[5] = 0.0
    embs[5, 0], q0 = 1.0, q.clone()
    q0[0] = 0.0                # orthogonal to frame 5
    for tau in (1.0, 0.07, 3.0):
        s = orc.score_external(q, embs, tau)
        assert abs(s[3].item() - 1 / tau) < 1e-5 / tau and abs(s[4].item() + 1 / tau) < 1e-5 / tau
        ref = torch.nn.functional.cosine_similarity(embs.double(), q.double()[None], dim=1) / tau
        np.testing.assert_allclose(s.double().numpy(), ref.numpy(), rtol=0, atol=2e-7 / tau)
        assert orc.score_external(q0, embs, tau)[5].item() == 0.0
        # positive rescaling of the question or of a frame changes nothing; tau only rescales
        np.testing.assert_allclose(orc.score_external(7 * q, embs, tau).numpy(), s.numpy(), atol=2e-6 / tau)
        np.testing.assert_allclose((orc.score_external(q, embs, 1.0) / tau).numpy(), s.numpy(), rtol=1e-6, atol=1e-9)
    # zero vectors are clamped, not NaN
    assert orc.score_external(torch.zeros(E), embs, 1.0).abs().max().item() == 0.0


def test_external_retrieval_selection_is_tau_invariant_and_blocks_average_frames():
    g = torch.Generator().manual_seed(10)
    E, T, W = 64, 50, 4
    embs = torch.randn(T, E, generator=g)
    q = torch.randn(E, generator=g)
    s1, i1, k1, _ = orc.retrieve_external(q, embs, 1.0, 8, T, W)
    s2, i2, k2, _ = orc.retrieve_external(q, embs, 0.05, 8, T, W)
    assert torch.equal(i1, i2) and k1 == k2 == 8
    brute = sorted(sorted(range(T - W), key=lambda f: (-s1[f].item(), f))[:8])
    assert i1.tolist() == brute
    assert all(f < T - W for f in i1.tolist())          # the window is not a candidate
    # blocks: the vector of a block is the mean of its frame vectors
    b = 4
    sb, ib, kb, _ = orc.retrieve_external(q, embs, 0.5, 8, T, W, b)
    n_blocks = (T - W) // b
    means = embs[: n_blocks * b].view(n_blocks, b, E).double().mean(dim=1)
    ref = torch.nn.functional.cosine_similarity(means, q.double()[None], dim=1) / 0.5
    np.testing.assert_allclose(sb.double().numpy(), ref.numpy(), atol=1e-6)
    top = sorted(sorted(range(n_blocks), key=lambda j: (-sb[j].item(), j))[:2])
    assert ib.tolist() == [j * b + f for j in top for f in range(b)] and kb == 8


# ----------------------------------------------------------------------------- quantised host tier (FP8 E4M3)
def test_e4m3_rounding_matches_the_format_and_the_library_conversion():
    # every code decodes to the value the format defines, and encodes back to itself
    for c in range(256):
        if (c & 0x7F) == 0x7F:
            continue  # NaN codes
        v = orc.e4m3_decode(c)
        e, m = (c >> 3) & 15, c & 7
        ref = (m / 8 * 2.0 ** -6) if e == 0 else (1 + m / 8) * 2.0 ** (e - 7)
        assert abs(v) == ref and (v < 0 or c < 128 or ref == 0)
        if ref != 0:
            assert orc.e4m3_encode(v) == c
    assert orc.e4m3_decode(0x7E) == 448.0 and orc.e4m3_decode(0x08) == 2.0 ** -6 and orc.e4m3_decode(0x01) == 2.0 ** -9
    # ties go to the even mantissa; beyond the largest value it saturates
    assert orc.e4m3_decode(orc.e4m3_encode(1.0625)) == 1.0      # midway 1.0 / 1.125 -> even (1.0)
    assert orc.e4m3_decode(orc.e4m3_encode(1.1875)) == 1.25     # midway 1.125 / 1.25 -> even (1.25)
    assert orc.e4m3_decode(orc.e4m3_encode(2.0 ** -10)) == 0.0  # midway 0 / 2^-9 -> even (0)
    assert orc.e4m3_decode(orc.e4m3_encode(3 * 2.0 ** -10)) == 2.0 ** -8
    assert orc.e4m3_decode(orc.e4m3_encode(1e4)) == 448.0 and orc.e4m3_decode(orc.e4m3_encode(-460.0)) == -448.0
    # the library's conversion (torch.float8_e4m3fn, round to nearest even) on a dense sweep of the finite range
    g = torch.Generator().manual_seed(4)
    x = torch.cat([torch.randn(20000, generator=g) * s for s in (1e-3, 0.02, 1.0, 30.0, 150.0)]).clamp(-448, 448)
    lib = x.to(torch.float8_e4m3fn).float()
    mine = torch.tensor([orc.e4m3_decode(orc.e4m3_encode(float(v))) for v in x.tolist()])
    assert torch.equal(lib, mine)


def test_fp8_roundtrip_of_page_rows():
    g = torch.Generator().manual_seed(5)
    x = bf16(torch.randn(64, 128, generator=g) * torch.logspace(-3, 2, 64)[:, None])
    y, scales = orc.fp8_roundtrip(x, want_scales=True)
    amax = x.float().abs().amax(dim=1)
    assert torch.equal(scales, amax / 448.0)
    # independent statement with the library's conversion
    ref = ((x.float() / scales[:, None]).to(torch.float8_e4m3fn).float() * scales[:, None]).to(torch.bfloat16)
    assert torch.equal(y, ref)
    # the row's largest element survives exactly, every element within half a code step of its binade
    idx = x.float().abs().argmax(dim=1)
    assert torch.equal(y[torch.arange(64), idx], x[torch.arange(64), idx])
    rel = ((y.float() - x.float()).abs() / amax[:, None]).max().item()
    assert rel <= 16.0 / 448.0 + 2.0 ** -8     # half a code step of the top binade (32 / 2 of 448), plus the bf16 rounding
    # an all-zero row stays zero (scale 1), and the operation is idempotent
    z = bf16(torch.zeros(2, 128))
    assert torch.equal(orc.fp8_roundtrip(z), z)
    assert torch.equal(orc.fp8_roundtrip(y), y)


# ----------------------------------------------------------------------------- Eq. 3 in full: X's own K/V, RoPE
def _complex_rope(x: np.ndarray, pos: int, theta: float) -> np.ndarray:
    """RoFormer's definition: (x_i + i x_{i+D/2}) * exp(i * pos * theta^(-2i/D)), an independent statement."""
    d = x.shape[-1]
    z = x[..., : d // 2] + 1j * x[..., d // 2:]
    ang = pos * theta ** (-2.0 * np.arange(d // 2) / d)
    z = z * np.exp(1j * ang)
    return np.concatenate([z.real, z.imag], axis=-1)


def test_rope_closed_forms():
    g = torch.Generator().manual_seed(3)
    x = torch.randn(128, dtype=torch.float64, generator=g)
    theta = 1e6
    assert torch.equal(orc.rope(x, 0, theta), x)                                   # position 0 is the identity
    for pos in (1, 7, 196, 14111):
        r = orc.rope(x, pos, theta)
        assert abs(r.norm().item() - x.norm().item()) < 1e-12                      # a rotation keeps the norm
        np.testing.assert_allclose(r.numpy(), _complex_rope(x.numpy(), pos, theta), rtol=0, atol=1e-9)
    # rotations compose: R(a) R(b) = R(a + b); and the first pair turns by exactly pos radians
    np.testing.assert_allclose(orc.rope(orc.rope(x, 5, theta), 11, theta).numpy(), orc.rope(x, 16, theta).numpy(),
                               atol=1e-12)
    e0 = torch.zeros(128, dtype=torch.float64)
    e0[0] = 1.0
    r = orc.rope(e0, 3, theta)
    assert abs(r[0].item() - math.cos(3.0)) < 1e-15 and abs(r[64].item() - math.sin(3.0)) < 1e-15
    # the dot product of a rotated query and key depends on the position difference only
    y = torch.randn(128, dtype=torch.float64, generator=g)
    d1 = torch.dot(orc.rope(x, 40, theta), orc.rope(y, 33, theta)).item()
    d2 = torch.dot(orc.rope(x, 1007, theta), orc.rope(y, 1000, theta)).item()
    assert abs(d1 - d2) < 1e-9


def _sdpa_full(q, k_ctx, v_ctx, k_self, v_self, theta, static_ctx=False):
    """torch's scaled_dot_product_attention in fp64 on [R, X] with an explicit mask, GQA by head repetition,
    rotary embedding by the complex-number form, rotated vectors rounded to bf16."""
    n_q, hq, d = q.shape
    hkv, n_ctx, _ = k_ctx.shape
    n_self = k_self.shape[0]
    G = hq // hkv

    def rot(x, pos):  # x: bf16 [..., D] at integer positions pos (broadcast on the leading dims)
        xd = x.double().numpy()
        if theta <= 0:
            return torch.from_numpy(xd)
        out = np.empty_like(xd)
        for idx in np.ndindex(xd.shape[:-1]):
            out[idx] = _complex_rope(xd[idx], int(pos[idx]), theta)
        return torch.from_numpy(out).float().to(torch.bfloat16).double()

    k_all = torch.cat([k_ctx.permute(1, 0, 2), k_self], dim=0)          # [n_ctx + n_self][hkv][d]
    v_all = torch.cat([v_ctx.permute(1, 0, 2), v_self], dim=0).double()
    n_all = n_ctx + n_self
    if static_ctx:  # every context token at position 0, token s of X at 1 + s
        pos_1d = np.concatenate([np.zeros(n_ctx, dtype=np.int64), 1 + np.arange(n_self)])
        pos_q1 = 1 + n_self - n_q + np.arange(n_q)
    else:
        pos_1d, pos_q1 = np.arange(n_all), n_ctx + n_self - n_q + np.arange(n_q)
    pos_k = np.broadcast_to(pos_1d[:, None], (n_all, hkv))
    pos_q = np.broadcast_to(pos_q1[:, None], (n_q, hq))
    kr, qr = rot(k_all, pos_k), rot(q, pos_q)
    kh = kr.permute(1, 0, 2).repeat_interleave(G, dim=0)                # [hq][n_all][d]
    vh = v_all.permute(1, 0, 2).repeat_interleave(G, dim=0)
    mask = torch.zeros(n_q, n_all, dtype=torch.bool)
    for n in range(n_q):
        mask[n, : n_ctx + n_self - n_q + n + 1] = True
    o = torch.nn.functional.scaled_dot_product_attention(qr.permute(1, 0, 2), kh, vh, attn_mask=mask)
    return o.permute(1, 0, 2)


def _full_inputs(seed, n_q, n_self, n_ctx, hq=4, hkv=2, d=128):
    g = torch.Generator().manual_seed(seed)
    r = lambda *sh: bf16(torch.randn(*sh, generator=g))
    return r(n_q, hq, d), r(hkv, n_ctx, d), r(hkv, n_ctx, d), r(n_self, hkv, d), r(n_self, hkv, d)


@pytest.mark.parametrize("theta", [0.0, 1e6])
def test_attend_full_matches_masked_sdpa(theta):
    for seed, (n_q, n_self, n_ctx) in enumerate([(5, 5, 12), (1, 9, 7), (3, 8, 0), (6, 6, 40)]):
        q, kc, vc, ks, vs = _full_inputs(seed, n_q, n_self, n_ctx)
        out, out_b = orc.attend_full(q, kc, vc, ks, vs, theta)
        ref = _sdpa_full(q, kc, vc, ks, vs, theta)
        np.testing.assert_allclose(out.double().numpy(), ref.numpy(), rtol=0, atol=2e-6)
        assert torch.equal(out_b, out.to(torch.bfloat16))


def test_attend_full_reduces_to_the_special_cases():
    q, kc, vc, ks, vs = _full_inputs(11, 4, 4, 10)
    # no retrieved context, no positions: plain causal self-attention; its first row is the first token's value
    empty = torch.empty(2, 0, 128, dtype=torch.bfloat16)
    out, _ = orc.attend_full(q, empty, empty, ks, vs, 0.0)
    ref = torch.nn.functional.scaled_dot_product_attention(
        q.double().permute(1, 0, 2), ks.double().permute(1, 0, 2).repeat_interleave(2, dim=0),
        vs.double().permute(1, 0, 2).repeat_interleave(2, dim=0), is_causal=True).permute(1, 0, 2)
    np.testing.assert_allclose(out.double().numpy(), ref.numpy(), atol=2e-6)
    for h in range(4):
        assert torch.equal(out[0, h], vs[0, h // 2].float())
    # the tokens of X that follow a query do not reach it
    ks2, vs2 = ks.clone(), vs.clone()
    ks2[3], vs2[3] = bf16(torch.ones(2, 128)), bf16(torch.full((2, 128), 5.0))
    out2, _ = orc.attend_full(q, kc, vc, ks2, vs2, 1e6)
    out1, _ = orc.attend_full(q, kc, vc, ks, vs, 1e6)
    assert torch.equal(out2[:3], out1[:3]) and not torch.equal(out2[3], out1[3])
    # a decode step (one query, X grown by one token) is the last row of the same computation done at once
    for theta in (0.0, 1e6):
        whole, _ = orc.attend_full(q, kc, vc, ks, vs, theta)
        last, _ = orc.attend_full(q[3:].contiguous(), kc, vc, ks, vs, theta)
        assert torch.equal(last[0], whole[3])
    # values all ones -> output all ones, with or without positions
    ones_c, ones_s = bf16(torch.ones(2, 10, 128)), bf16(torch.ones(4, 2, 128))
    for theta in (0.0, 1e4):
        o, _ = orc.attend_full(q, kc, ones_c, ks, ones_s, theta)
        assert (o - 1).abs().max().item() < 1e-6


def test_attend_full_positions_are_relative_and_ordered():
    """With rotary embedding the retrieved tokens count as consecutive tokens: the result changes when two
    context tokens swap places (it does not without positions), and a key far away in position that equals
    the query direction scores as the rotation by the distance says."""
    q, kc, vc, ks, vs = _full_inputs(5, 2, 2, 6)
    perm = [1, 0, 2, 3, 4, 5]
    a0, _ = orc.attend_full(q, kc, vc, ks, vs, 0.0)
    b0, _ = orc.attend_full(q, kc[:, perm].contiguous(), vc[:, perm].contiguous(), ks, vs, 0.0)
    np.testing.assert_allclose(a0.numpy(), b0.numpy(), atol=1e-6)
    a1, _ = orc.attend_full(q, kc, vc, ks, vs, 1e6)
    b1, _ = orc.attend_full(q, kc[:, perm].contiguous(), vc[:, perm].contiguous(), ks, vs, 1e6)
    assert (a1 - b1).abs().max().item() > 1e-3


# ----------------------------------------------------------------------------- input generator
def test_synthetic_inputs_have_the_stated_distribution():
    k = synth.frame(2503, synth.K, 0, 2, 196, 4, 128, off_scale=0.0).float()
    assert abs(k.mean().item()) < 0.01 and abs(k.std().item() - 1.0) < 0.01
    ko = synth.frame(2503, synth.K, 0, 2, 196, 4, 128, off_scale=0.5).float()
    off = ko.mean(1)  # per (layer, head, dim) frame mean ~ N(0, 0.5^2 + 1/196)
    assert abs(off.std().item() - math.sqrt(0.25 + 1 / 196)) < 0.03
    # stateless: a layer slice equals the same layer generated alone
    k1 = synth.frame(2503, synth.K, 0, 1, 196, 4, 128, off_scale=0.5, layer0=1)
    assert torch.equal(k1[0], synth.frame(2503, synth.K, 0, 2, 196, 4, 128, off_scale=0.5)[1])
    lens = synth.question_lengths(7, 64, 24, 64)
    assert min(lens) >= 24 and max(lens) <= 64 and len(set(lens)) > 10


def test_attend_full_static_positions_match_masked_sdpa_and_forget_the_context_order():
    """The static variant of the "Positional Encoding" paragraph: all retrieved tokens share one position.  Against
    fp64 SDPA with the complex-number rotation at positions (0, ..., 0, 1, 2, ...); and, unlike consecutive positions,
    the result must not change when the context tokens are permuted (with consecutive positions it does)."""
    theta = 1e6
    for seed, (n_q, n_self, n_ctx) in enumerate([(5, 5, 12), (1, 9, 7), (6, 6, 40)]):
        q, kc, vc, ks, vs = _full_inputs(100 + seed, n_q, n_self, n_ctx)
        o, _ = orc.attend_full(q, kc, vc, ks, vs, theta, static_ctx=True)
        ref = _sdpa_full(q, kc, vc, ks, vs, theta, static_ctx=True)
        assert (o.double() - ref).abs().max().item() < 2e-6
        perm = torch.randperm(n_ctx, generator=torch.Generator().manual_seed(seed))
        o_p, _ = orc.attend_full(q, kc[:, perm].contiguous(), vc[:, perm].contiguous(), ks, vs, theta, static_ctx=True)
        assert (o - o_p).abs().max().item() < 1e-6
        o_c, _ = orc.attend_full(q, kc, vc, ks, vs, theta)
        o_cp, _ = orc.attend_full(q, kc[:, perm].contiguous(), vc[:, perm].contiguous(), ks, vs, theta)
        assert (o_c - o_cp).abs().max().item() > 1e-3      # consecutive positions do depend on the order
        assert (o - o_c).abs().max().item() > 1e-3         # and the two variants differ
    # without a rotation the flag changes nothing
    q, kc, vc, ks, vs = _full_inputs(7, 4, 6, 9)
    a, _ = orc.attend_full(q, kc, vc, ks, vs, 0.0, static_ctx=True)
    b, _ = orc.attend_full(q, kc, vc, ks, vs, 0.0)
    assert torch.equal(a, b)
