"""Pins of the CPU oracle against what the definition and the mathematics fix.

The paper prints no worked value for this path, so every pin is definitional: brute force on
tiny inputs, closed forms, invariants and a hand-made example.  Each test is chosen so that a
plausible slip in the oracle (dropped term, wrong index, transposed operand, wrong divisor)
fails it.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
from tests.bruteforce import bf16_round, dense_softmax_attention, expand_block_mask, to_f64

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_qkv(rng, H, N, D, scale=1.0):
    return tuple(bf16_round(rng.standard_normal((H, N, D)) * scale) for _ in range(3))


# ---------------------------------------------------------------- pooling and scores

def test_pool_constant_blocks_and_tail_divisor():
    # block i holds the constant (i+1) in channel 0 and -(i+1)/2 in channel 1; tail block has 13 tokens
    N, D = 64 * 2 + 13, 4
    x = np.zeros((1, N, D), dtype=np.float32)
    for n in range(N):
        x[0, n, 0] = n // 64 + 1
        x[0, n, 1] = -(n // 64 + 1) / 2
    # channel 2: one spike per block -> mean = spike / count (count = 13 in the tail, not 64)
    x[0, 0, 2] = 64.0
    x[0, 64, 2] = 32.0
    x[0, 128, 2] = 26.0
    p = oracle.block_pool(bf16_round(x))
    assert p.shape == (1, 3, D)
    np.testing.assert_allclose(p[0, :, 0], [1, 2, 3], rtol=0, atol=0)
    np.testing.assert_allclose(p[0, :, 1], [-0.5, -1.0, -1.5], rtol=0, atol=0)
    np.testing.assert_allclose(p[0, :, 2], [1.0, 0.5, 2.0], rtol=0, atol=1e-15)
    np.testing.assert_allclose(p[0, :, 3], 0.0)


def test_scores_orientation_by_hand():
    # pooled Q rows are unit vectors e_i, pooled K rows are j * e_0 + e_1:
    # S[i, j] = j for i = 0, 1 for i = 1, 0 otherwise.  A transposed operand gives a different table.
    nb, D = 3, 4
    pq = np.zeros((1, nb, D)); pk = np.zeros((1, nb, D))
    for i in range(nb):
        pq[0, i, i] = 1.0
        pk[0, i, 0] = float(i)
        pk[0, i, 1] = 1.0
    S = oracle.block_scores(pq, pk)
    np.testing.assert_array_equal(S[0], [[0, 1, 2], [1, 1, 1], [0, 0, 0]])


def test_scores_from_tokens_hand_example():
    # two blocks; Q tokens of block 0 are all (2, 0), of block 1 all (0, 4); K block 0 all (1, 1), block 1 all (3, -1)
    N, D = 128, 2
    q = np.zeros((1, N, D), np.float32); k = np.zeros((1, N, D), np.float32)
    q[0, :64] = (2, 0); q[0, 64:] = (0, 4)
    k[0, :64] = (1, 1); k[0, 64:] = (3, -1)
    S = oracle.image_scores(bf16_round(q), bf16_round(k))
    np.testing.assert_array_equal(S[0], [[2, 6], [4, -4]])
    assert S.dtype == np.float32


# ---------------------------------------------------------------- mask selection

def _read_golden():
    scores, masks, cur = [], {}, None
    for line in open(os.path.join(GOLDEN, "hand_mask_5blocks.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line == "scores":
            cur = scores
        elif line.startswith("mask ratio"):
            cur = masks.setdefault(float(line.split()[-1]), [])
        else:
            cur.append([float(t) for t in line.split()])
    return np.array(scores), {r: np.array(m, dtype=np.uint8) for r, m in masks.items()}


def test_hand_example_mask():
    S, masks = _read_golden()
    for ratio, want in masks.items():
        got, gap = oracle.select_mask(S[None], n_text=64, ratio=ratio)
        np.testing.assert_array_equal(got[0], want, err_msg=f"ratio {ratio}")
    # the exact tie in row 2 at ratio 0.5 is reported through a zero gap
    _, gap = oracle.select_mask(S[None], n_text=64, ratio=0.5)
    assert gap[0, 2] == 0.0 and gap[0, 1] > 0 and math.isinf(gap[0, 0])


@pytest.mark.parametrize("nb,n_text", [(5, 64), (9, 100), (12, 0), (70, 333), (72, 512)])
def test_kept_count_identity_and_structure(nb, n_text):
    rng = np.random.default_rng(nb)
    S = rng.standard_normal((2, nb, nb))
    ntb = (n_text + 63) // 64
    prev = None
    for ratio in [1.0 / 63, 0.1, 0.25, 1 / 3, 0.5, 0.75, 0.999, 1.0]:
        mask, _ = oracle.select_mask(S, n_text, ratio)
        assert mask.shape == (2, nb, nb)
        for h in range(2):
            for i in range(nb):
                row = mask[h, i]
                if i < ntb:
                    assert row.sum() == nb          # text query rows are dense
                    continue
                n_forced = ntb + 1
                n_free = nb - n_forced
                k = min(n_free, max(0, math.ceil(ratio * n_free - 1e-6)))
                assert row.sum() == k + n_forced
                assert row[:ntb].all() and row[i] == 1
        if prev is not None:                       # nested in the ratio
            assert ((prev == 1) <= (mask == 1)).all()
        prev = mask
    assert prev.all()                               # ratio 1.0 keeps everything


def test_per_head_ratios_select_each_head_on_its_own():
    # a head's mask depends on that head's scores and ratio alone: brute force per head, and the
    # heads must not leak into each other (swapping two ratios swaps nothing but the counts)
    rng = np.random.default_rng(5)
    H, N, D, n_text = 3, 7 * 64 + 9, 16, 70
    qt, kt, _ = rand_qkv(rng, H, N, D)
    ratios = [0.2, 1.0, 0.6]
    S32, mask, gap = oracle.image_mask_heads(qt, kt, n_text, ratios)
    nb, ntb = 8, 2
    assert mask.shape == (H, nb, nb) and gap.shape == (H, nb)
    S = S32.astype(np.float64)
    for h, r in enumerate(ratios):
        for i in range(ntb, nb):
            free = [j for j in range(ntb, nb) if j != i]
            kk = oracle.keep_count(r, len(free))
            best = max(itertools.combinations(free, kk), key=lambda c: sum(S[h, i, j] for j in c))
            assert [j for j in free if mask[h, i, j]] == sorted(best)
            assert mask[h, i, :ntb].all() and mask[h, i, i]
        assert mask[h, :ntb].all()
    assert mask[1].all()
    # one ratio for all heads is the per-image rule
    _, m_same, _ = oracle.image_mask_heads(qt, kt, n_text, [0.6] * H)
    _, m_img, _ = oracle.image_mask(qt, kt, n_text, 0.6)
    assert (m_same == m_img).all() and (m_same[2] == mask[2]).all()


def test_keep_count_rounding():
    assert oracle.keep_count(0.5, 63) == 32
    assert oracle.keep_count(0.25, 63) == 16
    assert oracle.keep_count(0.25, 255) == 64
    assert oracle.keep_count(1.0, 63) == 63
    assert oracle.keep_count(float(np.float32(0.1)), 10) == 1      # 0.1f is a hair above 1/10
    assert oracle.keep_count(float(np.float32(0.2)), 5) == 1
    assert oracle.keep_count(1e-9, 10) == 0
    assert oracle.keep_count(0.5, 0) == 0
    assert oracle.keep_count(0.30000001, 10) == 3 and oracle.keep_count(0.31, 10) == 4


@pytest.mark.parametrize("nb,n_text,ratio", [(5, 64, 0.5), (6, 64, 0.5), (6, 0, 0.6), (6, 128, 0.34)])
def test_topk_maximises_score_sum_bruteforce(nb, n_text, ratio):
    rng = np.random.default_rng(7 * nb + n_text)
    S = rng.standard_normal((1, nb, nb))
    mask, _ = oracle.select_mask(S, n_text, ratio)
    ntb = (n_text + 63) // 64
    for i in range(ntb, nb):
        free = [j for j in range(nb) if j >= ntb and j != i]
        k = oracle.keep_count(ratio, len(free))
        best = max(itertools.combinations(free, k), key=lambda c: sum(S[0, i, j] for j in c))
        chosen = [j for j in free if mask[0, i, j]]
        assert sorted(best) == chosen


def test_zero_queries_tie_break_and_uniform_average():
    # Q = 0: every score ties, so the k lowest free indices are kept, and every softmax weight is
    # equal: the output is the plain mean of V over the kept valid tokens.
    rng = np.random.default_rng(3)
    H, N, D, n_text = 1, 64 * 6 + 13, 8, 64
    q = bf16_round(np.zeros((H, N, D)))
    k = bf16_round(rng.standard_normal((H, N, D)))
    v = bf16_round(rng.standard_normal((H, N, D)))
    res = oracle.sparse_joint_attention(q, k, v, n_text, 0.4, 0.37)
    nb = 7
    kk = oracle.keep_count(0.4, nb - 2)
    vf = to_f64(v)[0]
    for i in range(1, nb):
        free = [j for j in range(1, nb) if j != i]
        want = np.zeros(nb, np.uint8); want[0] = 1; want[i] = 1; want[free[:kk]] = 1
        np.testing.assert_array_equal(res["mask"][0, i], want)
        toks = np.concatenate([np.arange(64 * j, min(64 * j + 64, N)) for j in np.nonzero(want)[0]])
        np.testing.assert_allclose(res["out"][0, 64 * i], vf[toks].mean(axis=0), rtol=0, atol=1e-13)
    assert (res["gap"][0, 1:] == 0).all()


# ---------------------------------------------------------------- attention

@pytest.mark.parametrize("H,N,D,n_text", [(2, 320, 64, 64), (1, 64 * 3 + 13, 128, 64 + 13), (1, 150, 16, 0)])
def test_ratio_one_equals_dense_bruteforce(H, N, D, n_text):
    rng = np.random.default_rng(N)
    q, k, v = rand_qkv(rng, H, N, D)
    scale = 1.0 / math.sqrt(D)
    res = oracle.sparse_joint_attention(q, k, v, n_text, 1.0, scale)
    assert res["mask"].all()
    for h in range(H):
        want = dense_softmax_attention(to_f64(q)[h], to_f64(k)[h], to_f64(v)[h], scale)
        np.testing.assert_allclose(res["out"][h], want, rtol=0, atol=1e-12)


@pytest.mark.parametrize("N,n_text,ratio", [(64 * 4 + 13, 64 + 13, 0.5), (64 * 5, 64, 0.5), (64 * 6 + 1, 0, 0.3)])
def test_sparse_with_tails_equals_token_level_bruteforce(N, n_text, ratio):
    rng = np.random.default_rng(N + 1)
    H, D = 2, 32
    q, k, v = rand_qkv(rng, H, N, D)
    scale = 0.21
    res = oracle.sparse_joint_attention(q, k, v, n_text, ratio, scale)
    assert not res["mask"].all()
    for h in range(H):
        tm = expand_block_mask(res["mask"][h], N)
        want = dense_softmax_attention(to_f64(q)[h], to_f64(k)[h], to_f64(v)[h], scale, tm)
        np.testing.assert_allclose(res["out"][h], want, rtol=0, atol=1e-12)


def test_rows_are_convex_combinations():
    rng = np.random.default_rng(11)
    H, N, D, n_text = 1, 64 * 5 + 13, 16, 64
    q, k, v = rand_qkv(rng, H, N, D, scale=2.0)
    res = oracle.sparse_joint_attention(q, k, v, n_text, 0.5, 0.25)
    vf = to_f64(v)[0]
    for n in [0, 63, 64, 200, N - 1]:
        w = oracle.attention_weights(q, k, res["mask"], 0.25, 0, n)
        kept = expand_block_mask(res["mask"][0], N)[n]
        assert (w >= 0).all() and abs(w.sum() - 1.0) < 1e-12
        assert (w[~kept] == 0).all() and (w[kept] > 0).all()
        np.testing.assert_allclose(w @ vf, res["out"][0, n], rtol=0, atol=1e-12)
        assert (res["out"][0, n] <= vf[kept].max(axis=0) + 1e-12).all()
        assert (res["out"][0, n] >= vf[kept].min(axis=0) - 1e-12).all()


def test_invariant_to_permuting_keys_within_a_block():
    rng = np.random.default_rng(5)
    H, N, D, n_text = 1, 64 * 5, 32, 64
    q, k, v = rand_qkv(rng, H, N, D)
    perm = np.arange(N)
    for j in range(N // 64):
        perm[64 * j:64 * j + 64] = 64 * j + rng.permutation(64)
    a = oracle.sparse_joint_attention(q, k, v, n_text, 0.5, 0.2)
    b = oracle.sparse_joint_attention(q, k[:, perm], v[:, perm], n_text, 0.5, 0.2)
    np.testing.assert_array_equal(a["mask"], b["mask"])
    np.testing.assert_allclose(a["out"], b["out"], rtol=0, atol=1e-12)
    # permuting query tokens within a block permutes the output rows and leaves the mask alone
    c = oracle.sparse_joint_attention(q[:, perm], k, v, n_text, 0.5, 0.2)
    np.testing.assert_array_equal(a["mask"], c["mask"])
    np.testing.assert_allclose(a["out"][:, perm], c["out"], rtol=0, atol=1e-12)


def test_softmax_closed_forms():
    rng = np.random.default_rng(9)
    H, N, D, n_text = 1, 64 * 4 + 13, 8, 64
    q, k, v = rand_qkv(rng, H, N, D)
    # V constant -> output is that constant
    vc = bf16_round(np.broadcast_to(np.array([1.5, -2, 0.25, 3, 0, 1, -1, 7]), (H, N, D)).copy())
    res = oracle.sparse_joint_attention(q, k, vc, n_text, 0.5, 0.3)
    np.testing.assert_allclose(res["out"], to_f64(vc), rtol=0, atol=1e-13)
    # all K rows identical -> uniform weights -> mean of the kept V rows
    kc = bf16_round(np.broadcast_to(rng.standard_normal(D), (H, N, D)).copy())
    res = oracle.sparse_joint_attention(q, kc, v, n_text, 0.5, 0.3)
    for n in (70, N - 1):
        kept = expand_block_mask(res["mask"][0], N)[n]
        np.testing.assert_allclose(res["out"][0, n], to_f64(v)[0][kept].mean(axis=0), rtol=0, atol=1e-13)
    # one key with a huge logit margin -> output is that key's V row
    qd = np.zeros((H, N, D), np.float32); qd[..., 0] = 8.0
    kd = np.zeros((H, N, D), np.float32); kd[0, 17, 0] = 64.0          # token 17 is in text block 0: always kept
    res = oracle.sparse_joint_attention(bf16_round(qd), bf16_round(kd), v, n_text, 0.5, 1.0)
    np.testing.assert_allclose(res["out"][0], np.broadcast_to(to_f64(v)[0, 17], (N, D)), rtol=0, atol=1e-12)


def test_scale_is_applied_to_logits():
    # two keys, logits differ by scale * 1: weights are sigmoid(scale)
    H, N, D = 1, 2, 2
    q = bf16_round(np.array([[[1.0, 0.0], [1.0, 0.0]]]))
    k = bf16_round(np.array([[[1.0, 0.0], [0.0, 0.0]]]))
    v = bf16_round(np.array([[[1.0, 0.0], [0.0, 1.0]]]))
    mask = np.ones((1, 1, 1), np.uint8)
    out = oracle.masked_attention(q, k, v, mask, 0.5)
    w = 1.0 / (1.0 + math.exp(-0.5))
    np.testing.assert_allclose(out[0, 0], [w, 1 - w], rtol=0, atol=1e-15)


def test_query_block_range_and_gate():
    rng = np.random.default_rng(2)
    H, N, D, n_text = 2, 64 * 4, 16, 64
    q, k, v = rand_qkv(rng, H, N, D)
    full = oracle.sparse_joint_attention(q, k, v, n_text, 0.5, 0.25)
    part = oracle.masked_attention(q, k, v, full["mask"], 0.25, qb_lo=1, qb_hi=3, heads=[1])
    np.testing.assert_array_equal(part[1, 64:192], full["out"][1, 64:192])
    assert np.isnan(part[0]).all() and np.isnan(part[1, :64]).all() and np.isnan(part[1, 192:]).all()
    Q, K, V = q[None].repeat(3, 1, 1, 1), k[None].repeat(3, 1, 1, 1), v[None].repeat(3, 1, 1, 1)
    res = oracle.gated_step(Q, K, V, [0, 2, 1], [1.0, 0.5, 0.5], n_text, 0.25)
    assert res[0] is None and res[2] is None
    np.testing.assert_array_equal(res[1]["out"], full["out"])
