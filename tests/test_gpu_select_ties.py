"""Exact ties in the mask selection: equal block scores keep the lower key-block index.

rapid3_select_mask is called on hand-made score tensors (no pooling in between, so the ties are
exact on both sides) and compared with the oracle's selection bit for bit -- no near-tie
allowance.  Both code paths of the kernel are covered: ranking by counting (rows with at most
32 free candidates: nb = 5) and the radix select (nb = 72, 264, 1024)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2509_22323_b200 import binding, inputs
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "hand_mask_5blocks.txt")

# (nb, n_text, n_image): one text block at nb = 5, eight elsewhere
SHAPES = {5: (64, 256), 72: (512, 4096), 264: (512, 16384), 1024: (512, 65024)}
RATIOS = (0.5, 0.25, 0.1, 0.75, 1.0 / 63.0, 0.999)


def read_golden():
    scores, masks, cur = [], {}, None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line == "scores":
            cur = scores
        elif line.startswith("mask ratio"):
            cur = masks.setdefault(float(line.split()[-1]), [])
        else:
            cur.append([float(t) for t in line.split()])
    return np.array(scores, np.float32), {r: np.array(m, np.uint8) for r, m in masks.items()}


def gpu_select(nb, S, ratios):
    """S: [n_img, H, nb, nb] fp32 -> dense masks [n_img, H, nb, nb] uint8 (lists checked on the way)."""
    n_text, n_image = SHAPES[nb]
    n_img, H = S.shape[:2]
    ctx = binding.Context(n_img, H, 64, n_text, n_image)
    assert ctx.nb == nb
    bitmask, kept_idx, kept_cnt = ctx.rapid3_select_mask(torch.from_numpy(S).to(DEV), list(ratios))
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    dense = binding.bitmask_to_dense(bitmask, nb).numpy()
    parity.check_lists(kept_idx, kept_cnt, dense)
    parity.check_padding_bits(bitmask, nb)
    return dense


def assert_equals_oracle(nb, S, ratios, what):
    dense = gpu_select(nb, S, ratios)
    n_text = SHAPES[nb][0]
    for p, r in enumerate(ratios):
        want, _gap = oracle.select_mask(S[p].astype(np.float64), n_text, r)
        np.testing.assert_array_equal(dense[p], want, err_msg=f"{what}: nb {nb} image {p} ratio {r}")


def test_hand_example_with_its_exact_tie():
    S, masks = read_golden()
    ratios = sorted(masks)
    got = gpu_select(5, np.stack([S[None]] * len(ratios)), ratios)
    for p, r in enumerate(ratios):
        np.testing.assert_array_equal(got[p, 0], masks[r], err_msg=f"hand example, ratio {r}")


@pytest.mark.parametrize("nb", [5, 72, 264, 1024])
def test_all_equal_scores_keep_the_lowest_indices(nb):
    H = 2
    for value in (0.0, -0.0, 1.5, -3.25):
        S = np.full((len(RATIOS), H, nb, nb), value, np.float32)
        assert_equals_oracle(nb, S, RATIOS, f"all scores {value}")
    # +0 and -0 compare equal: a checkerboard of the two is still one big tie
    S = np.zeros((len(RATIOS), H, nb, nb), np.float32)
    S[..., ::2] = -0.0
    assert_equals_oracle(nb, S, RATIOS, "signed zeros")


@pytest.mark.parametrize("nb", [5, 72, 264, 1024])
def test_runs_of_equal_values_straddle_the_kth_place(nb):
    """Scores drawn from a handful of levels: every row has long runs of equal values, and at most
    ratios the k-th place falls inside one."""
    H = 2 if nb < 1024 else 1
    rng = np.random.default_rng(1000 + nb)
    for levels in (2, 3, 7):
        vals = rng.standard_normal(levels).astype(np.float32)
        S = vals[rng.integers(0, levels, size=(len(RATIOS), H, nb, nb))]
        assert_equals_oracle(nb, S, RATIOS, f"{levels} levels")
    # one distinct winner, everything else tied; and one distinct loser
    S = np.zeros((len(RATIOS), H, nb, nb), np.float32)
    cols = rng.integers(0, nb, size=nb)
    S[..., np.arange(nb), cols] = 2.0
    S[..., np.arange(nb), (cols + nb // 2) % nb] = -2.0
    assert_equals_oracle(nb, S, RATIOS, "winner + ties + loser")
    # ties between values whose fp32 bit patterns differ in the lowest bits only
    base = np.float32(0.3)
    near = np.array([base, np.nextafter(base, np.float32(1)), np.nextafter(base, np.float32(0))], np.float32)
    S = near[rng.integers(0, 3, size=(len(RATIOS), H, nb, nb))]
    assert_equals_oracle(nb, S, RATIOS, "neighbouring floats")
    # the same with negative scores (the order-preserving key flips all bits there)
    assert_equals_oracle(nb, -S, RATIOS, "neighbouring negative floats")


@pytest.mark.parametrize("shape", [(64, 16, 64), (128, 32, 128), (77, 24, 64)])
def test_gated_step_with_zero_queries(shape):
    """Q = 0: every block score is exactly 0, so the kept free blocks of every row are the k lowest
    indices, and the output is the plain mean of V over the kept valid tokens."""
    n_text, grid, D = shape
    wl = inputs.Workload("zeroq", 2, 2, D, n_text, grid, 2.0, (0.5, 0.25), seed=77)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    Q.zero_()
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    out = torch.zeros_like(Q)
    acts, ratios = [2, 2], [0.5, 0.25]
    ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    ref = oracle.gated_step(Q.cpu(), K.cpu(), V.cpu(), acts, ratios, wl.n_text, wl.softmax_scale)
    ws = ctx.workspace(2)
    assert float(ws[0].abs().max()) == 0.0
    dense = binding.bitmask_to_dense(ws[1], wl.n_blocks).numpy()
    nb, ntb = wl.n_blocks, (wl.n_text + 63) // 64
    for b in range(2):
        np.testing.assert_array_equal(dense[b], ref[b]["mask"])
        parity.compare_outputs(out[b], ref[b]["out"], f"zero queries img {b}")
    # closed form of the rule, written out: row i keeps the text blocks, itself and the k lowest other indices
    for b, r in enumerate(ratios):
        n_free = nb - ntb - 1
        k = oracle.keep_count(r, max(n_free, 0))
        for i in range(ntb, nb):
            free = [j for j in range(ntb, nb) if j != i]
            want = np.zeros(nb, np.uint8)
            want[:ntb] = 1
            want[i] = 1
            want[free[:k]] = 1
            np.testing.assert_array_equal(dense[b, 0, i], want)
