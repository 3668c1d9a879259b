"""rapid3_select_mask_mass (cumulative-mass block selection) against the oracle: per-row counts
and masks bit-exact except where the oracle reports a near tie (deciding sum within 1e-9 of the
target, or equal scores at the boundary), then attention over those masks."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_22323_b200 import binding, inputs
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"
MARGIN_EPS = 1e-9


def run_mass(wl, shares, scale):
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    scores = ctx.rapid3_block_scores(Q, K)
    row_keep, bitmask, kept_idx, kept_cnt = ctx.rapid3_select_mask_mass(scores, shares, scale)
    out = torch.full(Q.shape, 0x7FC1, dtype=torch.int16, device=DEV).view(torch.bfloat16)
    ctx.rapid3_sparse_joint_attn(Q, K, V, out, kept_idx=kept_idx, kept_cnt=kept_cnt, softmax_scale=wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    return (Q.cpu(), K.cpu(), V.cpu()), row_keep.cpu().numpy(), bitmask, kept_idx, kept_cnt, out


@pytest.mark.parametrize("name,B,H,D,n_text,grid,shares", [
    ("mass128", 3, 2, 128, 77, 24, (0.5, 0.9, 1.0)),
    ("mass64", 2, 3, 64, 128, 28, (0.25, 0.7)),
    ("mass_notext", 2, 2, 128, 0, 20, (0.05, 0.6)),
    ("mass_wide", 1, 2, 64, 64, 80, (0.5,)),            # 101 blocks: several 32-lane rounds per row
])
def test_mass_selection_against_oracle(name, B, H, D, n_text, grid, shares):
    wl = inputs.Workload(name, B, H, D, n_text, grid, 2.0, (0.5,) * B, rope=(D == 128), seed=71)
    scale = wl.softmax_scale * 4.0        # pooled scores are small: a sharper temperature spreads the counts
    (Q, K, V), row_keep, bitmask, kept_idx, kept_cnt, out = run_mass(wl, list(shares), scale)
    nb = wl.n_blocks
    gpu_mask = binding.bitmask_to_dense(bitmask, nb).numpy()
    parity.check_lists(kept_idx, kept_cnt, gpu_mask)
    ntb = (n_text + 63) // 64
    seen = set()
    for b, tau in enumerate(shares):
        S32, mask, gap, k, margin = oracle.image_mask_mass(Q[b], K[b], n_text, tau, scale)
        near = (margin <= MARGIN_EPS) | (gap <= parity.TIE_EPS)
        bad = (row_keep[b] != k) & ~near
        assert not bad.any(), f"{name} img {b}: counts differ at {np.argwhere(bad)[:5]}"
        if near.any():
            print(f"{name} img {b}: {int(near.sum())} near-tie rows")
        rows_differ = (gpu_mask[b] != mask).any(axis=-1)
        assert not (rows_differ & ~near).any(), f"{name} img {b}: masks differ at {np.argwhere(rows_differ & ~near)[:5]}"
        assert (kept_cnt[b].cpu().numpy()[:, ntb:] == row_keep[b][:, ntb:] + ntb + 1).all()
        seen.update(np.unique(k[:, ntb:]).tolist())
        ref = oracle.masked_attention(Q[b], K[b], V[b], gpu_mask[b], wl.softmax_scale)
        parity.compare_outputs(out[b], ref, f"{name} img {b} share {tau}")
    assert len(seen) > 2, "the cases must exercise different counts per row"


def test_mass_argument_checks():
    wl = inputs.Workload("mass_bad", 1, 2, 64, 64, 8, 2.0, (0.5,), seed=72)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    scores = ctx.rapid3_block_scores(Q, K)
    for share, scale in (([0.0], 1.0), ([1.5], 1.0), ([float("nan")], 1.0), ([0.5], -1.0), ([0.5], float("inf"))):
        with pytest.raises(binding.Rapid3Error) as e:
            ctx.rapid3_select_mask_mass(scores, share, scale)
        assert e.value.code == -1


@pytest.mark.parametrize("wl_name,shares", [("flux_1024", (0.9, 0.5, 0.2)), ("flux_2048", (0.5,))])
def test_mass_selection_full_size_masks(wl_name, shares):
    # the benchmark's shapes (72 and 264 blocks, 24 heads): counts and masks of every row
    wl = inputs.WORKLOADS[wl_name]
    Q, K, _ = inputs.make_qkv(wl, 0, device=DEV)
    n = len(shares)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    scores = ctx.rapid3_block_scores(Q, K, img_idx=list(range(n)))
    scale = wl.softmax_scale * 4.0
    row_keep, bitmask, kept_idx, kept_cnt = ctx.rapid3_select_mask_mass(scores, list(shares), scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    gpu_mask = binding.bitmask_to_dense(bitmask, wl.n_blocks).numpy()
    parity.check_lists(kept_idx, kept_cnt, gpu_mask)
    row_keep = row_keep.cpu().numpy()
    for b, tau in enumerate(shares):
        S32, mask, gap, k, margin = oracle.image_mask_mass(Q[b].cpu(), K[b].cpu(), wl.n_text, tau, scale)
        near = (margin <= MARGIN_EPS) | (gap <= parity.TIE_EPS)
        assert not ((row_keep[b] != k) & ~near).any()
        assert not ((gpu_mask[b] != mask).any(axis=-1) & ~near).any()
        print(f"{wl_name} img {b} share {tau}: counts {k[k > 0].min()}..{k.max()}, {int(near.sum())} near-tie rows")


def test_gated_step_with_mass_selection():
    """rapid3_gated_step_mass = gate + compaction + the staged mass path: same masks and outputs as the staged
    calls on the attending images, gated images untouched, a share of 1 is dense."""
    wl = inputs.Workload("mass_gate", 5, 2, 128, 64, 20, 2.0, (0.5,) * 5, rope=True, seed=73)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    acts, shares = [2, 1, 2, 2, 0], [0.6, 0.5, 1.0, 0.2, 0.5]
    scale = 4.0 * wl.softmax_scale
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    out = torch.full(Q.shape, 0x7FC1, dtype=torch.int16, device=DEV).view(torch.bfloat16)
    n0 = ctx.launch_count()
    ctx.rapid3_gated_step_mass(Q, K, V, out, acts, shares, scale, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0 and ctx.launch_count() - n0 == 5
    raw = out.view(torch.int16)
    assert (raw[1] == np.int16(0x7FC1)).all() and (raw[4] == np.int16(0x7FC1)).all()
    ws = ctx.workspace(2)
    gpu_mask = binding.bitmask_to_dense(ws[1], wl.n_blocks).numpy()
    for slot, b in enumerate([0, 3]):
        S32, mask, gap, k, margin = oracle.image_mask_mass(Q[b].cpu(), K[b].cpu(), wl.n_text, shares[b], scale)
        near = (margin <= MARGIN_EPS) | (gap <= parity.TIE_EPS)
        assert not ((gpu_mask[slot] != mask).any(axis=-1) & ~near).any()
        ref = oracle.masked_attention(Q[b].cpu(), K[b].cpu(), V[b].cpu(), gpu_mask[slot], wl.softmax_scale)
        parity.compare_outputs(out[b], ref, f"mass gate img {b}")
    full = np.ones((wl.heads, wl.n_blocks, wl.n_blocks), np.uint8)
    ref = oracle.masked_attention(Q[2].cpu(), K[2].cpu(), V[2].cpu(), full, wl.softmax_scale)
    parity.compare_outputs(out[2], ref, "mass gate dense img 2")
    with pytest.raises(binding.Rapid3Error):
        ctx.rapid3_gated_step_mass(Q, K, V, out, acts, [0.6, 0.5, 1.0, 0.0, 0.5], scale)
