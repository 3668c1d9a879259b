"""GPU parity: the CUDA path through the C ABI against the fp64 CPU oracle on the same bytes."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2509_22323_b200 import binding, inputs
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"
POISON = 0x7FC1  # a bf16 NaN pattern: unwritten or over-written output rows show up on the host


def poison_like(t):
    return torch.full(t.shape, POISON, dtype=torch.int16, device=t.device).view(torch.bfloat16)


def small_workload(name, B, H, D, n_text, grid, sigma, ratios, rope=False, seed=11):
    return inputs.Workload(name, B, H, D, n_text, grid, sigma, tuple(ratios), rope=rope, seed=seed)


SMALL = {
    "tiny": inputs.WORKLOADS["tiny"],
    # 13-token tail, mixed text/image block, odd number of blocks, several tiles per row
    "tail64": small_workload("tail64", 2, 3, 64, 77, 24, 2.0, (0.5, 0.25)),
    "tail128": small_workload("tail128", 2, 2, 128, 141, 28, 3.0, (0.5, 0.3), rope=True),
    "notext": small_workload("notext", 1, 2, 128, 0, 20, 2.0, (0.4,), rope=True),
    "one_block": small_workload("one_block", 1, 1, 64, 7, 5, 1.0, (0.5,)),
}


def run_stages(wl, step=0):
    Q, K, V = inputs.make_qkv(wl, step, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    scores = ctx.rapid3_block_scores(Q, K)
    bitmask, kept_idx, kept_cnt = ctx.rapid3_select_mask(scores, wl.keep_ratios)
    out = poison_like(Q)
    ctx.rapid3_sparse_joint_attn(Q, K, V, out, kept_idx=kept_idx, kept_cnt=kept_cnt, softmax_scale=wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    return ctx, (Q, K, V), scores, bitmask, kept_idx, kept_cnt, out


@pytest.mark.parametrize("name", list(SMALL))
def test_small_configs_every_stage(name):
    wl = SMALL[name]
    ctx, (Q, K, V), scores, bitmask, kept_idx, kept_cnt, out = run_stages(wl)
    nb = wl.n_blocks
    assert ctx.nb == nb
    gpu_mask = binding.bitmask_to_dense(bitmask, nb).numpy()
    parity.check_lists(kept_idx, kept_cnt, gpu_mask)
    parity.check_padding_bits(bitmask, nb)
    Qc, Kc, Vc = Q.cpu(), K.cpu(), V.cpu()
    for b, ratio in enumerate(wl.keep_ratios):
        S32, mask, gap = oracle.image_mask(Qc[b], Kc[b], wl.n_text, ratio)
        # fp64 accumulation on both sides, one rounding to fp32: equal up to an occasional last-place flip
        np.testing.assert_allclose(scores[b].cpu().numpy(), S32, rtol=2e-7, atol=1e-9)
        flips = parity.compare_masks(gpu_mask[b], mask, gap, f"{name} img {b}")
        # stage isolation: the attention is compared with the oracle run on the GPU's own mask
        ref = oracle.masked_attention(Qc[b], Kc[b], Vc[b], gpu_mask[b], wl.softmax_scale)
        parity.compare_outputs(out[b], ref, f"{name} img {b} ratio {ratio}")
        assert len(flips) == 0 or name != "tiny"


@pytest.mark.parametrize("name", ["tiny", "tail64", "tail128"])
def test_dense_call_equals_dense_attention(name):
    wl = SMALL[name]
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    out = poison_like(Q)
    ctx.rapid3_sparse_joint_attn(Q, K, V, out, softmax_scale=wl.softmax_scale)      # kept_idx = NULL: dense
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    full = np.ones((wl.heads, wl.n_blocks, wl.n_blocks), np.uint8)
    for b in range(wl.batch):
        ref = oracle.masked_attention(Q[b].cpu(), K[b].cpu(), V[b].cpu(), full, wl.softmax_scale)
        parity.compare_outputs(out[b], ref, f"{name} dense img {b}")


def test_image_list_compaction_leaves_other_images_untouched():
    wl = small_workload("list", 4, 2, 64, 64, 16, 2.0, (0.5, 0.5, 0.5, 0.5))
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    idx = [3, 1]
    scores = ctx.rapid3_block_scores(Q, K, img_idx=idx)
    bitmask, kept_idx, kept_cnt = ctx.rapid3_select_mask(scores, [0.5, 0.25])
    out = poison_like(Q)
    ctx.rapid3_sparse_joint_attn(Q, K, V, out, img_idx=idx, kept_idx=kept_idx, kept_cnt=kept_cnt,
                                 softmax_scale=wl.softmax_scale)
    torch.cuda.synchronize()
    raw = out.view(torch.int16).cpu()
    assert (raw[0] == np.int16(POISON)).all() and (raw[2] == np.int16(POISON)).all()
    gpu_mask = binding.bitmask_to_dense(bitmask, wl.n_blocks).numpy()
    for p, (b, r) in enumerate(zip(idx, [0.5, 0.25])):
        S32, mask, gap = oracle.image_mask(Q[b].cpu(), K[b].cpu(), wl.n_text, r)
        parity.compare_masks(gpu_mask[p], mask, gap, f"list img {b}")
        ref = oracle.masked_attention(Q[b].cpu(), K[b].cpu(), V[b].cpu(), gpu_mask[p], wl.softmax_scale)
        parity.compare_outputs(out[b], ref, f"list img {b}")


def test_gated_step_small():
    wl = small_workload("gate", 5, 2, 128, 64, 16, 2.0, (1.0, 0.5, 0.5, 0.25, 1.0), rope=True)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    actions = [binding.ACT_ATTEND, binding.ACT_SKIP, binding.ACT_ATTEND, binding.ACT_ATTEND, binding.ACT_REUSE]
    ratios = [1.0, 0.5, 0.5, 0.25, 1.0]
    out = poison_like(Q)
    n0 = ctx.launch_count()
    ctx.rapid3_gated_step(Q, K, V, out, actions, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    assert ctx.launch_count() - n0 == 4           # pool, scores, select, attention
    raw = out.view(torch.int16).cpu()
    for b in (1, 4):                              # gated images: bit-identical to the poison fill
        assert (raw[b] == np.int16(POISON)).all()
    ref = oracle.gated_step(Q.cpu(), K.cpu(), V.cpu(), actions, ratios, wl.n_text, wl.softmax_scale)
    ws_scores, ws_mask, ws_idx, ws_cnt = ctx.workspace(2)
    gpu_mask = binding.bitmask_to_dense(ws_mask, wl.n_blocks).numpy()
    for slot, b in enumerate((2, 3)):
        parity.compare_masks(gpu_mask[slot], ref[b]["mask"], ref[b]["gap"], f"gate img {b}")
    for b in (0, 2, 3):
        parity.compare_outputs(out[b], ref[b]["out"], f"gate img {b}")
    # all images gated: nothing is launched, nothing is written
    out2 = poison_like(Q)
    n1 = ctx.launch_count()
    ctx.rapid3_gated_step(Q, K, V, out2, [0, 1, 0, 1, 0], ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.launch_count() == n1
    assert (out2.view(torch.int16) == np.int16(POISON)).all()


def test_gated_step_host_buffers():
    wl = small_workload("gate_host", 3, 2, 64, 64, 16, 2.0, (1.0, 0.5, 0.25))
    Q, K, V = [t.pin_memory() for t in inputs.make_qkv(wl, 0, device="cpu")]
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    out = torch.full(Q.shape, POISON, dtype=torch.int16).view(torch.bfloat16).pin_memory()
    actions, ratios = [2, 1, 2], [1.0, 0.5, 0.25]
    up, down = ctx.rapid3_gated_step_host(Q, K, V, out, actions, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    img = Q[0].numel() * 2
    assert (up, down) == (2 * 3 * img, 2 * img)
    assert (out[1].view(torch.int16) == np.int16(POISON)).all()
    ref = oracle.gated_step(Q, K, V, actions, ratios, wl.n_text, wl.softmax_scale)
    for b in (0, 2):
        parity.compare_outputs(out[b], ref[b]["out"], f"host img {b}")


def test_argument_errors_are_codes_not_faults():
    ctx = binding.Context(2, 2, 64, 64, 256)
    Q = torch.zeros((2, 2, 320, 64), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(binding.Rapid3Error) as e:
        ctx.rapid3_select_mask(torch.zeros((1, 2, 5, 5), device=DEV), [1.5])
    assert e.value.code == -1
    with pytest.raises(binding.Rapid3Error):
        ctx.rapid3_block_scores(Q, Q, img_idx=[2])
    with pytest.raises(binding.Rapid3Error):
        ctx.rapid3_gated_step(Q, Q, Q, Q, [2, 7], [0.5, 0.5])
    with pytest.raises(binding.Rapid3Error):
        ctx.rapid3_gated_step(Q, Q, Q, Q, [2, 2, 2], [0.5, 0.5, 0.5])
    with pytest.raises(binding.Rapid3Error):
        ctx.rapid3_sparse_joint_attn(Q, Q, Q, Q, softmax_scale=-1.0)
    for bad in [dict(D=96), dict(n_text=0, n_image=0), dict(B_max=65)]:
        kw = dict(B_max=1, H=2, D=64, n_text=64, n_image=256)
        kw.update(bad)
        with pytest.raises(binding.Rapid3Error):
            binding.Context(**kw)


def test_profile_modes_bracket_the_right_kernels():
    wl = small_workload("prof", 2, 2, 64, 64, 12, 2.0, (0.5, 1.0))
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    out = poison_like(Q)
    for mode, want in ((1, (3, 3, 3, 3)), (2, (0, 0, 0, 3)), (0, (0, 0, 0, 0))):
        ctx.profile(mode)
        ctx.profile_read()
        for _ in range(3):
            ctx.rapid3_gated_step(Q, K, V, out, [2, 2], [0.5, 1.0], wl.softmax_scale)
        torch.cuda.synchronize()
        pr = ctx.profile_read()
        assert tuple(pr[k][1] for k in ("block_pool", "block_scores", "select_mask", "attention")) == want
        assert all(pr[k][0] > 0 for k in pr if pr[k][1]) and all(pr[k][0] == 0 for k in pr if not pr[k][1])
    with pytest.raises(binding.Rapid3Error):
        ctx.profile(3)
