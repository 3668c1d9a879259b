"""Edge cases of the CUDA path against the oracle: strided (packed QKV) tensors, the largest
sequence the library accepts, a text-only sequence, a keep ratio that rounds to one block."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_22323_b200 import binding, inputs
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"
POISON = 0x7FC1


def poison(shape):
    return torch.full(shape, POISON, dtype=torch.int16, device=DEV).view(torch.bfloat16)


def test_packed_qkv_strides():
    """Q, K, V as views of one packed [B, N, 3, H, D] buffer and the output as a view of a padded
    buffer with the same element strides: every kernel addresses through rapid3_shape's strides."""
    wl = inputs.Workload("packed", 2, 3, 128, 77, 24, 2.0, (1.0, 0.4), rope=True, seed=41)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    B, H, N, D = Q.shape
    packed = torch.zeros((B, N, 3, H, D), dtype=torch.bfloat16, device=DEV)
    for i, t in enumerate((Q, K, V)):
        packed[:, :, i] = t.permute(0, 2, 1, 3)
    q, k, v = (packed[:, :, i].permute(0, 2, 1, 3) for i in range(3))        # [B, H, N, D] views
    assert q.stride() == k.stride() == v.stride() and q.stride(3) == 1
    out_buf = poison((B, N, 3, H, D))
    out = out_buf[:, :, 1].permute(0, 2, 1, 3)
    assert out.stride() == q.stride()
    ctx = binding.Context(B, H, D, wl.n_text, wl.n_image, strides=q.stride()[:3])
    ctx.rapid3_gated_step(q, k, v, out, [2, 2], list(wl.keep_ratios), wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    raw = out_buf.view(torch.int16)
    assert (raw[:, :, 0] == np.int16(POISON)).all() and (raw[:, :, 2] == np.int16(POISON)).all()
    ref = oracle.gated_step(Q.cpu(), K.cpu(), V.cpu(), [2, 2], list(wl.keep_ratios), wl.n_text, wl.softmax_scale)
    gpu_mask = binding.bitmask_to_dense(ctx.workspace(1)[1], wl.n_blocks).numpy()[0]
    parity.compare_masks(gpu_mask, ref[1]["mask"], ref[1]["gap"], "packed img 1")
    for b in range(B):
        parity.compare_outputs(out[b].contiguous(), ref[b]["out"], f"packed img {b}")


def test_largest_sequence():
    """N = 65536 tokens (1024 blocks, the library's limit), one head, D = 64: masks of every row,
    attention on sampled query blocks (first, a middle one, the last)."""
    wl = inputs.Workload("max_n", 1, 1, 64, 0, 256, 8.0, (0.1,), rope=False, seed=43)
    assert wl.n_blocks == 1024
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(1, 1, 64, 0, wl.n_image)
    out = poison(Q.shape)
    ctx.rapid3_gated_step(Q, K, V, out, [2], [0.1], wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    assert not (out.view(torch.int16) == np.int16(POISON)).any()
    ws = ctx.workspace(1)
    gpu_mask = binding.bitmask_to_dense(ws[1], 1024).numpy()[0]
    parity.check_lists(ws[2], ws[3], binding.bitmask_to_dense(ws[1], 1024).numpy())
    q, k, v = Q[0].cpu(), K[0].cpu(), V[0].cpu()
    S32, mask, gap = oracle.image_mask(q, k, 0, 0.1)
    assert mask.sum(axis=-1).min() == 1 + 103          # diagonal + ceil(0.1 * 1023)
    parity.compare_masks(gpu_mask, mask, gap, "max_n")
    ref = parity.oracle_out_samples(q, k, v, gpu_mask, wl.softmax_scale, [0], [0, 511, 1023])
    parity.compare_outputs(out[0], ref, "max_n")


def test_text_only_sequence_is_dense():
    wl = inputs.Workload("text_only", 1, 2, 64, 200, 0, 1.0, (0.3,), seed=45)
    gen = torch.Generator(device="cpu").manual_seed(45)
    Q, K, V = (torch.randn((1, 2, 200, 64), generator=gen).to(torch.bfloat16).to(DEV) for _ in range(3))
    ctx = binding.Context(1, 2, 64, 200, 0)
    out = poison(Q.shape)
    ctx.rapid3_gated_step(Q, K, V, out, [2], [0.3], wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    full = np.ones((2, 4, 4), np.uint8)
    gpu_mask = binding.bitmask_to_dense(ctx.workspace(1)[1], 4).numpy()[0]
    assert (gpu_mask == full).all()                    # every block holds text: all forced
    ref = oracle.masked_attention(Q[0].cpu(), K[0].cpu(), V[0].cpu(), full, wl.softmax_scale)
    parity.compare_outputs(out[0], ref, "text_only")


def test_ratio_that_keeps_a_single_free_block():
    wl = inputs.Workload("one_free", 1, 2, 128, 64, 16, 2.0, (0.01,), rope=True, seed=47)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(1, 2, 128, wl.n_text, wl.n_image)
    out = poison(Q.shape)
    ctx.rapid3_gated_step(Q, K, V, out, [2], [0.01], wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    ref = oracle.gated_step(Q.cpu(), K.cpu(), V.cpu(), [2], [0.01], wl.n_text, wl.softmax_scale)[0]
    assert (ref["mask"][:, 1:].sum(axis=-1) == 3).all()  # text block + diagonal + one free block
    gpu_mask = binding.bitmask_to_dense(ctx.workspace(1)[1], wl.n_blocks).numpy()[0]
    parity.compare_masks(gpu_mask, ref["mask"], ref["gap"], "one_free")
    parity.compare_outputs(out[0], ref["out"], "one_free")


@pytest.mark.parametrize("n_text,what", [(64, "vertical pairs inside consecutive quads (text prefix not a whole quad)"),
                                         (256, "column quads (text prefix of one quad)")])
def test_two_block_grid_rows_quad_layouts(n_text, what):
    """A 128 x 128 token grid: one grid row spans two 64-token blocks and the kernel regroups the query
    blocks of a CTA by grid column.  Both regroupings: masks of every row, attention on sampled query
    blocks of both halves of a grid row, at the text boundary and at the end."""
    wl = inputs.Workload("grid128", 1, 2, 64, n_text, 128, 8.0, (0.25,), rope=False, seed=49)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(1, wl.heads, 64, n_text, wl.n_image)
    out = poison(Q.shape)
    ctx.rapid3_gated_step(Q, K, V, out, [2], [0.25], wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    assert not (out.view(torch.int16) == np.int16(POISON)).any()
    nb, ntb = wl.n_blocks, n_text // 64
    ws = ctx.workspace(1)
    dm = binding.bitmask_to_dense(ws[1], nb).numpy()
    parity.check_lists(ws[2], ws[3], dm)
    q, k, v = Q[0].cpu(), K[0].cpu(), V[0].cpu()
    S32, mask, gap = oracle.image_mask(q, k, n_text, 0.25)
    parity.compare_masks(dm[0], mask, gap, what)
    qblocks = [0, ntb, ntb + 1, ntb + 2, ntb + 7, ntb + 8, ntb + 13, nb // 2, nb - 8, nb - 2, nb - 1]
    ref = parity.oracle_out_samples(q, k, v, dm[0], wl.softmax_scale, [0, 1], qblocks)
    parity.compare_outputs(out[0], ref, what)
