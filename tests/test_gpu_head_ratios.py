"""rapid3_gated_step_heads: one keep ratio per (image, head) (Sec. 3.2, theta in R^{L x H}).
Masks are compared head by head with the oracle's per-head selection, outputs with the oracle's
masked attention."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_22323_b200 import binding, inputs
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"
POISON = 0x7FC1


def poison_like(t):
    return torch.full(t.shape, POISON, dtype=torch.int16, device=t.device).view(torch.bfloat16)


def run_heads(wl, acts, ratios):
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    out = poison_like(Q)
    n0 = ctx.launch_count()
    ctx.rapid3_gated_step_heads(Q, K, V, out, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    return ctx, (Q.cpu(), K.cpu(), V.cpu()), out, ctx.launch_count() - n0


@pytest.mark.parametrize("D,grid,n_text", [(128, 24, 77), (64, 28, 128)])
def test_per_head_ratios_against_oracle(D, grid, n_text):
    H = 3
    ratios = [[0.5, 0.25, 1.0], [1.0, 1.0, 1.0], [0.1, 0.9, 0.5], [0.3, 0.3, 0.3], [0.75, 1.0, 0.05]]
    acts = [2, 2, 2, 0, 2]
    wl = inputs.Workload("heads", 5, H, D, n_text, grid, 2.0, (0.5,) * 5, rope=True, seed=61)
    ctx, (Q, K, V), out, launches = run_heads(wl, acts, ratios)
    assert launches == 4
    sparse = [b for b, (a, r) in enumerate(zip(acts, ratios)) if a == 2 and min(r) < 1.0]
    assert sparse == [0, 2, 4]
    ws_scores, ws_mask, ws_idx, ws_cnt = ctx.workspace(len(sparse))
    gpu_mask = binding.bitmask_to_dense(ws_mask, wl.n_blocks).numpy()
    parity.check_lists(ws_idx, ws_cnt, gpu_mask)
    raw = out.view(torch.int16).cpu()
    assert (raw[3] == np.int16(POISON)).all()                       # the gated image is untouched
    nb, ntb = wl.n_blocks, (n_text + 63) // 64
    for slot, b in enumerate(sparse):
        S32, mask, gap = oracle.image_mask_heads(Q[b], K[b], n_text, ratios[b])
        parity.compare_masks(gpu_mask[slot], mask, gap, f"heads img {b}")
        for h, r in enumerate(ratios[b]):                            # kept counts follow each head's own ratio
            want = ntb + 1 + oracle.keep_count(float(np.float32(r)), nb - ntb - 1)
            assert (ws_cnt[slot, h, ntb:].cpu().numpy() == want).all()
        ref = oracle.masked_attention(Q[b], K[b], V[b], gpu_mask[slot], wl.softmax_scale)
        parity.compare_outputs(out[b], ref, f"heads img {b}")
    full = np.ones((H, nb, nb), np.uint8)                            # all heads at 1.0: dense, no scoring
    ref = oracle.masked_attention(Q[1], K[1], V[1], full, wl.softmax_scale)
    parity.compare_outputs(out[1], ref, "heads dense img 1")


def test_equal_head_ratios_equal_the_per_image_call():
    wl = inputs.Workload("heads_eq", 4, 4, 128, 64, 20, 2.0, (0.5,) * 4, rope=True, seed=62)
    acts, r_img = [2, 1, 2, 2], [0.4, 0.5, 1.0, 0.15]
    ctx_h, _, out_h, _ = run_heads(wl, acts, [[r] * wl.heads for r in r_img])
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx_i = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    out_i = poison_like(Q)
    ctx_i.rapid3_gated_step(Q, K, V, out_i, acts, r_img, wl.softmax_scale)
    torch.cuda.synchronize()
    assert torch.equal(out_h.view(torch.int16), out_i.view(torch.int16))
    for a, b in zip(ctx_h.workspace(2), ctx_i.workspace(2)):
        assert torch.equal(a, b)


def test_head_ratio_argument_checks():
    wl = inputs.Workload("heads_bad", 2, 2, 64, 64, 8, 2.0, (0.5, 0.5), seed=63)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    out = poison_like(Q)
    for bad in ([[0.5, 0.0], [0.5, 0.5]], [[0.5, 0.5], [1.5, 0.5]], [[float("nan"), 0.5], [0.5, 0.5]]):
        with pytest.raises(binding.Rapid3Error) as e:
            ctx.rapid3_gated_step_heads(Q, K, V, out, [2, 2], bad, wl.softmax_scale)
        assert e.value.code == -1
    ctx.rapid3_gated_step_heads(Q, K, V, out, [2, 0], [[0.5, 0.5], [7.0, -1.0]], wl.softmax_scale)   # gated: ignored
    torch.cuda.synchronize()
    assert (out.view(torch.int16)[1] == np.int16(POISON)).all()
