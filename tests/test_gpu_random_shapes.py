"""Seeded random shapes through the whole gated step: batch size, heads, head dimension, text length,
grid size, actions and keep ratios are drawn per seed; every mask row and every output element of the
attending images is compared with the oracle, gated images must stay untouched."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_22323_b200 import binding, inputs
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"
POISON = 0x7FC1


@pytest.mark.parametrize("seed", list(range(14)))
def test_random_shape(seed):
    rng = np.random.default_rng(1000 + seed)
    B = int(rng.integers(1, 5))
    H = int(rng.integers(1, 4))
    D = int(rng.choice([64, 128]))
    n_text = int(rng.choice([0, 1, 63, 64, 65, 77, 128, 200]))
    grid = int(rng.integers(3, 34))
    ratios = [float(rng.choice([1.0, 0.75, 0.5, 0.3, 0.1, 0.02])) for _ in range(B)]
    acts = [int(rng.choice([0, 1, 2, 2, 2])) for _ in range(B)]
    if 2 not in acts:
        acts[0] = 2
    wl = inputs.Workload(f"rand{seed}", B, H, D, n_text, grid, float(rng.choice([1.0, 2.0, 4.0])), tuple(ratios),
                         rope=bool(rng.integers(0, 2)), seed=200 + seed)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(B, H, D, n_text, wl.n_image)
    out = torch.full(Q.shape, POISON, dtype=torch.int16, device=DEV).view(torch.bfloat16)
    ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0, (B, H, D, n_text, grid, acts, ratios)
    sparse = [b for b in range(B) if acts[b] == 2 and ratios[b] < 1.0]
    gpu_mask = {}
    if sparse:
        ws = ctx.workspace(len(sparse))
        dm = binding.bitmask_to_dense(ws[1], wl.n_blocks).numpy()
        parity.check_lists(ws[2], ws[3], dm)
        parity.check_padding_bits(ws[1], wl.n_blocks)
        gpu_mask = {b: dm[s] for s, b in enumerate(sparse)}
    raw = out.view(torch.int16)
    for b in range(B):
        if acts[b] != 2:
            assert (raw[b] == np.int16(POISON)).all()
            continue
        q, k, v = Q[b].cpu(), K[b].cpu(), V[b].cpu()
        if ratios[b] < 1.0:
            S32, mask, gap = oracle.image_mask(q, k, n_text, ratios[b])
            parity.compare_masks(gpu_mask[b], mask, gap, f"seed {seed} img {b}")
            use = gpu_mask[b]
        else:
            use = np.ones((H, wl.n_blocks, wl.n_blocks), np.uint8)
        ref = oracle.masked_attention(q, k, v, use, wl.softmax_scale)
        # a strong blur on a small grid, re-normalised, makes values of ten and more: the bounds follow the magnitude
        parity.compare_outputs(out[b], ref, f"seed {seed} img {b} ({B},{H},{D},{n_text},{grid}) r={ratios[b]}",
                               scale_with_magnitude=True)
