"""Full-size workloads in the launch configuration the benchmark times (one rapid3_gated_step
per batch): block masks against the oracle on every head of every sparse image, attention
outputs on a seeded sample of (head, query-block) units the oracle computes one by one -- at
least 300 units per workload, over all heads, all four positions of a block in its quad, both
tiles of a thread block, text rows, image rows and the tail."""
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


UNITS_PER_IMAGE = {"sd3_1024": 200, "flux_1024": 160, "flux_2048": 400, "trajectory": 32}


def check_step(wl, ctx, step, sampled_images, units_per_image=None):
    Q, K, V = inputs.make_qkv(wl, step, device=DEV)
    acts, ratios = inputs.make_actions(wl, step)
    out = poison_like(Q)
    ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    raw = out.view(torch.int16)
    sparse = [b for b in range(wl.batch) if acts[b] == binding.ACT_ATTEND and ratios[b] < 1.0]
    gpu_masks = {}
    if sparse:
        ws = ctx.workspace(len(sparse))
        dm = binding.bitmask_to_dense(ws[1], wl.n_blocks).numpy()
        parity.check_lists(ws[2], ws[3], dm)
        gpu_masks = {b: dm[s] for s, b in enumerate(sparse)}
    flips = 0
    n_units = 0
    nb, ntb = wl.n_blocks, (wl.n_text + 63) // 64
    for b in range(wl.batch):
        if acts[b] != binding.ACT_ATTEND:
            assert (raw[b] == np.int16(POISON)).all(), f"gated image {b} was written"
            continue
        assert not (raw[b] == np.int16(POISON)).any(), f"image {b} has unwritten output"
        q, k, v = Q[b].cpu(), K[b].cpu(), V[b].cpu()
        if ratios[b] < 1.0:
            S32, mask, gap = oracle.image_mask(q, k, wl.n_text, ratios[b])
            flips += len(parity.compare_masks(gpu_masks[b], mask, gap, f"{wl.name} step {step} img {b}"))
            use = gpu_masks[b]
        else:
            use = np.ones((wl.heads, wl.n_blocks, wl.n_blocks), np.uint8)
        if b in sampled_images:
            units = parity.sample_units(wl.heads, nb, ntb, units_per_image or UNITS_PER_IMAGE[wl.name],
                                        inputs.sub_seed(wl.seed, 10, step, b) % (1 << 32))
            n_units += len(units)
            ref = parity.oracle_out_units(q, k, v, use, wl.softmax_scale, units)
            parity.compare_outputs(out[b], ref, f"{wl.name} step {step} img {b} ratio {ratios[b]} ({len(units)} units)")
    return flips, n_units


@pytest.mark.parametrize("name", ["sd3_1024", "flux_1024", "flux_2048"])
def test_full_size_single_step(name):
    wl = inputs.WORKLOADS[name]
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    flips, n_units = check_step(wl, ctx, 0, sampled_images=range(wl.batch))
    assert n_units >= 300
    print(f"{name}: {flips} near-tie flips, outputs compared on {n_units} (head, query-block) units")


def test_gated_trajectory():
    wl = inputs.WORKLOADS["trajectory"]
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    flips = 0
    n_units = 0
    n_active = 0
    for step in range(wl.steps):
        acts, _ = inputs.make_actions(wl, step)
        n_active += sum(a == binding.ACT_ATTEND for a in acts)
        # masks on every step; outputs on a seeded subset of (step, image) pairs
        sampled = [b for b in range(wl.batch) if inputs.sub_seed(wl.seed, 9, step, b) % 19 == 0]
        f, u = check_step(wl, ctx, step, sampled_images=sampled)
        flips += f
        n_units += u
    assert 120 <= n_active <= 190
    print(f"trajectory: {n_active} attending image-steps, {flips} near-tie flips, {n_units} output units compared")
