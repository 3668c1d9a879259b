"""The running-maximum correction of the online softmax under stress, and run-to-run determinism.

The attention kernel rescales its accumulator only when a row's maximum grows by more than a
threshold -- rare on the synthetic workloads once the first key blocks are past.  Here the keys
grow from block to block, so that nearly every row rescales at nearly every key block while the
products of the blocks before are still in flight: the result must equal the oracle's and must
be the same bits on every run."""
import pytest
import torch

import oracle
from paper_2509_22323_b200 import binding, inputs
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def ramped(wl, step, gain):
    """Q, K, V of the workload with the keys of block j scaled by 1 + gain * j."""
    Q, K, V = inputs.make_qkv(wl, step, device=DEV)
    blk = torch.arange(K.shape[2], device=DEV) // 64
    K = (K.float() * (1.0 + gain * blk.float())[None, None, :, None]).to(torch.bfloat16).contiguous()
    return Q, K, V


@pytest.mark.parametrize("D,grid,gain", [(64, 32, 3.0), (64, 24, 1.0), (128, 32, 3.0), (128, 24, 1.0)])
def test_growing_keys_against_the_oracle(D, grid, gain):
    wl = inputs.Workload("ramp", 2, 3, D, 77, grid, 2.0, (1.0, 0.5), rope=False, seed=501 + D + grid)
    Q, K, V = ramped(wl, 0, gain)
    acts, ratios = [inputs.ACT_ATTEND] * 2, [1.0, 0.5]
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    first = None
    for rep in range(6):
        out = torch.zeros_like(Q)
        ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale)
        torch.cuda.synchronize()
        assert ctx.last_status() == 0
        if first is None:
            first = out
        else:
            assert torch.equal(out.view(torch.int16), first.view(torch.int16)), f"run {rep} differs from run 0"
    ref = oracle.gated_step(Q.cpu(), K.cpu(), V.cpu(), acts, ratios, wl.n_text, wl.softmax_scale)
    for b in range(2):
        # the softmax is close to one-hot here, so outputs are as large as single value rows: the bounds follow them
        parity.compare_outputs(first[b], ref[b]["out"], f"growing keys D {D} img {b}", scale_with_magnitude=True)


@pytest.mark.parametrize("name", ["sd3_1024", "flux_1024", "flux_2048", "trajectory"])
def test_full_size_growing_keys_stay_inside_the_values_and_repeat(name):
    """Full size, where the oracle cannot follow: every output row is a convex combination of value
    rows, so it lies between the smallest and the largest value of its (image, head, channel); and
    two runs give the same bits."""
    wl = inputs.WORKLOADS[name]
    acts, ratios = inputs.make_actions(wl, 0)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    for step, gain in ((1, 0.0), (2, 0.0), (3, 0.0), (0, 0.25 if wl.n_blocks < 100 else 0.05)):
        Q, K, V = ramped(wl, step, gain)
        lo, hi = V.float().amin(dim=2, keepdim=True), V.float().amax(dim=2, keepdim=True)
        runs = []
        for rep in range(3):
            out = torch.zeros_like(Q)
            ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale)
            torch.cuda.synchronize()
            assert ctx.last_status() == 0
            runs.append(out)
        live = [b for b, a in enumerate(acts) if a == inputs.ACT_ATTEND]
        o = runs[0].float()[live]
        slack = 0.01 * (hi - lo)[live] + 1e-3                   # bf16 rounding of the output
        assert bool((o >= lo[live] - slack).all()) and bool((o <= hi[live] + slack).all()), f"{name} step {step}"
        for rep in (1, 2):
            assert torch.equal(runs[rep].view(torch.int16), runs[0].view(torch.int16)), f"{name} step {step} run {rep}"
        del Q, K, V, runs, o
