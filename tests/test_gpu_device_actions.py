"""rapid3_gated_step_device: policy actions and keep ratios stay on the GPU.  Masks and outputs
are checked against the oracle's gated step (Sec. 3.3: the heads sample their actions on the
device; the step they gate is the same one), and must also equal those of rapid3_gated_step
given the same decisions from the host."""
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


@pytest.mark.parametrize("case", [
    ("mixed", [2, 0, 2, 2, 1, 2], [0.5, 1.0, 1.0, 0.25, 0.5, 0.5]),
    ("all_sparse", [2, 2, 2, 2, 2, 2], [0.5, 0.25, 0.75, 0.3, 0.9, 0.1]),
    ("all_dense", [2, 2, 2, 2, 2, 2], [1.0] * 6),
    ("all_gated", [0, 1, 0, 1, 0, 1], [0.5] * 6),
])
def test_device_actions_equal_host_actions(case):
    name, acts, ratios = case
    wl = inputs.Workload("dev_" + name, 6, 2, 128, 77, 24, 2.0, tuple(ratios), rope=True, seed=51)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx_h = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    ctx_d = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    out_h, out_d = poison_like(Q), poison_like(Q)
    ctx_h.rapid3_gated_step(Q, K, V, out_h, acts, ratios, wl.softmax_scale)
    a_dev = torch.tensor(acts, dtype=torch.int32, device=DEV)
    r_dev = torch.tensor(ratios, dtype=torch.float32, device=DEV)
    ctx_d.rapid3_gated_step_device(Q, K, V, out_d, a_dev, r_dev, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx_h.last_status() == 0 and ctx_d.last_status() == 0
    assert torch.equal(out_h.view(torch.int16), out_d.view(torch.int16))
    n_sparse = sum(1 for a, r in zip(acts, ratios) if a == 2 and r < 1.0)
    if n_sparse:
        for wh, wd in zip(ctx_h.workspace(n_sparse), ctx_d.workspace(n_sparse)):
            assert torch.equal(wh, wd)
    for b, a in enumerate(acts):
        if a != 2:
            assert (out_d[b].view(torch.int16) == np.int16(POISON)).all()
    # against the oracle: masks of the sparse images (slots in ascending batch order), outputs of all attending ones
    ref = oracle.gated_step(Q.cpu(), K.cpu(), V.cpu(), acts, ratios, wl.n_text, wl.softmax_scale)
    sparse = [b for b, (a, r) in enumerate(zip(acts, ratios)) if a == 2 and r < 1.0]
    if sparse:
        ws = ctx_d.workspace(len(sparse))
        dense = binding.bitmask_to_dense(ws[1], wl.n_blocks).numpy()
        parity.check_lists(ws[2], ws[3], dense)
        for slot, b in enumerate(sparse):
            parity.compare_masks(dense[slot], ref[b]["mask"], ref[b]["gap"], f"device actions {name} img {b}")
    for b, a in enumerate(acts):
        if a == 2:
            assert not (out_d[b].view(torch.int16) == np.int16(POISON)).any()
            parity.compare_outputs(out_d[b], ref[b]["out"], f"device actions {name} img {b} ratio {ratios[b]}")


def test_device_actions_flag_invalid_decisions():
    wl = inputs.Workload("dev_bad", 3, 2, 64, 64, 16, 2.0, (0.5, 0.5, 0.5), seed=53)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    out = poison_like(Q)
    a_dev = torch.tensor([2, 7, 2], dtype=torch.int32, device=DEV)          # 7 is no action
    r_dev = torch.tensor([0.5, 0.5, 1.5], dtype=torch.float32, device=DEV)  # 1.5 is no keep ratio
    ctx.rapid3_gated_step_device(Q, K, V, out, a_dev, r_dev, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == -1
    raw = out.view(torch.int16)
    assert not (raw[0] == np.int16(POISON)).any()                           # the valid image was processed
    assert (raw[1] == np.int16(POISON)).all() and (raw[2] == np.int16(POISON)).all()


def test_device_actions_change_between_graph_replays():
    """The point of device-resident decisions: one captured graph serves every step of a trajectory, the
    policy writes new actions and ratios into the same device arrays between replays."""
    wl = inputs.Workload("dev_graph", 4, 2, 128, 64, 20, 2.0, (0.5,) * 4, rope=True, seed=55)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    a_dev = torch.tensor([2, 2, 2, 2], dtype=torch.int32, device=DEV)
    r_dev = torch.tensor([0.5, 0.5, 0.5, 0.5], dtype=torch.float32, device=DEV)
    out = poison_like(Q)
    ctx.rapid3_gated_step_device(Q, K, V, out, a_dev, r_dev, wl.softmax_scale)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ctx.rapid3_gated_step_device(Q, K, V, out, a_dev, r_dev, wl.softmax_scale)
    plans = [([2, 0, 2, 1], [1.0, 0.5, 0.25, 0.5]), ([0, 1, 0, 1], [0.5] * 4), ([2, 2, 2, 2], [0.1, 1.0, 1.0, 0.9]),
             ([1, 2, 0, 0], [0.5, 0.3, 0.5, 0.5])]
    for acts, ratios in plans:
        a_dev.copy_(torch.tensor(acts, dtype=torch.int32))
        r_dev.copy_(torch.tensor(ratios, dtype=torch.float32))
        out.view(torch.int16).fill_(POISON)
        graph.replay()
        torch.cuda.synchronize()
        assert ctx.last_status() == 0
        want = poison_like(Q)
        ctx_h = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
        ctx_h.rapid3_gated_step(Q, K, V, want, acts, ratios, wl.softmax_scale)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), want.view(torch.int16)), (acts, ratios)
        ref = oracle.gated_step(Q.cpu(), K.cpu(), V.cpu(), acts, ratios, wl.n_text, wl.softmax_scale)
        for b, a in enumerate(acts):
            if a == 2:
                parity.compare_outputs(out[b], ref[b]["out"], f"graph replay {acts} img {b}")
            else:
                assert (out[b].view(torch.int16) == np.int16(POISON)).all()
