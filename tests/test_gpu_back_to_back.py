"""Steps queued back to back on one stream, with nothing waiting in between.

Inside a step the kernels are launched as programmatic dependents of one another (each may start
while the one before it still runs and waits on the device for its end), so what a kernel reads of
its predecessor's output must be that step's data and not a cached copy of an earlier step's.
Every step here has inputs of its own, the steps run without any host synchronisation, and each
result must equal, bit for bit, the result of the same step run alone."""
import pytest
import torch

from paper_2509_22323_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def count_sparse(acts, ratios):
    return sum(1 for a, r in zip(acts, ratios) if a == inputs.ACT_ATTEND and r < 1.0)


def run_alone(wl, qkv, acts, ratios):
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    out = torch.zeros_like(qkv[0])
    ctx.rapid3_gated_step(*qkv, out, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    return out, [w.clone() for w in ctx.workspace(count_sparse(acts, ratios))[:2]]


@pytest.mark.parametrize("name,n_sets", [("sd3_1024", 4), ("flux_1024", 2), ("tiny", 4)])
def test_queued_steps_equal_steps_run_alone(name, n_sets):
    wl = inputs.WORKLOADS[name]
    sets = [inputs.make_qkv(wl, s, device=DEV) for s in range(n_sets)]
    plans = [inputs.make_actions(wl, s) for s in range(n_sets)]
    alone = [run_alone(wl, sets[s], *plans[s]) for s in range(n_sets)]
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    outs = [torch.zeros_like(sets[0][0]) for _ in range(n_sets)]
    rounds = 5
    for i in range(rounds * n_sets):                      # no synchronisation inside this loop
        s = i % n_sets
        ctx.rapid3_gated_step(*sets[s], outs[s], *plans[s], wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    for s in range(n_sets):
        assert torch.equal(outs[s].view(torch.int16), alone[s][0].view(torch.int16)), f"{name}: step with input set {s}"
    # the workspace holds the last step's scores and masks
    last = (rounds * n_sets - 1) % n_sets
    n_sparse = count_sparse(*plans[last])
    if n_sparse:
        ws = ctx.workspace(n_sparse)
        assert torch.equal(ws[0], alone[last][1][0])
        assert torch.equal(ws[1], alone[last][1][1])


def test_queued_scoring_calls_equal_calls_run_alone():
    """The same for the scoring entry points, whose two kernels are chained the same way."""
    wl = inputs.WORKLOADS["sd3_1024"]
    sets = [inputs.make_qkv(wl, s, device=DEV) for s in range(3)]
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    alone = []
    for q, k, _v in sets:
        alone.append(ctx.rapid3_block_scores(q, k).clone())
        torch.cuda.synchronize()
    got = []
    for rep in range(4):
        for q, k, _v in sets:
            s = ctx.rapid3_block_scores(q, k)
            if rep == 3:
                got.append(s.clone())
    torch.cuda.synchronize()
    for s in range(3):
        assert torch.equal(got[s], alone[s]), f"scoring call {s}"


def _variants(wl, n_sets):
    """name -> function (ctx, set index, q, k, v, out) issuing one step of that entry point."""
    acts, ratios = inputs.make_actions(wl, 0)
    g = torch.Generator(device="cpu").manual_seed(4242)
    head_ratios = [[float(min(1.0, max(0.05, r * f))) for f in (0.5 + torch.rand(wl.heads, generator=g)).tolist()]
                   for r in ratios]
    shares = [0.5 + 0.4 * i / max(1, wl.batch - 1) for i in range(wl.batch)]
    acts_dev = torch.tensor(acts, dtype=torch.int32, device=DEV)
    ratios_dev = torch.tensor(ratios, dtype=torch.float32, device=DEV)
    q_gain = (0.5 + torch.rand(wl.head_dim, generator=g)).to(DEV)
    k_gain = (0.5 + torch.rand(wl.head_dim, generator=g)).to(DEV)
    produced = [(torch.empty((wl.batch, wl.heads, wl.n_tokens, wl.head_dim), dtype=torch.bfloat16, device=DEV),
                 torch.empty((wl.batch, wl.heads, wl.n_tokens, wl.head_dim), dtype=torch.bfloat16, device=DEV))
                for _ in range(n_sets)]
    return {
        "heads": lambda c, s, q, k, v, o: c.rapid3_gated_step_heads(q, k, v, o, acts, head_ratios, wl.softmax_scale),
        "mass": lambda c, s, q, k, v, o: c.rapid3_gated_step_mass(q, k, v, o, acts, shares, wl.softmax_scale,
                                                                  wl.softmax_scale),
        "device": lambda c, s, q, k, v, o: c.rapid3_gated_step_device(q, k, v, o, acts_dev, ratios_dev,
                                                                      wl.softmax_scale),
        "fused": lambda c, s, q, k, v, o: c.rapid3_gated_step_fused(q, k, v, q_gain, k_gain, None, 1e-6,
                                                                    produced[s][0], produced[s][1], o, acts, ratios,
                                                                    wl.softmax_scale),
    }


@pytest.mark.parametrize("variant", ["heads", "mass", "device", "fused"])
@pytest.mark.parametrize("name", ["sd3_1024", "flux_1024"])
def test_queued_steps_of_the_other_entry_points(name, variant):
    wl = inputs.WORKLOADS[name]
    n_sets = 3
    sets = [inputs.make_qkv(wl, s, device=DEV) for s in range(n_sets)]
    step = _variants(wl, n_sets)[variant]
    alone = []
    for s in range(n_sets):
        ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
        out = torch.zeros_like(sets[0][0])
        step(ctx, s, *sets[s], out)
        torch.cuda.synchronize()
        assert ctx.last_status() == 0
        alone.append(out)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    outs = [torch.zeros_like(sets[0][0]) for _ in range(n_sets)]
    for i in range(4 * n_sets):
        step(ctx, i % n_sets, *sets[i % n_sets], outs[i % n_sets])
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    for s in range(n_sets):
        assert torch.equal(outs[s].view(torch.int16), alone[s].view(torch.int16)), f"{name} {variant}: input set {s}"
