"""Failure detection and context hygiene, without faulting or hanging anything.

* A bounded device-side wait that runs out: the failure-injection build of the attention kernel
  (its producer stops early, its waits give up after 4096 polls) must return, report
  RAPID3_ERR_TIMEOUT through the status word, and leave the context usable.
* The tensor-map cache of a context: one context fed more distinct buffers than it has cache
  slots must keep computing with the right tensors."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_22323_b200 import binding, inputs
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"
POISON = 0x7FC1
ERR_TIMEOUT = -5


def poison_like(t):
    return torch.full(t.shape, POISON, dtype=torch.int16, device=t.device).view(torch.bfloat16)


@pytest.mark.parametrize("D,stop_group", [(128, 0), (128, 2), (128, 5), (64, 1), (64, 3)])
def test_wait_that_runs_out_sets_the_status_and_returns(D, stop_group):
    wl = inputs.Workload("timeout", 2, 2, D, 64, 16, 2.0, (0.5, 1.0), rope=(D == 128), seed=91)   # nb = 5
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    acts, ratios = [2, 2], [0.5, 1.0]
    want = poison_like(Q)
    ctx.rapid3_gated_step(Q, K, V, want, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0

    scratch = poison_like(Q)
    ctx.rapid3_debug_inject_timeout(Q, K, V, scratch, stop_group, wl.softmax_scale)
    torch.cuda.synchronize()                       # the kernel returned: nothing waits for ever
    assert ctx.last_status() == ERR_TIMEOUT
    assert ctx.last_status() == 0                  # reading the status cleared it
    assert (scratch[1].view(torch.int16) == np.int16(POISON)).all()     # only image 0 was launched

    # the context still computes: bit-identical to before the failure, and right against the oracle
    out = poison_like(Q)
    ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    assert torch.equal(out.view(torch.int16), want.view(torch.int16))
    ref = oracle.gated_step(Q.cpu(), K.cpu(), V.cpu(), acts, ratios, wl.n_text, wl.softmax_scale)
    for b in range(2):
        parity.compare_outputs(out[b], ref[b]["out"], f"after a timeout, img {b}")


def test_injection_entry_refuses_bad_arguments():
    ctx = binding.Context(1, 1, 64, 64, 256)
    Q = torch.zeros((1, 1, 320, 64), dtype=torch.bfloat16, device=DEV)
    for bad in (-1, 6):
        with pytest.raises(binding.Rapid3Error):
            ctx.rapid3_debug_inject_timeout(Q, Q, Q, Q, bad)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0


def test_one_context_many_distinct_buffers():
    """Fixed Q, K, V and a new output tensor per call -- more distinct base pointers than the context
    caches tensor maps for -- then fresh Q/K/V as well: every call must equal a fresh context's result."""
    wl = inputs.Workload("maps", 2, 2, 128, 64, 16, 2.0, (0.5, 1.0), rope=True, seed=93)
    acts, ratios = [2, 2], [0.5, 1.0]
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    fresh = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    want = poison_like(Q)
    fresh.rapid3_gated_step(Q, K, V, want, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    outs = [poison_like(Q) for _ in range(12)]
    assert len({o.data_ptr() for o in outs}) == 12
    for o in outs:
        ctx.rapid3_gated_step(Q, K, V, o, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    for n, o in enumerate(outs):
        assert torch.equal(o.view(torch.int16), want.view(torch.int16)), f"call {n}"
    # rotate all four tensors
    for step in range(1, 6):
        Q2, K2, V2 = inputs.make_qkv(wl, step, device=DEV)
        a, b = poison_like(Q2), poison_like(Q2)
        ctx.rapid3_gated_step(Q2, K2, V2, a, acts, ratios, wl.softmax_scale)
        other = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
        other.rapid3_gated_step(Q2, K2, V2, b, acts, ratios, wl.softmax_scale)
        torch.cuda.synchronize()
        assert torch.equal(a.view(torch.int16), b.view(torch.int16)), f"step {step}"
    ref = oracle.gated_step(Q.cpu(), K.cpu(), V.cpu(), acts, ratios, wl.n_text, wl.softmax_scale)
    for b in range(2):
        parity.compare_outputs(outs[-1][b], ref[b]["out"], f"many buffers img {b}")
