"""rapid3_gated_step_fused: the Q/K producer (RMS norm, gain, rotary embedding, bf16 rounding) with
the block pooling folded in.  The produced Q/K are compared with the fp64 oracle element by element
(fp32 arithmetic on the GPU: equal up to an occasional flip of the last bf16 bit), and the rest of
the step with rapid3_gated_step run on those Q/K (bit-identical output and workspace) and with the
oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_22323_b200 import binding, inputs
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"
POISON = 0x7FC1
EPS = 1e-6


def poison_like(t):
    return torch.full(t.shape, POISON, dtype=torch.int16, device=t.device).view(torch.bfloat16)


def bits_f64(t):
    return t.to(torch.float64).cpu().numpy()


def make_case(wl, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    Qr, Kr, V = inputs.make_qkv(wl, 0, device=DEV)
    # raw projections: token-dependent magnitudes, so that the normalisation has something to do
    mag = torch.exp(torch.randn((wl.batch, wl.heads, wl.n_tokens, 1), generator=g)).to(DEV)
    Qr = (Qr.float() * mag).to(torch.bfloat16)
    Kr = (Kr.float() * mag.flip(2)).to(torch.bfloat16)
    q_gain = (0.5 + torch.rand(wl.head_dim, generator=g)).to(DEV)
    k_gain = (0.5 + torch.rand(wl.head_dim, generator=g)).to(DEV)
    ang = torch.rand((wl.n_tokens, wl.head_dim // 2), generator=g, dtype=torch.float64) * 6.283185307179586
    ang[:wl.n_text] = 0.0                                          # text tokens are not rotated
    rot = torch.stack([torch.cos(ang), torch.sin(ang)], dim=-1).float().contiguous().to(DEV)
    return Qr, Kr, V, q_gain, k_gain, rot


def check_produced(raw, got, gain, rot, what):
    want = oracle.qk_prepare(raw.cpu(), gain.cpu().numpy(), None if rot is None else rot.cpu().numpy(), EPS)
    w = (want.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    g = bits_f64(got)
    # tolerance: one step of the 8-bit significand (at most 2^-7 |w|) where the fp32 evaluation lands on the
    # other side of a rounding boundary, plus the fp32 error itself, which a rotation that nearly cancels
    # leaves relative to the pair's length L, not to the small result: <= 8 roundings of terms <= L
    L = np.repeat(np.hypot(w[..., 0::2], w[..., 1::2]), 2, axis=-1)
    tol = np.abs(w) * 2.0 ** -7 + L * 2.0 ** -20
    assert (np.abs(g - w) <= tol).all(), f"{what}: beyond one bf16 step + fp32 evaluation error"
    frac = float((g != w).mean())
    print(f"{what}: {frac:.2e} of the elements differ by one bf16 step")
    assert frac < 5e-3


@pytest.mark.parametrize("D,grid,n_text,in_place,with_rot", [(128, 24, 77, False, True), (64, 28, 128, True, True),
                                                            (128, 20, 0, False, False)])
def test_fused_producer_step(D, grid, n_text, in_place, with_rot):
    wl = inputs.Workload("fused", 4, 2, D, n_text, grid, 2.0, (0.5,) * 4, rope=False, seed=81)
    acts, ratios = [2, 0, 2, 2], [0.5, 0.5, 1.0, 0.25]
    Qr, Kr, V, q_gain, k_gain, rot = make_case(wl, 5)
    if not with_rot:
        rot = None
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    if in_place:
        q, k = Qr.clone(), Kr.clone()
        src_q, src_k = q, k
    else:
        q, k = poison_like(Qr), poison_like(Kr)
        src_q, src_k = Qr, Kr
    out = poison_like(Qr)
    n0 = ctx.launch_count()
    ctx.rapid3_gated_step_fused(src_q, src_k, V, q_gain, k_gain, rot, EPS, q, k, out, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    assert ctx.launch_count() - n0 == 4                            # producer, scores, select, attention
    for b, a in enumerate(acts):
        if a != 2:                                                 # gated: neither produced nor attended
            want_q = Qr[b] if in_place else poison_like(Qr[b])
            assert torch.equal(q[b].view(torch.int16), want_q.view(torch.int16))
            assert (out[b].view(torch.int16) == np.int16(POISON)).all()
            continue
        check_produced(Qr[b], q[b], q_gain, rot, f"Q img {b}")
        check_produced(Kr[b], k[b], k_gain, rot, f"K img {b}")
    # the rest of the step: identical to the unfused step on the produced Q/K (same means, same masks)
    ctx2 = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    out2 = poison_like(Qr)
    ctx2.rapid3_gated_step(q, k, V, out2, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
    for a, b in zip(ctx.workspace(2), ctx2.workspace(2)):
        assert torch.equal(a, b)
    # and against the oracle on the produced Q/K
    gpu_mask = binding.bitmask_to_dense(ctx.workspace(2)[1], wl.n_blocks).numpy()
    for slot, b in enumerate([0, 3]):
        S32, mask, gap = oracle.image_mask(q[b].cpu(), k[b].cpu(), wl.n_text, ratios[b])
        parity.compare_masks(gpu_mask[slot], mask, gap, f"fused img {b}")
        ref = oracle.masked_attention(q[b].cpu(), k[b].cpu(), V[b].cpu(), gpu_mask[slot], wl.softmax_scale)
        parity.compare_outputs(out[b], ref, f"fused img {b}")


def test_fused_producer_all_dense_and_argument_checks():
    wl = inputs.Workload("fused_dense", 2, 2, 64, 64, 8, 2.0, (1.0, 1.0), seed=82)
    Qr, Kr, V, q_gain, k_gain, rot = make_case(wl, 6)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    q, k, out = poison_like(Qr), poison_like(Kr), poison_like(Qr)
    n0 = ctx.launch_count()
    ctx.rapid3_gated_step_fused(Qr, Kr, V, q_gain, k_gain, rot, EPS, q, k, out, [2, 2], [1.0, 1.0], wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.launch_count() - n0 == 2                            # producer and attention only
    check_produced(Qr[1], q[1], q_gain, rot, "dense Q")
    full = np.ones((wl.heads, wl.n_blocks, wl.n_blocks), np.uint8)
    ref = oracle.masked_attention(q[0].cpu(), k[0].cpu(), V[0].cpu(), full, wl.softmax_scale)
    parity.compare_outputs(out[0], ref, "fused dense")
    with pytest.raises(binding.Rapid3Error) as e:
        ctx.rapid3_gated_step_fused(Qr, Kr, V, q_gain, k_gain, rot, -1.0, q, k, out, [2, 2], [1.0, 1.0])
    assert e.value.code == -1
    with pytest.raises(binding.Rapid3Error) as e:                  # misaligned gain pointer
        ctx.rapid3_gated_step_fused(Qr, Kr, V, torch.ones(65, device=DEV)[1:], k_gain, rot, EPS, q, k, out, [2, 2], [1.0, 1.0])
    assert e.value.code == -1
