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
    parity.check_padding_bits(ws[1], 1024)
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


def test_fused_producer_in_place_on_packed_projections():
    """The fused step run in place on a packed [B, N, 3, H, D] projection buffer (the layout a fused QKV
    projection writes): Q and K are normalised and rotated where they lie, V is read as it is."""
    wl = inputs.Workload("packed_fused", 2, 3, 128, 77, 24, 2.0, (1.0, 0.4), rope=False, seed=42)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    B, H, N, D = Q.shape
    packed = torch.zeros((B, N, 3, H, D), dtype=torch.bfloat16, device=DEV)
    for i, t in enumerate((Q * 3, K * 0.5, V)):
        packed[:, :, i] = t.permute(0, 2, 1, 3)
    q, k, v = (packed[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    raw_q, raw_k = q.contiguous(), k.contiguous()
    gen = torch.Generator(device="cpu").manual_seed(3)
    gain = (0.5 + torch.rand(D, generator=gen)).to(DEV)
    ang = torch.rand((N, D // 2), generator=gen, dtype=torch.float64) * 6.283185307179586
    rot = torch.stack([torch.cos(ang), torch.sin(ang)], dim=-1).float().contiguous().to(DEV)
    out = poison((B, H, N, D))
    ctx = binding.Context(B, H, D, wl.n_text, wl.n_image, strides=q.stride()[:3])
    ctx_out = binding.Context(B, H, D, wl.n_text, wl.n_image)             # contiguous twin for the comparison run
    # the output has its own (contiguous) strides here, so it goes through a packed buffer as well
    out_buf = poison((B, N, 3, H, D))
    out_v = out_buf[:, :, 0].permute(0, 2, 1, 3)
    ctx.rapid3_gated_step_fused(q, k, v, gain, gain, rot, 1e-6, q, k, out_v, [2, 2], list(wl.keep_ratios),
                                wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    for b in range(B):
        for raw, got, name in ((raw_q, q, "Q"), (raw_k, k, "K")):
            want = oracle.qk_prepare(raw[b].cpu(), gain.cpu().numpy(), rot.cpu().numpy(), 1e-6)
            w = (want.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
            g = got[b].contiguous().to(torch.float64).cpu().numpy()
            L = np.repeat(np.hypot(w[..., 0::2], w[..., 1::2]), 2, axis=-1)
            assert (np.abs(g - w) <= np.abs(w) * 2.0 ** -7 + L * 2.0 ** -20).all(), f"{name} img {b}"
            assert (g != w).mean() < 5e-3
    assert torch.equal(packed[:, :, 2].permute(0, 2, 1, 3), V)              # V untouched
    ctx_out.rapid3_gated_step(q.contiguous(), k.contiguous(), V, out, [2, 2], list(wl.keep_ratios), wl.softmax_scale)
    torch.cuda.synchronize()
    assert torch.equal(out_v.contiguous().view(torch.int16), out.view(torch.int16))


def test_mass_selection_at_the_largest_sequence():
    """1024 blocks: the weighted radix select of the cumulative-mass rule over 32 lane rounds per pass."""
    wl = inputs.Workload("max_n_mass", 1, 1, 64, 0, 256, 8.0, (0.1,), rope=False, seed=44)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(1, 1, 64, 0, wl.n_image)
    scores = ctx.rapid3_block_scores(Q, K)
    scale = 8.0 * wl.softmax_scale
    row_keep, bitmask, kept_idx, kept_cnt = ctx.rapid3_select_mask_mass(scores, [0.3], scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    dm = binding.bitmask_to_dense(bitmask, 1024).numpy()
    parity.check_lists(kept_idx, kept_cnt, dm)
    S32, mask, gap, k, margin = oracle.image_mask_mass(Q[0].cpu(), K[0].cpu(), 0, 0.3, scale)
    near = (margin <= 1e-9) | (gap <= parity.TIE_EPS)
    assert not ((row_keep[0].cpu().numpy() != k) & ~near).any()
    assert not ((dm[0] != mask).any(axis=-1) & ~near).any()
    assert k.min() >= 1 and k.max() > k.min()


def lists_from_mask(mask):
    """[n, H, nb, nb] 0/1 -> (kept_idx int32 padded with -1, kept_cnt int32) in the library's layout."""
    n, H, nb, _ = mask.shape
    idx = np.full((n, H, nb, nb), -1, np.int32)
    cnt = mask.sum(-1).astype(np.int32)
    for p in range(n):
        for h in range(H):
            for i in range(nb):
                js = np.nonzero(mask[p, h, i])[0]
                idx[p, h, i, :len(js)] = js
    return torch.from_numpy(idx).to(DEV), torch.from_numpy(cnt).to(DEV)


@pytest.mark.parametrize("D,n_text,grid", [(128, 77, 20), (64, 0, 23)])
def test_caller_supplied_lists_of_any_shape(D, n_text, grid):
    """Kept lists the selection kernel would never write: rows that keep nothing (zero output), rows without
    their diagonal or text blocks, single-block rows, whole quads that keep nothing, a full row."""
    wl = inputs.Workload("anylist", 2, 2, D, n_text, grid, 2.0, (0.5, 0.5), seed=50)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    nb = wl.n_blocks
    rng = np.random.default_rng(12)
    mask = (rng.random((2, 2, nb, nb)) < 0.3).astype(np.uint8)
    mask[0, 0, 1] = 0                                    # a row that keeps nothing
    mask[0, 1, 0:4] = 0                                  # a whole quad that keeps nothing
    mask[1, 0, 2] = 0
    mask[1, 0, 2, nb - 1] = 1                            # only the (ragged) last block
    mask[1, 1, 3] = 1                                    # a full row
    mask[1, 1, nb - 1] = 0
    mask[1, 1, nb - 1, 0] = 1                            # the tail query block sees only block 0
    kept_idx, kept_cnt = lists_from_mask(mask)
    ctx = binding.Context(2, 2, D, n_text, wl.n_image)
    out = poison(Q.shape)
    ctx.rapid3_sparse_joint_attn(Q, K, V, out, kept_idx=kept_idx, kept_cnt=kept_cnt, softmax_scale=wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    for b in range(2):
        ref = oracle.masked_attention(Q[b].cpu(), K[b].cpu(), V[b].cpu(), mask[b], wl.softmax_scale)
        parity.compare_outputs(out[b], ref, f"anylist img {b}")
    o = out.float().cpu().numpy()
    assert (o[0, 0, 64:128] == 0).all() and (o[0, 1, 0:256] == 0).all()          # nothing kept: exact zeros


def test_malformed_list_sets_the_status_word_and_nothing_else():
    wl = inputs.Workload("badlist", 1, 1, 64, 64, 12, 2.0, (0.5,), seed=51)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    nb = wl.n_blocks
    mask = np.ones((1, 1, nb, nb), np.uint8)
    kept_idx, kept_cnt = lists_from_mask(mask)
    kept_idx[0, 0, 1, 0] = nb + 5                        # out of range
    kept_idx[0, 0, 2, 1] = -7                            # negative
    kept_cnt[0, 0, 2] = nb + 100                         # count beyond the row (clamped)
    ctx = binding.Context(1, 1, 64, 64, wl.n_image)
    out = poison(Q.shape)
    ctx.rapid3_sparse_joint_attn(Q, K, V, out, kept_idx=kept_idx, kept_cnt=kept_cnt, softmax_scale=wl.softmax_scale)
    torch.cuda.synchronize()
    assert ctx.last_status() == -6                       # RAPID3_ERR_BAD_LIST, reported, no fault
    assert ctx.last_status() == 0                        # reading clears it
    assert torch.isfinite(out.float()).all()
    # the rows with well-formed lists are what they should be
    mask[0, 0, 1, 0] = 0
    mask[0, 0, 2, 1] = 0
    ref = oracle.masked_attention(Q[0].cpu(), K[0].cpu(), V[0].cpu(), mask[0], wl.softmax_scale, qb_lo=3, qb_hi=nb)
    parity.compare_outputs(out[0], ref, "badlist rows 3..")


@pytest.mark.parametrize("D", [64, 128])
def test_running_maximum_that_grows_with_every_key_block(D):
    """Logits that climb from block to block by far more than the lazy-rescale threshold (and a very
    sharp softmax): every block triggers the rescale of O and l.  Then the reverse order, where the
    first block holds the maximum and everything after it underflows."""
    wl = inputs.Workload("climb", 1, 2, D, 64, 16, 2.0, (1.0,), seed=52)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    nb = wl.n_blocks
    ramp = torch.arange(wl.n_tokens, device=DEV, dtype=torch.float32).div(64, rounding_mode="floor")
    q0 = Q[0].float()
    for direction in (1.0, -1.0):
        # k_n = (3 * block(n) * direction) * unit vector along the mean query + small noise
        u = q0.mean(dim=1, keepdim=True)
        u = u / u.norm(dim=-1, keepdim=True)
        Kc = (K[0].float() * 0.1 + direction * 3.0 * ramp[None, :, None] * u).to(torch.bfloat16)[None]
        Qc = (q0 * 0.1 + 4.0 * u).to(torch.bfloat16)[None]
        ctx = binding.Context(1, 2, D, 64, wl.n_image)
        out = poison(Q.shape)
        scale = 1.0                                             # logits step by about 12 per block: 2^17 in the exp2 domain
        ctx.rapid3_sparse_joint_attn(Qc, Kc, V, out, softmax_scale=scale)
        torch.cuda.synchronize()
        assert ctx.last_status() == 0
        full = np.ones((2, nb, nb), np.uint8)
        ref = oracle.masked_attention(Qc[0].cpu(), Kc[0].cpu(), V[0].cpu(), full, scale)
        parity.compare_outputs(out[0], ref, f"climb D={D} dir={direction}", scale_with_magnitude=True)
        # the softmax really is that sharp: almost all the mass sits in one block
        w = oracle.attention_weights(Qc[0].cpu(), Kc[0].cpu(), full, scale, 0, 100)
        top = w.reshape(-1)[: (wl.n_tokens // 64) * 64].reshape(-1, 64).sum(-1).max()
        assert top > 0.99


def test_two_contexts_on_two_streams():
    """Two contexts driven from two streams at once (each owns its workspace and tensor maps): both give
    what a single call gives."""
    wl = inputs.Workload("streams", 3, 2, 128, 64, 24, 2.0, (1.0, 0.5, 0.25), rope=True, seed=53)
    Q, K, V = inputs.make_qkv(wl, 0, device=DEV)
    acts, ratios = [2, 2, 2], list(wl.keep_ratios)
    ref_ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    ref = poison(Q.shape)
    ref_ctx.rapid3_gated_step(Q, K, V, ref, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    ctxs = [binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image) for _ in range(2)]
    outs = [poison(Q.shape) for _ in range(2)]
    streams = [torch.cuda.Stream() for _ in range(2)]
    for rep in range(5):
        for c, o, s in zip(ctxs, outs, streams):
            with torch.cuda.stream(s):
                c.rapid3_gated_step(Q, K, V, o, acts, ratios, wl.softmax_scale)
    torch.cuda.synchronize()
    for c, o in zip(ctxs, outs):
        assert c.last_status() == 0
        assert torch.equal(o.view(torch.int16), ref.view(torch.int16))
        for a, b in zip(c.workspace(2), ref_ctx.workspace(2)):
            assert torch.equal(a, b)


def test_gated_step_inside_a_cuda_graph():
    """The step makes no allocation, copy or synchronisation of its own, so it can be captured once and
    replayed: the replays read the buffers' current contents (fresh Q, K, V written in place)."""
    wl = inputs.Workload("graph", 3, 2, 128, 64, 20, 2.0, (1.0, 0.5, 0.25), rope=True, seed=54)
    acts, ratios = [2, 2, 2], list(wl.keep_ratios)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    Q, K, V = (t.clone() for t in inputs.make_qkv(wl, 0, device=DEV))
    out = poison(Q.shape)
    ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale)      # warm: tensor maps are encoded here
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ctx.rapid3_gated_step(Q, K, V, out, acts, ratios, wl.softmax_scale)
    for step in (1, 2):
        Qn, Kn, Vn = inputs.make_qkv(wl, step, device=DEV)
        Q.copy_(Qn); K.copy_(Kn); V.copy_(Vn)
        out.view(torch.int16).fill_(POISON)
        graph.replay()
        torch.cuda.synchronize()
        assert ctx.last_status() == 0
        want = poison(Q.shape)
        ctx2 = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
        ctx2.rapid3_gated_step(Qn, Kn, Vn, want, acts, ratios, wl.softmax_scale)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), want.view(torch.int16))
