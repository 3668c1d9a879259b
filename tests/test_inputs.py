"""Seeded input generator: shapes, determinism, statistics of the recipe."""
import numpy as np
import torch

from paper_2509_22323_b200 import inputs


def test_shapes_of_the_five_workloads():
    w = inputs.WORKLOADS
    assert (w["tiny"].n_tokens, w["tiny"].n_blocks) == (320, 5)
    assert (w["sd3_1024"].n_tokens, w["sd3_1024"].n_blocks) == (4429, 70)
    assert (w["flux_1024"].n_tokens, w["flux_1024"].n_blocks) == (4608, 72)
    assert (w["flux_2048"].n_tokens, w["flux_2048"].n_blocks) == (16896, 264)
    assert w["trajectory"].steps == 28 and w["trajectory"].batch == 8


def test_tiny_is_deterministic_and_per_image_regenerable():
    wl = inputs.WORKLOADS["tiny"]
    q1, k1, v1 = inputs.make_qkv(wl)
    q2, k2, v2 = inputs.make_qkv(wl)
    assert q1.dtype == torch.bfloat16 and q1.shape == (1, 2, 320, 64) and q1.is_contiguous()
    assert torch.equal(q1, q2) and torch.equal(k1, k2) and torch.equal(v1, v2)
    assert not torch.equal(q1, k1)
    assert torch.equal(inputs.make_tensor(wl, 1, 0, 0), k1[0])
    assert not torch.equal(inputs.make_tensor(wl, 1, 1, 0), k1[0])      # another step differs


def test_field_statistics():
    wl = inputs.Workload("t", 1, 2, 64, 64, 32, 4.0, (0.5,), rope=False, seed=5)
    v = inputs.make_tensor(wl, 2, 0, 0).float()
    img = v[:, 64:].reshape(2, 32, 32, 64)
    # unit-variance blurred field + 0.3 white noise -> std about sqrt(1 + 0.09)
    assert abs(img.std().item() - (1.09 ** 0.5)) < 0.15   # channel means of a small grid add a little
    # neighbouring tokens are strongly correlated (blur), text tokens are not
    a, b = img[:, :, :-1].flatten(), img[:, :, 1:].flatten()
    assert torch.corrcoef(torch.stack((a, b)))[0, 1] > 0.8
    t = v[:, :64]
    assert abs(t.std().item() - 1.0) < 0.05
    assert abs(torch.corrcoef(torch.stack((t[:, :-1].flatten(), t[:, 1:].flatten())))[0, 1]) < 0.05


def test_rope_keeps_pair_norms_and_leaves_text_and_v_alone():
    base = inputs.Workload("t", 1, 1, 64, 64, 8, 2.0, (0.5,), rope=False, seed=6)
    roped = inputs.Workload("t", 1, 1, 64, 64, 8, 2.0, (0.5,), rope=True, seed=6)
    for t in (0, 1):
        a, b = inputs.make_tensor(base, t, 0, 0).float(), inputs.make_tensor(roped, t, 0, 0).float()
        assert torch.equal(a[:, :64], b[:, :64])                  # text untouched
        na = a[:, 64:].reshape(1, 64, 32, 2).norm(dim=-1)
        nb = b[:, 64:].reshape(1, 64, 32, 2).norm(dim=-1)
        assert torch.allclose(na, nb, atol=0.05)
        assert torch.equal(a[:, 64], b[:, 64])                    # grid position (0, 0): zero angle
        assert not torch.equal(a[:, 64 + 9], b[:, 64 + 9])
    assert torch.equal(inputs.make_tensor(base, 2, 0, 0), inputs.make_tensor(roped, 2, 0, 0))


def test_actions_of_the_trajectory():
    wl = inputs.WORKLOADS["trajectory"]
    n_gate = n_att = 0
    hist = {}
    for s in range(wl.steps):
        acts, ratios = inputs.make_actions(wl, s)
        assert inputs.make_actions(wl, s) == (acts, ratios)
        for a, r in zip(acts, ratios):
            if a == inputs.ACT_ATTEND:
                n_att += 1
                hist[r] = hist.get(r, 0) + 1
                assert r in wl.ratio_set
            else:
                n_gate += 1
                assert a in (inputs.ACT_SKIP, inputs.ACT_REUSE)
    assert n_gate + n_att == 224
    assert 0.2 < n_gate / 224 < 0.4
    assert set(hist) == set(wl.ratio_set)
    acts, ratios = inputs.make_actions(inputs.WORKLOADS["flux_1024"], 0)
    assert acts == [2, 2, 2] and ratios == [1.0, 0.5, 0.25]
