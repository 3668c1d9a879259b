"""rapid3_block_scores_static: the scoring pass for hosts that cannot allocate device memory
(a serving process whose allocator already owns the whole GPU, a sampling loop that must not take
the device-wide synchronisation of an allocation).  It keeps its block means in a fixed array
inside the library, so two things are checked through the C ABI: that it returns exactly what the
context-based rapid3_block_scores returns, and that a second call right after the first is not
disturbed by what the first one left in the shared array (different images, different count).
Collected last on purpose: a failure here cannot hide the other tests' results under `-x`.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2509_22323_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_static_scores_match_context_scores_on_two_calls_in_a_row():
    wl = inputs.Workload("noalloc", 3, 3, 128, 77, 24, 2.0, (0.5, 0.5, 0.5), rope=True, seed=31)
    Q, K, _ = inputs.make_qkv(wl, 0, device=DEV)
    ctx = binding.Context(wl.batch, wl.heads, wl.head_dim, wl.n_text, wl.n_image)
    nb = wl.n_blocks
    calls = [None, [2, 0]]                     # all three images, then a re-ordered subset
    for idx in calls:
        n = wl.batch if idx is None else len(idx)
        want = ctx.rapid3_block_scores(Q, K, img_idx=idx, n_img=n)
        got = torch.full((n, wl.heads, nb, nb), float("nan"), dtype=torch.float32, device=DEV)
        binding.rapid3_block_scores_static(ctx.shape, Q, K, got, img_idx=idx, n_img=n)
        torch.cuda.synchronize()
        # same kernels, same fp64 accumulation and single rounding: the tolerance of the parity tests
        np.testing.assert_allclose(got.cpu().numpy(), want.cpu().numpy(), rtol=2e-7, atol=1e-9)
    assert ctx.last_status() == 0


def test_static_scores_reject_requests_beyond_the_fixed_array():
    limit = binding.static_scratch_bytes()
    assert limit == 16 << 20
    # 2 images of FLUX 2048^2 need 2 * 2 * 24 * 264 * 128 fp64 block means = 25.9 MB > 16 MiB
    N = 512 + 128 * 128
    shape = binding.Shape(2, 24, 128, 512, 128 * 128, 64, 24 * N * 128, N * 128, 128)
    dummy = torch.zeros(8, dtype=torch.bfloat16, device=DEV)   # never read: the call is refused on the host
    out = torch.zeros(8, dtype=torch.float32, device=DEV)
    with pytest.raises(binding.Rapid3Error) as e:
        binding.rapid3_block_scores_static(shape, dummy, dummy, out, n_img=2)
    assert e.value.code == -3
    with pytest.raises(binding.Rapid3Error):
        binding.rapid3_block_scores_static(shape, dummy, dummy, out, n_img=3)   # beyond B_max
