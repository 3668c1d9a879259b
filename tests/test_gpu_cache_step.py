"""Cache-Reuse data path on the GPU (rapid3_cache_step through the C ABI) against the oracle:
bit-exact, on a batch with all three actions, at FLUX / SD3 latent sizes and a ragged small size."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_22323_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("shape", [(8, 4096, 64), (2, 128, 128, 16), (3, 8), (5, 1000 * 8)])
def test_cache_step_bit_exact(shape):
    gen = torch.Generator(device="cpu").manual_seed(sum(shape))
    x, o, d = (torch.randn(shape, generator=gen).mul(3.0).to(torch.bfloat16) for _ in range(3))
    B = shape[0]
    actions = [(2, 1, 0, 1, 2, 2, 0, 1)[b % 8] for b in range(B)]
    o_ref, d_ref = oracle.cache_step(x, o, d, actions)
    xg, og, dg = x.to(DEV), o.to(DEV), d.to(DEV)
    binding.rapid3_cache_step(xg, og, dg, actions)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(og.cpu().view(torch.int16).numpy().view(np.uint16), o_ref)
    np.testing.assert_array_equal(dg.cpu().view(torch.int16).numpy().view(np.uint16), d_ref)


def test_cache_step_argument_errors():
    x = torch.zeros((2, 64), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(binding.Rapid3Error):
        binding.rapid3_cache_step(x, x, x, [2, 5])
    y = torch.zeros((2, 12), dtype=torch.bfloat16, device=DEV)          # 12 elements: not a multiple of 8
    with pytest.raises(binding.Rapid3Error):
        binding.rapid3_cache_step(y, y, y, [1, 1])
