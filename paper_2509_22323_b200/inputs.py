"""Seeded synthetic inputs for the policy-gated block-sparse joint attention path.

This module only *generates data*: Q/K/V tensors shaped like the joint
(text + image token) attention of an SD3/FLUX-class MMDiT block, and the
per-(step, image) policy actions of a gated denoising trajectory.  It holds none
of the method's arithmetic (no pooling, scoring, masking or attention), so both
the CUDA path and the CPU oracle may be fed from it.

Recipe (one image, one tensor of Q/K/V), all in fp32 before the final cast:
  * image tokens: an i.i.d. N(0,1) field on the G x G token grid per (head,
    channel), blurred with a separable Gaussian (std ``sigma`` tokens, radius
    ceil(3 sigma), reflect padding), re-normalised to unit standard deviation
    per (head, channel), plus 0.3 * N(0,1) white noise;
  * text tokens: i.i.d. N(0,1);
  * joint sequence = text tokens first, then image tokens in raster order;
  * optional 2-D rotary embedding on the image tokens of Q and K: the first D/2
    channels rotate with the grid row, the last D/2 with the grid column,
    adjacent channel pairs, base 10000; text tokens are not rotated;
  * cast to bf16 (round to nearest even).

Every (config seed, tensor, step, image) has its own 64-bit sub-seed obtained
with a splitmix64 mix, so any image of any step can be regenerated alone.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Sequence, Tuple

import torch

_MASK64 = (1 << 64) - 1

ACT_SKIP = 0
ACT_REUSE = 1
ACT_ATTEND = 2


def splitmix64(x: int) -> int:
    """One round of the splitmix64 output function on a 64-bit integer."""
    x = (x + 0x9E3779B97F4A7C15) & _MASK64
    z = x
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def sub_seed(seed: int, tensor: int, step: int, image: int) -> int:
    """Counter-based sub-seed for (config seed, tensor id, step, image)."""
    h = splitmix64(seed & _MASK64)
    for v in (tensor, step, image):
        h = splitmix64(h ^ ((v + 1) & _MASK64))
    return h


def _uniform01(h: int) -> float:
    return (h >> 11) * (1.0 / (1 << 53))


@dataclass(frozen=True)
class Workload:
    """Shape of one attention call plus the generator parameters."""

    name: str
    batch: int
    heads: int
    head_dim: int
    n_text: int
    grid: int                      # image tokens = grid * grid
    sigma: float
    keep_ratios: Tuple[float, ...]  # one per image
    rope: bool = False
    seed: int = 0
    steps: int = 1                 # > 1 only for the gated trajectory
    p_gate: float = 0.0            # probability that skip/reuse fires
    ratio_set: Tuple[float, ...] = field(default=(1.0, 0.5, 0.25))

    @property
    def n_image(self) -> int:
        return self.grid * self.grid

    @property
    def n_tokens(self) -> int:
        return self.n_text + self.n_image

    @property
    def n_blocks(self) -> int:
        return (self.n_tokens + 63) // 64

    @property
    def softmax_scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)


WORKLOADS = {
    "tiny": Workload("tiny", 1, 2, 64, 64, 16, 2.0, (0.5,), rope=False, seed=0),
    "sd3_1024": Workload("sd3_1024", 2, 24, 64, 333, 64, 4.0, (1.0, 0.5), rope=False, seed=1),
    "flux_1024": Workload("flux_1024", 3, 24, 128, 512, 64, 4.0, (1.0, 0.5, 0.25), rope=True, seed=2),
    "flux_2048": Workload("flux_2048", 1, 24, 128, 512, 128, 8.0, (0.25,), rope=True, seed=3),
    "trajectory": Workload("trajectory", 8, 24, 128, 512, 64, 4.0, (1.0,) * 8, rope=True, seed=4,
                           steps=28, p_gate=0.3),
}


def _gauss_kernel(sigma: float, device, dtype) -> torch.Tensor:
    radius = int(math.ceil(3.0 * sigma))
    x = torch.arange(-radius, radius + 1, device=device, dtype=dtype)
    w = torch.exp(-0.5 * (x / sigma) ** 2)
    return w / w.sum()


def _blur2d(field_: torch.Tensor, sigma: float) -> torch.Tensor:
    """Separable Gaussian blur of [C, G, G] with reflect padding."""
    w = _gauss_kernel(sigma, field_.device, field_.dtype)
    r = (w.numel() - 1) // 2
    x = field_.unsqueeze(1)                                   # [C,1,G,G]
    # reflect padding needs pad < size; fall back to repeated reflection for tiny grids
    def pad_reflect(t, pad_lr, pad_tb):
        while pad_lr > 0 or pad_tb > 0:
            pl = min(pad_lr, t.shape[-1] - 1)
            pt = min(pad_tb, t.shape[-2] - 1)
            t = torch.nn.functional.pad(t, (pl, pl, pt, pt), mode="reflect")
            pad_lr -= pl
            pad_tb -= pt
        return t
    x = pad_reflect(x, r, 0)
    x = torch.nn.functional.conv2d(x, w.view(1, 1, 1, -1))
    x = pad_reflect(x, 0, r)
    x = torch.nn.functional.conv2d(x, w.view(1, 1, -1, 1))
    return x.squeeze(1)


def _rope_image(x: torch.Tensor, grid: int) -> torch.Tensor:
    """2-D rotary embedding on image tokens.  x: [H, G*G, D] fp32."""
    H, n, D = x.shape
    half = D // 2
    npair = half // 2
    dev, dt = x.device, x.dtype
    freq = 10000.0 ** (-torch.arange(npair, device=dev, dtype=dt) / npair)   # [npair]
    rows = torch.arange(grid, device=dev, dtype=dt).repeat_interleave(grid)  # [n]
    cols = torch.arange(grid, device=dev, dtype=dt).repeat(grid)             # [n]
    out = torch.empty_like(x)
    for pos, lo in ((rows, 0), (cols, half)):
        ang = pos[:, None] * freq[None, :]                                   # [n, npair]
        c, s = torch.cos(ang), torch.sin(ang)
        seg = x[:, :, lo:lo + half].reshape(H, n, npair, 2)
        a, b = seg[..., 0], seg[..., 1]
        rot = torch.stack((a * c - b * s, a * s + b * c), dim=-1)
        out[:, :, lo:lo + half] = rot.reshape(H, n, half)
    return out


def make_tensor(wl: Workload, tensor: int, step: int, image: int, device="cpu") -> torch.Tensor:
    """One of Q (0), K (1), V (2) for one image of one step: bf16 [H, N, D]."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(sub_seed(wl.seed, tensor, step, image) & ((1 << 63) - 1))
    H, D, G, T = wl.heads, wl.head_dim, wl.grid, wl.n_text
    base = torch.randn(H * D, G, G, generator=gen, device=dev, dtype=torch.float32)
    blurred = _blur2d(base, wl.sigma)
    std = blurred.flatten(1).std(dim=1, unbiased=False).clamp_min(1e-12)
    blurred = blurred / std[:, None, None]
    noise = torch.randn(H * D, G, G, generator=gen, device=dev, dtype=torch.float32)
    img = (blurred + 0.3 * noise).reshape(H, D, G * G).transpose(1, 2).contiguous()  # [H, I, D]
    if wl.rope and tensor in (0, 1):
        img = _rope_image(img, G)
    txt = torch.randn(H, T, D, generator=gen, device=dev, dtype=torch.float32)
    return torch.cat((txt, img), dim=1).to(torch.bfloat16).contiguous()


def make_qkv(wl: Workload, step: int = 0, device="cpu", images: Sequence[int] | None = None):
    """Q, K, V as bf16 [B, H, N, D] (contiguous) for one step."""
    imgs = list(range(wl.batch)) if images is None else list(images)
    out = []
    for t in range(3):
        out.append(torch.stack([make_tensor(wl, t, step, b, device) for b in imgs], dim=0))
    return tuple(out)


def make_actions(wl: Workload, step: int) -> Tuple[List[int], List[float]]:
    """Per-image (action, keep ratio) for one step of the gated trajectory.

    With probability ``p_gate`` the image launches no attention (first half of
    that mass is a step skip, second half a cache reuse); otherwise it attends
    with a keep ratio drawn uniformly from ``ratio_set``.  For single-step
    workloads the fixed ``keep_ratios`` are returned and every image attends.
    """
    if wl.steps == 1:
        return [ACT_ATTEND] * wl.batch, [float(r) for r in wl.keep_ratios]
    acts, ratios = [], []
    for b in range(wl.batch):
        u1 = _uniform01(sub_seed(wl.seed, 7, step, b))
        u2 = _uniform01(sub_seed(wl.seed, 8, step, b))
        if u1 < wl.p_gate:
            acts.append(ACT_SKIP if u1 < 0.5 * wl.p_gate else ACT_REUSE)
            ratios.append(1.0)
        else:
            acts.append(ACT_ATTEND)
            ratios.append(float(wl.ratio_set[min(int(u2 * len(wl.ratio_set)), len(wl.ratio_set) - 1)]))
    return acts, ratios
