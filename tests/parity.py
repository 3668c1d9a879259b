"""Helpers shared by the GPU parity tests: run the CUDA path through the binding, run the
oracle on the same bytes, and compare (bit-exact masks with the near-tie protocol; outputs
within max-abs 2e-2 and mean-abs 2e-3)."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2509_22323_b200 import binding

MAX_ABS_TOL = 2e-2
MEAN_ABS_TOL = 2e-3
TIE_EPS = 1e-6


def compare_masks(gpu_mask: np.ndarray, ora_mask: np.ndarray, gap: np.ndarray, what: str = ""):
    """gpu_mask, ora_mask: [H, nb, nb] uint8; gap: [H, nb].  Rows whose last-kept / first-dropped
    scores differ by more than 0 and at most 1e-6 are near ties: a flip there is reported, every
    other row must match bit for bit -- including rows with gap exactly 0, where the scores are
    equal and the lower block index decides.  Returns the list of flipped near-tie rows."""
    diff_rows = np.argwhere((gpu_mask != ora_mask).any(axis=-1))
    flips = []
    for h, i in diff_rows:
        if 0.0 < gap[h, i] <= TIE_EPS:
            flips.append((int(h), int(i), float(gap[h, i])))
        else:
            raise AssertionError(f"{what}: mask row (head {h}, block {i}) differs, gap {gap[h, i]:.3e}\n"
                                 f"gpu {gpu_mask[h, i]}\nora {ora_mask[h, i]}")
    if flips:
        print(f"{what}: {len(flips)} near-tie rows flipped (reported, not hidden): {flips[:8]}")
    return flips


def check_lists(kept_idx: torch.Tensor, kept_cnt: torch.Tensor, dense_mask: np.ndarray):
    """The ascending kept list and the count must restate the bitmask exactly."""
    idx, cnt = kept_idx.cpu().numpy(), kept_cnt.cpu().numpy()
    nb = dense_mask.shape[-1]
    np.testing.assert_array_equal(cnt, dense_mask.sum(axis=-1))
    flat_m, flat_i, flat_c = dense_mask.reshape(-1, nb), idx.reshape(-1, nb), cnt.reshape(-1)
    for r in range(flat_m.shape[0]):
        want = np.nonzero(flat_m[r])[0]
        np.testing.assert_array_equal(flat_i[r, :flat_c[r]], want)
        assert (flat_i[r, flat_c[r]:] == -1).all()


def check_padding_bits(bitmask: torch.Tensor, nb: int):
    """Bits at and beyond nb in the last word(s) of every bitmask row are zero."""
    bm = bitmask.cpu().numpy().astype(np.uint64)
    words = bm.shape[-1]
    for w in range(words):
        lo = 64 * w
        if lo + 64 <= nb:
            continue
        valid = max(nb - lo, 0)
        pad = np.uint64(0xFFFFFFFFFFFFFFFF) if valid == 0 else ~np.uint64((1 << valid) - 1)
        assert not (bm[..., w] & pad).any(), f"bits >= {nb} set in word {w}"


def compare_outputs(gpu_out: torch.Tensor, ora_out: np.ndarray, what: str = "", scale_with_magnitude: bool = False):
    """gpu_out bf16 [..., N, D]; ora_out fp64 with NaN where the oracle was not evaluated.
    The two tolerances are absolute and presume outputs of a few units at most (the workloads' value
    distribution).  With scale_with_magnitude they grow with the largest output: rounding the exact
    result to bf16 alone costs up to 2^-8 of its magnitude (0.031 at |o| = 8), so for inputs that reach
    |o| > 4 the bounds become 2^-7 max|o| and 2^-10 max|o|."""
    g = gpu_out.to(torch.float64).cpu().numpy()
    sel = ~np.isnan(ora_out)
    assert sel.any(), "nothing to compare"
    assert np.isfinite(g[sel]).all(), f"{what}: non-finite GPU output"
    err = np.abs(g[sel] - ora_out[sel])
    mx, mean = float(err.max()), float(err.mean())
    print(f"{what}: max-abs {mx:.3e} mean-abs {mean:.3e} over {sel.sum()} values")
    max_tol, mean_tol = MAX_ABS_TOL, MEAN_ABS_TOL
    if scale_with_magnitude:
        big = float(np.abs(ora_out[sel]).max())
        max_tol, mean_tol = max(max_tol, big * 2.0 ** -7), max(mean_tol, big * 2.0 ** -10)
    assert mx <= max_tol, f"{what}: max-abs error {mx:.3e} > {max_tol}"
    assert mean <= mean_tol, f"{what}: mean-abs error {mean:.3e} > {mean_tol}"
    return mx, mean


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 numpy array of its bit patterns (one copy to the host)."""
    return np.ascontiguousarray(t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16))


def oracle_out_samples(q, k, v, mask, scale, heads, qblocks):
    """Oracle attention on the (head, query block) units heads x qblocks; NaN elsewhere."""
    return oracle_out_units(q, k, v, mask, scale, [(h, i) for h in heads for i in qblocks])


def oracle_out_units(q, k, v, mask, scale, units):
    """Oracle attention of one image on a list of (head, query block) units, each computed by one
    call of the oracle on that head alone; rows of every other unit stay NaN.  q, k, v: bf16
    [H, N, D] tensors (converted to bit patterns once)."""
    qb, kb, vb = bf16_bits(q), bf16_bits(k), bf16_bits(v)
    H, N, D = qb.shape
    out = np.full((H, N, D), np.nan)
    for h, i in units:
        part = oracle.masked_attention(qb[h:h + 1], kb[h:h + 1], vb[h:h + 1], mask[h:h + 1], scale, qb_lo=i, qb_hi=i + 1)
        out[h, 64 * i:64 * i + 64] = part[0, 64 * i:64 * i + 64]
    return out


def sample_units(n_heads: int, nb: int, ntb: int, count: int, seed: int):
    """Seeded sample of (head, query block) units of one image: per head the first and last text
    block, the first image block and the last two blocks (the tail), then uniformly drawn units up
    to `count`.  Every head and every position of a block within its quad of four is covered."""
    rng = np.random.default_rng(seed)
    units = set()
    for h in range(n_heads):
        for i in (0, ntb - 1, ntb, nb - 2, nb - 1):
            if 0 <= i < nb and (h + i) % 3 == 0:
                units.add((h, i))
        units.add((h, int(rng.integers(0, nb))))
    while len(units) < min(count, n_heads * nb):
        units.add((int(rng.integers(0, n_heads)), int(rng.integers(0, nb))))
    units = sorted(units)
    assert {h for h, _ in units} == set(range(n_heads))
    if nb >= 8 and count >= 64:
        assert {i % 4 for _, i in units} == {0, 1, 2, 3} and {(i // 2) % 2 for _, i in units} == {0, 1}
    return units
