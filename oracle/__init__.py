"""CPU fp64 oracle of the policy-gated block-sparse joint attention path.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The product path never imports this package.

The arithmetic lives in ``rapid3_oracle.c`` (plain C, fp64); this file compiles it
with gcc on first use and marshals numpy / torch arrays.  Per image the steps are
those the method defines (Sec. 3.2 "Level-3: Sparse-Attention" for the role of the
sparse attention and its per-step sparsity level; the block rule is this project's
reading, stated in the C file's header):

    pool -> scores -> (round to fp32) -> forced + top-k mask -> masked softmax attention

Block scores are rounded to fp32 before the top-k decision because that is the
precision in which the kernels take the same decision.

Parity status: pinned by definition-level tests only; unpinned against the paper,
which prints no value for this path.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rapid3_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_OUT_DIR, "librapid3_oracle.so")
_lib = None

BLOCK = 64
TIE_EPS = 1e-6


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared object (gcc, OpenMP)."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC):
        tmp = _LIB_PATH + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        f64p = ctypes.POINTER(ctypes.c_double)
        u8p = ctypes.POINTER(ctypes.c_uint8)
        ci, cd = ctypes.c_int, ctypes.c_double
        lib.oracle_block_pool.argtypes = [u16p, ci, ci, f64p]
        lib.oracle_block_scores.argtypes = [f64p, f64p, ci, ci, f64p]
        lib.oracle_keep_count.argtypes = [cd, ci]
        lib.oracle_keep_count.restype = ci
        lib.oracle_select_mask.argtypes = [f64p, ci, ci, cd, u8p, f64p]
        lib.oracle_select_mask_mass.argtypes = [f64p, ci, ci, cd, cd, u8p, f64p, ctypes.POINTER(ctypes.c_int32), f64p]
        lib.oracle_qk_prepare.argtypes = [u16p, ci, ci, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float),
                                          cd, u16p]
        lib.oracle_masked_attention.argtypes = [u16p, u16p, u16p, ci, ci, u8p, cd, ci, ci, f64p]
        lib.oracle_attention_weights.argtypes = [u16p, u16p, ci, ci, u8p, cd, ci, f64p]
        lib.oracle_num_threads.restype = ci
        _lib = lib
    return _lib


def _bits(x) -> np.ndarray:
    """bf16 torch tensor (or uint16 array) -> contiguous uint16 numpy array of bit patterns."""
    if isinstance(x, np.ndarray):
        assert x.dtype == np.uint16
        return np.ascontiguousarray(x)
    import torch
    assert x.dtype == torch.bfloat16
    return np.ascontiguousarray(x.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16))


def _p(a: np.ndarray, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def n_blocks(n_tokens: int) -> int:
    return (n_tokens + BLOCK - 1) // BLOCK


def n_text_blocks(n_text: int) -> int:
    """Blocks that contain at least one text token (text comes first in the joint sequence)."""
    return (n_text + BLOCK - 1) // BLOCK


def keep_count(ratio: float, n_free: int) -> int:
    return int(_load().oracle_keep_count(float(ratio), int(n_free)))


def block_pool(x) -> np.ndarray:
    """[H, N, D] bf16 -> [H, nb, D] fp64 block means."""
    xb = _bits(x)
    H, N, D = xb.shape
    nb = n_blocks(N)
    out = np.empty((H, nb, D), dtype=np.float64)
    lib = _load()
    for h in range(H):
        lib.oracle_block_pool(_p(xb[h], ctypes.c_uint16), N, D, _p(out[h], ctypes.c_double))
    return out


def block_scores(pq: np.ndarray, pk: np.ndarray) -> np.ndarray:
    """[H, nb, D] x [H, nb, D] -> [H, nb, nb] fp64 scores."""
    pq = np.ascontiguousarray(pq, dtype=np.float64)
    pk = np.ascontiguousarray(pk, dtype=np.float64)
    H, nb, D = pq.shape
    S = np.empty((H, nb, nb), dtype=np.float64)
    lib = _load()
    for h in range(H):
        lib.oracle_block_scores(_p(pq[h], ctypes.c_double), _p(pk[h], ctypes.c_double), nb, D,
                                _p(S[h], ctypes.c_double))
    return S


def select_mask(S: np.ndarray, n_text: int, ratio: float):
    """[H, nb, nb] scores -> (mask uint8 [H, nb, nb], gap fp64 [H, nb])."""
    S = np.ascontiguousarray(S, dtype=np.float64)
    H, nb, _ = S.shape
    mask = np.zeros((H, nb, nb), dtype=np.uint8)
    gap = np.empty((H, nb), dtype=np.float64)
    lib = _load()
    for h in range(H):
        lib.oracle_select_mask(_p(S[h], ctypes.c_double), nb, n_text_blocks(n_text), float(ratio),
                               _p(mask[h], ctypes.c_uint8), _p(gap[h], ctypes.c_double))
    return mask, gap


def select_mask_mass(S: np.ndarray, n_text: int, tau: float, scale: float):
    """Cumulative-mass selection: [H, nb, nb] scores -> (mask uint8 [H, nb, nb], gap fp64 [H, nb],
    k int32 [H, nb] free candidates kept per row, margin fp64 [H, nb])."""
    S = np.ascontiguousarray(S, dtype=np.float64)
    H, nb, _ = S.shape
    mask = np.zeros((H, nb, nb), dtype=np.uint8)
    gap = np.empty((H, nb), dtype=np.float64)
    k = np.empty((H, nb), dtype=np.int32)
    margin = np.empty((H, nb), dtype=np.float64)
    lib = _load()
    for h in range(H):
        lib.oracle_select_mask_mass(_p(S[h], ctypes.c_double), nb, n_text_blocks(n_text), float(tau), float(scale),
                                    _p(mask[h], ctypes.c_uint8), _p(gap[h], ctypes.c_double),
                                    _p(k[h], ctypes.c_int32), _p(margin[h], ctypes.c_double))
    return mask, gap, k, margin


def masked_attention(q, k, v, mask: np.ndarray, scale: float, qb_lo: int = 0, qb_hi: Optional[int] = None,
                     heads: Optional[Sequence[int]] = None) -> np.ndarray:
    """[H, N, D] bf16 Q, K, V and mask [H, nb, nb] -> fp64 [H, N, D].

    Only query blocks [qb_lo, qb_hi) of the listed heads are computed; other rows are NaN.
    """
    qb, kb, vb = _bits(q), _bits(k), _bits(v)
    H, N, D = qb.shape
    nb = n_blocks(N)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    assert mask.shape == (H, nb, nb)
    out = np.full((H, N, D), np.nan, dtype=np.float64)
    lib = _load()
    hi = nb if qb_hi is None else qb_hi
    for h in (range(H) if heads is None else heads):
        lib.oracle_masked_attention(_p(qb[h], ctypes.c_uint16), _p(kb[h], ctypes.c_uint16),
                                    _p(vb[h], ctypes.c_uint16), N, D, _p(mask[h], ctypes.c_uint8),
                                    float(scale), int(qb_lo), int(hi), _p(out[h], ctypes.c_double))
    return out


def attention_weights(q, k, mask: np.ndarray, scale: float, head: int, token: int) -> np.ndarray:
    """Softmax weights (over all N tokens, zeros where not kept) of one query token."""
    qb, kb = _bits(q), _bits(k)
    H, N, D = qb.shape
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    w = np.empty(N, dtype=np.float64)
    _load().oracle_attention_weights(_p(qb[head], ctypes.c_uint16), _p(kb[head], ctypes.c_uint16), N, D,
                                     _p(mask[head], ctypes.c_uint8), float(scale), int(token),
                                     _p(w, ctypes.c_double))
    return w


def image_scores(q, k) -> np.ndarray:
    """Pooled block scores of one image, rounded to fp32 (returned as fp32)."""
    return block_scores(block_pool(q), block_pool(k)).astype(np.float32)


def image_mask(q, k, n_text: int, ratio: float):
    """Scores (fp32), mask and near-tie flags of one image: the decision is taken on fp32 scores."""
    S32 = image_scores(q, k)
    mask, gap = select_mask(S32.astype(np.float64), n_text, ratio)
    return S32, mask, gap


def image_mask_mass(q, k, n_text: int, tau: float, scale: float):
    """Scores (fp32) and the cumulative-mass mask of one image; the weights are taken on the fp32
    scores with the scale as an fp32 number, the arithmetic itself is fp64."""
    S32 = image_scores(q, k)
    mask, gap, kk, margin = select_mask_mass(S32.astype(np.float64), n_text, tau, float(np.float32(scale)))
    return S32, mask, gap, kk, margin


def image_mask_heads(q, k, n_text: int, ratios: Sequence[float]):
    """The same with one keep ratio per head (Sec. 3.2: the sparsity head emits theta in R^{L x H}):
    head h is selected on its own scores with ratios[h]."""
    S32 = image_scores(q, k)
    assert len(ratios) == S32.shape[0]
    parts = [select_mask(S32[h:h + 1].astype(np.float64), n_text, float(r)) for h, r in enumerate(ratios)]
    return S32, np.concatenate([m for m, _ in parts]), np.concatenate([g for _, g in parts])


def sparse_joint_attention(q, k, v, n_text: int, ratio: float, scale: float, qb_lo: int = 0,
                           qb_hi: Optional[int] = None, heads: Optional[Sequence[int]] = None):
    """Whole path for one image: returns dict(scores, mask, gap, out)."""
    S32, mask, gap = image_mask(q, k, n_text, ratio)
    out = masked_attention(q, k, v, mask, scale, qb_lo, qb_hi, heads)
    return {"scores": S32, "mask": mask, "gap": gap, "out": out}


def gated_step(Q, K, V, actions: Sequence[int], ratios: Sequence[float], n_text: int, scale: float):
    """One policy-gated step over a batch [B, H, N, D].

    Images whose action is not "attend" (2) produce no output (None): a skipped step never
    runs and a cache reuse bypasses the attention.
    """
    res = []
    for b, (a, r) in enumerate(zip(actions, ratios)):
        res.append(sparse_joint_attention(Q[b], K[b], V[b], n_text, r, scale) if a == 2 else None)
    return res


# ----------------------------------------------------------------------------------------------
# Cache-Reuse data path (paper Sec. 3.2, "Level-2: Cache-Reuse": the conditional definition of
# O_t and the cached residual Delta = G(X) - X).  Plain numpy on bf16 bit patterns.  The paper
# fixes no precision; the sum / difference is taken in fp32 (one IEEE rounding) and then rounded
# to bf16 (round to nearest even), the arithmetic a bf16 pipeline has.

def _bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def cache_step(x, o, delta, actions: Sequence[int]):
    """x, o, delta: [B, ...] bf16 tensors (or uint16 bit arrays).  Returns (o_new, delta_new) as
    uint16 bit arrays: action 2 (attend) refreshes delta = o - x, action 1 (reuse) sets
    o = x + delta, action 0 (skip) leaves both as they were."""
    xb, ob, db = (_bits(t).copy() for t in (x, o, delta))
    for b, a in enumerate(actions):
        xf = _bf16_bits_to_f32(xb[b])
        if a == 2:
            db[b] = _f32_to_bf16_bits(_bf16_bits_to_f32(ob[b]) - xf)
        elif a == 1:
            ob[b] = _f32_to_bf16_bits(xf + _bf16_bits_to_f32(db[b]))
    return ob, db


# ----------------------------------------------------------------------------------------------
# Equivalent steps (paper Sec. 3.3, the cost term of the reward): K = sum_k (1 - C_k^cache) *
# (1 - C_k^sparse) over the steps the step policy keeps, rounded to the nearest integer.  A step
# that reuses the cache has C^sparse = 0 (no attention runs), a step that attends has C^cache = 0.

def equivalent_steps(actions: Sequence[int], c_cache: Sequence[float], c_sparse: Sequence[float]):
    total = 0.0
    for a, cc, cs in zip(actions, c_cache, c_sparse):
        if a == 0:                      # skipped: the step is not part of the trajectory
            continue
        C_cache = float(np.float32(cc)) if a == 1 else 0.0
        C_sparse = float(np.float32(cs)) if a == 2 else 0.0
        total += (1.0 - C_cache) * (1.0 - C_sparse)
    return total, int(np.floor(total + 0.5))


# ----------------------------------------------------------------------------------------------
# Q/K producer in front of the attention (RMS normalisation with a learned gain, then rotary
# embedding, one rounding to bf16); see oracle_qk_prepare in the C file.

def qk_prepare(x, gain: np.ndarray, rot: Optional[np.ndarray], eps: float) -> np.ndarray:
    """x: [H, N, D] bf16 (or uint16 bits); gain: [D] fp32; rot: [N, D/2, 2] fp32 (cos, sin) or None.
    Returns the bf16 bit patterns [H, N, D] (uint16)."""
    xb = _bits(x)
    H, N, D = xb.shape
    gain = np.ascontiguousarray(gain, dtype=np.float32)
    assert gain.shape == (D,)
    rp = None
    if rot is not None:
        rot = np.ascontiguousarray(rot, dtype=np.float32)
        assert rot.shape == (N, D // 2, 2)
        rp = _p(rot, ctypes.c_float)
    out = np.empty_like(xb)
    lib = _load()
    for h in range(H):
        lib.oracle_qk_prepare(_p(xb[h], ctypes.c_uint16), N, D, _p(gain, ctypes.c_float), rp, float(eps),
                              _p(out[h], ctypes.c_uint16))
    return out
