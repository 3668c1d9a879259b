"""Token-level brute-force attention used only to pin the oracle.

Written separately from the oracle: no blocks, no online tricks; a dense [N, N] boolean
token mask says which keys each query sees.
"""
import numpy as np
import torch


def bf16_round(x: np.ndarray) -> torch.Tensor:
    """fp array -> bf16 torch tensor (round to nearest even)."""
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)


def to_f64(x: torch.Tensor) -> np.ndarray:
    return x.to(torch.float64).numpy()


def dense_softmax_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: float,
                            token_mask: np.ndarray | None = None) -> np.ndarray:
    """Textbook softmax(q k^T * scale) v on fp64 [N, D] arrays with an optional [N, N] mask."""
    z = (q @ k.T) * scale
    if token_mask is not None:
        z = np.where(token_mask, z, -np.inf)
    z = z - z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p = p / p.sum(axis=1, keepdims=True)
    return p @ v


def expand_block_mask(block_mask: np.ndarray, n_tokens: int, block: int = 64) -> np.ndarray:
    """[nb, nb] block mask -> [N, N] token mask."""
    idx = np.arange(n_tokens) // block
    return block_mask[np.ix_(idx, idx)].astype(bool)
