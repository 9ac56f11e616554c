"""Small host-side helpers for the tests (bit views, nibble unpacking, dense tables)."""
import numpy as np
import torch


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """BF16 tensor -> uint16 numpy array of its bit patterns."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """uint16 BF16 bit patterns -> float64 values."""
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f32_to_bf16_tensor(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16)


def unpack_nibbles(plane: np.ndarray) -> np.ndarray:
    """u8 [...,64] -> u8 [...,128]; element 2j is the low nibble of byte j."""
    lo = plane & 15
    hi = plane >> 4
    return np.stack([lo, hi], axis=-1).reshape(plane.shape[:-1] + (128,))


def dequant(anchor, residual, meta, full: bool) -> np.ndarray:
    """float64 reconstruction zero + scale * level of plane rows [...,64] / meta [...,2]."""
    a = unpack_nibbles(anchor).astype(np.float64)
    if full:
        lvl = 16.0 * a + unpack_nibbles(residual).astype(np.float64)
    else:
        lvl = 16.0 * a + 8.0
    return meta[..., 1:2].astype(np.float64) + meta[..., 0:1].astype(np.float64) * lvl
