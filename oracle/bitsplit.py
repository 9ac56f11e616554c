"""CPU oracle of the other Anchor / Residual bit splits -- TEST INFRASTRUCTURE, like the rest of this package.

The paper splits the 8-bit code of Section 2.3's quantiser into its top 4 and bottom 4 bits (Section 4.1
stage 4) and names other splits as a direction (Conclusion).  Here the split point is a parameter: the
Anchor is the top A bits of the code, the Residual the bottom R = 8 - A bits, A in {2, 4, 6}; the code and
its (scale, zero) are those of the 4 + 4 path (oracle.split_quantize), so code = (anchor << R) | residual
whatever A is.  On the Anchor alone the reconstruction takes the middle of the bucket the Anchor names,
level = (anchor << R) + 2^(R-1) (Section 4.2, Anchor phase: 16 a + 8 for A = 4).

Packing, per 128-element row and per stream: element e's field occupies bits [e * w, (e + 1) * w) of the
row's 16 * w bytes, least-significant bit first (w = A for the Anchor plane, R for the Residual plane).
For w = 4 that is the two-nibbles-per-byte layout of the 4 + 4 planes: byte j = element 2j | element 2j+1 << 4.

Plain numpy, one field at a time; nothing here is shared with the CUDA library.
"""
from __future__ import annotations

import numpy as np

import oracle

D = 128


def pack_fields(fields: np.ndarray, width: int) -> np.ndarray:
    """fields: integer [..., 128], each < 2^width -> u8 [..., 16 * width], bit e * width + i of a row =
    bit i of element e."""
    f = np.asarray(fields, np.uint8)
    assert f.shape[-1] == D and 1 <= width <= 8 and int(f.max(initial=0)) < (1 << width)
    bits = (f[..., :, None] >> np.arange(width, dtype=np.uint8)) & 1          # [..., 128, width], LSB first
    return np.packbits(bits.reshape(f.shape[:-1] + (D * width,)), axis=-1, bitorder="little")


def unpack_fields(plane: np.ndarray, width: int) -> np.ndarray:
    """Inverse of pack_fields: u8 [..., 16 * width] -> u8 [..., 128]."""
    p = np.asarray(plane, np.uint8)
    assert p.shape[-1] == 16 * width
    bits = np.unpackbits(p, axis=-1, bitorder="little").reshape(p.shape[:-1] + (D, width))
    return (bits.astype(np.uint16) << np.arange(width, dtype=np.uint16)).sum(axis=-1).astype(np.uint8)


def split_quantize_bits(src_bf16_bits: np.ndarray, anchor_bits: int):
    """src_bf16_bits: uint16 [..., 128] -> (anchor u8 [..., 16 A], residual u8 [..., 16 R], meta f32 [..., 2],
    codes u8 [..., 128])."""
    assert anchor_bits in (2, 4, 6)
    r_bits = 8 - anchor_bits
    _, _, meta, codes = oracle.split_quantize(src_bf16_bits, want_codes=True)
    anchor = pack_fields(codes >> r_bits, anchor_bits)
    residual = pack_fields(codes & ((1 << r_bits) - 1), r_bits)
    return anchor, residual, meta, codes


def recombine_bits(anchor: np.ndarray, residual: np.ndarray | None, meta: np.ndarray, anchor_bits: int):
    """-> (levels u8 [..., 128], dequantised BF16 bit patterns uint16 [..., 128]).  levels = the full code
    (anchor << R) | residual, or with residual None the bucket mid-point (anchor << R) + 2^(R-1).  The
    dequantised value is bf16(fl(level * scale + zero)), the multiply-add rounded once, as in the 4 + 4 path
    (Section 4.2, refinement to Q_full)."""
    assert anchor_bits in (2, 4, 6)
    r_bits = 8 - anchor_bits
    a = unpack_fields(anchor, anchor_bits).astype(np.uint16)
    if residual is None:
        levels = (a << r_bits) + (1 << (r_bits - 1))
    else:
        levels = (a << r_bits) | unpack_fields(residual, r_bits)
    levels = levels.astype(np.uint8)
    # dequantisation by the C oracle's own routine (one fmaf, then round-to-nearest-even BF16): the levels go in
    # as the 4 + 4 planes of the same 8-bit values
    _, deq = oracle.recombine(pack_fields(levels >> 4, 4), pack_fields(levels & 15, 4), np.asarray(meta, np.float32))
    return levels, deq
