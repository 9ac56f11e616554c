"""Pins for oracle/bitsplit.py (Anchor / Residual splits other than 4 + 4) against things other than itself;
no GPU needed.

* A = 4 reproduces the planes of the 4 + 4 oracle (itself pinned by closed forms and an exact-rational brute
  force) byte for byte, and its Anchor-only / full reconstructions reproduce oracle.recombine's;
* the fields of a packed row, read back bit by bit with Python integers, are the code's top A and bottom R bits;
* (anchor << R) | residual is the 8-bit code for every A (Conclusion: the streams carry the code between them);
* the Anchor-only reconstruction is within 2^(R-1) scale of the full one (+ the BF16 rounding of both), and its error
  against the source shrinks as A grows: 2 < 4 < 6 bits;
* integer rows (min 0, max 255: scale 1) give levels equal to the values, so the fields are the values' bits.
"""
import numpy as np
import pytest

import oracle
import synth
from oracle import bitsplit
from util import bf16_bits, bits_to_f64, f32_to_bf16_tensor


def _rows(n=37, seed=3, recipe="normal_outlier4x8"):
    return bf16_bits(synth.kv_block_values(recipe, n, 2, 16, "cpu", "bitsplit", seed)).reshape(-1, 128)


def test_four_plus_four_is_the_main_path():
    x = _rows()
    a, r, m, codes = bitsplit.split_quantize_bits(x, 4)
    wa, wr, wm, wcodes = oracle.split_quantize(x, want_codes=True)
    assert np.array_equal(a, wa) and np.array_equal(r, wr) and np.array_equal(codes, wcodes)
    assert np.array_equal(m.view(np.uint32), wm.view(np.uint32))
    lv, deq = bitsplit.recombine_bits(a, r, m, 4)
    ocodes, odeq = oracle.recombine(wa, wr, wm)
    assert np.array_equal(lv, ocodes) and np.array_equal(deq, odeq)


@pytest.mark.parametrize("A", [2, 4, 6])
def test_fields_bit_by_bit_and_the_code_identity(A):
    R = 8 - A
    x = _rows(5, seed=A)
    a, r, m, codes = bitsplit.split_quantize_bits(x, A)
    assert a.shape == (x.shape[0], 16 * A) and r.shape == (x.shape[0], 16 * R)
    for row in range(0, x.shape[0], 29):
        big_a = int.from_bytes(a[row].tobytes(), "little")       # the row as one integer: bit i of byte j = bit 8j + i
        big_r = int.from_bytes(r[row].tobytes(), "little")
        for e in range(128):
            fa = (big_a >> (e * A)) & ((1 << A) - 1)
            fr = (big_r >> (e * R)) & ((1 << R) - 1)
            c = int(codes[row, e])
            assert fa == c >> R and fr == c & ((1 << R) - 1) and (fa << R) | fr == c
    assert np.array_equal(bitsplit.unpack_fields(a, A), codes >> R)
    lv, _ = bitsplit.recombine_bits(a, r, m, A)
    assert np.array_equal(lv, codes)
    lv_a, _ = bitsplit.recombine_bits(a, None, m, A)
    assert np.array_equal(lv_a, ((codes >> R) << R) + (1 << (R - 1)))


def test_anchor_only_error_bound_and_ordering():
    x = _rows(61, seed=9, recipe="lognormal_channels")
    xf = bits_to_f64(x)
    errs = {}
    for A in (2, 4, 6):
        R = 8 - A
        a, r, m, _ = bitsplit.split_quantize_bits(x, A)
        full = bits_to_f64(bitsplit.recombine_bits(a, r, m, A)[1])
        anch = bits_to_f64(bitsplit.recombine_bits(a, None, m, A)[1])
        scale = m[:, :1].astype(np.float64)
        assert np.all(np.abs(anch - full) <= (1 << (R - 1)) * scale + 2.0 ** -8 * (np.abs(full) + np.abs(anch)) + 1e-30)
        errs[A] = np.abs(anch - xf).mean()
        # the full reconstruction does not depend on the split
        assert np.array_equal(bitsplit.recombine_bits(a, r, m, A)[1], oracle.recombine(*oracle.split_quantize(x))[1])
    assert errs[6] < errs[4] < errs[2]


def test_integer_rows_give_the_values_bits():
    vals = np.array([[0.0, 255.0] + [float((7 * i) % 256) for i in range(126)]], np.float32)
    x = bf16_bits(f32_to_bf16_tensor(vals))
    for A in (2, 4, 6):
        R = 8 - A
        a, r, m, codes = bitsplit.split_quantize_bits(x, A)
        assert m[0, 0] == 1.0 and m[0, 1] == 0.0 and np.array_equal(codes[0], vals[0].astype(np.uint8))
        assert np.array_equal(bitsplit.unpack_fields(a, A)[0], vals[0].astype(np.uint8) >> R)
        assert np.array_equal(bitsplit.unpack_fields(r, R)[0], vals[0].astype(np.uint8) & ((1 << R) - 1))


def test_pack_unpack_round_trip_all_widths():
    g = np.random.default_rng(1)
    for w in (2, 4, 6):
        f = g.integers(0, 1 << w, size=(9, 128), dtype=np.uint8)
        assert np.array_equal(bitsplit.unpack_fields(bitsplit.pack_fields(f, w), w), f)
