"""Pins for the CPU oracle against things other than itself (no GPU needed).

Quantiser: closed forms (integer rows, ties), an exact-rational brute force, the scale/2 and
8.5*scale error bounds, bit identities of the split (Section 2.3; Section 4.1 stage 4;
Conclusion: INT4 + INT4 = INT8).  Attention: brute force with Python floats, torch's float64
scaled_dot_product_attention on the dequantised tensors, and invariants of softmax attention
(Section 2 equation).  Verify decision: properties of longest-agreeing-prefix (Section 4.3).
"""
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
import synth
from util import bf16_bits, bits_to_f64, dequant, f32_to_bf16_tensor, unpack_nibbles


def _row_bits(values) -> np.ndarray:
    v = np.asarray(values, np.float32)
    t = f32_to_bf16_tensor(v)
    assert np.array_equal(t.to(torch.float32).numpy(), v), "test row must be exact in BF16"
    return bf16_bits(t)


# ----------------------------------------------------------------------------- quantiser
def test_integer_rows_give_identity_codes_and_split_all_256():
    # rows with min 0 and max 255: scale = 1, inv = 1, code = value
    rows = []
    others = [v for v in range(1, 255)]
    for i in range(0, len(others), 126):
        chunk = others[i:i + 126]
        chunk = chunk + [1] * (126 - len(chunk))
        rows.append([0.0, 255.0] + [float(c) for c in chunk])
    rows = np.array(rows, np.float32)
    a, r, meta, codes = oracle.split_quantize(_row_bits(rows), want_codes=True)
    assert np.array_equal(codes, rows.astype(np.uint8))
    assert np.all(meta[:, 0] == 1.0) and np.all(meta[:, 1] == 0.0)
    seen = set(codes.reshape(-1).tolist())
    assert seen == set(range(256))
    ua, ur = unpack_nibbles(a), unpack_nibbles(r)
    assert np.array_equal(ua, codes >> 4) and np.array_equal(ur, codes & 15)
    assert np.array_equal((ua.astype(np.uint16) << 4) | ur, codes)
    # packing order: byte j = element 2j in the low nibble, 2j+1 in the high nibble
    assert np.array_equal(a[:, 0], (codes[:, 0] >> 4) | ((codes[:, 1] >> 4) << 4))
    assert np.array_equal(r[:, 5], (codes[:, 10] & 15) | ((codes[:, 11] & 15) << 4))
    assert a.shape == (rows.shape[0], 64) and r.shape == (rows.shape[0], 64)


def test_ties_round_half_to_even():
    vals = [0.0, 255.0] + [k + 0.5 for k in range(126)]
    a, r, meta, codes = oracle.split_quantize(_row_bits([vals]), want_codes=True)
    want = [0, 255] + [k if k % 2 == 0 else k + 1 for k in range(126)]
    assert codes[0].tolist() == want


def test_shifted_scaled_row_closed_form():
    # x = -3 + 0.5 * i, i in 0..127 -> range 63.5; code = RNE(i * 255/127) up to the FP32 steps,
    # checked against exact rationals built from the same FP32 inv.
    i = np.arange(128)
    x = (-3.0 + 0.5 * i).astype(np.float32)
    a, r, meta, codes = oracle.split_quantize(_row_bits([x]), want_codes=True)
    assert meta[0, 1] == np.float32(-3.0)
    assert meta[0, 0] == np.float32(63.5) / np.float32(255.0)
    inv = Fraction(float(np.float32(255.0) / np.float32(63.5)))
    for k in range(128):
        exact = Fraction(k, 2) * inv
        lo = math.floor(exact)
        frac = exact - lo
        want = lo + (1 if (frac > Fraction(1, 2) or (frac == Fraction(1, 2) and lo % 2 == 1)) else 0)
        assert codes[0, k] == want
    # and the plain formula i*255/127 agrees wherever it is not within 1e-3 of a tie
    ideal = i * 255.0 / 127.0
    clear = np.abs(ideal - np.floor(ideal) - 0.5) > 1e-3
    assert np.array_equal(codes[0][clear], np.rint(ideal[clear]).astype(np.uint8))


def _fraction_quantize_row(vals32):
    """Independent exact-rational quantiser for one row of float32 values."""
    mn, mx = min(vals32), max(vals32)
    rng = np.float32(mx) - np.float32(mn)
    if not rng >= np.float32(2.0 ** -100):
        return [0] * len(vals32), np.float32(0.0), np.float32(mn) + np.float32(0.0)
    scale = rng / np.float32(255.0)
    inv = np.float32(255.0) / rng
    out = []
    for v in vals32:
        u = np.float32(v) - np.float32(mn)
        exact = Fraction(float(u)) * Fraction(float(inv))
        lo = math.floor(exact)
        frac = exact - lo
        c = lo + (1 if (frac > Fraction(1, 2) or (frac == Fraction(1, 2) and lo % 2 == 1)) else 0)
        out.append(min(255, max(0, c)))
    return out, scale, np.float32(mn) + np.float32(0.0)


@pytest.mark.parametrize("recipe", ["normal_outlier4x8", "lognormal_channels", "student_t4"])
def test_quantiser_matches_exact_rational_brute_force(recipe):
    x = synth.kv_block_values(recipe, 1, 2, 4, "cpu", "pin", 1)          # 8 rows
    bits = bf16_bits(x).reshape(-1, 128)
    a, r, meta, codes = oracle.split_quantize(bits, want_codes=True)
    vals = (bits.astype(np.uint32) << 16).view(np.float32)
    for row in range(bits.shape[0]):
        want, scale, zero = _fraction_quantize_row(vals[row].tolist())
        assert codes[row].tolist() == want
        assert meta[row, 0] == scale and meta[row, 1] == zero


@pytest.mark.parametrize("recipe", ["normal_outlier4x8", "lognormal_channels", "student_t4",
                                    "normal_outlier2pct_x10"])
def test_error_bounds_full_and_anchor(recipe):
    x = synth.kv_block_values(recipe, 8, 8, 16, "cpu", "bound", 2)
    bits = bf16_bits(x).reshape(-1, 128)
    a, r, meta = oracle.split_quantize(bits)
    xv = bits_to_f64(bits)
    scale = meta[:, 0:1].astype(np.float64)
    assert np.all(np.abs(xv - dequant(a, r, meta, True)) <= scale * (0.5 + 1e-4))
    assert np.all(np.abs(xv - dequant(a, r, meta, False)) <= scale * (8.5 + 1e-4))
    # the range is really used: every row reaches code 0 and code 255
    codes, _ = oracle.recombine(a, r, meta)
    assert np.all(codes.min(axis=1) == 0) and np.all(codes.max(axis=1) == 255)
    # vNMSE ordering of Table 3: a 4-bit state is far worse than the 8-bit state
    e_full = np.mean((xv - dequant(a, r, meta, True)) ** 2)
    e_anchor = np.mean((xv - dequant(a, r, meta, False)) ** 2)
    assert e_anchor > 100 * e_full


def test_degenerate_rows():
    const = np.full((1, 128), 1.5, np.float32)
    a, r, meta, codes = oracle.split_quantize(_row_bits(const), want_codes=True)
    assert meta[0, 0] == 0.0 and meta[0, 1] == np.float32(1.5) and not codes.any()
    assert np.all(dequant(a, r, meta, True) == 1.5)
    negzero = np.full((1, 128), -0.0, np.float32)
    a, r, meta = oracle.split_quantize(_row_bits(negzero))
    assert meta[0, 1] == 0.0 and not np.signbit(meta[0, 1])
    # a sub-threshold range is treated as constant (no overflow in 255 / range)
    tiny = np.zeros((1, 128), np.float32)
    tiny[0, 3] = np.float32(2.0 ** -120)
    a, r, meta, codes = oracle.split_quantize(_row_bits(tiny), want_codes=True)
    assert meta[0, 0] == 0.0 and not codes.any()
    # empty input
    a, r, meta = oracle.split_quantize(np.zeros((0, 128), np.uint16))
    assert a.shape == (0, 64) and meta.shape == (0, 2)


def test_recombine_round_trip_and_bf16_dequant():
    x = synth.kv_block_values("lognormal_channels", 4, 2, 16, "cpu", "rt", 3)
    bits = bf16_bits(x).reshape(-1, 128)
    a, r, meta, codes = oracle.split_quantize(bits, want_codes=True)
    codes2, deq = oracle.recombine(a, r, meta)
    assert np.array_equal(codes, codes2)
    exact = meta[:, 1:2].astype(np.float64) + meta[:, 0:1].astype(np.float64) * codes
    got = bits_to_f64(deq)
    # FP32 multiply-add (rel 2^-24) then BF16 rounding (8 significant bits: half-ulp <= 2^-8 rel)
    assert np.all(np.abs(got - exact) <= np.abs(exact) * (2.0 ** -8 + 2.0 ** -22) + 1e-30)
    nz = exact != 0
    assert np.max(np.abs(got - exact)[nz] / np.abs(exact)[nz]) > 2.0 ** -10   # really BF16
    # an integer row dequantises to itself exactly
    row = np.array([[0.0, 255.0] + [float(v) for v in range(1, 127)]], np.float32)
    a, r, meta = oracle.split_quantize(_row_bits(row))
    _, deq = oracle.recombine(a, r, meta)
    assert np.array_equal(bits_to_f64(deq), row.astype(np.float64))


# ----------------------------------------------------------------------------- attention
# the C interface carries softmax_scale as a binary32 value; 1/sqrt(128) is rounded to it once
SM_SCALE = float(np.float32(1.0 / math.sqrt(128.0)))


def _small_case(seed, B=2, Hkv=2, G=2, n_q=1, lens=(37, 20), bt=16, shuffled=True,
                recipe="normal_outlier4x8"):
    lens_t = torch.tensor(lens, dtype=torch.int32)
    table, nb = synth.block_table(lens_t, bt, shuffled, "pin", seed)
    k = synth.kv_block_values(recipe, nb, Hkv, bt, "cpu", "pinK", seed)
    v = synth.kv_block_values(recipe, nb, Hkv, bt, "cpu", "pinV", seed)
    q = synth.queries(B, n_q, Hkv * G, "cpu", "pinQ", seed)
    kp = oracle.split_quantize(bf16_bits(k))
    vp = oracle.split_quantize(bf16_bits(v))
    return dict(q=q, kp=kp, vp=vp, table=table.numpy(), lens=lens_t.numpy(), Hkv=Hkv, G=G, bt=bt,
                n_q=n_q, B=B)


def _gather_dense(planes, table, lens, b, hkv, bt, full):
    """float64 [len][128] dequantised rows of sequence b, kv head hkv."""
    a, r, m = planes
    rows = []
    for t in range(int(lens[b])):
        blk = table[b, t // bt]
        rows.append(dequant(a[blk, hkv, t % bt], r[blk, hkv, t % bt], m[blk, hkv, t % bt], full))
    return np.stack(rows) if rows else np.zeros((0, 128))


@pytest.mark.parametrize("full", [False, True])
def test_attention_brute_force_python_floats(full):
    c = _small_case(11, lens=(19, 5))
    out = oracle.attention(full, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"], c["lens"],
                           c["Hkv"], c["bt"])
    qf = bits_to_f64(bf16_bits(c["q"]))
    for b in range(c["B"]):
        for h in range(c["Hkv"] * c["G"]):
            K = _gather_dense(c["kp"], c["table"], c["lens"], b, h // c["G"], c["bt"], full).tolist()
            V = _gather_dense(c["vp"], c["table"], c["lens"], b, h // c["G"], c["bt"], full).tolist()
            qv = qf[b, 0, h].tolist()
            s = [sum(qv[d] * K[t][d] for d in range(128)) * SM_SCALE for t in range(len(K))]
            mx = max(s)
            w = [math.exp(x - mx) for x in s]
            z = sum(w)
            for d in range(0, 128, 7):
                o = sum(w[t] * V[t][d] for t in range(len(K))) / z
                assert abs(out[b, 0, h, d] - o) <= 1e-12 * (1 + abs(o))


@pytest.mark.parametrize("full", [False, True])
@pytest.mark.parametrize("causal,n_q", [(False, 1), (False, 3), (True, 4)])
def test_attention_matches_torch_sdpa_float64(full, causal, n_q):
    c = _small_case(12, B=2, Hkv=2, G=4, n_q=n_q, lens=(70, 33))
    out = oracle.attention(full, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"], c["lens"],
                           c["Hkv"], c["bt"], causal=causal)
    qf = torch.from_numpy(bits_to_f64(bf16_bits(c["q"])))                      # [B][n_q][Hq][128]
    for b in range(c["B"]):
        L = int(c["lens"][b])
        K = torch.stack([torch.from_numpy(_gather_dense(c["kp"], c["table"], c["lens"], b, h,
                                                        c["bt"], full)) for h in range(c["Hkv"])])
        V = torch.stack([torch.from_numpy(_gather_dense(c["vp"], c["table"], c["lens"], b, h,
                                                        c["bt"], full)) for h in range(c["Hkv"])])
        Q = qf[b].permute(1, 0, 2).unsqueeze(0)                                # [1][Hq][n_q][128]
        mask = None
        if causal:
            j = torch.arange(n_q).view(n_q, 1)
            t = torch.arange(L).view(1, L)
            mask = t < (L - n_q + j + 1)
        ref = torch.nn.functional.scaled_dot_product_attention(
            Q, K.unsqueeze(0), V.unsqueeze(0), attn_mask=mask, enable_gqa=True, scale=SM_SCALE)
        ref = ref[0].permute(1, 0, 2).numpy()                                  # [n_q][Hq][128]
        assert np.allclose(out[b], ref, rtol=1e-11, atol=1e-12)


def test_attention_invariants():
    c = _small_case(13, B=1, Hkv=2, G=2, lens=(48,), shuffled=False)
    qb = bf16_bits(c["q"])
    # q = 0 -> uniform weights -> mean of V_hat
    out0 = oracle.attention(False, np.zeros_like(qb), c["kp"], c["vp"], c["table"], c["lens"],
                            c["Hkv"], c["bt"])
    for h in range(4):
        V = _gather_dense(c["vp"], c["table"], c["lens"], 0, h // 2, c["bt"], False)
        assert np.allclose(out0[0, 0, h], V.mean(axis=0), rtol=1e-12, atol=1e-13)
    # len = 1 -> V_hat of token 0
    out1 = oracle.attention(True, qb, c["kp"], c["vp"], c["table"], np.array([1], np.int32),
                            c["Hkv"], c["bt"])
    for h in range(4):
        V = _gather_dense(c["vp"], c["table"], np.array([1]), 0, h // 2, c["bt"], True)
        assert np.allclose(out1[0, 0, h], V[0], rtol=1e-13, atol=0)
    # outputs are convex combinations of V_hat rows
    out = oracle.attention(True, qb, c["kp"], c["vp"], c["table"], c["lens"], c["Hkv"], c["bt"])
    for h in range(4):
        V = _gather_dense(c["vp"], c["table"], c["lens"], 0, h // 2, c["bt"], True)
        assert np.all(out[0, 0, h] <= V.max(axis=0) + 1e-12)
        assert np.all(out[0, 0, h] >= V.min(axis=0) - 1e-12)
    # permuting whole blocks of tokens (with their rows) leaves non-causal attention unchanged
    perm = np.array([[2, 0, 1]], np.int32)
    outp = oracle.attention(True, qb, c["kp"], c["vp"], perm, c["lens"], c["Hkv"], c["bt"])
    assert np.allclose(out, outp, rtol=1e-12, atol=1e-13)
    # softmax_scale is honoured: scale 0 gives the mean again
    outs = oracle.attention(False, qb, c["kp"], c["vp"], c["table"], c["lens"], c["Hkv"], c["bt"],
                            softmax_scale=0.0)
    assert np.allclose(outs, out0, rtol=1e-12, atol=1e-13)
    # GQA mapping: q head h reads kv head h // G -> swapping the two KV heads' planes swaps
    # which q heads see which data
    sw = lambda p: tuple(None if x is None else np.ascontiguousarray(x[:, ::-1]) for x in p)
    qsw = np.ascontiguousarray(qb[:, :, [2, 3, 0, 1]])
    outsw = oracle.attention(True, qsw, sw(c["kp"]), sw(c["vp"]), c["table"], c["lens"], c["Hkv"],
                             c["bt"])
    assert np.allclose(outsw[:, :, [2, 3, 0, 1]], out, rtol=1e-12, atol=1e-13)


def test_causal_equals_truncated_non_causal_and_empty_visibility():
    c = _small_case(14, B=1, Hkv=1, G=2, n_q=3, lens=(21,))
    qb = bf16_bits(c["q"])
    outc = oracle.attention(True, qb, c["kp"], c["vp"], c["table"], c["lens"], 1, c["bt"],
                            causal=True)
    for j in range(3):
        o = oracle.attention(True, qb[:, j:j + 1], c["kp"], c["vp"], c["table"],
                             np.array([21 - 3 + j + 1], np.int32), 1, c["bt"])
        assert np.array_equal(o[0, 0], outc[0, j])
    # len 2 with 3 causal queries: query 0 sees nothing -> zeros
    o = oracle.attention(False, qb, c["kp"], c["vp"], c["table"], np.array([2], np.int32), 1,
                         c["bt"], causal=True)
    assert not o[0, 0].any() and o[0, 1].any()
    # len 0 -> zeros
    o = oracle.attention(False, qb, c["kp"], c["vp"], c["table"], np.array([0], np.int32), 1,
                         c["bt"])
    assert not o.any()


# ------------------------------------------------------------------------ verify decision
def test_verify_decision_properties():
    rng = np.random.default_rng(5)
    full = rng.standard_normal((3, 4, 8, 128))
    draft = full.astype(np.float32)
    fr, dev = oracle.verify_decision(full, draft, 1e-3, 1e-2)
    assert fr.tolist() == [4, 4, 4] and np.all(dev < 1e-3)
    # perturb position j of sequence 1 by 10x the tolerance -> first_reject = j
    for j in range(4):
        d2 = draft.copy()
        d2[1, j, 3, 17] += np.float32(10 * (1e-3 + 1e-2 * abs(full[1, j, 3, 17])))
        fr, dev = oracle.verify_decision(full, d2, 1e-3, 1e-2)
        assert fr.tolist() == [4, j, 4]
        assert 9.0 < dev[1, j] < 11.0
    # two perturbed positions: the first one wins
    d2 = draft.copy()
    d2[0, 3, 0, 0] += 1.0
    d2[0, 1, 0, 0] += 1.0
    fr, dev = oracle.verify_decision(full, d2, 1e-3, 1e-2)
    assert fr[0] == 1
    # dev is the plain formula
    want = np.max(np.abs(full - d2.astype(np.float64)) / (1e-3 + 1e-2 * np.abs(full)), axis=(2, 3))
    assert np.allclose(dev, want, rtol=1e-14)
    # monotone in atol: a looser tolerance never rejects earlier
    noisy = (full + 3e-3 * rng.standard_normal(full.shape)).astype(np.float32)
    last = -1
    for atol in [1e-4, 1e-3, 1e-2, 1e-1]:
        fr, _ = oracle.verify_decision(full, noisy, atol, 0.0)
        assert np.all(fr >= last)
        last = fr.copy()
    assert np.all(last == 4)
    # k = 1
    fr, dev = oracle.verify_decision(full[:, :1], draft[:, :1], 1e-3, 1e-2)
    assert fr.tolist() == [1, 1, 1]


def test_anchor_state_is_a_worse_draft_than_full_state():
    # Table 3 ordering on attention outputs: the Anchor-only (4-bit) error is far above the
    # 8-bit error, both measured against attention on the BF16 values.
    c = _small_case(15, B=1, Hkv=2, G=2, lens=(256,), shuffled=False)
    qb = bf16_bits(c["q"])
    oa = oracle.attention(False, qb, c["kp"], c["vp"], c["table"], c["lens"], 2, c["bt"])
    of = oracle.attention(True, qb, c["kp"], c["vp"], c["table"], c["lens"], 2, c["bt"])
    k = synth.kv_block_values("normal_outlier4x8", 16, 2, 16, "cpu", "pinK", 15).double()
    v = synth.kv_block_values("normal_outlier4x8", 16, 2, 16, "cpu", "pinV", 15).double()
    K = k.permute(1, 0, 2, 3).reshape(2, 256, 128)
    V = v.permute(1, 0, 2, 3).reshape(2, 256, 128)
    Q = torch.from_numpy(bits_to_f64(qb))[0].permute(1, 0, 2).unsqueeze(0)
    ref = torch.nn.functional.scaled_dot_product_attention(Q, K.unsqueeze(0), V.unsqueeze(0),
                                                           enable_gqa=True, scale=SM_SCALE)[0, :, 0].numpy()
    nm = lambda o: np.mean(np.sum((o - ref) ** 2, -1) / np.sum(ref ** 2, -1))
    assert nm(oa[0, 0]) > 20 * nm(of[0, 0])
    assert nm(of[0, 0]) < 1e-2


def test_attention_on_bf16_pages_equals_torch_sdpa_and_the_plane_oracle():
    """oracle.attention_bf16_pages (the paper's dequantise-to-pages decode path) against torch's float64
    scaled_dot_product_attention on the same rows (paged shuffled table, GQA, causal), and against the
    plane oracle up to the BF16 rounding of the dequantised rows."""
    import torch
    rng = np.random.default_rng(5)
    B, Hkv, G, n_q, bt, lens = 2, 2, 4, 3, 16, (50, 21)
    nb = sum((l + bt - 1) // bt for l in lens)
    x = rng.normal(0.0, 1.0, (2, nb, Hkv, bt, 128)).astype(np.float32)
    kb, vb = (np.asarray(bf16_bits(f32_to_bf16_tensor(x[i]))) for i in range(2))
    q = rng.normal(0.0, 1.0, (B, n_q, Hkv * G, 128)).astype(np.float32)
    qb = np.asarray(bf16_bits(f32_to_bf16_tensor(q)))
    perm = rng.permutation(nb).astype(np.int32)
    table = np.zeros((B, 4), np.int32)
    table[0, :4] = perm[:4]
    table[1, :2] = perm[4:6]
    lens_a = np.array(lens, np.int32)
    # quantise, recombine to BF16 pages with the oracle, attend on the pages
    kp, vp = oracle.split_quantize(kb), oracle.split_quantize(vb)
    k_pages, v_pages = oracle.recombine(*kp)[1], oracle.recombine(*vp)[1]
    for causal in (False, True):
        got = oracle.attention_bf16_pages(qb, k_pages, v_pages, table, lens_a, causal=causal)
        qf, kf, vf = (torch.from_numpy(bits_to_f64(a)) for a in (qb, k_pages, v_pages))
        for b in range(B):
            L = int(lens[b])
            rows = lambda pages: pages[torch.from_numpy(table[b, :(L + bt - 1) // bt].astype(np.int64))].permute(1, 0, 2, 3).reshape(Hkv, -1, 128)[:, :L]
            kk, vv = rows(kf), rows(vf)
            mask = torch.ones(n_q, L, dtype=torch.bool)
            if causal:
                for j in range(n_q):
                    mask[j, max(L - n_q + j + 1, 0):] = False
            want = torch.nn.functional.scaled_dot_product_attention(
                qf[b].permute(1, 0, 2)[None], kk[None], vv[None], attn_mask=mask, enable_gqa=True,
                scale=float(np.float32(1.0 / np.sqrt(128.0))))[0].permute(1, 0, 2)   # (the scale crosses the C ABI as binary32)
            assert np.allclose(got[b], want.numpy(), rtol=1e-9, atol=1e-12)
        # the BF16 rounding of the pages (2^-9 relative per element) is the only difference from the plane oracle
        ref = oracle.attention(True, qb, kp, vp, table, lens_a, Hkv, bt, causal=causal)
        assert np.max(np.abs(got - ref)) < 0.05 and np.max(np.abs(got - ref)) > 0.0
