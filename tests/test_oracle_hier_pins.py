"""Pins of the Algorithm 1 oracle (oracle/hier.py) against what the paper and the mathematics fix:
the stated bit-field properties of Section 4.1 stage 4, an exact-rational / high-precision restatement
of stages 1-3 on one page, the inverse alpha-law, and the ordering of Table 3 (Lynx < INT8 < INT4 on the
attention-output error).  CPU only."""
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np

import oracle
from oracle import hier
from util import bf16_bits, bits_to_f64, dequant, f32_to_bf16_tensor


def _pages(seed, n=3, P=256, H=128, outliers=True):
    rng = np.random.default_rng(seed)
    x = rng.normal(0.0, 1.0, (n, P, H))
    if outliers:                       # a few channels with a fixed large magnitude (Section 2.3)
        x[:, :, rng.choice(H, min(4, H - 1), replace=False)] *= 8.0
    return bits_to_f64(np.asarray(bf16_bits(f32_to_bf16_tensor(x.astype(np.float32)))))


def test_split_stream_fields_have_the_stated_ranges_and_identity():
    q = hier.hier_quantize(_pages(1))
    qa, qr, I = q["q_anc"].astype(int), q["q_res"].astype(int), q["I"].astype(int)
    assert qa.min() >= -8 and qa.max() <= 7 and qr.min() >= -8 and qr.max() <= 7     # two 4-bit fields
    assert I.min() >= 0 and I.max() <= 120
    v_mag = np.where(qa < 0, -qa - 1, qa)
    assert np.array_equal((v_mag << 4) - qr, I)                    # V_recon - Q_res == I
    assert set(np.unique(v_mag)) <= set(range(8))
    # sign-aware map: a negative entry never shares its anchor with a non-negative one (-0 is distinct)
    x = _pages(1)
    xn = (x - q["gamma_min"][:, None]) / (q["gamma_scale"][:, None] + hier.EPS)
    cent = xn.reshape(3, 8, 32, 128) - q["mu"][:, :, None]
    assert np.array_equal(qa.reshape(cent.shape) < 0, cent < 0)
    # every chunk has an entry of full magnitude (the one that defines sigma): I = 120 there, up to epsilon
    assert np.all(I.reshape(3, 8, 32, 128).max(axis=2) >= 119)


def test_stages_1_to_3_against_exact_rationals_and_high_precision_logarithms():
    x = _pages(2, n=1, P=64, H=3)                                   # small: pure-Python exact arithmetic
    q = hier.hier_quantize(x, chunk=32)
    getcontext().prec = 50
    eps, alpha = Fraction(hier.EPS), Fraction(hier.ALPHA)
    ln1a = (Decimal(1) + Decimal(hier.ALPHA)).ln()
    checked = 0
    for h in range(3):
        col = [Fraction(float(v)) for v in x[0, :, h]]
        gmin, gscale = min(col), max(col) - min(col)
        xn = [(v - gmin) / (gscale + eps) for v in col]
        assert abs(float(gmin) - q["gamma_min"][0, h]) == 0 and abs(float(gscale) - q["gamma_scale"][0, h]) < 1e-15
        for c in range(2):
            ch = xn[32 * c:32 * c + 32]
            mu = sum(ch) / 32
            cent = [v - mu for v in ch]
            sigma = max(abs(v) for v in cent)
            assert abs(float(mu) - q["mu"][0, c, h]) < 1e-14 and abs(float(sigma) - q["sigma"][0, c, h]) < 1e-14
            for i, v in enumerate(cent):
                xf = abs(v) / (sigma + eps)
                y = (Decimal(1) + Decimal(hier.ALPHA) * (Decimal(xf.numerator) / Decimal(xf.denominator))).ln() / ln1a * 120
                if abs(y - y.to_integral_value()) - Decimal("0.5") > Decimal("-1e-9"):
                    continue                                       # a tie within rounding noise
                assert int(y.to_integral_value(rounding="ROUND_HALF_EVEN")) == int(q["I"][0, 32 * c + i, h])
                checked += 1
    assert checked > 180


def test_inverse_alpha_law_and_reconstruction_errors():
    x = _pages(3)
    q = hier.hier_quantize(x)
    meta = (q["gamma_min"], q["gamma_scale"], q["mu"], q["sigma"])
    full = hier.hier_dequantize(q["q_anc"], q["q_res"], *meta)
    anchor = hier.hier_dequantize(q["q_anc"], None, *meta)
    # the alpha-law is monotone and its inverse inverts it: magnitudes reconstructed from the exact
    # (unrounded) y would be exact; with rounding the error in y is at most half a step
    xf = np.linspace(0.0, 1.0, 2001)
    y = np.log1p(hier.ALPHA * xf) / np.log1p(hier.ALPHA) * 120.0
    assert np.all(np.diff(y) > 0) and y[0] == 0.0 and abs(y[-1] - 120.0) < 1e-12
    back = np.expm1(y / 120.0 * np.log1p(hier.ALPHA)) / hier.ALPHA
    assert np.max(np.abs(back - xf)) < 1e-12
    # per element: |x^ - x| is bounded by half a step of y at that magnitude, in the element's own units
    unit = (q["sigma"][:, :, None, :] + hier.EPS).repeat(32, axis=2).reshape(x.shape) * (q["gamma_scale"][:, None, :] + hier.EPS)
    xfin = np.abs(x - (q["mu"][:, :, None, :].repeat(32, axis=2).reshape(x.shape) * (q["gamma_scale"][:, None, :] + hier.EPS)
                       + q["gamma_min"][:, None, :])) / unit
    step = np.log1p(hier.ALPHA) / 120.0 * (1.0 + hier.ALPHA * xfin) / hier.ALPHA     # d|x_final| / dy
    growth = np.exp(0.5 * np.log1p(hier.ALPHA) / 120.0)                             # the curve steepens within the step
    assert np.all(np.abs(full - x) <= 0.5 * step * growth * unit + 1e-9)
    # the Residual is a centred correction of at most 8 steps: Anchor-only is coarser, never closer on average
    assert np.abs(anchor - x).mean() > 4.0 * np.abs(full - x).mean()
    assert np.all(np.abs(anchor - x) <= 8.0 * step * growth ** 16 * unit + 1e-9)


def _attend(q, k, v):
    s = (q @ k.T) / np.sqrt(128.0)
    w = np.exp(s - s.max(axis=1, keepdims=True))
    return (w / w.sum(axis=1, keepdims=True)) @ v


def test_table3_ordering_of_the_attention_output_error():
    # Table 3 orders the schemes by the normalised error of the attention outputs: Lynx (8 bits,
    # hierarchical) below uniform INT8 below uniform INT4, and Lynx's Anchor alone (4 bits) below INT4.
    # Here on synthetic rows with outlier channels, uniform = this repository's per-token linear quantiser.
    rng = np.random.default_rng(11)
    n_tok = 1024
    k = _pages(21, n=4).reshape(n_tok, 128)
    v = _pages(22, n=4).reshape(n_tok, 128)
    qv = rng.normal(0.0, 1.0, (16, 128))
    ref = _attend(qv, k, v)

    def vnmse(kk, vv):
        o = _attend(qv, kk, vv)
        return float(np.mean(np.sum((o - ref) ** 2, axis=1) / np.sum(ref ** 2, axis=1)))

    def hier_rt(x, anchor_only):
        qh = hier.hier_quantize(x.reshape(4, 256, 128))
        return hier.hier_dequantize(qh["q_anc"], None if anchor_only else qh["q_res"], qh["gamma_min"], qh["gamma_scale"],
                                    qh["mu"], qh["sigma"]).reshape(n_tok, 128)

    def linear_rt(x, full):
        a, r, m = oracle.split_quantize(np.asarray(bf16_bits(f32_to_bf16_tensor(x.astype(np.float32)))))
        return dequant(a, r, m, full)
    e_lynx = vnmse(hier_rt(k, False), hier_rt(v, False))
    e_lynx4 = vnmse(hier_rt(k, True), hier_rt(v, True))
    e_int8 = vnmse(linear_rt(k, True), linear_rt(v, True))
    e_int4 = vnmse(linear_rt(k, False), linear_rt(v, False))
    assert e_lynx < e_int8 < e_int4, (e_lynx, e_int8, e_int4)
    assert e_lynx4 < e_int4, (e_lynx4, e_int4)
