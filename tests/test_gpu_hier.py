"""GPU parity of lynx_hier_quantize / lynx_hier_dequantize (Algorithm 1 and its inverse) against the
binary64 oracle (oracle/hier.py).  The kernels compute in binary32, so a raw integer may differ from
the oracle's by one where the companded value lies within binary32 noise of a rounding tie; everywhere
else codes are identical, and reconstructions agree to a fraction of a quantisation step."""
import numpy as np
import pytest
import torch

import synth
from oracle import hier
from util import bf16_bits, bits_to_f64

pytestmark = pytest.mark.gpu


def _nib(packed):         # u8 [...,64] -> signed 4-bit values int [...,128]
    lo, hi = packed & 15, packed >> 4
    v = np.stack([lo, hi], axis=-1).reshape(packed.shape[:-1] + (128,)).astype(np.int64)
    return np.where(v > 7, v - 16, v)


# 1000 pages: more than the quantiser's grid (three CTAs per SM), so CTAs walk through several pages
@pytest.mark.parametrize("recipe,n_pages", [("normal_outlier4x8", 5), ("student_t4", 37), ("lognormal_channels", 300),
                                            ("normal_outlier4x8", 1000)])
def test_hier_quantize_and_dequantize_match_the_oracle(recipe, n_pages):
    # pages of 256 tokens x 128 channels (one KV head each)
    x = synth.kv_block_values(recipe, n_pages, 1, 256, "cpu", "hier", n_pages).reshape(n_pages, 256, 128)
    _check_against_oracle(x)


def test_hier_degenerate_pages():
    """Channels that are constant over a page or over a chunk (range / deviation 0: only epsilon keeps the
    divisions finite), a single outlier in an otherwise constant channel, a page of zeros, negative zero,
    values of very different magnitude in neighbouring channels."""
    g = torch.Generator().manual_seed(11)
    x = torch.randn(6, 256, 128, generator=g)
    x[0, :, 0:8] = 3.25                      # constant over the page
    x[0, :, 8] = -0.0
    x[1, 64:96, 16:24] = -1.5                # constant over one chunk
    x[1, :, 24] = 0.0
    x[1, 200, 24] = 7.0                      # one outlier in a constant channel
    x[2] = 0.0                               # a page of zeros
    x[3, :, 0::2] *= 1.0e-3                  # small next to large: the two channels of a word
    x[3, :, 1::2] *= 1.0e3
    x[4] = torch.round(x[4] * 2.0) / 2.0     # many equal values, ties in the statistics
    x[5, :, 40] = torch.linspace(-1.0, 1.0, 256)
    _check_against_oracle(x.to(torch.bfloat16))


def _check_against_oracle(x):
    import paper_2607_01831_b200 as lynx
    lynx.load()
    n_pages = x.shape[0]
    got = lynx.hier_quantize(x.cuda())
    torch.cuda.synchronize()
    xf = bits_to_f64(bf16_bits(x))
    want = hier.hier_quantize(xf)
    # metadata: binary32 against binary64
    for name in ("gamma_min", "gamma_scale", "mu", "sigma"):
        g = getattr(got, name).cpu().numpy().astype(np.float64)
        assert np.allclose(g, want[name], rtol=2e-6, atol=2e-7), name
    qa, qr = _nib(got.q_anc.cpu().numpy()), _nib(got.q_res.cpu().numpy())
    v_mag = np.where(qa < 0, -qa - 1, qa)
    I_gpu = (v_mag << 4) - qr
    I_ref = want["I"].astype(np.int64)
    assert qa.min() >= -8 and qa.max() <= 7 and qr.min() >= -8 and qr.max() <= 7
    diff = I_gpu != I_ref
    assert np.all(np.abs(I_gpu - I_ref) <= 1)
    assert diff.mean() < 2e-3, f"{diff.mean():.2e} of the raw integers differ"
    # where they differ the oracle's companded value is within noise of a tie
    meta = (want["gamma_min"], want["gamma_scale"], want["mu"], want["sigma"])
    xn = (xf - meta[0][:, None]) / (meta[1][:, None] + hier.EPS)
    cent = xn.reshape(n_pages, 8, 32, 128) - meta[2][:, :, None]
    xfin = (cent / (meta[3][:, :, None] + hier.EPS)).reshape(xf.shape)
    y = np.log1p(hier.ALPHA * np.abs(xfin)) / np.log1p(hier.ALPHA) * 120.0
    assert np.all(np.abs(np.abs(y[diff] - np.floor(y[diff])) - 0.5) < 2e-2)
    # signs: identical except for centred values within binary32 noise of zero
    sdiff = (qa < 0) != (want["q_anc"].astype(np.int64) < 0)
    assert np.all(np.abs(xfin[sdiff]) < 1e-4)
    # reconstruction: both streams, and the Anchor alone, against the oracle's reconstruction
    for anchor_only in (False, True):
        rec = lynx.hier_dequantize(got, anchor_only=anchor_only)
        torch.cuda.synchronize()
        r_gpu = bits_to_f64(bf16_bits(rec))
        r_ref = hier.hier_dequantize(want["q_anc"], None if anchor_only else want["q_res"], *meta)
        unit = ((meta[3][:, :, None, :] + hier.EPS).repeat(32, axis=2).reshape(xf.shape)
                * (meta[1][:, None, :] + hier.EPS))
        step = np.log1p(hier.ALPHA) / 120.0 * (1.0 + hier.ALPHA * np.abs(xfin)) / hier.ALPHA * unit   # one code step
        tol = 1.5 * step + 2.0 ** -8 * np.abs(r_ref) + 1e-6          # a step where I differs, BF16 rounding elsewhere
        if anchor_only:      # a raw integer that differs across a multiple of 16 moves the Anchor by a whole interval
            tol = np.where(diff, 36.0 * step, tol)
        assert np.all(np.abs(r_gpu - r_ref) <= tol), float(np.max(np.abs(r_gpu - r_ref) / tol))
        close = np.abs(r_gpu - r_ref) <= 2.0 ** -8 * np.abs(r_ref) + 1e-4 * unit + 1e-6
        assert close.mean() > 0.995
    # and the round trip itself: the full reconstruction is far closer to the input than the Anchor's
    full = bits_to_f64(bf16_bits(lynx.hier_dequantize(got)))
    anch = bits_to_f64(bf16_bits(lynx.hier_dequantize(got, anchor_only=True)))
    assert np.abs(full - xf).mean() * 4.0 < np.abs(anch - xf).mean()


def test_hier_pages_feed_the_bf16_attention():
    # the paper's flow end to end: Algorithm 1, dequantise to BF16 pages, attend on the pages
    import oracle
    import paper_2607_01831_b200 as lynx
    Hkv, G, L = 2, 4, 1000
    n_pg = (L + 255) // 256
    kx = synth.kv_block_values("normal_outlier4x8", n_pg * Hkv, 1, 256, "cpu", "hierK").reshape(n_pg * Hkv, 256, 128)
    vx = synth.kv_block_values("normal_outlier4x8", n_pg * Hkv, 1, 256, "cpu", "hierV").reshape(n_pg * Hkv, 256, 128)
    q = synth.queries(1, 1, Hkv * G, "cpu", "hierQ")
    pages = {}
    for name, x in (("k", kx), ("v", vx)):
        h = lynx.hier_quantize(x.cuda())
        pages[name] = lynx.hier_dequantize(h).view(n_pg, Hkv, 256, 128)      # [block][head][token][128], block = page
    geo = lynx.Geometry(Hkv * G, Hkv, 256, n_pg, n_pg)
    table = torch.arange(n_pg, dtype=torch.int32).view(1, n_pg).cuda()
    lens = torch.tensor([L], dtype=torch.int32).cuda()
    got = lynx.bf16_attention(geo, q.cuda(), pages["k"], pages["v"], table, lens)
    ref = oracle.attention_bf16_pages(bf16_bits(q), bf16_bits(pages["k"]), bf16_bits(pages["v"]),
                                      table.cpu().numpy(), lens.cpu().numpy())
    g = got.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(g - ref) <= 2e-3 + 1e-2 * np.abs(ref))
    # and against attention on the unquantised rows: the 8-bit hierarchical state is a close approximation
    exact = oracle.attention_bf16_pages(bf16_bits(q), bf16_bits(kx.view(n_pg, Hkv, 256, 128)),
                                        bf16_bits(vx.view(n_pg, Hkv, 256, 128)), table.cpu().numpy(), lens.cpu().numpy())
    assert np.sqrt(np.mean((g - exact) ** 2) / np.mean(exact ** 2)) < 0.1
