"""CPU oracle of the paper's own quantiser, Algorithm 1 "Lynx Hierarchical Quantization" (Section 4.1)
and of its inverse (Section 4.1 stage 3, the inverse alpha-law) -- TEST INFRASTRUCTURE, like the rest
of this package: plain numpy in binary64, the algorithm's stages in the paper's order and notation.

A page block X is P consecutive tokens of one KV head, H = 128 channels each; the algorithm treats
every channel on its own ("per-channel"): page-level min / range over the P tokens, then chunks of C
consecutive tokens with their own mean and max-magnitude, an alpha-law companding of the normalised
values to 7-bit magnitudes, and the split into a 4-bit Anchor (sign-aware two's complement) and a
4-bit centred Residual.

Readings taken where Algorithm 1 is silent or at odds with itself (PARITY UNPINNED for these: no
printed example fixes them; the pins in tests/test_oracle_pins.py cover what the text does fix):
  * alpha = 255, epsilon = 1e-6 (neither is given; the text only calls it "the standard alpha-law").
  * axis: "axis=1" of the page block is the token axis (per-channel statistics); "axis=2" on the
    two-dimensional chunk view can only mean its last axis (the C entries of a chunk).
  * S = Sign(X_cent), not Sign(X_view): X_view is non-negative after stage 1, so its sign carries
    nothing, while stage 3 drops the sign of X_cent.  Sign(0) counts as +1.
  * magnitude scale 120 instead of 2^7 - 1 = 127: with I up to 127 the biased value I + 7 reaches 134
    and V_mag = 8, so Q_anc would span [-9, 8] (more than 4 bits) and Q_res [-15, 7].  Scaling to
    127 - 7 = 120 keeps every stated property (V_mag in [0, 7], Q_anc in [-8, 7], Q_res a centred
    correction in [-8, 7], V_recon - Q_res = I) and changes only that constant, in both directions.
  * Round = round half to even (numpy rint); ties have measure zero for real data.
  * the metadata (gamma_min, gamma_scale, mu, sigma) stay binary64 here; a kernel will have to fix
    their storage type.
"""
from __future__ import annotations

import numpy as np

ALPHA = 255.0
EPS = 1.0e-6
YMAX = 120.0        # see the module docstring (the paper prints 2^7 - 1)


def hier_quantize(x_pages: np.ndarray, chunk: int = 32, alpha: float = ALPHA, eps: float = EPS) -> dict:
    """x_pages: float [n_pages][P tokens][H channels] (P a multiple of `chunk`).
    Returns q_anc, q_res (int8, same shape, values in [-8, 7]), the raw integers I (uint8), and the
    metadata gamma_min, gamma_scale [n_pages][H], mu, sigma [n_pages][P/chunk][H]."""
    x = np.asarray(x_pages, np.float64)
    n, P, H = x.shape
    assert P % chunk == 0
    # Stage 1: per-channel, page-level normalisation (statistics over the page's tokens)
    g_min = x.min(axis=1)                                   # [n][H]
    g_scale = x.max(axis=1) - g_min
    xn = (x - g_min[:, None, :]) / (g_scale[:, None, :] + eps)
    # Stage 2: per-channel, chunk-wise isolation (chunks of `chunk` consecutive tokens of a channel)
    xv = xn.reshape(n, P // chunk, chunk, H)
    mu = xv.mean(axis=2)                                    # [n][P/C][H]
    x_cent = xv - mu[:, :, None, :]
    sigma = np.abs(x_cent).max(axis=2)
    x_final = x_cent / (sigma[:, :, None, :] + eps)
    # Stage 3: alpha-law magnitudes, raw integers, signs
    y = np.log1p(alpha * np.abs(x_final)) / np.log1p(alpha) * YMAX
    I = np.rint(y).astype(np.int64)
    S = np.where(x_cent < 0.0, -1, 1).astype(np.int64)
    # Stage 4: split-stream construction
    I_bias = I + 7
    v_mag = I_bias >> 4
    v_recon = v_mag << 4
    q_res = v_recon - I
    q_anc = v_mag * S + np.minimum(S, 0)
    shp = (n, P, H)
    return dict(q_anc=q_anc.reshape(shp).astype(np.int8), q_res=q_res.reshape(shp).astype(np.int8),
                I=I.reshape(shp).astype(np.uint8), gamma_min=g_min, gamma_scale=g_scale, mu=mu, sigma=sigma)


def hier_dequantize(q_anc: np.ndarray, q_res: np.ndarray | None, gamma_min: np.ndarray, gamma_scale: np.ndarray,
                    mu: np.ndarray, sigma: np.ndarray, alpha: float = ALPHA, eps: float = EPS) -> np.ndarray:
    """Inverse of hier_quantize.  q_res=None reconstructs from the Anchor stream alone (the Residual,
    a centred correction, taken as zero).  Returns float64 [n_pages][P][H]."""
    qa = np.asarray(q_anc, np.int64)
    n, P, H = qa.shape
    chunks = mu.shape[1]
    C = P // chunks
    S = np.where(qa < 0, -1, 1)
    v_mag = np.where(qa < 0, -qa - 1, qa)                   # undo the two's-complement map
    I = (v_mag << 4) - (0 if q_res is None else np.asarray(q_res, np.int64))
    mag = np.expm1(I / YMAX * np.log1p(alpha)) / alpha      # |x_final| = ((1 + alpha)^(I / YMAX) - 1) / alpha
    x_final = (S * mag).reshape(n, chunks, C, H)
    x_cent = x_final * (sigma[:, :, None, :] + eps)
    xn = (x_cent + mu[:, :, None, :]).reshape(n, P, H)
    return xn * (gamma_scale[:, None, :] + eps) + gamma_min[:, None, :]
