"""CPU oracle of decode attention over a quantised prefix followed by a BF16 tail -- TEST
INFRASTRUCTURE, like the rest of this package: plain numpy in binary64, one (sequence, query, head) at
a time, written from the definitions.

The prefix is the transferred KV cache in the Lynx planes (Section 4.1 stage 4 packing; dequantised
value = level * scale + zero of the linear grouped quantiser of Section 2.3, with level = 16 a + 8 on
the Anchor alone (Section 4.2, Anchor phase) or 16 a + r once the Residual has arrived); the tail holds
the tokens the decode node generated itself, which never went through the quantiser and stay BF16
pages.  Attention is Section 2's softmax(q K^T scale) V over the concatenation [prefix ; tail].

Also here: the log-sum-exp of a set of scores and the textbook rule that joins two softmax-weighted
averages over disjoint key sets from their log-sum-exps, which is how a kernel for the prefix and a
kernel for the tail can be combined.
"""
from __future__ import annotations

import numpy as np

D = 128


def _bf16_f64(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def dequantised_rows(full: bool, planes, blocks: np.ndarray, hkv: int, length: int) -> np.ndarray:
    """Rows [length][128] of one (sequence, KV head): token t = row t % block_tokens of block
    blocks[t // block_tokens].  planes = (anchor u8 [nb][Hkv][bt][64], residual or None, meta f32
    [nb][Hkv][bt][2] = (scale, zero)); byte j of a row = element 2j (low nibble) | element 2j+1 << 4."""
    anchor, residual, meta = planes
    a = np.asarray(anchor)[blocks, hkv].reshape(-1, 64)[:length].astype(np.int64)
    m = np.asarray(meta)[blocks, hkv].reshape(-1, 2)[:length].astype(np.float64)
    a_el = np.stack([a & 15, a >> 4], axis=-1).reshape(-1, D)
    if full:
        r = np.asarray(residual)[blocks, hkv].reshape(-1, 64)[:length].astype(np.int64)
        level = 16 * a_el + np.stack([r & 15, r >> 4], axis=-1).reshape(-1, D)
    else:
        level = 16 * a_el + 8
    return level.astype(np.float64) * m[:, :1] + m[:, 1:2]


def prefix_tail_attention(full: bool, q_bf16_bits: np.ndarray, k_planes, v_planes, block_table: np.ndarray,
                          seq_lens: np.ndarray, k_tail_bits: np.ndarray, v_tail_bits: np.ndarray,
                          tail_table: np.ndarray, tail_lens: np.ndarray, causal_tail: bool = False,
                          softmax_scale: float | None = None) -> dict:
    """q_bf16_bits uint16 [B][n_q][Hq][128]; prefix planes and block_table / seq_lens as in
    oracle.attention; tail pages uint16 [nb_t][Hkv][bt_t][128] with tail_table int32 [B][max_t] and
    tail_lens int32 [B].  Every query sees the whole prefix; of the tail it sees all tokens or, with
    causal_tail, the first tail_len - n_q + j + 1 (the n_q queries are the tail's last n_q tokens).
    Returns out float64 [B][n_q][Hq][128] (zeros where a query sees nothing) and the natural-log
    log-sum-exps lse_prefix, lse_tail, lse [B][n_q][Hq] (-inf for an empty set)."""
    q = _bf16_f64(q_bf16_bits)
    B, n_q, Hq, d = q.shape
    kt, vt = _bf16_f64(k_tail_bits), _bf16_f64(v_tail_bits)
    Hkv, bt = np.asarray(k_planes[0]).shape[1], np.asarray(k_planes[0]).shape[2]
    bt_t = kt.shape[2]
    assert d == D and Hq % Hkv == 0 and kt.shape[1] == Hkv
    G = Hq // Hkv
    if softmax_scale is None:
        softmax_scale = 1.0 / np.sqrt(np.float64(D))
    scale = np.float64(np.float32(softmax_scale))
    out = np.zeros((B, n_q, Hq, D), np.float64)
    lse = {k: np.full((B, n_q, Hq), -np.inf) for k in ("lse_prefix", "lse_tail", "lse")}

    def logsumexp(s):
        return -np.inf if s.size == 0 else s.max() + np.log(np.exp(s - s.max()).sum())

    for b in range(B):
        n_pre = min(max(int(seq_lens[b]), 0), block_table.shape[1] * bt)
        n_tail = min(max(int(tail_lens[b]), 0), tail_table.shape[1] * bt_t)
        blocks = np.asarray(block_table[b, :(n_pre + bt - 1) // bt], np.int64)
        tblocks = np.asarray(tail_table[b, :(n_tail + bt_t - 1) // bt_t], np.int64)
        for h in range(Hq):
            kp = dequantised_rows(full, k_planes, blocks, h // G, n_pre)
            vp = dequantised_rows(full, v_planes, blocks, h // G, n_pre)
            ktl = kt[tblocks, h // G].reshape(-1, D)[:n_tail]
            vtl = vt[tblocks, h // G].reshape(-1, D)[:n_tail]
            for j in range(n_q):
                lim = max(n_tail - n_q + j + 1, 0) if causal_tail else n_tail
                s_pre = (kp @ q[b, j, h]) * scale
                s_tail = (ktl[:lim] @ q[b, j, h]) * scale
                lse["lse_prefix"][b, j, h] = logsumexp(s_pre)
                lse["lse_tail"][b, j, h] = logsumexp(s_tail)
                s = np.concatenate([s_pre, s_tail])
                lse["lse"][b, j, h] = logsumexp(s)
                if s.size == 0:
                    continue
                w = np.exp(s - s.max())
                out[b, j, h] = (w / w.sum()) @ np.concatenate([vp, vtl[:lim]])
    return dict(out=out, **lse)


def lse_merge(out_a: np.ndarray, lse_a: np.ndarray, out_b: np.ndarray, lse_b: np.ndarray):
    """Two softmax-weighted averages over disjoint key sets, each with the natural-log log-sum-exp of its
    scores, joined into the average over the union: weights e^lse_a and e^lse_b, normalised.  out_*
    [..., 128], lse_* [...]; an empty set has lse = -inf and contributes nothing; if both are empty the
    result is zero with lse = -inf.  Returns (out, lse)."""
    la, lb = np.asarray(lse_a, np.float64), np.asarray(lse_b, np.float64)
    m = np.maximum(la, lb)
    safe = np.where(np.isfinite(m), m, 0.0)
    wa, wb = np.exp(la - safe), np.exp(lb - safe)
    tot = wa + wb
    inv = np.where(tot > 0.0, 1.0 / np.where(tot > 0.0, tot, 1.0), 0.0)
    out = (np.asarray(out_a, np.float64) * (wa * inv)[..., None] + np.asarray(out_b, np.float64) * (wb * inv)[..., None])
    with np.errstate(divide="ignore"):
        lse = np.where(tot > 0.0, safe + np.log(np.where(tot > 0.0, tot, 1.0)), -np.inf)
    return out, lse
