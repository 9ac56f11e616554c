"""CPU oracle of token-level verification (Section 4.3; the speculative-sampling rule of Section 2.4's
references) -- TEST INFRASTRUCTURE, like the rest of this package: plain numpy in binary64, one sequence
and one position at a time.

The decode instance drafts tokens s_1..s_k from the Anchor-state distributions p_1..p_k; the verification
pass on the full-precision state yields q_1..q_{k+1}.  Token s_i is accepted with probability
min(1, q_i(s_i) / p_i(s_i)); the first rejected position j is corrected by a token drawn from the residual
distribution norm(max(0, q_j - p_j)); if every draft is accepted a bonus token is drawn from q_{k+1}.  The
output sequence is then distributed as if sampled from q alone (the losslessness the paper relies on).

Readings (the paper leaves the rule to its references, and prints it only in a commented-out passage with
p and q in the other roles):
  * the random numbers are inputs: u[b, i] decides position i (accepted iff u * p_i(s_i) < q_i(s_i): no
    division, p = 0 with q > 0 accepts, p = q = 0 rejects), r[b] draws the correction or the bonus token by
    inverse CDF over the vocabulary in index order: the smallest x with cumsum(w)[x] > r * sum(w);
  * a residual that is zero everywhere (q_j <= p_j for all x, only possible through rounding) falls back to
    w = q_j.
"""
from __future__ import annotations

import numpy as np


def token_verify(p_probs: np.ndarray, q_probs: np.ndarray, draft_tokens: np.ndarray, u: np.ndarray,
                 r: np.ndarray):
    """p_probs [B][k][V], q_probs [B][k+1][V], draft_tokens int [B][k], u [B][k], r [B].
    Returns (n_accepted int32 [B], next_token int32 [B], margin float64 [B]); `margin` is how far the two
    decisions of sequence b were from flipping (relative distance of the acceptance tests and of r * sum(w)
    from the nearest CDF step), for tests that compare with lower-precision implementations."""
    p = np.asarray(p_probs, np.float64)
    q = np.asarray(q_probs, np.float64)
    B, k, V = p.shape
    assert q.shape == (B, k + 1, V)
    n_acc = np.zeros(B, np.int32)
    nxt = np.zeros(B, np.int32)
    margin = np.full(B, np.inf)
    for b in range(B):
        j = k
        for i in range(k):
            s = int(draft_tokens[b, i])
            lhs, rhs = float(u[b, i]) * p[b, i, s], q[b, i, s]
            scale = max(abs(lhs), abs(rhs), 1e-300)
            margin[b] = min(margin[b], abs(lhs - rhs) / scale)
            if not lhs < rhs:
                j = i
                break
        n_acc[b] = j
        w = np.maximum(q[b, j] - p[b, j], 0.0) if j < k else q[b, k].copy()
        if j < k and not w.sum() > 0.0:
            w = q[b, j].copy()
        c = np.cumsum(w)
        t = float(r[b]) * c[-1]
        x = int(np.searchsorted(c, t, side="right"))
        x = min(x, V - 1)
        nxt[b] = x
        steps = np.abs(c - t) / max(c[-1], 1e-300)
        margin[b] = min(margin[b], float(steps.min()))
    return n_acc, nxt, margin
