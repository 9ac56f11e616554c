"""Pins of the token-level verification oracle (Section 4.3) against facts that do not come from it."""
import numpy as np

from oracle.token_verify import token_verify


def _dist(rng, *shape):
    x = rng.random(shape) ** 3
    return x / x.sum(axis=-1, keepdims=True)


def test_identical_distributions_accept_everything_and_draw_the_bonus_from_q():
    rng = np.random.default_rng(1)
    B, k, V = 5, 6, 37
    q = _dist(rng, B, k + 1, V)
    s = rng.integers(0, V, (B, k))
    for b in range(B):                                     # tokens the draft could have drawn
        for i in range(k):
            s[b, i] = int(np.argmax(q[b, i]))
    u = rng.random((B, k)) * 0.999
    r = rng.random(B)
    n, nxt, _ = token_verify(q[:, :k], q, s, u, r)
    assert n.tolist() == [k] * B                           # ratio 1: u < 1 always accepts
    for b in range(B):                                     # bonus: inverse CDF of q_{k+1}, written out
        c, t = 0.0, r[b] * q[b, k].sum()
        for x in range(V):
            c += q[b, k, x]
            if c > t:
                break
        assert nxt[b] == x


def test_one_hot_target_rejects_a_different_draft_and_corrects_to_its_token():
    B, k, V = 3, 4, 11
    p = np.full((B, k, V), 1.0 / V)
    q = np.zeros((B, k + 1, V))
    q[..., 7] = 1.0
    s = np.full((B, k), 2)
    s[1, 0] = 7                                            # sequence 1 drafted the right first token
    n, nxt, _ = token_verify(p, q, s, np.full((B, k), 0.5), np.array([0.0, 0.5, 0.999]))
    assert n.tolist() == [0, 1, 0] and nxt.tolist() == [7, 7, 7]


def test_acceptance_threshold_is_q_over_p():
    V = 4
    p = np.array([[[0.5, 0.5, 0.0, 0.0]]])
    q = np.array([[[0.2, 0.8, 0.0, 0.0], [0.25, 0.25, 0.25, 0.25]]])
    s = np.array([[0]])                                    # ratio q/p = 0.4
    assert token_verify(p, q, s, np.array([[0.39]]), np.array([0.1]))[0].tolist() == [1]
    n, nxt, _ = token_verify(p, q, s, np.array([[0.41]]), np.array([0.1]))
    assert n.tolist() == [0] and nxt.tolist() == [1]       # residual max(0, q - p) = (0, 0.3, 0, 0)
    s = np.array([[1]])                                    # ratio 1.6 -> always accepted
    assert token_verify(p, q, s, np.array([[0.999]]), np.array([0.6]))[0].tolist() == [1]
    assert token_verify(p, q, s, np.array([[0.999]]), np.array([0.6]))[1].tolist() == [2]   # bonus: cdf .25 .5 .75 1


def test_output_distribution_is_the_target_distribution():
    # the losslessness of Section 2.4: with drafts drawn from p and the rule above, the first output token is
    # distributed as q_1, whatever p is (Monte Carlo on a small vocabulary, 5 sigma)
    rng = np.random.default_rng(7)
    V, N = 6, 200_000
    p1, q = _dist(rng, V), _dist(rng, 2, V)
    s = rng.choice(V, size=N, p=p1)
    P = np.broadcast_to(p1, (N, 1, V))
    Q = np.broadcast_to(q, (N, 2, V))
    n, nxt, _ = token_verify(P, Q, s[:, None], rng.random((N, 1)), rng.random(N))
    first = np.where(n == 1, s, nxt)
    freq = np.bincount(first, minlength=V) / N
    assert np.all(np.abs(freq - q[0]) < 5 * np.sqrt(q[0] * (1 - q[0]) / N) + 1e-4)
    # and the second token, given that the first was accepted, as q_2
    acc = n == 1
    freq2 = np.bincount(nxt[acc], minlength=V) / acc.sum()
    assert np.all(np.abs(freq2 - q[1]) < 5 * np.sqrt(q[1] * (1 - q[1]) / acc.sum()) + 1e-4)


def test_zero_residual_falls_back_to_the_target_row():
    p = np.array([[[0.5, 0.5]]])
    q = np.array([[[0.5, 0.5], [1.0, 0.0]]])
    n, nxt, _ = token_verify(p, q, np.array([[0]]), np.array([[1.0]]), np.array([0.75]))   # u p = q: not accepted
    assert n.tolist() == [0] and nxt.tolist() == [1]
