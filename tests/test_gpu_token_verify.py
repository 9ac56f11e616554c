"""lynx_token_verify (Section 4.3 at token level) against the binary64 oracle."""
import numpy as np
import pytest
import torch

from oracle.token_verify import token_verify as oracle_token_verify

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lynx():
    import paper_2607_01831_b200 as L
    L.load()
    return L


def _dists(rng, B, k, V, sharp):
    """Target distributions q and Anchor-state distributions p = softmax of perturbed logits."""
    logits = rng.standard_normal((B, k + 1, V)) * sharp
    q = np.exp(logits - logits.max(-1, keepdims=True))
    q /= q.sum(-1, keepdims=True)
    lp = logits[:, :k] + 0.3 * rng.standard_normal((B, k, V))
    p = np.exp(lp - lp.max(-1, keepdims=True))
    p /= p.sum(-1, keepdims=True)
    return p.astype(np.float32), q.astype(np.float32)


@pytest.mark.parametrize("B,k,V,sharp", [(64, 8, 1000, 2.0), (16, 4, 128256, 3.0), (32, 64, 257, 1.0),
                                          (8, 1, 5, 0.5), (24, 16, 32000, 6.0)])
def test_token_verify_matches_oracle(lynx, B, k, V, sharp):
    rng = np.random.default_rng(B * 1000 + k)
    p, q = _dists(rng, B, k, V, sharp)
    s = np.stack([[rng.choice(V, p=p[b, i].astype(np.float64) / p[b, i].astype(np.float64).sum()) for i in range(k)]
                  for b in range(B)]).astype(np.int32)
    u = rng.random((B, k)).astype(np.float32)
    r = rng.random(B).astype(np.float32)
    want_n, want_x, margin = oracle_token_verify(p, q, s, u, r)
    got_n, got_x = lynx.token_verify(torch.from_numpy(p).cuda(), torch.from_numpy(q).cuda(),
                                     torch.from_numpy(s).cuda(), torch.from_numpy(u).cuda(),
                                     torch.from_numpy(r).cuda())
    torch.cuda.synchronize()
    got_n, got_x = got_n.cpu().numpy(), got_x.cpu().numpy()
    # FP32 sums against binary64: compare the sequences whose decisions are not within rounding of a threshold
    clear = margin > 1e-4
    assert clear.sum() >= B // 2, "too few sequences outside the guard band"
    assert np.array_equal(got_n[clear], want_n[clear])
    assert np.array_equal(got_x[clear], want_x[clear])
    assert np.all((got_x >= 0) & (got_x < V)) and np.all((got_n >= 0) & (got_n <= k))
    assert len(set(want_n.tolist())) > 1 or k == 1           # both accepted and rejected windows occur


def test_token_verify_closed_cases_and_errors(lynx):
    B, k, V = 3, 4, 11
    p = torch.full((B, k, V), 1.0 / V, device="cuda")
    q = torch.zeros(B, k + 1, V, device="cuda")
    q[..., 7] = 1.0
    s = torch.full((B, k), 2, dtype=torch.int32, device="cuda")
    s[1, 0] = 7
    n, x = lynx.token_verify(p, q, s, torch.full((B, k), 0.5, device="cuda"),
                             torch.tensor([0.0, 0.5, 0.999], device="cuda"))
    assert n.cpu().tolist() == [0, 1, 0] and x.cpu().tolist() == [7, 7, 7]
    # identical distributions: everything accepted, the bonus token from q_{k+1}
    qq = torch.rand(B, k + 1, V, device="cuda")
    qq /= qq.sum(-1, keepdim=True)
    ss = qq[:, :k].argmax(-1).to(torch.int32)
    n, x = lynx.token_verify(qq[:, :k].contiguous(), qq, ss, torch.rand(B, k, device="cuda") * 0.99,
                             torch.full((B,), 0.5, device="cuda"))
    assert n.cpu().tolist() == [k] * B
    cdf = qq[:, k].double().cumsum(-1).cpu().numpy()
    for b in range(B):
        assert x.cpu().tolist()[b] == int(np.searchsorted(cdf[b], 0.5 * cdf[b, -1], side="right"))
    L = lynx.load()
    assert L.lynx_token_verify(None, None, None, None, None, 0, 1, 1, None, None, None) == 0
    assert L.lynx_token_verify(None, None, None, None, None, 1, 1, 1, None, None, None) == 1    # NULL
    assert L.lynx_token_verify(p.data_ptr(), q.data_ptr(), s.data_ptr(), p.data_ptr(), p.data_ptr(), 1, 65, 8,
                               s.data_ptr(), s.data_ptr(), None) == 2                            # k > 64
