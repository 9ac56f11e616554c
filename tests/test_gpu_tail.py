"""GPU parity of the log-sum-exps the attention calls leave in their workspaces, and of decode attention over a
quantised prefix followed by a BF16 tail (prefix call + BF16-page call + lynx_lse_merge), against the binary64
oracle (oracle/tail.py).  Outputs within |gpu - ref| <= 2e-3 + 1e-2 |ref| as for every attention call; the
log-sum-exps within 2e-4 (integer kernels, BF16 kernel) or 3e-3 (FP16 kernel, 33..64 columns): a relative
error e of a softmax sum moves its logarithm by e."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import tail
from util import bf16_bits

pytestmark = pytest.mark.gpu
ATOL, RTOL = 2e-3, 1e-2


@pytest.fixture(scope="module")
def lynx():
    import paper_2607_01831_b200 as m
    m.load()
    return m


def _close(got, ref, what):
    err = np.abs(got - ref)
    worst = float(np.max(err / (ATOL + RTOL * np.abs(ref))))
    assert np.all(np.isfinite(got)) and worst <= 1.0, f"{what}: worst error/bound {worst:.3f}"


def _lse_close(got, ref, tol, what):
    assert np.array_equal(np.isneginf(got), np.isneginf(ref)), what + ": empty rows differ"
    fin = np.isfinite(ref)
    assert np.all(np.isfinite(got[fin])), what + ": non-finite log-sum-exp"
    if fin.any():
        worst = float(np.max(np.abs(got[fin] - ref[fin])))
        assert worst <= tol, f"{what}: log-sum-exp off by {worst:.2e}"


def _case(lynx, seed, Hkv, G, n_q, lens, tail_lens, bt=16, bt_t=16, recipe="normal_outlier4x8"):
    B = len(lens)
    lens_t, tl = torch.tensor(lens, dtype=torch.int32), torch.tensor(tail_lens, dtype=torch.int32)
    table, nb = synth.block_table(torch.clamp(lens_t, min=1), bt, True, "gt", seed)
    ttable, nbt = synth.block_table(torch.clamp(tl, min=1), bt_t, True, "gt2", seed)
    k = synth.kv_block_values(recipe, nb, Hkv, bt, "cpu", "gtK", seed)
    v = synth.kv_block_values(recipe, nb, Hkv, bt, "cpu", "gtV", seed)
    kt = synth.kv_block_values(recipe, nbt, Hkv, bt_t, "cpu", "gtKt", seed)
    vt = synth.kv_block_values(recipe, nbt, Hkv, bt_t, "cpu", "gtVt", seed)
    q = synth.queries(B, n_q, Hkv * G, "cpu", "gtQ", seed)
    K, V = lynx.split_quantize(k.cuda()), lynx.split_quantize(v.cuda())
    geo = lynx.Geometry(Hkv * G, Hkv, bt, nb, table.shape[1])
    geo_t = lynx.Geometry(Hkv * G, Hkv, bt_t, nbt, ttable.shape[1])
    return dict(B=B, n_q=n_q, geo=geo, geo_t=geo_t, q=q, K=K, V=V, kt=kt, vt=vt, table=table, lens=lens_t, ttable=ttable,
                tlens=tl, kp=oracle.split_quantize(bf16_bits(k)), vp=oracle.split_quantize(bf16_bits(v)))


def _oracle(c, full, causal_tail, lens=None, tlens=None):
    return tail.prefix_tail_attention(full, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                                      (c["lens"] if lens is None else lens).numpy(), bf16_bits(c["kt"]), bf16_bits(c["vt"]),
                                      c["ttable"].numpy(), (c["tlens"] if tlens is None else tlens).numpy(),
                                      causal_tail=causal_tail)


# columns = n_q * G: 4 / 8 / 16 / 32 (integer kernels; verification takes 32 as two passes), 64 (FP16 kernel for
# verification, two slices for anchor); a 40000-token sequence spans many CTAs (partial slots, two-level merge)
@pytest.mark.parametrize("G,n_q,lens", [(4, 1, (700, 0, 33)), (4, 2, (40000, 5)), (8, 2, (130, 2100)), (4, 8, (3000, 3)),
                                        (8, 8, (900, 70)), (1, 3, (1, 257))])
def test_log_sum_exps_of_the_plane_attention(lynx, G, n_q, lens):
    c = _case(lynx, 100 + G * n_q, 2, G, n_q, lens, (0,) * len(lens))
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    ws = lynx.make_workspace(c["geo"], c["B"], n_q, "cuda")
    for causal in (False, True):
        # the oracle's "tail" is empty; its causal limit is then expressed through shortened prefix lengths per query
        for full in (False, True):
            if full:
                got, _, _ = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, ws, causal=causal)
            else:
                got = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, ws, causal=causal)
            lse = lynx.workspace_lse(c["geo"], c["B"], n_q, ws).cpu().numpy().astype(np.float64)
            assert lynx.load().lynx_check(ws.data_ptr(), None) == 0
            ref_lse = np.empty_like(lse)
            ref_out = np.empty((c["B"], n_q, 2 * G, 128))
            for j in range(n_q):   # query j sees len - n_q + j + 1 tokens when causal
                seen = torch.clamp(c["lens"] - (n_q - j - 1), min=0) if causal else c["lens"]
                cj = dict(c, q=c["q"][:, j:j + 1].contiguous())
                r = _oracle(cj, full, False, lens=seen.to(torch.int32))
                ref_lse[:, j], ref_out[:, j] = r["lse_prefix"][:, 0], r["out"][:, 0]
            _close(got.cpu().numpy().astype(np.float64), ref_out, f"out full={full} causal={causal}")
            _lse_close(lse, ref_lse, 3e-3 if full and n_q * G > 32 else 2e-4, f"G={G} n_q={n_q} full={full} causal={causal}")


@pytest.mark.parametrize("G,n_q,lens,tail_lens,bt_t", [(4, 1, (5000, 300, 0, 0), (37, 0, 260, 0), 16),
                                                       (4, 2, (2100, 64), (2, 130), 16),
                                                       (8, 1, (999, 17), (1, 4100), 32),
                                                       (2, 4, (1500, 40), (4, 77), 48)])
@pytest.mark.parametrize("full", [False, True])
def test_prefix_in_planes_plus_bf16_tail(lynx, G, n_q, lens, tail_lens, bt_t, full):
    """Decode (n_q = 1) and short windows (the n_q queries are the tail's last tokens: causal inside the tail,
    every query sees the whole prefix).  Sequences with an empty prefix, an empty tail, or both."""
    c = _case(lynx, 200 + G + n_q, 2, G, n_q, lens, tail_lens, bt_t=bt_t, recipe="lognormal_channels")
    qd = c["q"].cuda()
    ws = lynx.make_workspace(c["geo"], c["B"], n_q, "cuda")
    if full:
        pre, _, _ = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], c["table"].cuda(), c["lens"].cuda(), ws,
                                                causal=False)
    else:
        pre = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], c["table"].cuda(), c["lens"].cuda(), ws, causal=False)
    lse_pre = lynx.workspace_lse(c["geo"], c["B"], n_q, ws)
    n = int(lynx.load().lynx_bf16_workspace_bytes(c["geo_t"]._c(), c["B"], n_q))
    ws_t = torch.empty(n, dtype=torch.uint8, device="cuda")
    tl = lynx.bf16_attention(c["geo_t"], qd, c["kt"].cuda(), c["vt"].cuda(), c["ttable"].cuda(), c["tlens"].cuda(),
                             workspace=ws_t, causal=True)
    lse_tl = lynx.bf16_workspace_lse(c["geo_t"], c["B"], n_q, ws_t)
    out, lse = lynx.lse_merge(pre, lse_pre, tl, lse_tl, want_lse=True)
    torch.cuda.synchronize()
    ref = _oracle(c, full, True)
    _lse_close(lse_pre.cpu().numpy().astype(np.float64), ref["lse_prefix"], 2e-4, "prefix")
    _lse_close(lse_tl.cpu().numpy().astype(np.float64), ref["lse_tail"], 2e-4, "tail")
    _lse_close(lse.cpu().numpy().astype(np.float64), ref["lse"], 2e-4, "joined")
    _close(out.cpu().numpy().astype(np.float64), ref["out"], f"prefix + tail G={G} n_q={n_q} full={full}")
    # in place, without the joined log-sum-exp
    same = lynx.lse_merge(pre, lse_pre, tl, lse_tl, out=pre)
    assert same.data_ptr() == pre.data_ptr() and torch.equal(same, out)


def test_lse_merge_against_the_oracle_rule_and_its_edge_cases(lynx):
    g = torch.Generator().manual_seed(5)
    rows = 1003
    a, b = torch.randn(rows, 128, generator=g), torch.randn(rows, 128, generator=g)
    la, lb = torch.randn(rows, generator=g) * 20.0, torch.randn(rows, generator=g) * 20.0
    la[0] = lb[1] = -np.inf          # one empty part: the other's row, bit for bit
    la[2] = lb[2] = -np.inf          # both empty: zeros and -inf
    a[0] = np.nan                    # whatever an empty part's row holds stays out
    b[2] = np.inf
    la[3], lb[3] = 80.0, -80.0       # far apart
    la[4] = lb[4] = 3.0              # equal
    out, lse = lynx.lse_merge(a.cuda(), la.cuda(), b.cuda(), lb.cuda(), want_lse=True)
    ref, ref_lse = tail.lse_merge(np.where(np.isfinite(a.numpy()), a.numpy(), 0.0).astype(np.float64), la.numpy(),
                                  np.where(np.isfinite(b.numpy()), b.numpy(), 0.0).astype(np.float64), lb.numpy())
    got, got_lse = out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got))
    assert np.max(np.abs(got - ref)) <= 1e-5
    assert np.array_equal(np.isneginf(got_lse), np.isneginf(ref_lse))
    fin = np.isfinite(ref_lse)
    assert np.max(np.abs(got_lse[fin] - ref_lse[fin])) <= 1e-5 * (1 + np.max(np.abs(ref_lse[fin])))
    assert torch.equal(out[0].cpu(), b[0]) and torch.equal(out[1].cpu(), a[1]) and not out[2].any()
    assert torch.equal(out[3].cpu(), a[3])
    # argument checks: NULL, alignment, negative size; an empty call launches nothing
    L = lynx.load()
    x = a.cuda()
    assert L.lynx_lse_merge(None, la.cuda().data_ptr(), x.data_ptr(), la.cuda().data_ptr(), 4, x.data_ptr(), None, None) == 1
    assert L.lynx_lse_merge(x.data_ptr() + 4, la.cuda().data_ptr(), x.data_ptr(), la.cuda().data_ptr(), 4, x.data_ptr(), None, None) == 3
    assert L.lynx_lse_merge(x.data_ptr(), la.cuda().data_ptr(), x.data_ptr(), la.cuda().data_ptr(), -1, x.data_ptr(), None, None) == 2
    assert L.lynx_lse_merge(None, None, None, None, 0, None, None, None) == 0


def test_verify_decision_on_outputs_in_memory(lynx):
    g = torch.Generator().manual_seed(9)
    B, k, Hq = 37, 5, 12
    f = torch.randn(B, k, Hq, 128, generator=g)
    d = f + 0.02 * torch.randn(B, k, Hq, 128, generator=g) * (torch.rand(B, k, 1, 1, generator=g) < 0.5)
    d[3] = f[3]                                  # a window that agrees everywhere
    d[4, 0, 2, 7] += 5.0                         # and one rejected at its first position
    exercised = 0
    for atol, rtol in [(0.05, 0.05), (0.1, 0.0), (0.2, 0.1), (1e-3, 1e-2)]:
        want_fr, want_dev = oracle.verify_decision(f.numpy().astype(np.float64), d.numpy(), atol, rtol)
        fr, dev = lynx.verify_decision(f.cuda(), d.cuda(), atol, rtol)
        assert np.allclose(dev.cpu().numpy(), want_dev, rtol=1e-5, atol=1e-7)
        clear = np.all(np.abs(want_dev - 1.0) > 1e-4, axis=1)      # (binary32 against binary64 at the threshold)
        exercised += int(clear.sum())
        assert np.array_equal(fr.cpu().numpy()[clear], want_fr[clear])
        assert int(fr[3]) == k and int(fr[4]) == 0
    assert exercised >= 100
    L = lynx.load()
    x = f.cuda()
    fr = torch.empty(B, dtype=torch.int32, device="cuda")
    dv = torch.empty(B, k, device="cuda")
    assert L.lynx_verify_decision(x.data_ptr(), None, B, k, Hq, 0.1, 0.1, fr.data_ptr(), dv.data_ptr(), None) == 1
    assert L.lynx_verify_decision(x.data_ptr(), x.data_ptr(), B, 65, Hq, 0.1, 0.1, fr.data_ptr(), dv.data_ptr(), None) == 2
    assert L.lynx_verify_decision(x.data_ptr(), x.data_ptr(), B, k, Hq, 0.0, 0.1, fr.data_ptr(), dv.data_ptr(), None) == 2
    assert L.lynx_verify_decision(x.data_ptr() + 4, x.data_ptr(), B, k, Hq, 0.1, 0.1, fr.data_ptr(), dv.data_ptr(), None) == 3
    assert L.lynx_verify_decision(None, None, 0, k, Hq, 0.1, 0.1, None, None, None) == 0


def test_a_window_is_verified_over_prefix_and_tail(lynx):
    """Section 4.3 with a BF16 tail: drafts on the Anchor prefix + tail, the full-state pass on prefix + tail, the
    agreement test on the joined outputs -- against the oracle's decision on its own joined outputs."""
    G, k = 4, 4      # 16 columns: one launch of the integer kernels, two slices of the BF16-page kernel
    c = _case(lynx, 321, 2, G, k, (1800, 90, 0), (6, 40, 9), recipe="student_t4")
    qd = c["q"].cuda()
    ws = lynx.make_workspace(c["geo"], c["B"], k, "cuda")
    ws_t = torch.empty(int(lynx.load().lynx_bf16_workspace_bytes(c["geo_t"]._c(), c["B"], k)), dtype=torch.uint8, device="cuda")
    tl = lynx.bf16_attention(c["geo_t"], qd, c["kt"].cuda(), c["vt"].cuda(), c["ttable"].cuda(), c["tlens"].cuda(),
                             workspace=ws_t, causal=True)
    lse_tl = lynx.bf16_workspace_lse(c["geo_t"], c["B"], k, ws_t).clone()
    lse_pre = lynx.workspace_lse(c["geo"], c["B"], k, ws)
    anchor = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], c["table"].cuda(), c["lens"].cuda(), ws, causal=False)
    draft = lynx.lse_merge(anchor, lse_pre, tl, lse_tl)
    full, _, _ = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], c["table"].cuda(), c["lens"].cuda(), ws, causal=False)
    joined = lynx.lse_merge(full, lse_pre, tl, lse_tl)
    ref_a, ref_f = _oracle(c, False, True)["out"], _oracle(c, True, True)["out"]
    _close(draft.cpu().numpy().astype(np.float64), ref_a, "draft over prefix + tail")
    _close(joined.cpu().numpy().astype(np.float64), ref_f, "full state over prefix + tail")
    exercised = 0
    for atol, rtol in [(2e-2, 2e-2), (5e-2, 5e-2), (1e-1, 1e-1), (3e-1, 1e-1), (1.0, 0.0), (3e-3, 0.0)]:
        want_fr, want_dev = oracle.verify_decision(ref_f, ref_a.astype(np.float32), atol, rtol)
        if np.all(np.abs(want_dev - 1.0) > 0.05):
            exercised += 1
            fr, dev = lynx.verify_decision(joined, draft, atol, rtol)
            assert np.array_equal(fr.cpu().numpy(), want_fr), (atol, rtol, want_dev)
    assert exercised >= 1
