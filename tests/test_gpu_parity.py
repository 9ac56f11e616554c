"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element.

Codes, planes, metadata bits and accept/reject indices must match bit-exactly; attention
outputs within |gpu - ref| <= 2e-3 + 1e-2 |ref| against the float64 oracle.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from util import bf16_bits, f32_to_bf16_tensor

pytestmark = pytest.mark.gpu

ATOL, RTOL = 2e-3, 1e-2


@pytest.fixture(scope="module")
def lynx():
    import paper_2607_01831_b200 as m
    m.load()
    return m


def _planes_np(p):
    return (p.anchor.cpu().numpy(), None if p.residual is None else p.residual.cpu().numpy(),
            p.meta.cpu().numpy())


def _assert_planes_equal(got, want):
    ga, gr, gm = got
    wa, wr, wm = want
    assert np.array_equal(ga, wa), "anchor plane differs"
    assert np.array_equal(gr, wr), "residual plane differs"
    assert np.array_equal(gm.view(np.uint32), wm.view(np.uint32)), "meta bits differ"


# ------------------------------------------------------------------------- split-quantise
@pytest.mark.parametrize("recipe", ["normal_outlier4x8", "lognormal_channels", "student_t4",
                                    "normal_outlier2pct_x10"])
@pytest.mark.parametrize("n_blocks", [1, 37, 300])
def test_split_quantize_bit_exact(lynx, recipe, n_blocks):
    x = synth.kv_block_values(recipe, n_blocks, 8, 16, "cpu", "sq", n_blocks)
    x = x.reshape(-1, 128)[: x.numel() // 128 - 3]          # ragged tail: not a multiple of 64 rows
    got = lynx.split_quantize(x.cuda())
    torch.cuda.synchronize()
    _assert_planes_equal(_planes_np(got), oracle.split_quantize(bf16_bits(x)))


def test_split_quantize_special_rows(lynx):
    rows = [
        [0.0, 255.0] + [float(v) for v in range(1, 127)],
        [0.0, 255.0] + [k + 0.5 for k in range(126)],          # ties -> even
        [1.5] * 128,                                           # constant row
        [-0.0] * 128,                                          # minus zero
        [0.0] * 127 + [2.0 ** -120],                           # sub-threshold range
        [-3.0 + 0.5 * i for i in range(128)],
        [1.0e38] * 64 + [-1.0e38] * 64,                        # huge but finite range
    ]
    x = f32_to_bf16_tensor(np.array(rows, np.float32))
    got = lynx.split_quantize(x.cuda())
    torch.cuda.synchronize()
    _assert_planes_equal(_planes_np(got), oracle.split_quantize(bf16_bits(x)))


def test_split_quantize_block_ids_only_touch_listed_blocks(lynx):
    nb, hkv, bt = 20, 4, 16
    x = synth.kv_block_values("student_t4", nb, hkv, bt, "cpu", "ids", 1)
    ids = torch.tensor([3, 17, 0, 9, 25, -1], dtype=torch.int32)     # 25 and -1 are skipped
    out = lynx.alloc_planes((nb, hkv, bt), "cuda")
    out.anchor.fill_(0xAB); out.residual.fill_(0xCD); out.meta.fill_(-7.0)
    lynx.split_quantize(x.cuda(), out=out, block_ids=ids.cuda(), rows_per_block=hkv * bt)
    torch.cuda.synchronize()
    wa, wr, wm = oracle.split_quantize(bf16_bits(x))
    ga, gr, gm = _planes_np(out)
    listed = [3, 17, 0, 9]
    for b in range(nb):
        if b in listed:
            assert np.array_equal(ga[b], wa[b]) and np.array_equal(gr[b], wr[b])
            assert np.array_equal(gm[b].view(np.uint32), wm[b].view(np.uint32))
        else:
            assert np.all(ga[b] == 0xAB) and np.all(gr[b] == 0xCD) and np.all(gm[b] == -7.0)


def test_split_quantize_empty_and_errors(lynx):
    L = lynx.load()
    assert L.lynx_split_quantize(None, 0, None, 0, 0, None, None, None, None) == 0
    x = torch.zeros(4, 128, dtype=torch.bfloat16, device="cuda")
    p = lynx.alloc_planes((4,), "cuda")
    assert L.lynx_split_quantize(x.data_ptr(), 4, None, 0, 0, None, p.residual.data_ptr(),
                                 p.meta.data_ptr(), None) == 1                      # NULL
    assert L.lynx_split_quantize(x.data_ptr() + 2, 3, None, 0, 0, p.anchor.data_ptr(),
                                 p.residual.data_ptr(), p.meta.data_ptr(), None) == 3  # alignment
    assert L.lynx_split_quantize(x.data_ptr(), -1, None, 0, 0, p.anchor.data_ptr(),
                                 p.residual.data_ptr(), p.meta.data_ptr(), None) == 2  # shape
    assert L.lynx_status_string(3).decode().startswith("pointer")


# ------------------------------------------------------------------------------ recombine
def test_recombine_bit_exact(lynx):
    x = synth.kv_block_values("lognormal_channels", 61, 8, 16, "cpu", "rc", 1).reshape(-1, 128)[:-5]
    p = lynx.split_quantize(x.cuda())
    codes, deq = lynx.recombine(p, want_codes=True, want_bf16=True)
    codes_only, _ = lynx.recombine(p, want_codes=True, want_bf16=False)
    _, deq_only = lynx.recombine(p, want_codes=False, want_bf16=True)
    torch.cuda.synchronize()
    wa, wr, wm, wcodes = oracle.split_quantize(bf16_bits(x), want_codes=True)
    ocodes, odeq = oracle.recombine(wa, wr, wm)
    assert np.array_equal(ocodes, wcodes)
    assert np.array_equal(codes.cpu().numpy(), ocodes)
    assert np.array_equal(codes_only.cpu().numpy(), ocodes)
    assert np.array_equal(bf16_bits(deq), odeq)
    assert np.array_equal(bf16_bits(deq_only), odeq)
    # the identity the split is defined by
    a = p.anchor.cpu().numpy(); r = p.residual.cpu().numpy()
    lo = ((a & 15).astype(np.uint16) << 4) | (r & 15)
    hi = ((a >> 4).astype(np.uint16) << 4) | (r >> 4)
    assert np.array_equal(np.stack([lo, hi], -1).reshape(-1, 128), ocodes)


# ------------------------------------------------------------------------------ attention
def _case(lynx, seed, B, Hkv, G, n_q, lens, bt=16, shuffled=True, recipe="normal_outlier4x8"):
    lens_t = torch.tensor(lens, dtype=torch.int32)
    cap = [max(int(l), 1) for l in lens]
    table, nb = synth.block_table(torch.tensor(cap, dtype=torch.int32), bt, shuffled, "gp", seed)
    k = synth.kv_block_values(recipe, nb, Hkv, bt, "cpu", "gpK", seed)
    v = synth.kv_block_values(recipe, nb, Hkv, bt, "cpu", "gpV", seed)
    q = synth.queries(B, n_q, Hkv * G, "cpu", "gpQ", seed)
    K = lynx.split_quantize(k.cuda())
    V = lynx.split_quantize(v.cuda())
    torch.cuda.synchronize()
    kp, vp = oracle.split_quantize(bf16_bits(k)), oracle.split_quantize(bf16_bits(v))
    _assert_planes_equal(_planes_np(K), kp)
    geo = lynx.Geometry(Hkv * G, Hkv, bt, nb, table.shape[1])
    ws = lynx.make_workspace(geo, B, n_q, "cuda")
    return dict(geo=geo, ws=ws, q=q, K=K, V=V, kp=kp, vp=vp, table=table, lens=lens_t, Hkv=Hkv, bt=bt)


def _close(got, ref, what):
    err = np.abs(got - ref)
    bound = ATOL + RTOL * np.abs(ref)
    assert np.all(np.isfinite(got)), what + ": non-finite output"
    worst = float(np.max(err / bound))
    assert worst <= 1.0, f"{what}: worst error/bound {worst:.3f}, max abs err {err.max():.3e}"
    return float(err.max())


ATTN_CASES = [
    # B, Hkv, G, n_q, lens, bt, shuffled, recipe
    (1, 8, 4, 1, (4096,), 16, False, "normal_outlier4x8"),         # config-1 shape, several chunks
    (2, 2, 4, 1, (1000, 37), 16, True, "lognormal_channels"),      # ragged, not multiples of 16
    (3, 2, 8, 1, (1, 15, 17), 16, True, "student_t4"),             # tiny lengths, G = 8
    (2, 1, 1, 1, (300, 0), 16, True, "normal"),                    # G = 1 and an empty sequence
    (1, 2, 2, 3, (777,), 32, True, "normal_outlier2pct_x10"),      # 32-token blocks, n_q = 3
    (1, 2, 4, 4, (2500,), 16, True, "student_t4"),                 # 16 columns
    (1, 1, 4, 8, (1300,), 16, True, "lognormal_channels"),         # 32 columns
    (1, 1, 8, 8, (900,), 64, True, "normal_outlier4x8"),           # 64 columns, 64-token blocks
    (1, 1, 16, 1, (500,), 16, False, "normal"),                    # G = 16
]


@pytest.mark.parametrize("case", ATTN_CASES, ids=[str(i) for i in range(len(ATTN_CASES))])
@pytest.mark.parametrize("causal", [False, True])
def test_anchor_attention_matches_oracle(lynx, case, causal):
    B, Hkv, G, n_q, lens, bt, shuffled, recipe = case
    c = _case(lynx, 100 + len(lens) + n_q, B, Hkv, G, n_q, lens, bt, shuffled, recipe)
    out = lynx.anchor_attention(c["geo"], c["q"].cuda(), c["K"], c["V"], c["table"].cuda(),
                                c["lens"].cuda(), c["ws"], causal=causal)
    lynx.check(c["ws"])
    ref = oracle.attention(False, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                           c["lens"].numpy(), Hkv, bt, causal=causal)
    _close(out.cpu().numpy().astype(np.float64), ref, "anchor attention")
    # a second call on the same workspace gives the same bits (counters reset themselves)
    out2 = lynx.anchor_attention(c["geo"], c["q"].cuda(), c["K"], c["V"], c["table"].cuda(),
                                 c["lens"].cuda(), c["ws"], causal=causal)
    lynx.check(c["ws"])
    assert torch.equal(out, out2)


@pytest.mark.parametrize("case", ATTN_CASES, ids=[str(i) for i in range(len(ATTN_CASES))])
@pytest.mark.parametrize("causal", [True, False])
def test_merge_verify_matches_oracle_and_decides_identically(lynx, case, causal):
    B, Hkv, G, k, lens, bt, shuffled, recipe = case
    c = _case(lynx, 200 + len(lens) + k, B, Hkv, G, k, lens, bt, shuffled, recipe)
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    draft = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=causal)
    draft_np = draft.cpu().numpy()
    ref = oracle.attention(True, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                           c["lens"].numpy(), Hkv, bt, causal=causal)
    # thresholds: pick (atol, rtol) so that every oracle dev is outside the guard band around 1
    exercised = 0
    for atol, rtol in [(2e-2, 2e-2), (5e-2, 5e-2), (1e-1, 1e-1), (3e-1, 1e-1), (1.0, 0.0), (3e-3, 0.0)]:
        want_fr, want_dev = oracle.verify_decision(ref, draft_np, atol, rtol)
        if np.all(np.abs(want_dev - 1.0) > 0.05):
            exercised += 1
            out, fr, dev = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"],
                                                       draft_out=draft, atol=atol, rtol=rtol,
                                                       causal=causal)
            lynx.check(c["ws"])
            _close(out.cpu().numpy().astype(np.float64), ref, "merge-verify attention")
            assert np.array_equal(fr.cpu().numpy(), want_fr), (atol, rtol, want_dev)
            assert np.allclose(dev.cpu().numpy(), want_dev, rtol=0.05, atol=1e-3)
    assert exercised >= 1, "every threshold set fell inside the guard band: no index was compared"
    # the full result fed back as its own draft is accepted everywhere
    out, _, _ = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=causal)
    _close(out.cpu().numpy().astype(np.float64), ref, "merge-verify attention (no draft)")
    out2, fr, dev = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"],
                                                draft_out=out, atol=1e-3, rtol=1e-2, causal=causal)
    lynx.check(c["ws"])
    assert torch.equal(out, out2)
    assert fr.cpu().tolist() == [k] * B and float(dev.max()) == 0.0
    # perturbing position j of sequence 0 makes it the first rejection
    for j in range(k):
        bad = out.clone()
        bad[0, j, 1 % (Hkv * G), 5] += 1.0
        _, fr, _ = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"],
                                               draft_out=bad, atol=1e-3, rtol=1e-2, causal=causal)
        assert int(fr[0]) == j


@pytest.mark.parametrize("seed", range(6))
def test_short_heavy_tailed_contexts_keep_a_margin(lynx, seed):
    # a few tokens with heavy-tailed values: one token dominates, so the rounding of its weight to
    # FP16 is not averaged away; the two FP16 weight terms must keep the error well inside the bound
    c = _case(lynx, 400 + seed, 4, 2, 8, 1, (1, 15, 17, 3), 16, True, "student_t4")
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    for full in (False, True):
        if full:
            got = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"])[0]
        else:
            got = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"])
        lynx.check(c["ws"])
        ref = oracle.attention(full, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                               c["lens"].numpy(), 2, 16, causal=full)
        got = got.cpu().numpy().astype(np.float64)
        worst = float(np.max(np.abs(got - ref) / (ATOL + RTOL * np.abs(ref))))
        assert worst <= 0.5, f"full={full}: worst error/bound {worst:.3f}"


@pytest.mark.parametrize("recipe", ["student_t4", "normal_outlier2pct_x10"])
def test_single_token_context_returns_its_value_row(lynx, recipe):
    # softmax over one token is 1, so the output is that token's dequantised V row: FP32 rounding
    # only, whatever the magnitude of the row (the FP16 rounding of the weight cancels exactly)
    B, Hkv, G = 6, 2, 4
    c = _case(lynx, 500, B, Hkv, G, 1, (1,) * B, 16, True, recipe)
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    from util import dequant
    for full in (False, True):
        if full:
            got = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"])[0]
        else:
            got = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"])
        lynx.check(c["ws"])
        got = got.cpu().numpy().astype(np.float64)
        va, vr, vm = c["vp"]
        for b in range(B):
            blk = int(c["table"][b, 0])
            for h in range(Hkv * G):
                row = dequant(va[blk, h // G, 0], vr[blk, h // G, 0], vm[blk, h // G, 0], full)
                size = abs(float(vm[blk, h // G, 0, 1])) + 255.0 * float(vm[blk, h // G, 0, 0])
                assert np.max(np.abs(got[b, 0, h] - row)) <= 4e-6 * size + 1e-30


def test_anchor_then_verify_window_like_the_decoder(lynx):
    # k draft steps on the Anchor state with growing context, then one verify pass on Q_full
    B, Hkv, G, k, L = 1, 2, 4, 4, 1203
    c = _case(lynx, 301, B, Hkv, G, k, (L,), 16, True, "lognormal_channels")
    qd, td = c["q"].cuda(), c["table"].cuda()
    ws1 = lynx.make_workspace(c["geo"], B, 1, "cuda")
    draft = torch.empty(B, k, Hkv * G, 128, dtype=torch.float32, device="cuda")
    for j in range(k):
        lens_j = torch.tensor([L - k + j + 1], dtype=torch.int32).cuda()
        draft[:, j:j + 1] = lynx.anchor_attention(c["geo"], qd[:, j:j + 1].contiguous(), c["K"], c["V"],
                                                  td, lens_j, ws1)
    ref_draft = oracle.attention(False, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                                 c["lens"].numpy(), Hkv, 16, causal=True)
    _close(draft.cpu().numpy().astype(np.float64), ref_draft, "stepwise drafts vs causal anchor")
    ref = oracle.attention(True, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                           c["lens"].numpy(), Hkv, 16, causal=True)
    want_fr, want_dev = oracle.verify_decision(ref, draft.cpu().numpy(), 0.5, 0.0)
    assert np.all(np.abs(want_dev - 1.0) > 0.05)
    out, fr, dev = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, c["lens"].cuda(),
                                               c["ws"], draft_out=draft, atol=0.5, rtol=0.0)
    lynx.check(c["ws"])
    _close(out.cpu().numpy().astype(np.float64), ref, "verify")
    assert np.array_equal(fr.cpu().numpy(), want_fr)


def test_attention_argument_errors_and_bad_block_table(lynx):
    c = _case(lynx, 302, 1, 2, 4, 1, (100,), 16, True, "normal")
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    with pytest.raises(lynx.LynxError):                      # workspace too small
        lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"][:128])
    bad_geo = lynx.Geometry(8, 2, 24, c["geo"].num_blocks, c["geo"].max_blocks_per_seq)
    with pytest.raises(lynx.LynxError):                      # block_tokens not a multiple of 16
        lynx.anchor_attention(bad_geo, qd, c["K"], c["V"], td, ld, c["ws"])
    assert lynx.workspace_bytes(bad_geo, 1, 1) == 0
    q17 = torch.zeros(1, 17, 8, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lynx.LynxError):                      # too many query positions
        lynx.anchor_attention(c["geo"], q17, c["K"], c["V"], td, ld, c["ws"])
    # an out-of-range block id is clamped on the device and reported by lynx_check
    bad_table = td.clone()
    bad_table[0, 1] = 10_000
    lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], bad_table, ld, c["ws"])
    with pytest.raises(lynx.LynxError, match="block id"):
        lynx.check(c["ws"])
    lynx.check(c["ws"])                                      # the status word was cleared
    out = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"])
    lynx.check(c["ws"])
    ref = oracle.attention(False, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                           c["lens"].numpy(), 2, 16)
    _close(out.cpu().numpy().astype(np.float64), ref, "after a bad table")


def test_long_context_multi_chunk_sampled(lynx):
    # one KV head pair at 40k tokens: many chunks per (sequence, head), ragged end
    B, Hkv, G, k, L = 1, 2, 4, 4, 40_003
    c = _case(lynx, 303, B, Hkv, G, k, (L,), 16, True, "lognormal_channels")
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    out_a = lynx.anchor_attention(c["geo"], qd[:, :1].contiguous(), c["K"], c["V"], td, ld,
                                  lynx.make_workspace(c["geo"], B, 1, "cuda"))
    out_v, _, _ = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"])
    lynx.check(c["ws"])
    ref_a = oracle.attention(False, bf16_bits(c["q"][:, :1]), c["kp"], c["vp"], c["table"].numpy(),
                             c["lens"].numpy(), Hkv, 16)
    ref_v = oracle.attention(True, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                             c["lens"].numpy(), Hkv, 16, causal=True)
    _close(out_a.cpu().numpy().astype(np.float64), ref_a, "anchor 40k")
    _close(out_v.cpu().numpy().astype(np.float64), ref_v, "verify 40k")


# ----------- verify with 17..64 columns (17..32: two passes of the integer kernel; 33..64: the FP16 tcgen05 kernel)
WIDE_CASES = [
    # B, Hkv, G, k, lens, bt, recipe
    (4, 2, 4, 8, (1, 15, 17, 0), 16, "student_t4"),              # 32 columns (two slices): tiny, ragged and empty sequences
    (2, 2, 8, 8, (63, 130), 16, "normal_outlier2pct_x10"),       # 64 columns around one and two 64-token units
    (1, 2, 4, 5, (700,), 32, "lognormal_channels"),              # 20 columns: slices of 4 positions + 1
    (1, 2, 8, 5, (333,), 16, "normal_outlier4x8"),               # 40 columns, padded to 64
    (1, 1, 3, 11, (513,), 16, "normal"),                         # 33 columns, group of 3, 11 positions
    (3, 1, 16, 4, (64, 128, 65), 64, "student_t4"),              # 64 columns from G = 16, exact unit multiples
]


@pytest.mark.parametrize("case", WIDE_CASES, ids=[str(i) for i in range(len(WIDE_CASES))])
@pytest.mark.parametrize("causal", [True, False])
def test_wide_verify_matches_oracle_and_decides_identically(lynx, case, causal):
    B, Hkv, G, k, lens, bt, recipe = case
    c = _case(lynx, 600 + k + G, B, Hkv, G, k, lens, bt, True, recipe)
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    ref = oracle.attention(True, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                           c["lens"].numpy(), Hkv, bt, causal=causal)
    out, _, _ = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=causal)
    lynx.check(c["ws"])
    _close(out.cpu().numpy().astype(np.float64), ref, "wide verify")
    out2, _, _ = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=causal)
    assert torch.equal(out, out2)                 # same bits on a second call (deterministic merges)
    # a draft that differs from the full result at known positions: identical decisions
    rng = np.random.default_rng(7)
    draft = torch.from_numpy((ref + rng.normal(0.0, 0.02, ref.shape)).astype(np.float32))
    draft[0, k // 2] += 0.5
    exercised = 0
    for atol, rtol in [(0.2, 0.0), (0.1, 0.1), (0.3, 0.1), (1.0, 0.0)]:
        want_fr, want_dev = oracle.verify_decision(ref, draft.numpy(), atol, rtol)
        if np.all(np.abs(want_dev - 1.0) > 0.05):
            exercised += 1
            _, fr, dev = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"],
                                                     draft_out=draft.cuda(), atol=atol, rtol=rtol,
                                                     causal=causal)
            lynx.check(c["ws"])
            assert np.array_equal(fr.cpu().numpy(), want_fr), (atol, rtol, want_dev)
            assert np.allclose(dev.cpu().numpy(), want_dev, rtol=0.05, atol=2e-3)
    assert exercised >= 1, "every threshold set fell inside the guard band: no index was compared"


def test_wide_verify_long_context_many_pieces(lynx):
    # 32 and 64 columns at 40k tokens: every (sequence, head) is split over several CTAs, so the
    # partial slots, the last-contributor merge and the decision tickets are exercised
    for G, k in ((4, 8), (8, 8)):
        B, Hkv, L = 2, 2, 40_003
        c = _case(lynx, 700 + G, B, Hkv, G, k, (L, 9_000), 16, True, "lognormal_channels")
        qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
        ref = oracle.attention(True, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                               c["lens"].numpy(), Hkv, 16, causal=True)
        out, fr, dev = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"],
                                                   draft_out=torch.from_numpy(ref.astype(np.float32)).cuda(),
                                                   atol=0.05, rtol=0.0)
        lynx.check(c["ws"])
        _close(out.cpu().numpy().astype(np.float64), ref, f"wide verify 40k, {k * G} columns")
        assert fr.cpu().tolist() == [k] * B      # the oracle's own result as draft is accepted
        assert float(dev.max()) < 0.1


def test_long_context_partial_slots_merge_in_two_levels(lynx):
    # 40k tokens on two KV heads: every head is split over some 40 CTAs, more than one group of
    # partial slots, so the group tickets and the merge of the group results are exercised (anchor
    # and merge-verify at 4, 8 and 16 columns); the lengths differ, so the plain cut of the work is used
    B, Hkv, G, L = 2, 2, 4, 40_003
    for k in (1, 2, 4):
        c = _case(lynx, 740 + k, B, Hkv, G, k, (L, 9_000), 16, True, "lognormal_channels")
        qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
        for rep in range(2):   # the tickets reset themselves: a second call on the same workspace
            ra = oracle.attention(False, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                                  c["lens"].numpy(), Hkv, 16, causal=True)
            a = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=True)
            lynx.check(c["ws"])
            _close(a.cpu().numpy().astype(np.float64), ra, f"anchor 40k, {k * G} columns, call {rep}")
            rf = oracle.attention(True, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                                  c["lens"].numpy(), Hkv, 16, causal=True)
            out, fr, dev = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"],
                                                       draft_out=torch.from_numpy(rf.astype(np.float32)).cuda(),
                                                       atol=0.05, rtol=0.0)
            lynx.check(c["ws"])
            _close(out.cpu().numpy().astype(np.float64), rf, f"verify 40k, {k * G} columns, call {rep}")
            assert fr.cpu().tolist() == [k] * B


@pytest.mark.parametrize("B,Hkv,G,k,L", [(1, 8, 4, 1, 40_003), (1, 8, 4, 4, 20_001), (1, 2, 4, 2, 40_003),
                                         (2, 4, 8, 1, 33_000), (1, 8, 4, 8, 12_345), (3, 8, 2, 2, 7_777)])
def test_equal_length_sequences_use_the_aligned_cut(lynx, B, Hkv, G, k, L):
    # all sequences equally long and few (sequence, head) segments: every segment gets whole CTAs of its
    # own (18 per head for one layer of 8 heads; 74 per head with 2 heads: two merge levels; 6 for 24
    # segments).  Anchor and merge-verify, twice on the same workspace (tickets reset themselves).
    c = _case(lynx, 7600 + Hkv * k, B, Hkv, G, k, (L,) * B, 16, True, "lognormal_channels")
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    ra = oracle.attention(False, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(), c["lens"].numpy(),
                          Hkv, 16, causal=True)
    rf = oracle.attention(True, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(), c["lens"].numpy(),
                          Hkv, 16, causal=True)
    for rep in range(2):
        a = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=True)
        lynx.check(c["ws"])
        _close(a.cpu().numpy().astype(np.float64), ra, f"anchor, aligned cut, call {rep}")
        out, fr, dev = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=True,
                                                   draft_out=torch.from_numpy(rf.astype(np.float32)).cuda(),
                                                   atol=0.05, rtol=0.0)
        lynx.check(c["ws"])
        _close(out.cpu().numpy().astype(np.float64), rf, f"verify, aligned cut, call {rep}")
        assert fr.cpu().tolist() == [k] * B


@pytest.mark.parametrize("B,Hkv,G,k,lens", [(2, 2, 4, 24, (1500, 37)), (1, 2, 1, 40, (900,)), (2, 1, 8, 20, (300, 0)),
                                            (1, 1, 2, 64, (2100,)), (1, 2, 16, 5, (700,))])
def test_windows_beyond_one_launch_run_as_slices(lynx, B, Hkv, G, k, lens):
    # up to 64 drafted positions per call (the cap Section 5.1 states): more than 16 positions or 64 columns
    # are verified in slices of whole positions, anchor calls likewise; outputs against the oracle, and the
    # first rejected position over the WHOLE window identical to the oracle's
    c = _case(lynx, 9100 + k, B, Hkv, G, k, lens, 16, True, "lognormal_channels")
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    ra = oracle.attention(False, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(), c["lens"].numpy(),
                          Hkv, 16, causal=True)
    rf = oracle.attention(True, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(), c["lens"].numpy(),
                          Hkv, 16, causal=True)
    draft = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=True)
    lynx.check(c["ws"])
    _close(draft.cpu().numpy().astype(np.float64), ra, "anchor attention, sliced window")
    draft_np = draft.cpu().numpy()
    exercised = 0
    for atol, rtol in [(2e-2, 2e-2), (5e-2, 5e-2), (1e-1, 1e-1), (3e-1, 1e-1), (1.0, 0.0), (3e-3, 0.0)]:
        want_fr, want_dev = oracle.verify_decision(rf, draft_np, atol, rtol)
        if np.all(np.abs(want_dev - 1.0) > 0.05):
            exercised += 1
            out, fr, dev = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"],
                                                       draft_out=draft, atol=atol, rtol=rtol, causal=True)
            lynx.check(c["ws"])
            _close(out.cpu().numpy().astype(np.float64), rf, "merge-verify attention, sliced window")
            assert np.array_equal(fr.cpu().numpy(), want_fr), (atol, rtol, want_dev)
            assert np.allclose(dev.cpu().numpy(), want_dev, rtol=0.05, atol=1e-3)
    assert exercised >= 1
    # a perturbation in a later slice is found as the first rejection of the whole window
    out, _, _ = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=True)
    j = k - 2
    bad = out.clone()
    bad[0, j, 0, 5] += 1.0
    _, fr, dev = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], draft_out=bad,
                                             atol=1e-2, rtol=1e-2, causal=True)
    assert fr.cpu().tolist()[0] == j and fr.cpu().tolist()[1:] == [k] * (B - 1)
    with pytest.raises(lynx.LynxError):   # beyond the window cap
        lynx.workspace_bytes(c["geo"], B, 65) or lynx.make_workspace(c["geo"], B, 65, "cuda")


def test_wide_verify_single_token_returns_its_value_row(lynx):
    # the two weight terms on the tcgen05 path: one attended token gives its V row to FP32 rounding
    B, Hkv, G, k = 3, 1, 8, 8
    c = _case(lynx, 800, B, Hkv, G, k, (1,) * B, 16, True, "student_t4")
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    out, _, _ = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=False)
    lynx.check(c["ws"])
    from util import dequant
    va, vr, vm = c["vp"]
    got = out.cpu().numpy().astype(np.float64)
    for b in range(B):
        blk = int(c["table"][b, 0])
        row = dequant(va[blk, 0, 0], vr[blk, 0, 0], vm[blk, 0, 0], True)
        size = abs(float(vm[blk, 0, 0, 1])) + 255.0 * float(vm[blk, 0, 0, 0])
        assert np.max(np.abs(got[b] - row[None, None, :])) <= 4e-6 * size + 1e-30


@pytest.mark.parametrize("long_batches", [False, True])
def test_seeded_random_shapes_all_variants(lynx, long_batches):
    # a seeded sweep over shapes (KV heads, GQA group, positions, block size, ragged lengths) that
    # reaches every kernel variant: 1..64 columns, anchor and verify, causal or not; once with short
    # contexts and once with ragged batches of up to 47001 tokens (pieces of hundreds of units,
    # partial slots, empty and one-token sequences next to long ones)
    rng = np.random.default_rng(20250607 + int(long_batches))
    recipes = ["normal_outlier4x8", "lognormal_channels", "student_t4", "normal_outlier2pct_x10", "normal"]
    pool = [0, 1, 17, 300, 5000, 12345, 20000, 33333, 47001] if long_batches else \
        [0, 1, 5, 16, 63, 64, 65, 200, 777, 1500, 3100]
    done = 0
    exercised = 0
    while done < (8 if long_batches else 14):
        Hkv = int(rng.choice([1, 2, 3]))
        G = int(rng.choice([1, 2, 3, 4, 6, 8, 16]))
        k = int(rng.integers(1, 17))
        if k * G > 64:
            continue
        B = int(rng.integers(2, 6)) if long_batches else int(rng.integers(1, 4))
        bt = int(rng.choice([16, 32, 64]))
        lens = tuple(int(x) for x in rng.choice(pool, size=B))
        causal = bool(rng.integers(0, 2))
        c = _case(lynx, 900 + done, B, Hkv, G, k, lens, bt, True, recipes[done % len(recipes)])
        qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
        what = f"B={B} Hkv={Hkv} G={G} k={k} bt={bt} lens={lens} causal={causal}"
        ref_a = oracle.attention(False, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                                 c["lens"].numpy(), Hkv, bt, causal=causal)
        out_a = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=causal)
        lynx.check(c["ws"])
        _close(out_a.cpu().numpy().astype(np.float64), ref_a, "anchor " + what)
        ref_f = oracle.attention(True, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                                 c["lens"].numpy(), Hkv, bt, causal=causal)
        out_f, fr, dev = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"],
                                                     draft_out=out_a, atol=0.25, rtol=0.05, causal=causal)
        lynx.check(c["ws"])
        _close(out_f.cpu().numpy().astype(np.float64), ref_f, "verify " + what)
        want_fr, want_dev = oracle.verify_decision(ref_f, out_a.cpu().numpy(), 0.25, 0.05)
        if np.all(np.abs(want_dev - 1.0) > 0.05):
            assert np.array_equal(fr.cpu().numpy(), want_fr), what
            exercised += 1
        done += 1
    assert exercised >= done // 2, f"only {exercised} of {done} shapes had their indices compared"


@pytest.mark.parametrize("bt,G,k,lens", [(48, 4, 4, (1000, 5, 48, 49)), (112, 2, 16, (4000,)),
                                         (256, 4, 2, (513, 255))])
def test_block_sizes_that_are_no_power_of_two_or_large(lynx, bt, G, k, lens):
    # any multiple of 16 tokens per block is accepted: three 16-token sub-blocks per block, seven,
    # sixteen; sequences that end inside a block, in its first and in its last sub-block
    Hkv = 2
    c = _case(lynx, 7100 + bt, len(lens), Hkv, G, k, lens, bt, True, "student_t4")
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    for causal in (False, True):
        ref_a = oracle.attention(False, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                                 c["lens"].numpy(), Hkv, bt, causal=causal)
        out_a = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=causal)
        ref_f = oracle.attention(True, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                                 c["lens"].numpy(), Hkv, bt, causal=causal)
        out_f = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=causal)[0]
        lynx.check(c["ws"])
        _close(out_a.cpu().numpy().astype(np.float64), ref_a, f"anchor bt={bt} causal={causal}")
        _close(out_f.cpu().numpy().astype(np.float64), ref_f, f"verify bt={bt} causal={causal}")


@pytest.mark.parametrize("scale", [0.3, 0.02])
def test_custom_softmax_scale(lynx, scale):
    # softmax_scale other than 1/sqrt(128): sharper and flatter attention than the default, on the
    # mma.sync kernels (4 and 16 columns) and the tcgen05 kernel (32 columns)
    Hkv, G = 2, 4
    for k in (1, 4, 8):
        c = _case(lynx, 7300 + k, 2, Hkv, G, k, (700, 65), 16, True, "lognormal_channels")
        qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
        s32 = float(np.float32(scale))
        ref_a = oracle.attention(False, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                                 c["lens"].numpy(), Hkv, 16, causal=True, softmax_scale=s32)
        out_a = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=True,
                                      softmax_scale=s32)
        ref_f = oracle.attention(True, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(),
                                 c["lens"].numpy(), Hkv, 16, causal=True, softmax_scale=s32)
        out_f = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=True,
                                            softmax_scale=s32)[0]
        lynx.check(c["ws"])
        _close(out_a.cpu().numpy().astype(np.float64), ref_a, f"anchor scale={scale} k={k}")
        _close(out_f.cpu().numpy().astype(np.float64), ref_f, f"verify scale={scale} k={k}")


# ------------------------------------------------------------------ input ranges at the edges
@pytest.mark.parametrize("qscale", [8.0, 32.0, 128.0])
@pytest.mark.parametrize("recipe", ["student_t4", "normal"])
def test_scaled_queries(lynx, qscale, recipe):
    # queries far larger than the N(0,1) ones of the other tests (max |q| up to ~500): attention
    # becomes one-hot-like and any error in the logits shows.  The integer kernels carry the query
    # as 22-bit fixed point relative to its largest entry, the FP16 kernels as exact FP16 after a
    # power-of-two scale: 4, 16, 32 and 64 columns, anchor and merge-verify.
    Hkv = 2
    for G, k in ((4, 1), (4, 4), (4, 8), (8, 8)):
        c = _case(lynx, 8100 + k + G, 2, Hkv, G, k, (1500, 333), 16, True, recipe)
        q = (c["q"].float() * qscale).to(torch.bfloat16)
        qd, td, ld = q.cuda(), c["table"].cuda(), c["lens"].cuda()
        for full in (False, True):
            ref = oracle.attention(full, bf16_bits(q), c["kp"], c["vp"], c["table"].numpy(), c["lens"].numpy(),
                                   Hkv, 16, causal=True)
            if full:
                got = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=True)[0]
            else:
                got = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=True)
            lynx.check(c["ws"])
            _close(got.cpu().numpy().astype(np.float64), ref, f"qscale={qscale} {recipe} cols={k * G} full={full}")


def _scaled_value_case(lynx, seed, G, k, vscale):
    """A case whose V rows are scaled by `vscale` before quantisation (K unchanged)."""
    B, Hkv, bt, lens = 2, 2, 16, (700, 65)
    lens_t = torch.tensor(lens, dtype=torch.int32)
    table, nb = synth.block_table(lens_t, bt, True, "vr", seed)
    kx = synth.kv_block_values("normal", nb, Hkv, bt, "cpu", "vrK", seed)
    vx = (synth.kv_block_values("normal", nb, Hkv, bt, "cpu", "vrV", seed).float() * vscale).to(torch.bfloat16)
    q = synth.queries(B, k, Hkv * G, "cpu", "vrQ", seed)
    K, V = lynx.split_quantize(kx.cuda()), lynx.split_quantize(vx.cuda())
    kp, vp = oracle.split_quantize(bf16_bits(kx)), oracle.split_quantize(bf16_bits(vx))
    geo = lynx.Geometry(Hkv * G, Hkv, bt, nb, table.shape[1])
    return dict(geo=geo, ws=lynx.make_workspace(geo, B, k, "cuda"), q=q, K=K, V=V, kp=kp, vp=vp, table=table,
                lens=lens_t, Hkv=Hkv, bt=bt)


@pytest.mark.parametrize("vscale", [1.0e-3, 400.0, 1.0e30])
def test_value_rows_of_any_range_on_the_integer_kernels(lynx, vscale):
    # the integer kernels fold log2(scale_v) into the weights' exponent, so the magnitude of the V rows
    # (here ranges of ~1e-2, ~3000 and ~1e31) does not matter: relative accuracy as for ordinary rows
    for G, k, full in ((4, 1, False), (4, 4, False), (8, 8, False), (4, 2, True), (4, 4, True), (4, 8, True)):
        c = _scaled_value_case(lynx, 8300 + k, G, k, vscale)
        qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
        ref = oracle.attention(full, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(), c["lens"].numpy(),
                               c["Hkv"], 16, causal=True)
        if full:
            got = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=True)[0]
        else:
            got = lynx.anchor_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=True)
        lynx.check(c["ws"])
        got = got.cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got))
        err = np.abs(got - ref) / (ATOL * vscale + RTOL * np.abs(ref))     # the tolerance scaled with the rows
        assert float(err.max()) <= 1.0, (vscale, G, k, full, float(err.max()))


def test_value_range_limit_of_the_fp16_verify_kernels_is_reported(lynx):
    # merge-verify with 33..64 columns per launch carries the weights in FP16: value rows whose scale reaches
    # 16 (a range above 4080) would overflow them.  Just below the limit the result is within tolerance;
    # above it lynx_check reports LYNX_ERR_RANGE instead of a silent Inf / NaN.
    G, k = 8, 8
    c = _scaled_value_case(lynx, 8400, G, k, 400.0)      # ranges ~3000: scale_v ~ 12
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    assert float(c["vp"][2][..., 0].max()) < 16.0
    ref = oracle.attention(True, bf16_bits(c["q"]), c["kp"], c["vp"], c["table"].numpy(), c["lens"].numpy(),
                           c["Hkv"], 16, causal=True)
    got = lynx.merge_verify_attention(c["geo"], qd, c["K"], c["V"], td, ld, c["ws"], causal=True)[0]
    lynx.check(c["ws"])
    err = np.abs(got.cpu().numpy().astype(np.float64) - ref) / (ATOL * 400.0 + RTOL * np.abs(ref))
    assert float(err.max()) <= 1.0
    c = _scaled_value_case(lynx, 8401, G, k, 4000.0)     # ranges ~30000: scale_v ~ 120
    assert float(c["vp"][2][..., 0].max()) > 16.0
    lynx.merge_verify_attention(c["geo"], c["q"].cuda(), c["K"], c["V"], c["table"].cuda(), c["lens"].cuda(),
                                c["ws"], causal=True)
    with pytest.raises(lynx.LynxError, match="range"):
        lynx.check(c["ws"])
    lynx.check(c["ws"])                                   # the status word was cleared


def test_status_word_bits_map_to_their_statuses(lynx):
    # what a kernel records when a bounded wait runs out (or a block id / value range is bad) is one bit
    # of the workspace's status word; no wait is made to run out on the GPU here: the bits are written
    # from the host and lynx_check must report, in order of severity, and clear them
    c = _case(lynx, 8500, 1, 2, 4, 1, (100,), 16, True, "normal")
    word = c["ws"][:4].view(torch.int32)
    for bits, name in ((2, "status 8"), (1, "status 7"), (4, "status 9"), (7, "status 8"), (5, "status 7")):
        word.fill_(bits)
        with pytest.raises(lynx.LynxError, match=name):
            lynx.check(c["ws"])
        lynx.check(c["ws"])                                   # cleared by the report
    out = lynx.anchor_attention(c["geo"], c["q"].cuda(), c["K"], c["V"], c["table"].cuda(), c["lens"].cuda(), c["ws"])
    lynx.check(c["ws"])                                       # and the workspace is still usable
    assert bool(torch.isfinite(out).all())


# ------------------------------------------------- the paper's own flow: BF16 pages + attention on them
@pytest.mark.parametrize("G,n_q,lens,bt", [(4, 1, (4099, 37), 16), (8, 1, (2500, 0), 32), (4, 2, (777, 1), 16),
                                           (1, 1, (300, 5000), 16), (2, 1, (70,), 48)])
def test_bf16_pages_attention_matches_oracle(lynx, G, n_q, lens, bt):
    # lynx_recombine writes the dequantised BF16 pages (bit-exact against the oracle's), lynx_bf16_attention
    # attends on them: compared with the float64 oracle on the same pages
    Hkv = 2
    c = _case(lynx, 9000 + G + n_q, len(lens), Hkv, G, n_q, lens, bt, True, "lognormal_channels")
    _, k_pages = lynx.recombine(c["K"], want_codes=False, want_bf16=True)
    _, v_pages = lynx.recombine(c["V"], want_codes=False, want_bf16=True)
    ok_pages, ov_pages = oracle.recombine(*c["kp"])[1], oracle.recombine(*c["vp"])[1]
    assert np.array_equal(bf16_bits(k_pages), ok_pages) and np.array_equal(bf16_bits(v_pages), ov_pages)
    qd, td, ld = c["q"].cuda(), c["table"].cuda(), c["lens"].cuda()
    for causal in (False, True):
        got = lynx.bf16_attention(c["geo"], qd, k_pages, v_pages, td, ld, causal=causal)
        ref = oracle.attention_bf16_pages(bf16_bits(c["q"]), ok_pages, ov_pages, c["table"].numpy(),
                                          c["lens"].numpy(), causal=causal)
        _close(got.cpu().numpy().astype(np.float64), ref, f"bf16 pages G={G} n_q={n_q} causal={causal}")
    with pytest.raises(lynx.LynxError):        # more than 64 query positions
        lynx.bf16_attention(c["geo"], torch.zeros(len(lens), 65, Hkv * G, 128, dtype=torch.bfloat16, device="cuda"),
                            k_pages, v_pages, td, ld)


def test_bf16_pages_attention_windows_run_as_slices(lynx):
    # 5 positions x 4 heads per KV head = 20 columns: slices of 2, 2 and 1 positions; causal limits per position
    Hkv, G, n_q, lens, bt = 2, 4, 5, (700, 3, 0), 16
    c = _case(lynx, 9100, len(lens), Hkv, G, n_q, lens, bt, True, "student_t4")
    _, k_pages = lynx.recombine(c["K"], want_codes=False, want_bf16=True)
    _, v_pages = lynx.recombine(c["V"], want_codes=False, want_bf16=True)
    for causal in (False, True):
        got = lynx.bf16_attention(c["geo"], c["q"].cuda(), k_pages, v_pages, c["table"].cuda(), c["lens"].cuda(), causal=causal)
        ref = oracle.attention_bf16_pages(bf16_bits(c["q"]), oracle.recombine(*c["kp"])[1], oracle.recombine(*c["vp"])[1],
                                          c["table"].numpy(), c["lens"].numpy(), causal=causal)
        _close(got.cpu().numpy().astype(np.float64), ref, f"bf16 pages in slices, causal={causal}")


# ------------------------------------------------------------------------ degenerate key / value rows
@pytest.mark.parametrize("G,n_q", [(4, 1), (4, 2), (4, 4), (8, 8), (2, 1)])
def test_degenerate_key_and_value_rows(lynx, G, n_q):
    """Rows the quantiser and the kernels treat specially, mixed into ordinary ones: constant rows (scale 0: the
    row is its zero point), rows of zeros and of -0, rows 10^-4 times and 50 times the ordinary size (the large
    keys take nearly all the softmax mass), large value rows, a run of identical keys (uniform weights among
    them), and a sequence whose queries are zero (uniform weights over everything).  Anchor and full state at
    4 / 8 / 16 / 64 columns, the BF16-page kernel on the dequantised pages where it takes the shape."""
    Hkv, bt, lens = 2, 16, (300, 45)
    B = len(lens)
    lens_t = torch.tensor(lens, dtype=torch.int32)
    table, nb = synth.block_table(lens_t, bt, True, "dg", G * n_q)
    g = torch.Generator().manual_seed(77 + G * n_q)
    k = torch.randn(nb, Hkv, bt, 128, generator=g)
    v = torch.randn(nb, Hkv, bt, 128, generator=g)

    def rows(x, b, t0, t1):          # view of tokens [t0, t1) of sequence b: list of (block, row) slices
        return [(int(table[b, t // bt]), t % bt) for t in range(t0, min(t1, lens[b]))]
    for b in range(B):
        for blk, r in rows(k, b, 0, 10):
            k[blk, :, r] = 2.5
            v[blk, :, r] = -1.25
        for blk, r in rows(k, b, 10, 20):
            k[blk, :, r] = 0.0
            v[blk, :, r] = 0.0
        for blk, r in rows(k, b, 20, 25):
            k[blk, :, r] = -0.0
            v[blk, :, r] = -0.0
        for blk, r in rows(k, b, 30, 40):
            k[blk, :, r] *= 1.0e-4
            v[blk, :, r] *= 1.0e-4
        for blk, r in rows(k, b, 40, 44):
            k[blk, :, r] *= 50.0
        for blk, r in rows(k, b, 50, 60):
            v[blk, :, r] *= 100.0
        same = torch.randn(Hkv, 128, generator=g)
        for blk, r in rows(k, b, 100, 200):
            k[blk, :, r] = same
    k, v = k.to(torch.bfloat16), v.to(torch.bfloat16)
    q = synth.queries(B, n_q, Hkv * G, "cpu", "dgQ", G)
    q[1] = 0.0
    K, V = lynx.split_quantize(k.cuda()), lynx.split_quantize(v.cuda())
    kp, vp = oracle.split_quantize(bf16_bits(k)), oracle.split_quantize(bf16_bits(v))
    _assert_planes_equal(_planes_np(K), kp)
    _assert_planes_equal(_planes_np(V), vp)
    geo = lynx.Geometry(Hkv * G, Hkv, bt, nb, table.shape[1])
    ws = lynx.make_workspace(geo, B, n_q, "cuda")
    qd, td, ld = q.cuda(), table.cuda(), lens_t.cuda()
    for causal in (False, True):
        out = lynx.anchor_attention(geo, qd, K, V, td, ld, ws, causal=causal)
        lynx.check(ws)
        ref = oracle.attention(False, bf16_bits(q), kp, vp, table.numpy(), lens_t.numpy(), Hkv, bt, causal=causal)
        _close(out.cpu().numpy().astype(np.float64), ref, f"anchor, degenerate rows, causal={causal}")
        full, _, _ = lynx.merge_verify_attention(geo, qd, K, V, td, ld, ws, causal=causal)
        lynx.check(ws)
        ref = oracle.attention(True, bf16_bits(q), kp, vp, table.numpy(), lens_t.numpy(), Hkv, bt, causal=causal)
        _close(full.cpu().numpy().astype(np.float64), ref, f"full state, degenerate rows, causal={causal}")
        if n_q * G <= 8:
            _, k_pages = lynx.recombine(K, want_codes=False, want_bf16=True)
            _, v_pages = lynx.recombine(V, want_codes=False, want_bf16=True)
            got = lynx.bf16_attention(geo, qd, k_pages, v_pages, td, ld, causal=causal)
            ref = oracle.attention_bf16_pages(bf16_bits(q), oracle.recombine(*kp)[1], oracle.recombine(*vp)[1],
                                              table.numpy(), lens_t.numpy(), causal=causal)
            _close(got.cpu().numpy().astype(np.float64), ref, f"BF16 pages, degenerate rows, causal={causal}")
