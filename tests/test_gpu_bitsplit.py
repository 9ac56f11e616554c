"""GPU parity of lynx_split_quantize_bits / lynx_recombine_bits (Anchor / Residual splits 2 + 6, 4 + 4, 6 + 2)
against the CPU oracle (oracle/bitsplit.py): planes, metadata bits, codes and BF16 pages bit for bit; A = 4
against lynx_split_quantize's own planes; the pages through lynx_bf16_attention against the oracle's attention
on the oracle's pages."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import bitsplit
from util import bf16_bits, f32_to_bf16_tensor

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lynx():
    import paper_2607_01831_b200 as m
    m.load()
    return m


@pytest.mark.parametrize("A", [2, 4, 6])
@pytest.mark.parametrize("recipe,n_blocks", [("normal_outlier4x8", 1), ("student_t4", 37), ("lognormal_channels", 700)])
def test_planes_codes_and_pages_bit_exact(lynx, A, recipe, n_blocks):
    x = synth.kv_block_values(recipe, n_blocks, 8, 16, "cpu", "bs", n_blocks)
    x = x.reshape(-1, 128)[: x.numel() // 128 - 3]          # ragged tail: not a multiple of the rows per CTA trip
    a, r, m = lynx.split_quantize_bits(x.cuda(), A)
    wa, wr, wm, wcodes = bitsplit.split_quantize_bits(bf16_bits(x), A)
    assert np.array_equal(a.cpu().numpy(), wa), "anchor plane differs"
    assert np.array_equal(r.cpu().numpy(), wr), "residual plane differs"
    assert np.array_equal(m.cpu().numpy().view(np.uint32), wm.view(np.uint32)), "meta bits differ"
    for res, wres in ((r, wr), (None, None)):               # both streams, and the Anchor alone
        want_lv, want_deq = bitsplit.recombine_bits(wa, wres, wm, A)
        codes, deq = lynx.recombine_bits(a, res, m, A)
        assert np.array_equal(codes.cpu().numpy(), want_lv) and np.array_equal(bf16_bits(deq), want_deq)
        codes_only, none = lynx.recombine_bits(a, res, m, A, want_bf16=False)
        none2, deq_only = lynx.recombine_bits(a, res, m, A, want_codes=False)
        assert none is None and none2 is None
        assert torch.equal(codes_only, codes) and torch.equal(deq_only, deq)
    assert np.array_equal(lynx.recombine_bits(a, r, m, A)[0].cpu().numpy(), wcodes)


def test_four_plus_four_writes_the_main_planes(lynx):
    x = synth.kv_block_values("normal_outlier2pct_x10", 50, 4, 16, "cpu", "bs4", 1).reshape(-1, 128).cuda()
    a, r, m = lynx.split_quantize_bits(x, 4)
    p = lynx.split_quantize(x)
    assert torch.equal(a, p.anchor) and torch.equal(r, p.residual) and torch.equal(m.view(torch.int32), p.meta.view(torch.int32))
    _, deq = lynx.recombine_bits(a, r, m, 4, want_codes=False)
    _, deq_main = lynx.recombine(p, want_codes=False, want_bf16=True)
    assert torch.equal(deq.view(torch.int16), deq_main.view(torch.int16))


@pytest.mark.parametrize("A", [2, 6])
def test_special_rows(lynx, A):
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
    a, r, m = lynx.split_quantize_bits(x.cuda(), A)
    wa, wr, wm, _ = bitsplit.split_quantize_bits(bf16_bits(x), A)
    assert np.array_equal(a.cpu().numpy(), wa) and np.array_equal(r.cpu().numpy(), wr)
    assert np.array_equal(m.cpu().numpy().view(np.uint32), wm.view(np.uint32))
    for res, wres in ((r, wr), (None, None)):
        want_lv, want_deq = bitsplit.recombine_bits(wa, wres, wm, A)
        codes, deq = lynx.recombine_bits(a, res, m, A)
        assert np.array_equal(codes.cpu().numpy(), want_lv) and np.array_equal(bf16_bits(deq), want_deq)


@pytest.mark.parametrize("A", [2, 6])
def test_pages_of_a_split_feed_the_bf16_attention(lynx, A):
    # Anchor-only pages (what a decode node holds before the Residual lands) and full pages, attended by
    # lynx_bf16_attention; the oracle attends on its own pages
    Hkv, G, bt, lens = 2, 4, 16, (900, 45)
    lens_t = torch.tensor(lens, dtype=torch.int32)
    table, nb = synth.block_table(lens_t, bt, True, "bsatt", A)
    k = synth.kv_block_values("normal_outlier4x8", nb, Hkv, bt, "cpu", "bsK", A)
    v = synth.kv_block_values("normal_outlier4x8", nb, Hkv, bt, "cpu", "bsV", A)
    q = synth.queries(len(lens), 1, Hkv * G, "cpu", "bsQ", A)
    geo = lynx.Geometry(Hkv * G, Hkv, bt, nb, table.shape[1])
    ka, kr, km = lynx.split_quantize_bits(k.cuda(), A)
    va, vr, vm = lynx.split_quantize_bits(v.cuda(), A)
    oka, okr, okm, _ = bitsplit.split_quantize_bits(bf16_bits(k), A)
    ova, ovr, ovm, _ = bitsplit.split_quantize_bits(bf16_bits(v), A)
    for full in (False, True):
        _, kp = lynx.recombine_bits(ka, kr if full else None, km, A, want_codes=False)
        _, vp = lynx.recombine_bits(va, vr if full else None, vm, A, want_codes=False)
        okp = bitsplit.recombine_bits(oka, okr if full else None, okm, A)[1]
        ovp = bitsplit.recombine_bits(ova, ovr if full else None, ovm, A)[1]
        assert np.array_equal(bf16_bits(kp), okp) and np.array_equal(bf16_bits(vp), ovp)
        got = lynx.bf16_attention(geo, q.cuda(), kp, vp, table.cuda(), lens_t.cuda())
        ref = oracle.attention_bf16_pages(bf16_bits(q), okp, ovp, table.numpy(), lens_t.numpy())
        err = np.abs(got.cpu().numpy().astype(np.float64) - ref)
        assert np.all(err <= 2e-3 + 1e-2 * np.abs(ref)), float(np.max(err / (2e-3 + 1e-2 * np.abs(ref))))


def test_argument_errors(lynx):
    L = lynx.load()
    x = torch.zeros(4, 128, dtype=torch.bfloat16, device="cuda")
    a = torch.zeros(4, 96, dtype=torch.uint8, device="cuda")
    r = torch.zeros(4, 96, dtype=torch.uint8, device="cuda")
    m = torch.zeros(4, 2, device="cuda")
    assert L.lynx_split_quantize_bits(x.data_ptr(), 4, 3, a.data_ptr(), r.data_ptr(), m.data_ptr(), None) == 4    # unsupported split
    assert L.lynx_split_quantize_bits(x.data_ptr(), 4, 6, None, r.data_ptr(), m.data_ptr(), None) == 1            # NULL
    assert L.lynx_split_quantize_bits(x.data_ptr() + 2, 3, 6, a.data_ptr(), r.data_ptr(), m.data_ptr(), None) == 3  # alignment
    assert L.lynx_split_quantize_bits(x.data_ptr(), -1, 6, a.data_ptr(), r.data_ptr(), m.data_ptr(), None) == 2    # shape
    assert L.lynx_split_quantize_bits(None, 0, 6, None, None, None, None) == 0                                      # empty
    assert L.lynx_recombine_bits(a.data_ptr(), r.data_ptr(), m.data_ptr(), 4, 6, None, None, None) == 1             # no output
    assert L.lynx_recombine_bits(a.data_ptr(), r.data_ptr(), None, 4, 6, None, x.data_ptr(), None) == 1             # BF16 without meta
    assert L.lynx_recombine_bits(a.data_ptr(), r.data_ptr(), m.data_ptr(), 4, 5, None, x.data_ptr(), None) == 4
