"""Pins for oracle/tail.py (attention over a quantised prefix followed by a BF16 tail; the log-sum-exp
join of two partial attentions) against things other than itself; no GPU needed.

* an empty tail reduces it to the C oracle's attention over the planes (itself pinned by brute force),
  an empty prefix to the BF16-pages attention;
* torch's float64 scaled_dot_product_attention over the explicit concatenation of the dequantised prefix
  (tests/util.dequant) and the tail rows, causal mask included;
* closed forms of the log-sum-exp: n equal scores give s + log n; a single key gives its score;
* the join rule: joining the two parts' own attentions by their log-sum-exps gives the attention over
  the union, and the joined log-sum-exp is that of all scores; an empty part changes nothing.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import tail
from util import bf16_bits, bits_to_f64, dequant

SM_SCALE = float(np.float32(1.0 / math.sqrt(128.0)))   # the boundary takes the scale as a float


def _case(seed, B=2, Hkv=2, G=2, n_q=1, lens=(37, 20), tail_lens=(9, 17), bt=16, bt_t=16):
    lens_t = torch.tensor(lens, dtype=torch.int32)
    table, nb = synth.block_table(lens_t, bt, True, "tailpin", seed)
    k = synth.kv_block_values("normal_outlier4x8", nb, Hkv, bt, "cpu", "tailK", seed)
    v = synth.kv_block_values("normal_outlier4x8", nb, Hkv, bt, "cpu", "tailV", seed)
    tl = torch.tensor(tail_lens, dtype=torch.int32)
    ttable, nbt = synth.block_table(tl, bt_t, True, "tailpin2", seed)
    kt = synth.kv_block_values("normal_outlier4x8", max(nbt, 1), Hkv, bt_t, "cpu", "tailKt", seed)
    vt = synth.kv_block_values("normal_outlier4x8", max(nbt, 1), Hkv, bt_t, "cpu", "tailVt", seed)
    q = synth.queries(B, n_q, Hkv * G, "cpu", "tailQ", seed)
    return dict(q=bf16_bits(q), kp=oracle.split_quantize(bf16_bits(k)), vp=oracle.split_quantize(bf16_bits(v)),
                table=table.numpy(), lens=lens_t.numpy(), kt=bf16_bits(kt), vt=bf16_bits(vt),
                ttable=ttable.numpy(), tlens=tl.numpy(), B=B, Hkv=Hkv, G=G, n_q=n_q, bt=bt, bt_t=bt_t)


def _run(c, full, causal_tail=False, lens=None, tlens=None):
    return tail.prefix_tail_attention(full, c["q"], c["kp"], c["vp"], c["table"], c["lens"] if lens is None else lens,
                                      c["kt"], c["vt"], c["ttable"], c["tlens"] if tlens is None else tlens,
                                      causal_tail=causal_tail)


@pytest.mark.parametrize("full", [False, True])
def test_empty_tail_is_the_plane_attention(full):
    c = _case(1, n_q=2)
    got = _run(c, full, tlens=np.zeros(c["B"], np.int32))
    want = oracle.attention(full, c["q"], c["kp"], c["vp"], c["table"], c["lens"], c["Hkv"], c["bt"])
    assert np.allclose(got["out"], want, rtol=1e-12, atol=1e-13)
    assert np.all(np.isneginf(got["lse_tail"])) and np.array_equal(got["lse"], got["lse_prefix"])


@pytest.mark.parametrize("causal", [False, True])
def test_empty_prefix_is_the_bf16_page_attention(causal):
    c = _case(2, n_q=3)
    got = _run(c, True, causal_tail=causal, lens=np.zeros(c["B"], np.int32))
    want = oracle.attention_bf16_pages(c["q"], c["kt"], c["vt"], c["ttable"], c["tlens"], causal=causal)
    assert np.allclose(got["out"], want, rtol=1e-12, atol=1e-13)
    assert np.all(np.isneginf(got["lse_prefix"]))


@pytest.mark.parametrize("full", [False, True])
@pytest.mark.parametrize("causal,n_q", [(False, 1), (True, 4)])
def test_matches_torch_sdpa_on_the_concatenation(full, causal, n_q):
    c = _case(3, n_q=n_q, lens=(45, 16), tail_lens=(21, 6))
    got = _run(c, full, causal_tail=causal)
    qf = torch.from_numpy(bits_to_f64(c["q"]))
    ktf, vtf = bits_to_f64(c["kt"]), bits_to_f64(c["vt"])
    for b in range(c["B"]):
        n_pre, n_tail = int(c["lens"][b]), int(c["tlens"][b])
        K, V = [], []
        for h in range(c["Hkv"]):
            rows_k, rows_v = [], []
            for t in range(n_pre):
                blk = c["table"][b, t // c["bt"]]
                rows_k.append(dequant(c["kp"][0][blk, h, t % c["bt"]], c["kp"][1][blk, h, t % c["bt"]],
                                      c["kp"][2][blk, h, t % c["bt"]], full))
                rows_v.append(dequant(c["vp"][0][blk, h, t % c["bt"]], c["vp"][1][blk, h, t % c["bt"]],
                                      c["vp"][2][blk, h, t % c["bt"]], full))
            for t in range(n_tail):
                blk = c["ttable"][b, t // c["bt_t"]]
                rows_k.append(ktf[blk, h, t % c["bt_t"]])
                rows_v.append(vtf[blk, h, t % c["bt_t"]])
            K.append(np.stack(rows_k))
            V.append(np.stack(rows_v))
        K, V = torch.from_numpy(np.stack(K)), torch.from_numpy(np.stack(V))
        Q = qf[b].permute(1, 0, 2).unsqueeze(0)
        mask = None
        if causal:
            j = torch.arange(n_q).view(n_q, 1)
            t = torch.arange(n_pre + n_tail).view(1, -1)
            mask = t < (n_pre + n_tail - n_q + j + 1)
        ref = torch.nn.functional.scaled_dot_product_attention(Q, K.unsqueeze(0), V.unsqueeze(0), attn_mask=mask,
                                                               enable_gqa=True, scale=SM_SCALE)
        assert np.allclose(got["out"][b], ref[0].permute(1, 0, 2).numpy(), rtol=1e-11, atol=1e-12)
        # the log-sum-exp of all scores, against torch.logsumexp on the same masked score matrix
        Kg = K.repeat_interleave(c["G"], dim=0)
        s = torch.einsum("hjd,htd->hjt", Q[0], Kg) * SM_SCALE
        if mask is not None:
            s = s.masked_fill(~mask.unsqueeze(0), -math.inf)
        assert np.allclose(got["lse"][b], torch.logsumexp(s, dim=-1).permute(1, 0).numpy(), rtol=1e-12, atol=1e-12)


def test_log_sum_exp_closed_forms():
    # zero queries: every score is 0, so lse = log(number of keys seen), and the output is the mean of V
    c = _case(4, n_q=2, lens=(33, 7), tail_lens=(5, 12))
    c["q"] = np.zeros_like(c["q"])
    got = _run(c, True, causal_tail=True)
    for b in range(c["B"]):
        for j in range(2):
            seen_tail = int(c["tlens"][b]) - 2 + j + 1
            assert np.allclose(got["lse_prefix"][b, j], math.log(int(c["lens"][b])), rtol=0, atol=1e-13)
            assert np.allclose(got["lse_tail"][b, j], math.log(seen_tail), rtol=0, atol=1e-13)
            assert np.allclose(got["lse"][b, j], math.log(int(c["lens"][b]) + seen_tail), rtol=0, atol=1e-13)
    # a single key: lse is its score, the output its value row
    one = _run(c | {"q": _case(4)["q"][:, :1]}, True, lens=np.zeros(2, np.int32), tlens=np.ones(2, np.int32))
    qf, ktf, vtf = bits_to_f64(_case(4)["q"]), bits_to_f64(c["kt"]), bits_to_f64(c["vt"])
    for b in range(2):
        blk = c["ttable"][b, 0]
        for h in range(c["Hkv"] * c["G"]):
            s = float(ktf[blk, h // c["G"], 0] @ qf[b, 0, h]) * SM_SCALE
            assert abs(one["lse"][b, 0, h] - s) <= 1e-12 * (1 + abs(s))
            assert np.allclose(one["out"][b, 0, h], vtf[blk, h // c["G"], 0], rtol=1e-13, atol=0)


@pytest.mark.parametrize("full", [False, True])
def test_join_of_the_parts_is_the_attention_over_the_union(full):
    c = _case(5, n_q=3, lens=(50, 0), tail_lens=(8, 11))
    both = _run(c, full, causal_tail=True)
    pre = oracle.attention(full, c["q"], c["kp"], c["vp"], c["table"], c["lens"], c["Hkv"], c["bt"])
    tl = oracle.attention_bf16_pages(c["q"], c["kt"], c["vt"], c["ttable"], c["tlens"], causal=True)
    out, lse = tail.lse_merge(pre, both["lse_prefix"], tl, both["lse_tail"])
    assert np.allclose(out, both["out"], rtol=1e-11, atol=1e-12)
    assert np.allclose(lse, both["lse"], rtol=1e-12, atol=1e-12)
    # an empty part changes nothing, two empty parts give zero
    ninf = np.full(lse.shape, -np.inf)
    o2, l2 = tail.lse_merge(pre, both["lse_prefix"], np.full_like(pre, 123.0), ninf)
    seen = np.isfinite(both["lse_prefix"])
    assert np.array_equal(o2[seen], pre[seen]) and np.array_equal(l2, both["lse_prefix"])
    o3, l3 = tail.lse_merge(pre, ninf, tl, ninf)
    assert not o3.any() and np.all(np.isneginf(l3))
    # symmetric in its two parts
    o4, l4 = tail.lse_merge(tl, both["lse_tail"], pre, both["lse_prefix"])
    assert np.allclose(o4, out, rtol=1e-13, atol=1e-14) and np.allclose(l4, lse, rtol=1e-14, atol=0)
