"""Parity at a full-size workload, in the launch configuration bench.py times: config 3
(32 layers x 8 KV heads x 131072 tokens, layers flattened into the batch), checked on sampled
layers the oracle can compute one by one: planes bit-exact, drafts and verified outputs within
tolerance, accept/reject indices identical when outside the guard band."""
import os
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

pytestmark = pytest.mark.gpu
ATOL, RTOL = 2e-3, 1e-2


def _bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def test_config3_full_size_sampled_layers():
    import bench
    import oracle
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * 2 ** 30:
        pytest.skip("needs ~30 GB of device memory")
    wlk = bench.Workload(3, torch.device("cuda", 0))
    wl = wlk.wl
    wlk.step()
    torch.cuda.synchronize()
    for w in wlk.windows:
        wlk.lynx.check(w["ws"])
    nbl, Hkv, bt = wlk.nb_layer, wl.num_kv_heads, wl.block_tokens
    table = torch.arange(nbl, dtype=torch.int32).view(1, nbl).numpy()
    lens = np.array([wl.context], np.int32)
    win = wlk.windows[0]                       # k = 2
    k = win["k"]
    for layer in (0, wl.layers - 1):
        sl = slice(layer * nbl, (layer + 1) * nbl)
        planes = {}
        for which in "KV":
            want = oracle.split_quantize(_bits(wlk.src[which][sl]))
            got = wlk.planes[which]
            assert np.array_equal(got.anchor[sl].cpu().numpy(), want[0])
            assert np.array_equal(got.residual[sl].cpu().numpy(), want[1])
            assert np.array_equal(got.meta[sl].cpu().numpy().view(np.uint32), want[2].view(np.uint32))
            planes[which] = want
        q = _bits(win["q"][layer:layer + 1])
        ref_a = oracle.attention(False, q, planes["K"], planes["V"], table, lens, Hkv, bt, causal=True)
        ref_f = oracle.attention(True, q, planes["K"], planes["V"], table, lens, Hkv, bt, causal=True)
        draft = win["draft"][layer:layer + 1].cpu().numpy()
        full = win["out_full"][layer:layer + 1].cpu().numpy()
        for got, ref in ((draft, ref_a), (full, ref_f)):
            g = got.astype(np.float64)
            assert np.all(np.abs(g - ref) <= ATOL + RTOL * np.abs(ref)), float(np.abs(g - ref).max())
        want_fr, want_dev = oracle.verify_decision(ref_f, draft, 0.5, 0.1)
        if np.all(np.abs(want_dev - 1.0) > 0.05):
            assert int(win["first_reject"][layer]) == int(want_fr[0])
        assert np.allclose(win["dev"][layer].cpu().numpy(), want_dev[0], rtol=0.05, atol=1e-3)
