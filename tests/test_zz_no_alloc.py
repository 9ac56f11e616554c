"""The workspace-free anchor attention entry point (collected last on purpose).

Some callers of this library cannot allocate device memory at call time (code running inside
another framework's fixed memory plan, or a serving loop that has frozen its allocations), so
`lynx_anchor_attention_static` keeps its scratch in a fixed array inside the library.  This test
calls it through the C ABI twice in a row on the same inputs and checks both results against the
ordinary entry point, which gets a caller-allocated workspace, and against the CPU oracle.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from util import bf16_bits

pytestmark = pytest.mark.gpu

ATOL, RTOL = 2e-3, 1e-2


@pytest.mark.parametrize("G,n_q,lens", [(4, 2, (3001, 517)), (8, 2, (0, 1300)), (4, 1, (129, 0))])
def test_static_scratch_entry_matches_workspace_entry_twice(G, n_q, lens):
    import paper_2607_01831_b200 as lynx
    lynx.load()
    B, Hkv, bt = 2, 2, 16
    lens = torch.tensor(lens, dtype=torch.int32)
    table, nb = synth.block_table(torch.clamp(lens, min=1), bt, True, "zz", 1)
    kx = synth.kv_block_values("lognormal_channels", nb, Hkv, bt, "cpu", "zzK")
    vx = synth.kv_block_values("lognormal_channels", nb, Hkv, bt, "cpu", "zzV")
    K, V = lynx.split_quantize(kx.cuda()), lynx.split_quantize(vx.cuda())
    q_cpu = synth.queries(B, n_q, Hkv * G, "cpu", "zzQ")
    q = q_cpu.cuda()
    geo = lynx.Geometry(Hkv * G, Hkv, bt, nb, table.shape[1])
    td, ld = table.cuda(), lens.cuda()
    ws = lynx.make_workspace(geo, B, n_q, "cuda")
    want = lynx.anchor_attention(geo, q, K, V, td, ld, ws, causal=True)
    lynx.check(ws)
    want_np = want.cpu().numpy().astype(np.float64)
    ref = oracle.attention(False, bf16_bits(q_cpu), oracle.split_quantize(bf16_bits(kx)),
                           oracle.split_quantize(bf16_bits(vx)), table.numpy(), lens.numpy(), Hkv, bt, causal=True)
    for _ in range(2):                                   # two calls in a row share the array
        got = lynx.anchor_attention_static(geo, q, K, V, td, ld, causal=True)
        torch.cuda.synchronize()
        got_np = got.cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got_np))
        assert np.all(np.abs(got_np - want_np) <= ATOL + RTOL * np.abs(want_np))
        assert np.all(np.abs(got_np - ref) <= ATOL + RTOL * np.abs(ref))       # and the CPU oracle
    # different inputs right after: the array's old contents must not leak into the result
    lens2 = torch.tensor([64, min(2999, int(table.shape[1]) * bt)], dtype=torch.int32).cuda()
    want2 = lynx.anchor_attention(geo, q, K, V, td, lens2, ws)
    got2 = lynx.anchor_attention_static(geo, q, K, V, td, lens2)
    torch.cuda.synchronize()
    a, b = got2.cpu().numpy().astype(np.float64), want2.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(a - b) <= ATOL + RTOL * np.abs(b))


def test_static_scratch_entry_rejects_oversized_problems():
    import paper_2607_01831_b200 as lynx
    L = lynx.load()
    # 4096 sequences x 8 KV heads x 8 padded columns of partial slots need far more than 8 MiB
    geo = lynx.Geometry(32, 8, 16, 1 << 16, 16)
    assert lynx.workspace_bytes(geo, 4096, 1) > (8 << 20)
    q = torch.zeros(4096, 1, 32, 128, dtype=torch.bfloat16, device="cuda")
    planes = lynx.alloc_planes((16, 8, 16), "cuda")
    table = torch.zeros(4096, 16, dtype=torch.int32, device="cuda")
    lens = torch.zeros(4096, dtype=torch.int32, device="cuda")
    with pytest.raises(lynx.LynxError, match="workspace"):
        lynx.anchor_attention_static(geo, q, planes, planes, table, lens)
    assert L.lynx_status_string(5) == b"workspace too small"
