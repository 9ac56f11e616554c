"""Host-side logic of bench.py: reporting helpers, and the max-over-ranks reduction on two gloo
ranks (the multi-GPU path shards independent problems; its only cross-rank step is timing)."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
import synth  # noqa: E402


def test_kernel_table_and_job_value():
    times = {"anchor_attention": [1.0, 3.0], "merge_verify_attention[k=4]": [4.0],
             "merge_verify_attention[k=8]": [8.0]}
    lb = {"anchor_attention": 72e6, "merge_verify_attention": 136e6, "split_quantize": 392e6}
    tab = bench.kernel_table(times, lb, steps=1, ms_per_step=16.0, peak=6547.2)
    assert tab["anchor_attention"]["avg_ms"] == 2.0 and tab["anchor_attention"]["min_ms"] == 1.0
    assert tab["anchor_attention"]["GBps"] == pytest.approx(72e6 / 2e-3 / 1e9)
    assert tab["merge_verify_attention[k=8]"]["GBps"] == pytest.approx(136e6 / 8e-3 / 1e9)
    assert tab["anchor_attention"]["frac_of_measured"] == pytest.approx(36.0 / 6547.2)
    assert sum(v["share_of_step"] for v in tab.values()) == pytest.approx(1.0)
    assert bench.base_kind("merge_verify_attention[k=4]") == "merge_verify_attention"
    assert bench.job_value(10 ** 9, 1.0, 1) == pytest.approx(1000.0)
    assert bench.job_value(10 ** 9, 1.0, 8) == pytest.approx(8000.0)      # weak scaling: N x per-GPU
    assert set(bench.TRAFFIC_RATIO) == set(bench.BYTES_PER_ROW)


def test_workload_table_matches_the_stated_configs():
    w = synth.WORKLOADS
    assert (w[3].layers, w[3].context, w[3].num_kv_heads, w[3].num_q_heads, w[3].k_list) == (32, 131072, 8, 32, (2, 4, 8))
    assert (w[5].layers, w[5].batch, w[5].num_q_heads, w[5].k_list) == (80, 2, 64, (8,))
    assert w[4].ragged and w[4].shuffled_blocks and w[4].batch == 16 and w[4].min_context == 8192
    lens = synth.seq_lens(16, 8192, 65536, "c4_serving_mix", 0)
    assert lens.min() >= 8192 and lens.max() <= 65536 and len(set(lens.tolist())) > 8
    table, nb = synth.block_table(lens, 16, True, "c4_serving_mix", 0)
    used = torch.cat([table[b, :(int(lens[b]) + 15) // 16] for b in range(16)])
    assert used.numel() == nb and torch.unique(used).numel() == nb           # a permutation of the pool


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                     # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, dist, torch.device("cpu"))
    q.put((rank, ms, bench.job_value(10 ** 9, ms, world)))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [15.0, 15.0]       # both ranks report the slowest time
    assert got[0][2] == pytest.approx(2 * 1e9 / 15e-3 / 1e9)
