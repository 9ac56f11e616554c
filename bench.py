#!/usr/bin/env python
"""Benchmark of the Lynx hot path on B200: split-quantise, anchor decode attention, merge-verify.

One "step" is one pass of the whole hot path over one synthetic batch of the chosen workload:
split-quantise the whole BF16 KV cache (K and V, all layers), then for every speculation depth
k of the workload: k anchor decode steps on the Anchor planes (growing context) followed by
one merge-verify pass over the k drafted positions with its accept/reject index.

Prints ONE JSON line (the fields are described in the repository's design notes).  `--impl reference` times the CPU
oracle on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import synth  # noqa: E402

METRIC = "split-quant & anchor/verify decode-attn HBM GB/s (% of B200 peak); tokens/s"
BYTES_PER_ROW = {"split_quantize": 392, "anchor_attention": 72, "merge_verify_attention": 136}
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------- workload set-up
class Workload:
    """All device state of one configuration, layers flattened into the batch dimension."""

    def __init__(self, cfg_id: int, device, rank: int = 0, layers: int = 0):
        import dataclasses

        import paper_2607_01831_b200 as lynx
        self.lynx = lynx
        wl = synth.WORKLOADS[cfg_id]
        if layers:   # a reduced copy of the workload (profiling captures), never the bench default
            wl = dataclasses.replace(wl, layers=layers, name=f"{wl.name}[layers={layers}]")
        self.wl, self.cfg_id, self.device = wl, cfg_id, device
        bt, Hkv = wl.block_tokens, wl.num_kv_heads
        if wl.ragged:
            lens = synth.seq_lens(wl.batch, wl.min_context, wl.context, wl.name, rank)
        else:
            lens = torch.full((wl.batch,), wl.context, dtype=torch.int32)
        table, nb_layer = synth.block_table(lens, bt, wl.shuffled_blocks, wl.name, rank)
        self.lens_cpu, self.nb_layer = lens, nb_layer
        L = wl.layers
        self.B = L * wl.batch
        offs = (torch.arange(L, dtype=torch.int32) * nb_layer).view(L, 1, 1)
        self.table = (table.unsqueeze(0) + offs).reshape(self.B, -1).contiguous().to(device)
        self.lens_flat_cpu = lens.repeat(L)
        self.geo = lynx.Geometry(wl.num_q_heads, Hkv, bt, L * nb_layer, table.shape[1])
        # BF16 source cache, generated per layer into one flat allocation per tensor
        self.src = {}
        for which in "KV":
            buf = torch.empty(L * nb_layer, Hkv, bt, 128, dtype=torch.bfloat16, device=device)
            for l in range(L):
                synth.kv_block_values(wl.recipe, nb_layer, Hkv, bt, device, wl.name, which, l, rank,
                                      out=buf[l * nb_layer:(l + 1) * nb_layer])
            self.src[which] = buf
        self.planes = {w: lynx.alloc_planes((L * nb_layer, Hkv, bt), device) for w in "KV"}
        self.block_ids = None
        if wl.shuffled_blocks:   # newly arrived blocks, in arrival (table) order, every layer
            ids = [table[b, :(int(lens[b]) + bt - 1) // bt] for b in range(wl.batch)]
            ids = torch.cat(ids).to(torch.int32)
            self.block_ids = (ids.unsqueeze(0) + offs.view(L, 1)).reshape(-1).contiguous().to(device)
        # windows: (k, [lens tensor per draft step], q [B][k][Hq][128], draft, ws)
        reps = max(1, wl.anchor_steps // max(wl.k_list)) if wl.anchor_steps else 1
        self.windows = []
        for k in wl.k_list:
            q = synth.queries(self.B, k, wl.num_q_heads, device, wl.name, "q", k, rank)
            step_lens = [(self.lens_flat_cpu - k + j + 1).clamp(min=0).to(torch.int32).to(device)
                         for j in range(k)]
            qs = [q[:, j:j + 1].contiguous() for j in range(k)]
            self.windows.append(dict(
                k=k, q=q, qs=qs, step_lens=step_lens, reps=reps,
                step_out=[torch.empty(self.B, 1, wl.num_q_heads, 128, dtype=torch.float32, device=device)
                          for _ in range(k)],
                draft=torch.empty(self.B, k, wl.num_q_heads, 128, dtype=torch.float32, device=device),
                out_full=torch.empty(self.B, k, wl.num_q_heads, 128, dtype=torch.float32, device=device),
                first_reject=torch.empty(self.B, dtype=torch.int32, device=device),
                dev=torch.empty(self.B, k, dtype=torch.float32, device=device),
                ws=lynx.make_workspace(self.geo, self.B, k, device)))
        self.lens_flat = self.lens_flat_cpu.to(device)
        self.ws1 = lynx.make_workspace(self.geo, self.B, 1, device)
        # algorithmic bytes per launch kind
        rows_kv = 2 * L * Hkv * int(lens.sum())          # K rows + V rows over all layers
        self.rows_kv = rows_kv
        self.tokens_ctx = L * int(lens.sum())
        self.launch_rows = {"split_quantize": L * nb_layer * Hkv * bt, "anchor_attention": rows_kv,
                            "merge_verify_attention": rows_kv}
        torch.cuda.synchronize()

    # one pass of the hot path; `rec` (optional) receives (kind, start_event, end_event)
    def step(self, rec=None):
        lynx = self.lynx

        def timed(kind, fn):
            if rec is None:
                return fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            r = fn()
            b.record()
            rec.append((kind, a, b))
            return r

        for w in "KV":
            timed("split_quantize", lambda w=w: lynx.split_quantize(
                self.src[w], out=self.planes[w], block_ids=self.block_ids,
                rows_per_block=self.wl.num_kv_heads * self.wl.block_tokens if self.block_ids is not None else 0))
        K, V = self.planes["K"], self.planes["V"]
        n = 2
        for win in self.windows:
            for _ in range(win["reps"]):
                for j in range(win["k"]):
                    timed("anchor_attention", lambda j=j: lynx.anchor_attention(
                        self.geo, win["qs"][j], K, V, self.table, win["step_lens"][j], self.ws1,
                        out=win["step_out"][j]))
                    win["draft"][:, j:j + 1].copy_(win["step_out"][j])
                timed(f"merge_verify_attention[k={win['k']}]", lambda: lynx.merge_verify_attention(
                    self.geo, win["q"], K, V, self.table, self.lens_flat, win["ws"], draft_out=win["draft"],
                    atol=0.5, rtol=0.1, causal=True, out_full=win["out_full"],
                    first_reject=win["first_reject"], dev=win["dev"]))
                n += win["k"] + self.verify_kernels(win["k"])
        return n

    def verify_kernels(self, k):
        """Kernels of one merge-verify call: one attention launch per slice of the window (the library takes up
        to 16 columns per launch on the integer kernel and runs 17..32 columns as two such passes; up to 16
        positions and 64 columns on the FP16 kernel), plus the decision kernel when there is more than one."""
        G = self.wl.num_q_heads // self.wl.num_kv_heads
        cols = k * G
        if 16 < cols <= 32 and 16 // G > 0:
            per = 16 // G
        elif k <= 16 and cols <= 64:
            per = k
        else:
            per = min(16, max(1, 64 // G))
        slices = -(-k // per)
        return slices + (1 if slices > 1 else 0)

    def launches_per_step(self):
        return 2 + sum(w["reps"] * (w["k"] + self.verify_kernels(w["k"])) for w in self.windows)

    def bytes_per_step(self):
        b = 2 * self.launch_rows["split_quantize"] * BYTES_PER_ROW["split_quantize"]
        for w in self.windows:
            b += w["reps"] * (w["k"] * self.rows_kv * BYTES_PER_ROW["anchor_attention"]
                              + self.rows_kv * BYTES_PER_ROW["merge_verify_attention"])
        return b


# ------------------------------------------------------------------------------ clock sampling
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 c[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# --------------------------------------------------------------------------------- CPU oracle
class OracleSample:
    """One layer of the workload on the host, for timing the oracle as it stands."""

    def __init__(self, cfg_id: int, k_list=None):
        import numpy as np
        wl = synth.WORKLOADS[cfg_id]
        self.wl, self.np = wl, np
        bt, Hkv = wl.block_tokens, wl.num_kv_heads
        if wl.ragged:
            self.lens = synth.seq_lens(wl.batch, wl.min_context, wl.context, wl.name, 0)
        else:
            self.lens = torch.full((wl.batch,), wl.context, dtype=torch.int32)
        self.table, nb = synth.block_table(self.lens, bt, wl.shuffled_blocks, wl.name, 0)
        bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
        self.kb = bits(synth.kv_block_values(wl.recipe, nb, Hkv, bt, "cpu", wl.name, "K", 0, 0))
        self.vb = bits(synth.kv_block_values(wl.recipe, nb, Hkv, bt, "cpu", wl.name, "V", 0, 0))
        self.k_list = tuple(k_list if k_list is not None else wl.k_list)
        self.q = {k: bits(synth.queries(wl.batch, k, wl.num_q_heads, "cpu", wl.name, "q", k, 0))
                  for k in self.k_list}
        self.rows_q = 2 * nb * Hkv * bt
        self.rows_a = 2 * Hkv * int(self.lens.sum())

    def run(self):
        """One pass: split-quantise K and V, then per k: k anchor steps and one verify.
        Returns (seconds, algorithmic bytes, description)."""
        import oracle
        np, wl = self.np, self.wl
        t0 = time.perf_counter()
        kp = oracle.split_quantize(self.kb)
        vp = oracle.split_quantize(self.vb)
        t1 = time.perf_counter()
        nbytes = self.rows_q * BYTES_PER_ROW["split_quantize"]
        tab, lens = self.table.numpy(), self.lens.numpy()
        for k in self.k_list:
            q = self.q[k]
            draft = np.empty((wl.batch, k, wl.num_q_heads, 128), np.float32)
            for j in range(k):
                lj = np.maximum(lens - k + j + 1, 0).astype(np.int32)
                draft[:, j] = oracle.attention(False, q[:, j:j + 1], kp, vp, tab, lj, wl.num_kv_heads,
                                               wl.block_tokens)[:, 0]
            of = oracle.attention(True, q, kp, vp, tab, lens, wl.num_kv_heads, wl.block_tokens, causal=True)
            oracle.verify_decision(of, draft, 0.5, 0.1)
            nbytes += self.rows_a * (k * BYTES_PER_ROW["anchor_attention"] + BYTES_PER_ROW["merge_verify_attention"])
        t2 = time.perf_counter()
        desc = (f"{wl.name}: 1 of {wl.layers} layers, all {wl.num_kv_heads} KV heads, full context: "
                f"split-quantise K+V ({t1 - t0:.2f} s), then for k in {list(self.k_list)}: k anchor steps + 1 "
                f"merge-verify ({t2 - t1:.2f} s); same algorithmic bytes per row as the GPU arm")
        return t2 - t0, nbytes, desc


def oracle_sample(cfg_id: int, k_list=None):
    """Times the oracle on one layer of the workload.  Returns (GB/s, description, threads, s)."""
    import oracle
    smp = OracleSample(cfg_id, k_list)
    secs = nbytes = 0.0
    passes = 0
    while secs < 10.0 and passes < 8:       # about 10-30 s of CPU work
        s1, b1, desc = smp.run()
        secs, nbytes, passes = secs + s1, nbytes + b1, passes + 1
    desc = f"{passes} pass(es) of: " + desc
    return nbytes / secs / 1e9, desc, oracle.threads(), secs


# ---------------------------------------------------------------------- reporting helpers
# DRAM bytes ncu measured for one launch, as a multiple of the algorithmic bytes of that launch
# (dram__bytes_read.sum + dram__bytes_write.sum over 72 / 136 / 392 B per row; captures on an
# 8-layer copy of config 3, summarised under profiles/).  Traffic grows in proportion to the
# rows a launch processes, so a full launch is scaled by the rows.
TRAFFIC_RATIO = {"anchor_attention": 1.005, "merge_verify_attention": 1.005, "split_quantize": 0.990}


def base_kind(kind: str) -> str:
    return kind.split("[")[0]


def max_over_ranks(ms: float, dist=None, device=None) -> float:
    """Whole-job time of a step sequence: the slowest rank's device time."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(step_bytes: int, ms_per_step: float, world: int) -> float:
    """GB/s of the whole job: every rank runs the same per-GPU workload (weak scaling)."""
    return world * step_bytes / (ms_per_step * 1e-3) / 1e9


def kernel_table(times_ms: dict, launch_bytes: dict, steps: int, ms_per_step: float, peak: float):
    """times_ms: kind -> list of per-launch durations.  Returns per-kind statistics."""
    out = {}
    for kind, ts in times_ms.items():
        avg = sum(ts) / len(ts)
        nbytes = launch_bytes[base_kind(kind)]
        gbs = nbytes / (avg * 1e-3) / 1e9
        out[kind] = {"launches": len(ts), "avg_ms": avg, "min_ms": min(ts), "GBps": gbs,
                     "frac_of_measured": gbs / peak, "frac_of_nominal_8TBps": gbs / NOMINAL_HBM_GBS,
                     "share_of_step": sum(ts) / steps / ms_per_step,
                     "algorithmic_bytes_per_launch": nbytes}
    return out


# --------------------------------------------------------------------------------------- main
def run_reference(args):
    """The CPU oracle as the reference arm: each step is a bounded sample of the workload (one
    layer; split-quantise, then the first speculation depth's anchor steps and verify)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    wl = synth.WORKLOADS[args.config]
    smp = OracleSample(args.config, k_list=wl.k_list[:1])
    vals, desc = [], ""
    for i in range(args.warmup + args.steps):
        secs, nbytes, desc = smp.run()
        if i >= args.warmup:
            vals.append(nbytes / secs / 1e9)
    value = len(vals) / sum(1.0 / v for v in vals)
    threads = oracle.threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "note": "CPU oracle on host cores, bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="lynx", choices=["lynx", "reference"])
    ap.add_argument("--config", type=int, default=3, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--layers", type=int, default=0,
                    help="run a reduced copy of the workload with this many layers (for ncu captures)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-context", action="store_true", help="skip the context measurements after the timed steps")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "lynx" else args.warmup
    if args.impl == "reference":
        return run_reference(args)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    wlk = Workload(args.config, device, rank, args.layers)
    wl = wlk.wl

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        wlk.step()
    barrier()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    rec = []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    n_launch = 0
    for _ in range(args.steps):
        n_launch += wlk.step(rec)
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if sampler else None
    ms = max_over_ranks(ms, dist, device)
    lynx = wlk.lynx
    for w in wlk.windows:
        lynx.check(w["ws"])
    lynx.check(wlk.ws1)

    ms_per_step = ms / args.steps
    step_bytes = wlk.bytes_per_step()
    value = job_value(step_bytes, ms_per_step, world)
    peak, peak_kind = measured_peak()

    per = {}
    for kind, a, b in rec:
        per.setdefault(kind, []).append(a.elapsed_time(b))
    launch_bytes = {k_: wlk.launch_rows[k_] * BYTES_PER_ROW[k_] for k_ in BYTES_PER_ROW}
    kernels = kernel_table(per, launch_bytes, args.steps, ms_per_step, peak)
    for kind, st in kernels.items():
        if kind == "split_quantize":     # context tokens (K and V of all layers) per second
            st["tokens_per_s"] = wlk.tokens_ctx / (2 * st["avg_ms"] * 1e-3)
        elif kind == "anchor_attention":  # decode steps x sequences per second, all layers
            st["tokens_per_s"] = wl.batch / (st["avg_ms"] * 1e-3)
        else:                             # verified positions per second, all layers
            k_of = int(kind.split("=")[1].rstrip("]"))
            st["tokens_per_s"] = wl.batch * k_of / (st["avg_ms"] * 1e-3)
    # shares by kernel (all verify depths together) pick the dominant kernel
    share = {}
    for kind, st in kernels.items():
        share[base_kind(kind)] = share.get(base_kind(kind), 0.0) + st["share_of_step"]
    dom = max(share, key=share.get)
    dom_ts = [t for kind, ts in per.items() if base_kind(kind) == dom for t in ts]
    dom_gbs = launch_bytes[dom] / (sum(dom_ts) / len(dom_ts) * 1e-3) / 1e9
    roof = {"bound": "hbm", "kernel": dom, "achieved": dom_gbs, "peak": peak, "unit": "GB/s",
            "frac": dom_gbs / peak,
            "peak_source": "measured copy rate (MEASURED_PEAKS.json hbm_gbs)" if peak_kind == "measured"
            else "fallback 6.65 TB/s (MEASURED_PEAKS.json absent)",
            "traffic": launch_bytes[dom] * TRAFFIC_RATIO[dom],
            "traffic_source": "ncu dram__bytes_read+write on a 6-layer copy of config 3, scaled by rows",
            "algorithmic_bytes_per_launch": launch_bytes[dom], "share_of_step": share[dom],
            "launches": len(dom_ts), "avg_launch_ms": sum(dom_ts) / len(dom_ts)}

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8 x s8 -> s32 (Q.K^T) and u8 x u8 -> s32 (P.V) on tcgen05 kind::i8; f16 -> f32 on tcgen05 for verify with 33..64 columns per launch; f32 softmax and quantiser",
        "data": "synthetic",
        "config": {"workload": wl.name, "layers": wl.layers, "batch": wl.batch, "context": wl.context,
                   "num_kv_heads": wl.num_kv_heads, "num_q_heads": wl.num_q_heads, "k": list(wl.k_list),
                   "block_tokens": wl.block_tokens, "layers_flattened_into_batch": True,
                   "l2": "inputs larger than L2 (no flush)" if step_bytes > 1e9 else "inputs fit in L2",
                   "step": "split-quantise K,V; per k: k anchor steps then 1 merge-verify"},
        "gpu_launches": n_launch, "frac_of_measured_peak": value / world / peak,
        "frac_of_nominal_8TBps": value / world / NOMINAL_HBM_GBS,
        "kernels": kernels, "roofline": roof, "clocks": clocks,
    }

    if rank == 0 and world == 1 and not args.no_context:
        line["per_layer_launches"] = run_per_layer(wlk, peak)
        line["recombine"] = run_recombine(wlk, peak)
        line["bf16_pages"] = run_bf16_pages(wlk, peak)
        line["hierarchical"] = run_hier(wlk, peak)
        line["progressive"] = run_progressive(wlk)
        line["token_verify"] = run_token_verify(wlk, peak)
        line["bf16_tail"] = run_tail(wlk)
        line["bit_splits"] = run_bit_splits(wlk, peak)
    if rank == 0 and world == 1 and not args.no_e2e:
        line["e2e"] = run_e2e(wlk, args.e2e_steps, step_bytes)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, desc, threads, secs = oracle_sample(args.config)
        line["cpu_baseline"] = {"value": v, "unit": "GB/s", "cores": threads, "kind": "oracle",
                                "sample": desc, "seconds": secs}
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


def run_progressive(wlk: "Workload", max_layers: int = 8, cap: int = 64, k: int = 4):
    """Context: progressive arrival (Section 4.2, Residual Phase; Section 4.2 "Speculative Decoder").  The
    Anchor planes of up to 8 layers are resident; their Residual planes arrive from pinned host memory on
    a second stream, layer by layer (the stand-in for the NIC queue of lower priority), while the decoder
    drafts on the Anchor state: one anchor decode step over all layers per token, the host polling the
    Residual's arrival before each next token as the paper's decoder does, up to `cap` drafts.  When the
    Residual is in, one merge-verify pass checks the last k drafted positions.  Reported against the same
    work done one after the other.  Not part of `value`."""
    lynx, wl, dev = wlk.lynx, wlk.wl, wlk.device
    layers = min(wl.layers, max_layers)
    Bs, nb = layers * wl.batch, layers * wlk.nb_layer
    K, V = wlk.planes["K"], wlk.planes["V"]
    host = {w: pl.residual[:nb].cpu().pin_memory() for w, pl in (("K", K), ("V", V))}
    late = {w: torch.zeros_like(pl.residual[:nb]) for w, pl in (("K", K), ("V", V))}     # where the Residual lands
    Ka, Va = (lynx.Planes(pl.anchor[:nb], late[w], pl.meta[:nb]) for w, pl in (("K", K), ("V", V)))
    geo = lynx.Geometry(wl.num_q_heads, wl.num_kv_heads, wl.block_tokens, nb, wlk.table.shape[1])
    table = wlk.table[:Bs].contiguous()
    lens_full = wlk.lens_flat[:Bs].contiguous()
    win = next(w for w in wlk.windows if w["k"] == k) if any(w["k"] == k for w in wlk.windows) else wlk.windows[0]
    k = win["k"]
    q1 = win["qs"][0][:Bs].contiguous()
    qk = win["q"][:Bs].contiguous()
    ws1, wsk = lynx.make_workspace(geo, Bs, 1, dev), lynx.make_workspace(geo, Bs, k, dev)
    out1 = torch.empty(Bs, 1, wl.num_q_heads, 128, dtype=torch.float32, device=dev)
    draft = torch.zeros(Bs, k, wl.num_q_heads, 128, dtype=torch.float32, device=dev)
    outk = torch.empty_like(draft)
    fr = torch.empty(Bs, dtype=torch.int32, device=dev)
    dv = torch.empty(Bs, k, dtype=torch.float32, device=dev)
    step_lens = [(lens_full - cap + j + 1).contiguous() for j in range(cap)]
    copy_stream = torch.cuda.Stream(device=dev)
    per_layer = wlk.nb_layer

    def transfer():
        with torch.cuda.stream(copy_stream):
            for l in range(layers):
                sl = slice(l * per_layer, (l + 1) * per_layer)
                for w in "KV":
                    late[w][sl].copy_(host[w][sl], non_blocking=True)
            ev = torch.cuda.Event()
            ev.record(copy_stream)
        return ev

    def anchor_step(j):
        lynx.anchor_attention(geo, q1, Ka, Va, table, step_lens[j], ws1, out=out1)

    def verify():
        lynx.merge_verify_attention(geo, qk, Ka, Va, table, lens_full, wsk, draft_out=draft, atol=0.5, rtol=0.1,
                                    causal=True, out_full=outk, first_reject=fr, dev=dv)
    import time
    for _ in range(2):          # warm-up of every piece
        transfer().synchronize(); anchor_step(0); verify(); torch.cuda.synchronize()
    t0 = time.perf_counter(); transfer().synchronize(); t_h2d = time.perf_counter() - t0
    t0 = time.perf_counter()
    for j in range(8):
        anchor_step(j); torch.cuda.synchronize()
    t_step = (time.perf_counter() - t0) / 8
    t0 = time.perf_counter(); verify(); torch.cuda.synchronize(); t_ver = time.perf_counter() - t0
    # overlapped: drafts run while the Residual arrives
    for w in "KV":
        late[w].zero_()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    ev = transfer()
    n = 0
    while n < cap and not ev.query():
        anchor_step(n); torch.cuda.current_stream().synchronize()     # (a decoder needs the token before the next step)
        n += 1
    t_draft_end = time.perf_counter() - t0
    ev.synchronize()
    verify(); torch.cuda.synchronize()
    t_total = time.perf_counter() - t0
    lynx.check(wsk); lynx.check(ws1)
    ok = bool(torch.equal(late["K"], K.residual[:nb]) and torch.equal(late["V"], V.residual[:nb]))
    serial = t_h2d + n * t_step + t_ver
    return {"layers": layers, "residual_bytes": int(2 * late["K"].numel()), "h2d_alone_ms": t_h2d * 1e3,
            "anchor_step_ms": t_step * 1e3, "verify_ms": t_ver * 1e3, "drafts_while_waiting": n, "draft_cap": cap,
            "drafting_ended_ms": t_draft_end * 1e3, "overlapped_total_ms": t_total * 1e3, "one_after_the_other_ms": serial * 1e3,
            "transfer_hidden_frac": min(1.0, n * t_step / t_h2d) if t_h2d > 0 else None,
            "residual_arrived_intact": ok, "timing": "host wall clock around synchronised steps (context only)"}


def run_token_verify(wlk: "Workload", peak: float, batch: int = 256, k: int = 8, vocab: int = 128256):
    """Context: token-level verification (Section 4.3) of `batch` windows of k drafts over a Llama-3-sized
    vocabulary; synthetic distributions, the uniforms supplied.  Not part of `value`."""
    lynx = wlk.lynx
    g = torch.Generator(device=wlk.device)
    g.manual_seed(1234)
    logits = torch.randn(batch, k + 1, vocab, generator=g, device=wlk.device) * 3.0
    q = torch.softmax(logits, -1)
    p = torch.softmax(logits[:, :k] + 0.3 * torch.randn(batch, k, vocab, generator=g, device=wlk.device), -1)
    del logits
    s = torch.multinomial(p.view(-1, vocab), 1, generator=g).view(batch, k).to(torch.int32)
    u = torch.rand(batch, k, generator=g, device=wlk.device)
    r = torch.rand(batch, generator=g, device=wlk.device)
    for _ in range(3):
        n_acc, nxt = lynx.token_verify(p, q, s, u, r)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 20
    e0.record()
    for _ in range(reps):
        n_acc, nxt = lynx.token_verify(p, q, s, u, r)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    # bytes that must move: one or two vocabulary rows per window (the correction or the bonus row), read twice
    # at worst by the slice sums and the walk of one slice; counted once
    rows = int((n_acc < k).sum().item()) * 2 + int((n_acc == k).sum().item())
    gb = rows * vocab * 4 / (ms * 1e-3) / 1e9
    return {"windows": batch, "k": k, "vocab": vocab, "ms": ms, "mean_accepted": float(n_acc.float().mean().item()),
            "bytes": rows * vocab * 4, "GBps": gb, "frac_of_measured": gb / peak}


def run_hier(wlk: "Workload", peak: float, max_pages: int = 16384):
    """Context: the paper's own quantiser (Algorithm 1) and its inverse on the first rows of the BF16
    K source viewed as pages of 256 tokens (1 GiB at most).  Not part of `value`."""
    lynx = wlk.lynx
    src = wlk.src["K"].view(-1, 128)
    n = min(src.shape[0] // 256, max_pages)
    x = src[: n * 256].view(n, 256, 128)
    h = lynx.hier_quantize(x)
    out = torch.empty(n, 256, 128, dtype=torch.bfloat16, device=wlk.device)

    def time_ms(fn, reps=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps
    lib, stream = lynx.load(), torch.cuda.current_stream().cuda_stream

    def quant():
        st = lib.lynx_hier_quantize(x.data_ptr(), n, h.q_anc.data_ptr(), h.q_res.data_ptr(), h.gamma_min.data_ptr(),
                                    h.gamma_scale.data_ptr(), h.mu.data_ptr(), h.sigma.data_ptr(), stream)
        if st != 0:
            raise RuntimeError(f"lynx_hier_quantize: status {st}")
    res = {"pages": n}
    meta = (2 * 128 + 2 * 8 * 128) * 4
    for name, fn, bytes_pp in (("quantize", quant, 256 * 256 + 2 * 256 * 64 + meta),
                               ("dequantize", lambda: lynx.hier_dequantize(h, out=out), 2 * 256 * 64 + meta + 256 * 256),
                               ("dequantize_anchor_only", lambda: lynx.hier_dequantize(h, anchor_only=True, out=out),
                                256 * 64 + meta + 256 * 256)):
        ms = time_ms(fn)
        g = n * bytes_pp / (ms * 1e-3) / 1e9
        res[name] = {"ms": ms, "bytes_per_page": bytes_pp, "GBps": g, "frac_of_measured": g / peak}
    return res


def run_bf16_pages(wlk: "Workload", peak: float, max_layers: int = 8):
    """Context: the decode path the paper describes (Section 4.2: dequantise to BF16 pages, the engine's
    attention reads 256 bytes per row) against the fused call on the same full-precision state (136
    bytes per row), one decode step (n_q = 1) on up to 8 layers of the workload: lynx_recombine of K
    and V to pages, lynx_bf16_attention on them, lynx_merge_verify_attention with k = 1.  Not part of
    `value`."""
    lynx, wl = wlk.lynx, wlk.wl
    layers = min(wl.layers, max_layers)
    Bs = layers * wl.batch
    nb = layers * wlk.nb_layer
    dev = wlk.device

    def first(pl):
        return lynx.Planes(pl.anchor[:nb], pl.residual[:nb], pl.meta[:nb])
    K, V = first(wlk.planes["K"]), first(wlk.planes["V"])
    geo = lynx.Geometry(wl.num_q_heads, wl.num_kv_heads, wl.block_tokens, nb, wlk.table.shape[1])
    table, lens = wlk.table[:Bs].contiguous(), wlk.lens_flat[:Bs].contiguous()
    q = wlk.windows[0]["qs"][0][:Bs].contiguous()
    ws = lynx.make_workspace(geo, Bs, 1, dev)
    pages = {w: torch.empty(nb, wl.num_kv_heads, wl.block_tokens, 128, dtype=torch.bfloat16, device=dev) for w in "KV"}
    import ctypes
    wsb = torch.empty(int(lynx.load().lynx_bf16_workspace_bytes(ctypes.byref(geo._c()), Bs, 1)),
                      dtype=torch.uint8, device=dev)
    out_a = torch.empty(Bs, 1, wl.num_q_heads, 128, dtype=torch.float32, device=dev)
    out_b = torch.empty_like(out_a)
    lib = lynx.load()
    stream = torch.cuda.current_stream().cuda_stream

    def recombine():
        for w, pl in (("K", K), ("V", V)):
            st = lib.lynx_recombine(pl.anchor.data_ptr(), pl.residual.data_ptr(), pl.meta.data_ptr(),
                                    pl.anchor.numel() // 64, None, pages[w].data_ptr(), stream)
            if st != 0:
                raise RuntimeError(f"lynx_recombine: status {st}")

    def bf16():
        lynx.bf16_attention(geo, q, pages["K"], pages["V"], table, lens, workspace=wsb, out=out_b)

    def fused():
        lynx.merge_verify_attention(geo, q, K, V, table, lens, ws, causal=True, out_full=out_a)

    def time_ms(fn, reps=5):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps
    rows = 2 * wl.num_kv_heads * int(wlk.lens_flat_cpu[:Bs].sum())     # K rows + V rows the step attends to
    rows_pool = 2 * nb * wl.num_kv_heads * wl.block_tokens
    t_rec, t_bf, t_fu = time_ms(recombine), time_ms(bf16), time_ms(fused)
    lynx.check(ws)
    diff = float((out_a - out_b).abs().max())

    def entry(ms, bytes_):
        g = bytes_ / (ms * 1e-3) / 1e9
        return {"ms": ms, "bytes": bytes_, "GBps": g, "frac_of_measured": g / peak}
    return {"layers": layers, "rows": rows,
            "recombine_to_pages": entry(t_rec, rows_pool * (136 + 256)),
            "bf16_attention": entry(t_bf, rows * 256),
            "fused_full_state_decode": entry(t_fu, rows * 136),
            "roofline": {"bound": "hbm", "kernel": "bf16_attention", "achieved": rows * 256 / (t_bf * 1e-3) / 1e9,
                         "peak": peak, "unit": "GB/s", "frac": rows * 256 / (t_bf * 1e-3) / 1e9 / peak},
            "speedup_fused_vs_bf16_attention": t_bf / t_fu,
            "speedup_fused_vs_recombine_plus_bf16_attention": (t_rec + t_bf) / t_fu,
            "max_abs_difference_of_outputs": diff}


def run_tail(wlk: "Workload", max_layers: int = 8, tail_tokens: int = 1024):
    """Context: one decode step (n_q = 1) on the Anchor state of up to 8 layers of the workload when every
    sequence is followed by `tail_tokens` tokens the decode node generated itself (BF16 pages, Section 4.2
    keeps them out of the quantiser): lynx_anchor_attention on the prefix, lynx_bf16_attention on the tail,
    lynx_lse_merge of the two by the log-sum-exps the calls leave in their workspaces.  Reports what the tail
    adds to the prefix call.  Not part of `value`."""
    import ctypes
    lynx, wl = wlk.lynx, wlk.wl
    layers = min(wl.layers, max_layers)
    Bs, nb, dev = layers * wl.batch, layers * wlk.nb_layer, wlk.device
    K = lynx.Planes(wlk.planes["K"].anchor[:nb], None, wlk.planes["K"].meta[:nb])
    V = lynx.Planes(wlk.planes["V"].anchor[:nb], None, wlk.planes["V"].meta[:nb])
    geo = lynx.Geometry(wl.num_q_heads, wl.num_kv_heads, wl.block_tokens, nb, wlk.table.shape[1])
    table, lens = wlk.table[:Bs].contiguous(), wlk.lens_flat[:Bs].contiguous()
    q = wlk.windows[0]["qs"][0][:Bs].contiguous()
    ws = lynx.make_workspace(geo, Bs, 1, dev)
    # the tail: `tail_tokens` BF16 tokens per sequence in pages of the workload's block size (seeded values)
    bt = wl.block_tokens
    per = (tail_tokens + bt - 1) // bt
    geo_t = lynx.Geometry(wl.num_q_heads, wl.num_kv_heads, bt, Bs * per, per)
    gen = torch.Generator(device=dev)
    gen.manual_seed(20260701)
    pages = [torch.randn(Bs * per, wl.num_kv_heads, bt, 128, device=dev, generator=gen).to(torch.bfloat16) for _ in "KV"]
    ttable = torch.arange(Bs * per, dtype=torch.int32, device=dev).view(Bs, per)
    tlens = torch.full((Bs,), tail_tokens, dtype=torch.int32, device=dev)
    ws_t = torch.empty(int(lynx.load().lynx_bf16_workspace_bytes(ctypes.byref(geo_t._c()), Bs, 1)), dtype=torch.uint8, device=dev)
    out_p = torch.empty(Bs, 1, wl.num_q_heads, 128, dtype=torch.float32, device=dev)
    out_t, out = torch.empty_like(out_p), torch.empty_like(out_p)
    lse_p, lse_t = lynx.workspace_lse(geo, Bs, 1, ws), lynx.bf16_workspace_lse(geo_t, Bs, 1, ws_t)

    def prefix():
        lynx.anchor_attention(geo, q, K, V, table, lens, ws, out=out_p)

    def tail():
        lynx.bf16_attention(geo_t, q, pages[0], pages[1], ttable, tlens, workspace=ws_t, causal=True, out=out_t)

    def merge():
        lynx.lse_merge(out_p, lse_p, out_t, lse_t, out=out)

    def all3():
        prefix(); tail(); merge()

    def time_ms(fn, reps=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps
    t = {name: time_ms(fn) for name, fn in (("prefix_anchor_attention", prefix), ("tail_bf16_attention", tail),
                                             ("lse_merge", merge), ("all_three", all3))}
    lynx.check(ws)
    share = float(torch.exp(lse_t - torch.logaddexp(lse_p, lse_t)).mean())
    return {"layers": layers, "sequences": Bs, "tail_tokens": tail_tokens, "ms": t,
            "tail_adds": t["all_three"] / t["prefix_anchor_attention"] - 1.0, "mean_softmax_mass_on_tail": share}


def run_bit_splits(wlk: "Workload", peak: float, max_rows: int = 4 << 20):
    """Context: the Anchor / Residual split at other bit positions (Conclusion: splits other than INT4 + INT4) on
    the first rows of the BF16 K source, at most 4 Mi rows: lynx_split_quantize_bits for 2 + 6 and 6 + 2 bits
    (392 bytes per row, as for 4 + 4), lynx_recombine_bits to BF16 pages from both streams and from the Anchor
    alone.  Not part of `value`."""
    lynx = wlk.lynx
    src = wlk.src["K"].view(-1, 128)
    rows = min(src.shape[0], max_rows)
    x = src[:rows]
    lib, stream = lynx.load(), torch.cuda.current_stream().cuda_stream
    deq = torch.empty(rows, 128, dtype=torch.bfloat16, device=wlk.device)

    def time_ms(fn, reps=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps
    out = {"rows": rows}
    for A in (2, 6):
        a, r, m = lynx.split_quantize_bits(x, A)

        def quant():
            st = lib.lynx_split_quantize_bits(x.data_ptr(), rows, A, a.data_ptr(), r.data_ptr(), m.data_ptr(), stream)
            if st != 0:
                raise RuntimeError(f"lynx_split_quantize_bits: status {st}")

        def pages(res):
            st = lib.lynx_recombine_bits(a.data_ptr(), res.data_ptr() if res is not None else None, m.data_ptr(), rows, A,
                                         None, deq.data_ptr(), stream)
            if st != 0:
                raise RuntimeError(f"lynx_recombine_bits: status {st}")
        for name, fn, bpr in (("split_quantize", quant, 256 + 128 + 8), ("pages_from_both_streams", lambda: pages(r), 136 + 256),
                              ("pages_from_the_anchor", lambda: pages(None), 16 * A + 8 + 256)):
            ms = time_ms(fn)
            g = rows * bpr / (ms * 1e-3) / 1e9
            out[f"{A}+{8 - A} {name}"] = {"ms": ms, "bytes_per_row": bpr, "GBps": g, "frac_of_measured": g / peak}
    return out


def run_recombine(wlk: "Workload", peak: float, max_rows: int = 4 << 20):
    """Context: the stand-alone refinement `lynx_recombine` (Anchor + Residual -> 8-bit codes and/or
    dequantised BF16 rows, the layout a stock BF16 attention would read) on the first rows of the
    K planes, at most 4 Mi rows (1 GiB of BF16 output).  Not part of `value`."""
    lynx = wlk.lynx
    K = wlk.planes["K"]
    rows = min(K.anchor.numel() // 64, max_rows)
    a, r, m = K.anchor.view(-1, 64)[:rows], K.residual.view(-1, 64)[:rows], K.meta.view(-1, 2)[:rows]
    codes = torch.empty(rows, 128, dtype=torch.uint8, device=wlk.device)
    deq = torch.empty(rows, 128, dtype=torch.bfloat16, device=wlk.device)
    lib = lynx.load()
    stream = torch.cuda.current_stream().cuda_stream
    out = {"rows": rows}
    for name, c, d, bpr in (("bf16", None, deq, 136 + 256), ("codes", codes, None, 136 + 128),
                            ("codes+bf16", codes, deq, 136 + 128 + 256)):
        def call():
            st = lib.lynx_recombine(a.data_ptr(), r.data_ptr(), m.data_ptr(), rows,
                                    c.data_ptr() if c is not None else None,
                                    d.data_ptr() if d is not None else None, stream)
            if st != 0:
                raise RuntimeError(f"lynx_recombine: status {st}")
        for _ in range(3):
            call()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 10
        e0.record()
        for _ in range(reps):
            call()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        gbs = rows * bpr / (ms * 1e-3) / 1e9
        out[name] = {"ms": ms, "bytes_per_row": bpr, "GBps": gbs, "frac_of_measured": gbs / peak}
    return out


def run_per_layer(wlk: "Workload", peak: float):
    """Context for the flattened numbers: one anchor decode step and one verify pass issued the
    way a decoder has to, one launch per layer (batch = the workload's sequences), back to back
    on one stream.  Not part of `value`."""
    lynx, wl = wlk.lynx, wlk.wl
    L, Bs = wl.layers, wl.batch
    win = wlk.windows[0]
    k = win["k"]
    geo = wlk.geo
    ws1 = lynx.make_workspace(geo, Bs, 1, wlk.device)
    wsk = lynx.make_workspace(geo, Bs, k, wlk.device)
    K, V = wlk.planes["K"], wlk.planes["V"]
    views = []
    for l in range(L):
        sl = slice(l * Bs, (l + 1) * Bs)
        views.append((win["qs"][k - 1][sl], win["q"][sl], wlk.table[sl], wlk.lens_flat[sl], win["step_out"][k - 1][sl],
                      win["draft"][sl], win["out_full"][sl], win["first_reject"][sl], win["dev"][sl]))

    def anchor_all():
        for q1, qk, tb, ln, o1, dr, of, fr, dv in views:
            lynx.anchor_attention(geo, q1, K, V, tb, ln, ws1, out=o1)

    def verify_all():
        for q1, qk, tb, ln, o1, dr, of, fr, dv in views:
            lynx.merge_verify_attention(geo, qk, K, V, tb, ln, wsk, draft_out=dr, atol=0.5, rtol=0.1,
                                        causal=True, out_full=of, first_reject=fr, dev=dv)

    out = {}
    for name, fn, bpr in (("anchor_attention", anchor_all, BYTES_PER_ROW["anchor_attention"]),
                          (f"merge_verify_attention[k={k}]", verify_all, BYTES_PER_ROW["merge_verify_attention"])):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 5
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        gbs = wlk.rows_kv * bpr / (ms * 1e-3) / 1e9
        out[name] = {"launches": L, "ms_all_layers": ms, "us_per_layer": ms * 1e3 / L, "GBps": gbs,
                     "frac_of_measured": gbs / peak}
        # the same launches replayed from one CUDA graph (no host work between them)
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                fn()
            for _ in range(2):
                graph.replay()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(reps):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            gms = e0.elapsed_time(e1) / reps
            out[name]["cuda_graph_us_per_layer"] = gms * 1e3 / L
            del graph
        except Exception as exc:   # capture is an extra: the eager figure above stands on its own
            out[name]["cuda_graph_us_per_layer"] = None
            out[name]["cuda_graph_error"] = str(exc)[:200]
            torch.cuda.synchronize()
    lynx.check(ws1)
    lynx.check(wsk)
    return out


def run_e2e(wlk: "Workload", steps: int, step_bytes: int):
    """The same step driven from HOST buffers: every step copies the BF16 KV cache and the queries
    from pinned host memory to the device, runs the path, and reads the verified outputs and the
    accept/reject indices back."""
    host_src = {w: torch.empty(wlk.src[w].shape, dtype=torch.bfloat16, pin_memory=True) for w in "KV"}
    for w in "KV":
        host_src[w].copy_(wlk.src[w])
    host_q = [win["q"].cpu().pin_memory() for win in wlk.windows]
    host_out = [torch.empty(win["out_full"].shape, dtype=torch.float32, pin_memory=True) for win in wlk.windows]
    host_fr = [torch.empty(win["first_reject"].shape, dtype=torch.int32, pin_memory=True) for win in wlk.windows]
    h2d = sum(t.numel() * t.element_size() for t in host_src.values()) + sum(t.numel() * 2 for t in host_q)
    d2h = sum(t.numel() * 4 for t in host_out) + sum(t.numel() * 4 for t in host_fr)

    def one():
        for w in "KV":
            wlk.src[w].copy_(host_src[w], non_blocking=True)
        for win, hq in zip(wlk.windows, host_q):
            win["q"].copy_(hq, non_blocking=True)
            for j in range(win["k"]):
                win["qs"][j].copy_(win["q"][:, j:j + 1])
        wlk.step()
        for win, ho, hf in zip(wlk.windows, host_out, host_fr):
            ho.copy_(win["out_full"], non_blocking=True)
            hf.copy_(win["first_reject"], non_blocking=True)

    one()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        one()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    return {"value": step_bytes / (ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": ms, "steps": steps,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}


if __name__ == "__main__":
    main()
