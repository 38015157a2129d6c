#!/usr/bin/env python
"""Benchmark of the AdaSD hot path on B200.

One step = one decode round of the workload, i.e. one pass of the whole hot path:
K draft steps (adasd_draft_entropy on [B,V]), one adasd_verify with the fused
threshold update, and (fixed-window workloads) one adasd_vanilla_verify on the same
inputs.  The headline `value` is the metric's own figure: logit rows read by
adasd_verify per second of adasd_verify time (a row = one length-V logit row), inputs
resident in HBM, CUDA events around every verify launch of the timed steps.  The rate of
the whole step (all call kinds) is reported beside it under `config`.  `e2e` is the same
verify metric through the C ABI from pinned HOST buffers, copies inside the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C1|C2|C3|C4|C5]
                    [--prefill N] [--impl reference]

  C3, C4   batched fixed-window rounds, issued call by call (the default, C4, is the workload
           the metric is quoted on); --prefill N imports N entries into both KDE lists of every
           sequence first, to show the cost the paper names (Sec. 4.4: KDE cost grows with the
           collected samples)
  C1, C2   single-stream rounds: microseconds per call from CUDA-graph replays
  C5       the whole adaptive round (input generation, K draft steps with the device-side active
           mask, verification with the fused update) captured ONCE in a CUDA graph and replayed
           for every round of the workload: rounds/s of that graph and of a generator-only graph

With N > 1 (under torchrun) every rank runs its own batch of sequences: the path
shards over sequences with no collective on the data path (weak scaling).
`--impl reference` times the float64 CPU oracle on a bounded sample of the same
workload on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

METRIC = "verify_logit_rows_per_s"
UNIT = "rows/s"
# DRAM bytes of one verify launch (dram__bytes_read.sum + dram__bytes_write.sum) per algorithmic
# byte, from the ncu capture of workload C3 summarised under profiles/ (144.14 MB against
# 139.54 MB); traffic grows in proportion to the rows read, so other workloads scale by it.
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.033


def measured_peak_gbs():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock/throttle samples during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx, self.proc = gpu_index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.idx)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                  "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def step_rows(wl) -> dict:
    """Logit rows read by one step, per call kind (fixed window K)."""
    B, K = wl.B, wl.K
    return {"draft": B * K, "verify": B * (2 * K + 1), "vanilla": B * (2 * K + 1)}


def sfu_figures(B: int, K: int, V: int, verify_ms: float, clocks) -> dict:
    """Special-function (XU) throughput of the verify launch: nominal peak = 148 SMs x 16
    results per clock x the SM clock sampled during the run (1965 MHz if none was sampled)."""
    ops = (3 * B * K + B) * V
    mhz = (clocks or {}).get("sm_mhz") or 1965.0
    peak = 148 * 16 * mhz * 1e6
    achieved = ops / (verify_ms * 1e-3)
    return {"bound": "alu", "achieved": achieved / 1e12, "peak": peak / 1e12, "unit": "Tops/s",
            "frac": achieved / peak, "ops_per_launch": ops}


def cuts_on(args, wl) -> bool:
    """A top-k or top-p cut is set (temperature alone adds no launch)."""
    if not args.warpers:
        return False
    _, k, p = args.warpers
    return (0 < k < wl.V) or p < 1.0


def vanilla_launches(wl, sm_count: int) -> int:
    """Kernels one adasd_vanilla_verify call launches: with enough bf16 rows to fill the GPU
    it runs three (log-sum-exps of all rows, accept test, sampling of one
    position per sequence), else one."""
    streaming = wl.dtype == synth.BF16 and wl.V % 8 == 0 and wl.V >= 8192
    return 3 if streaming and wl.B * (2 * wl.K + 1) >= 2 * sm_count else 1


# ------------------------------------------------------------------------------ N ranks

def rank_workload(wl, rank: int, sets: int):
    """The shard of rank `rank`: sequences are independent, so every rank owns its own batch of
    the workload's shape (weak scaling) from its own seed; no data ever crosses ranks."""
    return wl.scaled(seed=wl.seed + 1000 * rank, rounds=max(sets, 1))


def max_over_ranks(values, dist, device):
    """Element-wise maximum over the ranks of a few timings (the job is as slow as its slowest rank)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_rate(world: int, units_per_rank_step: int, steps: int, ms: float) -> float:
    """Units all ranks processed in `steps` steps divided by the (max over ranks) time."""
    return world * units_per_rank_step * steps / (ms * 1e-3)


# ------------------------------------------------------------------------------ our arm

def run_ours(args) -> dict:
    import torch
    import paper_2512_11280_b200 as adasd

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    wl = synth.WORKLOADS[args.workload]
    if args.workload in ("C1", "C2"):
        return run_single_stream(args, torch, adasd, wl, rank, world, local, dev, dist)
    if args.workload == "C5":
        return run_adaptive_graph(args, torch, adasd, wl, rank, world, local, dev, dist)
    # every rank owns its own sequences: same shapes, different seed
    wl = rank_workload(wl, rank, args.sets)
    B, K, V = wl.B, wl.K, wl.V
    tdt = torch.bfloat16 if wl.dtype == synth.BF16 else torch.float32
    ctx = adasd.Context(B, V, K, dtype=wl.dtype,
                        list_capacity=args.prefill + (args.steps + args.warmup + 64) * K + 64, device=local)
    if args.prefill > 0:
        prefill_lists(ctx, B, args.prefill)
    if args.warpers:
        ctx.set_warpers(*args.warpers)
    gs = synth.GpuSynth(wl, str(dev))

    # input sets resident in HBM, cycled so that consecutive steps never share data;
    # one set is larger than L2 for the batched workloads (C3 139 MB, C4 1.28 GB)
    nset = max(args.sets, 1)
    zd = [torch.empty((B, K, V), dtype=tdt, device=dev) for _ in range(nset)]
    zt = [torch.empty((B, K + 1, V), dtype=tdt, device=dev) for _ in range(nset)]
    f32 = dict(dtype=torch.float32, device=dev)
    i32 = dict(dtype=torch.int32, device=dev)
    U = [gs.new_round_uniforms() for _ in range(nset)]
    u_d = [torch.empty((K, B), **f32) for _ in range(nset)]
    for s in range(nset):
        gs.draft_rows(s, zd[s])
        gs.target_rows(s, zt[s])
        gs.round_uniforms(s, U[s])
        u_d[s].copy_(U[s]["draft"].T)
    Hk = torch.zeros((K, B), **f32)
    tokk = torch.zeros((K, B), **i32)
    stopk = torch.zeros((K, B), dtype=torch.uint8, device=dev)
    dlen = torch.zeros(B, **i32)
    x = torch.zeros((B, K), **i32)
    al, nt, val, vnt = (torch.zeros(B, **i32) for _ in range(4))
    torch.cuda.synchronize()

    ev_pairs = []

    def step(s: int, timed_kernel: bool = False, zd_s=None, zt_s=None):
        zds = zd[s] if zd_s is None else zd_s
        zts = zt[s] if zt_s is None else zt_s
        for k in range(K):
            ctx.draft_entropy(zds[:, k, :], Hk[k], u=u_d[s][k], token_out=tokk[k], stop_out=stopk[k],
                              draft_len=dlen, row_stride=K * V)
        x.copy_(tokk.T)
        if timed_kernel:
            e0 = torch.cuda.Event(enable_timing=True)
            e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
        ctx.verify(zds, zts, x, U[s]["target"], U[s]["accept"], al, nt, fuse_update=True)
        if timed_kernel:
            e1.record()
            ev_pairs.append((e0, e1))
        ctx.vanilla_verify(zds, zts, x, U[s]["vanilla_accept"], U[s]["resample"], val, vnt)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for w in range(args.warmup):
        step(w % nset)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(args.steps):
        step((args.warmup + i) % nset, timed_kernel=True)
    t1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms = t0.elapsed_time(t1)
    verify_ms = statistics.mean(a.elapsed_time(b) for a, b in ev_pairs)
    status = ctx.status()
    if status != 0:
        raise RuntimeError(f"device status word {status} after the timed region")
    if not (0 <= int(al.min()) and int(al.max()) <= K and 0 <= int(nt.min()) and int(nt.max()) < V):
        raise RuntimeError("accept_len / next_token out of range")

    # ---- end to end from pinned host buffers (copies inside the timed region)
    e2e_steps = max(2, min(args.e2e_steps, args.steps))
    hd = torch.empty((B, K, V), dtype=tdt).pin_memory()
    ht = torch.empty((B, K + 1, V), dtype=tdt).pin_memory()
    hd.copy_(zd[0])
    ht.copy_(zt[0])
    h_out = torch.empty((2, B), dtype=torch.int32).pin_memory()
    d_out = torch.empty((2, B), **i32)
    zd_e = torch.empty_like(zd[0])
    zt_e = torch.empty_like(zt[0])

    def e2e_step():
        zd_e.copy_(hd, non_blocking=True)
        zt_e.copy_(ht, non_blocking=True)
        ctx.verify(zd_e, zt_e, x, U[0]["target"], U[0]["accept"], al, nt, fuse_update=True)
        d_out[0].copy_(al)
        d_out[1].copy_(nt)
        h_out.copy_(d_out, non_blocking=True)

    e2e_step()
    barrier()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)

    # the K draft calls of a round as one CUDA graph (issued one by one from Python the interpreter's
    # time per call would be the measurement): microseconds per adasd_draft_entropy call
    def drafts():
        for s in range(nset):
            for k in range(K):
                ctx.draft_entropy(zd[s][:, k, :], Hk[k], u=u_d[s][k], token_out=tokk[k], stop_out=stopk[k],
                                  draft_len=dlen, row_stride=K * V)
    side = torch.cuda.Stream()
    g_d = graph_of(torch, drafts, side)
    time_replays(torch, g_d, 3, side)
    draft_ms = time_replays(torch, g_d, 10, side) / (nset * K)

    ms, e2e_ms, verify_ms, draft_ms = max_over_ranks([ms, e2e_ms, verify_ms, draft_ms], dist, dev)

    rows = step_rows(wl)
    rows_step = sum(rows.values())
    row_bytes = wl.row_bytes
    peak, peak_kind = measured_peak_gbs()
    verify_bytes = rows["verify"] * row_bytes
    achieved = verify_bytes / (verify_ms * 1e-3) / 1e9
    h2d = (hd.numel() + ht.numel()) * hd.element_size()
    out = {
        "metric": METRIC, "value": whole_job_rate(world, rows["verify"], 1, verify_ms), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 (bf16 logits, fp32 arithmetic)" if wl.dtype == synth.BF16 else "f32",
        "data": "synthetic",
        "config": {"workload": f"{args.workload}: B={B} K={K} V={V} {'bf16' if wl.dtype == synth.BF16 else 'fp32'} "
                               f"fixed window, per step {K} draft_entropy + verify(fused update) + vanilla_verify",
                   "rows_per_step": rows, "bytes_per_step": rows_step * row_bytes,
                   "sequences_per_gpu": B, "input_sets": nset,
                   "l2": f"inputs larger than L2: {nset} sets of {(2 * K + 1) * B * row_bytes / 1e6:.0f} MB cycled",
                   "value_is": "rows read by adasd_verify / adasd_verify time (mean of the timed launches, max over ranks)",
                   "step_rows_per_s_all_calls": whole_job_rate(world, rows_step, args.steps, ms),
                   "kde_list_prefill": args.prefill,
                   "warpers": None if not args.warpers else
                   {"temperature": args.warpers[0], "top_k": args.warpers[1], "top_p": args.warpers[2],
                    "note": "with top-k / top-p on, every call first finds one cutoff logit per row "
                            "(row_cutoff_kernel): the times include it, the bytes count the rows once"},
                   "draft_entropy": {"us_per_call": 1e3 * draft_ms, "bytes_per_call": B * row_bytes,
                                     "gbs": B * row_bytes / (draft_ms * 1e-3) / 1e9,
                                     "frac_of_peak": B * row_bytes / (draft_ms * 1e-3) / 1e9 / peak,
                                     "timing": f"one CUDA graph of {nset * K} calls, 10 replays"},
                   "hbm_gbs_all_calls": world * rows_step * row_bytes * args.steps / (ms * 1e-3) / 1e9},
        "e2e": {"value": whole_job_rate(world, rows["verify"], e2e_steps, e2e_ms), "unit": UNIT,
                "what": "pinned host logits -> device, adasd_verify through the C ABI, results -> host",
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": h_out.numel() * 4,
                "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps},
        # with a top-k / top-p cut every draft call adds two launches (the one-pass cutoff kernel and the
        # radix kernel for the rows it hands over), verify and vanilla verify four each (target and draft rows)
        "gpu_launches": args.steps * (K + 1 + vanilla_launches(wl, torch.cuda.get_device_properties(dev).multi_processor_count)
                                      + (2 * K + 8 if cuts_on(args, wl) else 0)),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": "adasd_verify", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_8TBs_nominal": achieved / 8000.0,
                     "algorithmic_bytes_per_launch": verify_bytes, "ms_per_launch": verify_ms,
                     "traffic": NCU_TRAFFIC_PER_ALGORITHMIC_BYTE * verify_bytes,
                     "traffic_source": "ncu capture of C3, scaled by the rows of this workload",
                     # the pipe that ncu shows busiest: 2 ex2 + 1 lg2 per logit pair, 1 ex2 per bonus logit
                     "special_function_pipe": sfu_figures(B, K, V, verify_ms, clocks)},
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = oracle_sample(synth.WORKLOADS[args.workload], args.cpu_seconds)
    if dist is not None:
        dist.destroy_process_group()
    return out if rank == 0 else None


def prefill_lists(ctx, B: int, n: int) -> None:
    """n entries in L_D^A and L_D^R (and a few rejected entropies) of every sequence: the state of
    a long decoding run, so that the KDE sums of the verify tail have n terms per list."""
    rng = np.random.default_rng(7)
    for b in range(B):
        LA = np.clip(rng.normal(0.25, 0.12, n), 0.01, 0.99)
        LR = np.clip(rng.normal(0.65, 0.15, n), 0.01, 0.99)
        ctx.state_import(b, 0.0, rng.uniform(1.0, 4.0, 16), LA, LR)


def common_fields(args, world, wl, name, extra_cfg, value, ms_per_step, verify_ms, verify_rows, launches,
                  clocks, e2e):
    peak, peak_kind = measured_peak_gbs()
    verify_bytes = verify_rows * wl.row_bytes
    achieved = verify_bytes / (verify_ms * 1e-3) / 1e9
    cfg = {"workload": name, "sequences_per_gpu": wl.B,
           "value_is": "rows read by adasd_verify / adasd_verify time (mean of the timed launches)"}
    cfg.update(extra_cfg)
    return {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None,
            "dtype": "f32 (bf16 logits, fp32 arithmetic)" if wl.dtype == synth.BF16 else "f32",
            "data": "synthetic", "config": cfg, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": "adasd_verify", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "algorithmic_bytes_per_launch": verify_bytes, "ms_per_launch": verify_ms,
                         "traffic": None,
                         "note": "latency-bound launch: a few rows per call" if wl.B == 1 else
                                 "windows vary from round to round: bytes are the mean over the timed rounds"}}


def graph_of(torch, fn, stream):
    """Captures fn() once on `stream` (after one eager pass) and returns the CUDA graph."""
    with torch.cuda.stream(stream):
        fn()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            fn()
    torch.cuda.synchronize()
    return g


def time_replays(torch, g, n, stream) -> float:
    """Milliseconds per replay of a captured graph (n replays between two events)."""
    with torch.cuda.stream(stream):
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            g.replay()
        e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n


def run_single_stream(args, torch, adasd, wl, rank, world, local, dev, dist) -> dict:
    """C1 / C2: one sequence; a round is K draft calls on [1,V] and one verify call.  The calls are
    latency bound, so they are timed as replays of CUDA graphs (issued one by one from Python the
    interpreter's ~14 us per call would be the measurement): a graph of the K draft calls, a graph
    of the verify call, and a graph of the whole round.  Several input sets are cycled."""
    wl = rank_workload(wl, rank, args.sets)
    B, K, V = wl.B, wl.K, wl.V
    tdt = torch.bfloat16 if wl.dtype == synth.BF16 else torch.float32
    nset = max(args.sets, 2)
    ctx = adasd.Context(B, V, K, dtype=wl.dtype, list_capacity=1 << 16, device=local)
    gs = synth.GpuSynth(wl, str(dev))
    f32, i32 = dict(dtype=torch.float32, device=dev), dict(dtype=torch.int32, device=dev)
    zd = [torch.empty((B, K, V), dtype=tdt, device=dev) for _ in range(nset)]
    zt = [torch.empty((B, K + 1, V), dtype=tdt, device=dev) for _ in range(nset)]
    U = [gs.new_round_uniforms() for _ in range(nset)]
    ud = [torch.empty((K, B), **f32) for _ in range(nset)]
    for s in range(nset):
        gs.draft_rows(s, zd[s])
        gs.target_rows(s, zt[s])
        gs.round_uniforms(s, U[s])
        ud[s].copy_(U[s]["draft"].T)
    Hk, tokk = torch.zeros((K, B), **f32), torch.zeros((K, B), **i32)
    stopk = torch.zeros((K, B), dtype=torch.uint8, device=dev)
    active = torch.ones(B, dtype=torch.uint8, device=dev)
    dlen, x = torch.zeros(B, **i32), torch.zeros((B, K), **i32)
    al, nt = torch.zeros(B, **i32), torch.zeros(B, **i32)
    adaptive = wl.adaptive_window

    def drafts():
        for s in range(nset):
            dlen.zero_()
            active.fill_(1)
            for k in range(K):
                ctx.draft_entropy(zd[s][:, k, :], Hk[k], u=ud[s][k], token_out=tokk[k],
                                  active=active if adaptive else None, stop_out=stopk[k],
                                  draft_len=dlen, row_stride=K * V)

    def verifies():
        for s in range(nset):
            ctx.verify(zd[s], zt[s], x, U[s]["target"], U[s]["accept"], al, nt,
                       draft_len=None, fuse_update=True)

    def rounds():
        for s in range(nset):
            dlen.zero_()
            active.fill_(1)
            for k in range(K):
                ctx.draft_entropy(zd[s][:, k, :], Hk[k], u=ud[s][k], token_out=tokk[k],
                                  active=active if adaptive else None, stop_out=stopk[k],
                                  draft_len=dlen, row_stride=K * V)
            x.copy_(tokk.T)
            ctx.verify(zd[s], zt[s], x, U[s]["target"], U[s]["accept"], al, nt,
                       draft_len=dlen if adaptive else None, fuse_update=True)

    side = torch.cuda.Stream()
    g_d, g_v, g_r = (graph_of(torch, f, side) for f in (drafts, verifies, rounds))
    reps = max(args.steps, 20)
    for g in (g_d, g_v, g_r):
        time_replays(torch, g, max(args.warmup, 3), side)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms_d = time_replays(torch, g_d, reps, side) / nset
    ms_v = time_replays(torch, g_v, reps, side) / nset
    ms_r = time_replays(torch, g_r, reps, side) / nset
    clocks = sampler.stop() if rank == 0 else None
    if ctx.status() != 0:
        raise RuntimeError("device status word set after the timed region")

    # end to end: one round's logits from pinned host memory, verify through the C ABI, results back
    hd, ht = zd[0].cpu().pin_memory(), zt[0].cpu().pin_memory()
    h_out = torch.empty((2, B), dtype=torch.int32).pin_memory()
    d_out = torch.empty((2, B), **i32)

    def e2e_step():
        zd[0].copy_(hd, non_blocking=True)
        zt[0].copy_(ht, non_blocking=True)
        ctx.verify(zd[0], zt[0], x, U[0]["target"], U[0]["accept"], al, nt, fuse_update=True)
        d_out[0].copy_(al)
        d_out[1].copy_(nt)
        h_out.copy_(d_out, non_blocking=True)

    e2e_step()
    torch.cuda.synchronize()
    n_e2e = 20
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n_e2e):
        e2e_step()
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1) / n_e2e
    ms_r, ms_v, e2e_ms = max_over_ranks([ms_r, ms_v, e2e_ms], dist, dev)

    vrows = B * (2 * K + 1)
    extra = {"rows_per_round": {"draft": B * K, "verify": vrows},
             "timing": f"CUDA-graph replays, {nset} input sets per graph, {reps} replays",
             "us_per_draft_call": 1e3 * ms_d / K, "us_per_verify_call": 1e3 * ms_v,
             "us_per_round": 1e3 * ms_r, "rounds_per_s": world * 1e3 / ms_r,
             "l2": "single-stream rows (1.4-6.4 MB a round) fit in L2; the calls are launch-latency bound"}
    e2e = {"value": world * vrows / (e2e_ms * 1e-3), "unit": UNIT,
           "h2d_bytes_per_step": (hd.numel() + ht.numel()) * hd.element_size(), "d2h_bytes_per_step": h_out.numel() * 4,
           "steps": n_e2e, "ms_per_step": e2e_ms,
           "what": "pinned host logits -> device, adasd_verify through the C ABI, results -> host"}
    out = common_fields(args, world, wl, f"{args.workload}: B={B} K={K} V={V} single stream, graph replays", extra,
                        world * vrows / (ms_v * 1e-3), ms_r, ms_v, vrows, reps * nset * (K + 2), clocks, e2e)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = oracle_sample(synth.WORKLOADS[args.workload], args.cpu_seconds, max_rounds=64)
    if dist is not None:
        dist.destroy_process_group()
    return out if rank == 0 else None


def run_adaptive_graph(args, torch, adasd, wl, rank, world, local, dev, dist) -> dict:
    """C5: the whole adaptive round captured once in a CUDA graph (inputs of the round the device
    counter names, K draft steps with the device-side active mask, verification with the fused
    threshold update) and replayed for every round of the workload; the same with the generator
    alone, so that the library's share of a round is visible.  Per-call verify times come from an
    eager pass over a sample of rounds (CUDA events around each verify launch)."""
    R = args.rounds if args.rounds > 0 else wl.rounds
    wl = wl.scaled(seed=wl.seed + 1000 * rank)
    B, K, V = wl.B, wl.K, wl.V

    def build():
        ctx = adasd.Context(B, V, K, dtype=wl.dtype, list_capacity=R * K + 64, device=local)
        gs = synth.GpuSynth(wl, str(dev))
        f32, i32 = dict(dtype=torch.float32, device=dev), dict(dtype=torch.int32, device=dev)
        t = dict(ctx=ctx, gs=gs,
                 zd=torch.empty((B, K, V), dtype=torch.bfloat16, device=dev),
                 zt=torch.empty((B, K + 1, V), dtype=torch.bfloat16, device=dev),
                 U=gs.new_round_uniforms(), ud=torch.empty((K, B), **f32),
                 Hk=torch.zeros((K, B), **f32), tokk=torch.zeros((K, B), **i32),
                 stopk=torch.zeros((K, B), dtype=torch.uint8, device=dev),
                 active=torch.ones(B, dtype=torch.uint8, device=dev), dlen=torch.zeros(B, **i32),
                 x=torch.zeros((B, K), **i32), al=torch.zeros(B, **i32), nt=torch.zeros(B, **i32),
                 acc=torch.zeros((2, B), dtype=torch.int64, device=dev), ev=[])
        return t

    def generate(t):
        t["gs"].draft_rows(0, t["zd"], use_round_dev=True)
        t["gs"].target_rows(0, t["zt"], use_round_dev=True)
        t["gs"].round_uniforms(0, t["U"], use_round_dev=True)
        t["ud"].copy_(t["U"]["draft"].T)

    def library(t, timed=False):
        t["dlen"].zero_()
        t["active"].fill_(1)
        for k in range(K):
            t["ctx"].draft_entropy(t["zd"][:, k, :], t["Hk"][k], u=t["ud"][k], token_out=t["tokk"][k],
                                   active=t["active"], stop_out=t["stopk"][k], draft_len=t["dlen"],
                                   row_stride=K * V)
        t["x"].copy_(t["tokk"].T)
        if timed:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        t["ctx"].verify(t["zd"], t["zt"], t["x"], t["U"]["target"], t["U"]["accept"], t["al"], t["nt"],
                        draft_len=t["dlen"], fuse_update=True)
        if timed:
            e1.record()
            t["ev"].append((e0, e1))
        t["acc"][0] += t["dlen"]
        t["acc"][1] += t["al"]

    # eager sample: per-launch verify time and the rows it read (windows vary)
    t = build()
    sample = min(R, 64)
    for _ in range(sample):
        generate(t)
        library(t, timed=True)
        t["gs"].advance_round(1)
    torch.cuda.synchronize()
    verify_ms = statistics.mean(a.elapsed_time(b) for a, b in t["ev"][3:])
    mean_kt_sample = float(t["acc"][0].sum()) / (sample * B)
    t["ctx"].close()

    # the whole round in one graph, replayed R times
    t = build()
    side = torch.cuda.Stream()

    def whole():
        generate(t)
        library(t)
        t["gs"].advance_round(1)

    def gen_only():
        generate(t)
        t["gs"].advance_round(1)

    g = graph_of(torch, whole, side)
    t["ctx"].reset()
    t["gs"].round_dev.zero_()
    t["acc"].zero_()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms_round = time_replays(torch, g, R, side)
    clocks = sampler.stop() if rank == 0 else None
    status = t["ctx"].status()
    if status != 0:
        raise RuntimeError(f"device status word {status} after the replays")
    mean_kt = float(t["acc"][0].sum()) / (R * B)
    mean_acc = float(t["acc"][1].sum()) / (R * B)
    T, nE, nA, nR = t["ctx"].get_thresholds()
    torch.cuda.synchronize()
    g2 = graph_of(torch, gen_only, side)
    t["gs"].round_dev.zero_()
    ms_gen = time_replays(torch, g2, R, side)
    def drafts():
        for k in range(K):
            t["ctx"].draft_entropy(t["zd"][:, k, :], t["Hk"][k], u=t["ud"][k], token_out=t["tokk"][k],
                                   stop_out=t["stopk"][k], draft_len=t["dlen"], row_stride=K * V)
    g3 = graph_of(torch, drafts, side)
    time_replays(torch, g3, 3, side)
    draft_ms = time_replays(torch, g3, 20, side) / K
    ms_round, ms_gen, verify_ms, draft_ms = max_over_ranks([ms_round, ms_gen, verify_ms, draft_ms], dist, dev)

    # end to end: one round's logits from pinned host memory
    hd, ht = t["zd"].cpu().pin_memory(), t["zt"].cpu().pin_memory()
    h_out = torch.empty((2, B), dtype=torch.int32).pin_memory()
    d_out = torch.empty((2, B), dtype=torch.int32, device=dev)

    def e2e_step():
        t["zd"].copy_(hd, non_blocking=True)
        t["zt"].copy_(ht, non_blocking=True)
        t["ctx"].verify(t["zd"], t["zt"], t["x"], t["U"]["target"], t["U"]["accept"], t["al"], t["nt"],
                        draft_len=t["dlen"], fuse_update=True)
        d_out[0].copy_(t["al"])
        d_out[1].copy_(t["nt"])
        h_out.copy_(d_out, non_blocking=True)

    e2e_step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(3):
        e2e_step()
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1) / 3
    last_rows = float((2 * t["dlen"] + 1).sum())

    vrows = B * (2 * mean_kt_sample + 1)
    extra = {"rounds": R, "rounds_per_s": world * 1e3 / ms_round, "ms_per_round": ms_round,
             "generator_only_rounds_per_s": world * 1e3 / ms_gen, "generator_only_ms_per_round": ms_gen,
             "library_ms_per_round": ms_round - ms_gen,
             "mean_window": mean_kt, "mean_accept_len": mean_acc,
             "draft_entropy": {"us_per_call": 1e3 * draft_ms, "bytes_per_call": B * wl.row_bytes,
                               "gbs": B * wl.row_bytes / (draft_ms * 1e-3) / 1e9,
                               "frac_of_peak": B * wl.row_bytes / (draft_ms * 1e-3) / 1e9 / measured_peak_gbs()[0],
                               "timing": f"every row active: one CUDA graph of {K} calls, 20 replays"},
             "list_sizes_at_end": {"nE_max": int(nE.max()), "nA_max": int(nA.max()), "nR_max": int(nR.max())},
             "T_G_mean_at_end": float(T.mean()),
             "verify_sample": f"first {sample} rounds issued call by call, mean window {mean_kt_sample:.2f}",
             "l2": f"every round generates {(2 * K + 1) * B * wl.row_bytes / 1e6:.0f} MB of fresh logits (larger than L2)",
             "timing": "one CUDA graph of the whole round (generator, 16 draft steps with the active mask, verify with "
                       "the fused update, round counter), replayed for every round"}
    e2e = {"value": world * last_rows / (e2e_ms * 1e-3), "unit": UNIT,
           "h2d_bytes_per_step": (hd.numel() + ht.numel()) * hd.element_size(), "d2h_bytes_per_step": h_out.numel() * 4,
           "steps": 3, "ms_per_step": e2e_ms,
           "what": "pinned host logits -> device, adasd_verify through the C ABI, results -> host"}
    out = common_fields(args, world, wl, f"C5: B={B} Kmax={K} V={V} adaptive windows, {R} rounds in one replayed graph",
                        extra, world * vrows / (verify_ms * 1e-3), ms_round, verify_ms, vrows, R * (K + 1), clocks, e2e)
    out["steps"] = R
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = oracle_sample(synth.WORKLOADS["C5"], args.cpu_seconds)
    if dist is not None:
        dist.destroy_process_group()
    return out if rank == 0 else None


# ------------------------------------------------------------------------------ oracle arm

def oracle_sample(wl, seconds: float, max_rounds: int = 4) -> dict:
    """The oracle, as it stands, on the metric's own work: the AdaSD verify round (Algorithm 1,
    verification and update) of whole sequences of the workload, round after round, until about
    `seconds` of CPU work are done.  Input generation and the draft tokens are not timed.
    Returns verify rows/s on the host cores."""
    import oracle
    cores = len(os.sched_getaffinity(0))
    K = wl.K
    oracle.lib()
    rows, dt, nseq, rounds = 0, 0.0, 0, 0
    chunk = 16                                     # sequences generated and timed at a time
    states = [oracle.SequenceState(capacity=1 << 15) for _ in range(wl.B)]
    while dt < seconds and rounds < max_rounds:
        U = synth.round_uniforms_cpu(wl, rounds)
        ud, ut, ua = U["draft"], U["target"], U["accept"]
        for b0 in range(0, wl.B, chunk):
            bl = np.arange(b0, min(b0 + chunk, wl.B), dtype=np.int32)
            hd, ht = synth.host_round(wl, rounds, bl)
            for n, b in enumerate(bl):
                x = [oracle.draft_step(hd[n, k], float(ud[b, k]), 0.0)["token"] for k in range(K)]
                t0 = time.perf_counter()
                oracle.verify_round(states[b], hd[n], ht[n], x, ut[b], ua[b])
                dt += time.perf_counter() - t0
                rows += 2 * K + 1
            nseq += len(bl)
            if dt >= seconds:
                break
        rounds += 1
    return {"value": rows / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"verify rounds of {nseq} sequence-rounds of the workload ({rows} rows, {dt:.1f} s of oracle "
                      f"time; input generation and draft tokens excluded); OpenMP over positions inside the round",
            "seconds": dt}


def run_reference(args) -> dict:
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return None
    wl = synth.WORKLOADS[args.workload]
    K = wl.K
    rows = step_rows(wl)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(wl, 0.5, 1)
    total_rows, secs = 0, 0.0
    steps = max(1, min(args.steps, 6))
    for _ in range(steps):
        s = oracle_sample(wl, 4.0, 1)
        total_rows += s["value"] * s["seconds"]
        secs += s["seconds"]
    value = total_rows / secs
    cores = len(os.sched_getaffinity(0))
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": secs / steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": f"{args.workload}: B={wl.B} K={K} V={wl.V}; each step is a bounded "
                                   f"sample: about 4 s of oracle verify rounds on sequences of round 0 "
                                   f"({2 * K + 1} rows per sequence of the {rows['verify']} one adasd_verify call reads)"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "about 4 s of oracle time per step, sequences of round 0"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C4", choices=["C1", "C2", "C3", "C4", "C5"])
    ap.add_argument("--prefill", type=int, default=0,
                    help="entries imported into both KDE lists of every sequence before timing (C3, C4)")
    ap.add_argument("--warpers", default="", help="C3/C4: temperature,top_k,top_p of the adjusted distribution, e.g. 0.8,50,0.95")
    ap.add_argument("--rounds", type=int, default=0, help="C5: rounds replayed (0 = all 1024)")
    ap.add_argument("--sets", type=int, default=4, help="input sets resident in HBM")
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="oracle time in the cpu_baseline sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.warpers:
        t, k, p_ = args.warpers.split(",")
        args.warpers = (float(t), int(k), float(p_))
        if args.workload not in ("C3", "C4"):
            ap.error("--warpers applies to the fixed-window workloads C3 and C4")
    out = run_reference(args) if args.impl == "reference" else run_ours(args)
    if out is not None:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
