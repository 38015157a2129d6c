#!/usr/bin/env python
"""Benchmark of the AdaSD hot path on B200.

One step = one decode round of the workload, i.e. one pass of the whole hot path:
K draft steps (adasd_draft_entropy on [B,V]), one adasd_verify with the fused
threshold update, and one adasd_vanilla_verify on the same inputs.  The metric is
logit rows read per second (a row = one length-V logit row) with the inputs already
resident in HBM; the `e2e` figure pushes the same step through the C ABI from pinned
host buffers, copies included.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C4] [--impl reference]

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
# byte, from the ncu capture of workload C3 summarised under profiles/ (143.91 MB against
# 139.54 MB); traffic grows in proportion to the rows read, so other workloads scale by it.
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.031


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
    if wl.adaptive_window:
        raise SystemExit("bench.py times the fixed-window workloads (C3, C4)")
    # every rank owns its own sequences: same shapes, different seed
    wl = rank_workload(wl, rank, args.sets)
    B, K, V = wl.B, wl.K, wl.V
    tdt = torch.bfloat16 if wl.dtype == synth.BF16 else torch.float32
    ctx = adasd.Context(B, V, K, dtype=wl.dtype, list_capacity=(args.steps + args.warmup + 64) * K + 64,
                        device=local)
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
    h_out = torch.empty((4, B), dtype=torch.int32).pin_memory()
    d_out = torch.empty((4, B), **i32)
    zd_e = torch.empty_like(zd[0])
    zt_e = torch.empty_like(zt[0])

    def e2e_step():
        zd_e.copy_(hd, non_blocking=True)
        zt_e.copy_(ht, non_blocking=True)
        step(0, zd_s=zd_e, zt_s=zt_e)
        d_out[0].copy_(al)
        d_out[1].copy_(nt)
        d_out[2].copy_(val)
        d_out[3].copy_(vnt)
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

    ms, e2e_ms = max_over_ranks([ms, e2e_ms], dist, dev)

    rows = step_rows(wl)
    rows_step = sum(rows.values())
    row_bytes = wl.row_bytes
    peak, peak_kind = measured_peak_gbs()
    verify_bytes = rows["verify"] * row_bytes
    achieved = verify_bytes / (verify_ms * 1e-3) / 1e9
    h2d = (hd.numel() + ht.numel()) * hd.element_size()
    out = {
        "metric": METRIC, "value": whole_job_rate(world, rows_step, args.steps, ms), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 (bf16 logits, fp32 arithmetic)" if wl.dtype == synth.BF16 else "f32",
        "data": "synthetic",
        "config": {"workload": f"{args.workload}: B={B} K={K} V={V} {'bf16' if wl.dtype == synth.BF16 else 'fp32'} "
                               f"fixed window, per step {K} draft_entropy + verify(fused update) + vanilla_verify",
                   "rows_per_step": rows, "bytes_per_step": rows_step * row_bytes,
                   "sequences_per_gpu": B, "input_sets": nset,
                   "l2": f"inputs larger than L2: {nset} sets of {(2 * K + 1) * B * row_bytes / 1e6:.0f} MB cycled",
                   "hbm_gbs_all_calls": world * rows_step * row_bytes * args.steps / (ms * 1e-3) / 1e9},
        "e2e": {"value": whole_job_rate(world, rows_step, e2e_steps, e2e_ms), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": h_out.numel() * 4,
                "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps},
        "gpu_launches": args.steps * (K + 1 + vanilla_launches(wl, torch.cuda.get_device_properties(dev).multi_processor_count)),
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


# ------------------------------------------------------------------------------ oracle arm

def oracle_sample(wl, seconds: float, max_rounds: int = 4) -> dict:
    """The oracle, as it stands, on whole rounds of the workload (every sequence: K draft
    steps, the AdaSD verify round and the vanilla round) until about `seconds` of CPU work
    are done.  Input generation is not timed.  Returns rows/s on the host cores."""
    import oracle
    cores = len(os.sched_getaffinity(0))
    K = wl.K
    oracle.lib()
    rows, dt, nseq, rounds = 0, 0.0, 0, 0
    chunk = 16                                     # sequences generated and timed at a time
    states = [oracle.SequenceState(capacity=4096) for _ in range(wl.B)]
    while dt < seconds and rounds < max_rounds:
        U = synth.round_uniforms_cpu(wl, rounds)
        ud, ut, ua = U["draft"], U["target"], U["accept"]
        for b0 in range(0, wl.B, chunk):
            bl = np.arange(b0, min(b0 + chunk, wl.B), dtype=np.int32)
            hd, ht = synth.host_round(wl, rounds, bl)
            t0 = time.perf_counter()
            for n, b in enumerate(bl):
                x = [oracle.draft_step(hd[n, k], float(ud[b, k]), 0.0)["token"] for k in range(K)]
                oracle.verify_round(states[b], hd[n], ht[n], x, ut[b], ua[b])
                oracle.vanilla_round(hd[n], ht[n], x, U["vanilla_accept"][b], float(U["resample"][b]))
                rows += K + 2 * (2 * K + 1)
            dt += time.perf_counter() - t0
            nseq += len(bl)
            if dt >= seconds:
                break
        rounds += 1
    return {"value": rows / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{nseq} sequence-rounds of the workload ({rows} rows, {dt:.1f} s of oracle time, "
                      f"input generation excluded); OpenMP over positions inside the verify round",
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
                                   f"sample: about 4 s of oracle time on sequences of round 0 "
                                   f"({K + 2 * (2 * K + 1)} rows per sequence of the {sum(rows.values())} a full step reads)"},
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
    ap.add_argument("--workload", default="C4", choices=["C3", "C4"])
    ap.add_argument("--sets", type=int, default=4, help="input sets resident in HBM")
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="oracle time in the cpu_baseline sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    out = run_reference(args) if args.impl == "reference" else run_ours(args)
    if out is not None:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
