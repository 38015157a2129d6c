"""The N > 1 path of bench.py on CPU: two gloo ranks.

The hot path shards over sequences with no exchange step, so what N ranks share is host
logic only: which batch a rank owns, the max-over-ranks timing and the whole-job rate.
Rank 0 alone reports.
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
import synth  # noqa: E402


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        base = synth.WORKLOADS["C3"].scaled(name="mr", B=3, K=2, V=64, rounds=4)
        wl = bench.rank_workload(base, rank, sets=2)
        zd, zt = synth.host_round(wl, 0)[:2]
        # every rank times its own steps; the job takes as long as its slowest rank
        my_ms, my_e2e = 10.0 * (rank + 1), 100.0 / (rank + 1)
        dist.barrier()
        ms, e2e = bench.max_over_ranks([my_ms, my_e2e], dist, torch.device("cpu"))
        rows_step = sum(bench.step_rows(wl).values())
        value = bench.whole_job_rate(world, rows_step, 5, ms)
        np.savez(os.path.join(out_dir, f"r{rank}.npz"), zd=np.asarray(zd), zt=np.asarray(zt), ms=ms, e2e=e2e,
                 value=value, rows_step=rows_step, seed=wl.seed, shape=np.array([wl.B, wl.K, wl.V]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_own_their_batches_and_agree_on_the_job_rate(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [np.load(tmp_path / f"r{k}.npz") for k in range(world)]
    # same shapes, different seeds, different logits: nothing is shared, nothing is split
    assert (r[0]["shape"] == r[1]["shape"]).all() and int(r[0]["seed"]) != int(r[1]["seed"])
    assert r[0]["zd"].shape == r[1]["zd"].shape and not np.array_equal(r[0]["zd"], r[1]["zd"])
    assert not np.array_equal(r[0]["zt"], r[1]["zt"])
    # the maximum over ranks, element by element, seen by both
    for k in range(world):
        assert float(r[k]["ms"]) == 20.0 and float(r[k]["e2e"]) == 100.0
    # whole-job rate: the rows of both ranks over the slowest rank's time
    rows_step = int(r[0]["rows_step"])
    assert rows_step == 3 * 2 + 2 * 3 * (2 * 2 + 1)
    assert float(r[0]["value"]) == pytest.approx(2 * rows_step * 5 / 20e-3)
    assert float(r[0]["value"]) == float(r[1]["value"])


def test_single_rank_needs_no_process_group():
    assert bench.max_over_ranks([1.5, 2.5], None, torch.device("cpu")) == [1.5, 2.5]
    assert bench.whole_job_rate(1, 100, 4, 2.0) == pytest.approx(200000.0)


def test_reference_arm_leaves_other_ranks_idle(monkeypatch):
    # under torchrun the oracle arm runs on rank 0 only; the others return at once
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")

    class A:
        workload, steps, warmup = "C3", 1, 0
    assert bench.run_reference(A()) is None
