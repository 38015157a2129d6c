"""Seeded synthetic inputs for the AdaSD hot path (input generation only).

This package feeds the same seeded logits and uniforms to the CUDA library and to
the CPU oracle.  It contains none of the method's arithmetic: no softmax, entropy,
divergence, sampling or threshold logic.  The recipe is the Zipf-offset Gaussian
generator ``z_d = s * N(0,1) - ln(rank_v)``, ``z_t = z_d + N(0, tau^2)``; the
Gaussian is a 65536-entry quantile table indexed by a 64-bit integer mix, and every
fp32 operation is rounded on its own, so host and device rows are bit-identical.

The synthetic rows stand in for real draft/target model logits over the Llama-3
(V=128256) and Qwen-2.5 (V=151936) vocabularies, which are not available offline.
"""
from __future__ import annotations

import ctypes
import functools
import os
import subprocess
from dataclasses import dataclass, replace
from typing import Callable, Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_CPU_SO = os.path.join(_HERE, "libsynth_cpu.so")
_GPU_SO = os.path.join(_HERE, "libsynth_gpu.so")

BF16, FP32 = 0, 1
GAUSS_N = 1 << 16

# sub-streams of the uniform stream
U_DRAFT, U_TARGET, U_ACCEPT, U_RESAMPLE, U_VANILLA_ACCEPT = 0, 1, 2, 3, 4


def _newer(target: str, *sources: str) -> bool:
    if not os.path.exists(target):
        return False
    t = os.path.getmtime(target)
    return all(os.path.getmtime(s) <= t for s in sources)


def build_cpu(force: bool = False) -> str:
    src = os.path.join(_HERE, "synth_cpu.c")
    hdr = os.path.join(_HERE, "synth_core.h")
    if force or not _newer(_CPU_SO, src, hdr):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
             "-fno-fast-math", "-o", _CPU_SO, src])
    return _CPU_SO


def build_gpu(force: bool = False) -> str:
    src = os.path.join(_HERE, "synth_gpu.cu")
    hdr = os.path.join(_HERE, "synth_core.h")
    if force or not _newer(_GPU_SO, src, hdr):
        subprocess.check_call(
            ["nvcc", "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a",
             "-lineinfo", "-Xcompiler", "-fPIC", "-shared", "--fmad=false", "-o", _GPU_SO, src])
    return _GPU_SO


@functools.lru_cache(maxsize=None)
def _cpu():
    lib = ctypes.CDLL(build_cpu())
    c = ctypes
    lib.synth_permutation_rank.argtypes = [c.c_uint64, c.c_int32, c.c_void_p]
    lib.synth_permutation_rank.restype = None
    lib.synth_rows_cpu.argtypes = [c.c_int32, c.c_uint64, c.c_uint32, c.c_int64, c.c_void_p,
                                   c.c_void_p, c.c_void_p, c.c_void_p, c.c_int32, c.c_void_p,
                                   c.c_void_p, c.c_int32, c.c_void_p, c.c_int64]
    lib.synth_rows_cpu.restype = None
    lib.synth_uniforms_cpu.argtypes = [c.c_uint64, c.c_uint32, c.c_uint32, c.c_int32, c.c_int32,
                                       c.c_void_p]
    lib.synth_uniforms_cpu.restype = None
    lib.synth_param_bits.argtypes = [c.c_uint64, c.c_uint32, c.c_int32, c.c_int32, c.c_uint32,
                                     c.c_void_p]
    lib.synth_param_bits.restype = None
    return lib


@functools.lru_cache(maxsize=None)
def _gpu():
    lib = ctypes.CDLL(build_gpu())
    c = ctypes
    lib.synth_rows_gpu.argtypes = [c.c_int32, c.c_uint64, c.c_uint32, c.c_void_p, c.c_int32,
                                   c.c_int32, c.c_int32, c.c_void_p, c.c_void_p, c.c_int64,
                                   c.c_int32, c.c_int32, c.c_void_p, c.c_void_p, c.c_int32,
                                   c.c_void_p, c.c_int64, c.c_int64, c.c_void_p]
    lib.synth_rows_gpu.restype = c.c_int
    lib.synth_uniforms_gpu.argtypes = [c.c_uint64, c.c_uint32, c.c_uint32, c.c_void_p, c.c_int32,
                                       c.c_int32, c.c_void_p, c.c_void_p]
    lib.synth_uniforms_gpu.restype = c.c_int
    lib.synth_counter_add_gpu.argtypes = [c.c_void_p, c.c_uint32, c.c_void_p]
    lib.synth_counter_add_gpu.restype = c.c_int
    return lib


# ----------------------------------------------------------------------------- tables

@functools.lru_cache(maxsize=8)
def gauss_table() -> np.ndarray:
    """fp32 standard-normal quantiles at (j + 1/2) / 65536."""
    from scipy.special import ndtri
    q = (np.arange(GAUSS_N, dtype=np.float64) + 0.5) / GAUSS_N
    return np.ascontiguousarray(ndtri(q).astype(np.float32))


@functools.lru_cache(maxsize=8)
def rank_table(seed: int, V: int) -> np.ndarray:
    """rank[v] in 1..V: seeded permutation of the vocabulary's Zipf ranks."""
    out = np.empty(V, dtype=np.int32)
    _cpu().synth_permutation_rank(seed, V, out.ctypes.data)
    return out


@functools.lru_cache(maxsize=8)
def lnrank_table(seed: int, V: int) -> np.ndarray:
    return np.ascontiguousarray(np.log(rank_table(seed, V).astype(np.float64)).astype(np.float32))


# ----------------------------------------------------------------------------- host generator

def param_uniform(seed: int, round_: int, B: int, K: int, j: int) -> np.ndarray:
    """[B,K] float64 uniforms in [0,1) for parameter draw number j of a round."""
    bits = np.empty((B, K), dtype=np.uint64)
    _cpu().synth_param_bits(seed, round_, B, K, j, bits.ctypes.data)
    return (bits >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def rows_cpu(kind: int, seed: int, round_: int, b: np.ndarray, k: np.ndarray, s: np.ndarray,
             tau: Optional[np.ndarray], V: int, dtype: int) -> np.ndarray:
    """Rows (b[r], k[r]) of a round: uint16 bf16 bits or float32, shape [n, V]."""
    b = np.ascontiguousarray(b, dtype=np.int32)
    k = np.ascontiguousarray(k, dtype=np.int32)
    s = np.ascontiguousarray(s, dtype=np.float32)
    n = b.shape[0]
    out = np.empty((n, V), dtype=np.uint16 if dtype == BF16 else np.float32)
    tau_p = None
    if tau is not None:
        tau = np.ascontiguousarray(tau, dtype=np.float32)
        tau_p = tau.ctypes.data
    g = gauss_table()
    ln = lnrank_table(seed, V)
    _cpu().synth_rows_cpu(kind, seed, round_, n, b.ctypes.data, k.ctypes.data, s.ctypes.data,
                          tau_p, V, g.ctypes.data, ln.ctypes.data, dtype, out.ctypes.data, V)
    return out


def uniforms_cpu(seed: int, substream: int, round_: int, B: int, n: int) -> np.ndarray:
    out = np.empty((B, n), dtype=np.float32)
    _cpu().synth_uniforms_cpu(seed, substream, round_, B, n, out.ctypes.data)
    return out


def round_uniforms_cpu(wl: "Workload", round_: int) -> dict:
    """All uniforms of one round, float32.

    draft [B,K], target [B,K+1], accept [B,K], vanilla_accept [B,K], resample [B].
    Common random numbers: target[:, i] == draft[:, i] for i < K, so that the draft
    token x_i = invCDF(q_i, u) and the target sample y_i = invCDF(p_i, u) agree when
    p_i and q_i are close - the stand-in for a real draft model agreeing with its
    target.  With independent uniforms two samples from a 128k-token vocabulary
    almost never coincide and every round would end at its first candidate.
    """
    B, K = wl.B, wl.K
    d = uniforms_cpu(wl.seed, U_DRAFT, round_, B, K)
    t = uniforms_cpu(wl.seed, U_TARGET, round_, B, K + 1)
    t[:, :K] = d
    return dict(draft=d, target=t,
                accept=uniforms_cpu(wl.seed, U_ACCEPT, round_, B, K),
                vanilla_accept=uniforms_cpu(wl.seed, U_VANILLA_ACCEPT, round_, B, K),
                resample=uniforms_cpu(wl.seed, U_RESAMPLE, round_, B, 1)[:, 0].copy())


# ----------------------------------------------------------------------------- workloads

@dataclass(frozen=True)
class Workload:
    """One of the five benchmark workloads (or a scaled-down copy for tests)."""
    name: str
    seed: int
    B: int
    K: int            # window: draft positions per round (Kmax when adaptive)
    V: int
    dtype: int
    rounds: int
    adaptive_window: bool   # True: the entropy stop check sets K_t <= K each round
    vanilla: bool           # also run the vanilla comparison mode on the same inputs
    recipe: str
    tau0: float = 0.0       # recipe "fixed_tau": the target noise of every position

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)

    def params(self, round_: int) -> Tuple[np.ndarray, np.ndarray]:
        """(s, tau) as float32 [B, K+1] for one round (position K is the bonus row)."""
        B, K1 = self.B, self.K + 1
        if self.recipe == "cycle":
            s = np.array([0.5, 2.0, 6.0], dtype=np.float64)[np.arange(K1) % 3]
            t = np.array([0.1, 1.0, 3.0], dtype=np.float64)[np.arange(K1) % 3]
            s = np.broadcast_to(s, (B, K1))
            t = np.broadcast_to(t, (B, K1))
        elif self.recipe == "uniform":
            s = 0.5 + 5.5 * param_uniform(self.seed, round_, B, K1, 0)
            t = 0.1 + 2.9 * param_uniform(self.seed, round_, B, K1, 1)
        elif self.recipe == "peaked_mixture":
            sel = param_uniform(self.seed, round_, B, K1, 0)
            mid = 1.0 + 3.0 * param_uniform(self.seed, round_, B, K1, 1)
            s = np.where(sel < 0.1, 12.0, np.where(sel < 0.2, 0.2, mid))
            t = 0.05 + 3.95 * param_uniform(self.seed, round_, B, K1, 2)
        elif self.recipe == "fixed_tau":
            # nearly equal draft and target rows: the small-distance regime
            s = 0.5 + 5.5 * param_uniform(self.seed, round_, B, K1, 0)
            t = np.full((B, K1), self.tau0)
        elif self.recipe == "drift":
            s = 0.5 + 5.5 * param_uniform(self.seed, round_, B, K1, 0)
            frac = round_ / max(self.rounds - 1, 1)
            t = np.full((B, K1), 0.2 + 2.8 * frac)
        else:
            raise ValueError(self.recipe)
        return (np.ascontiguousarray(s, dtype=np.float32),
                np.ascontiguousarray(t, dtype=np.float32))

    def all_params(self) -> Tuple[np.ndarray, np.ndarray]:
        """(s, tau) float32 [rounds, B, K+1] for the whole run."""
        ss, tt = zip(*(self.params(r) for r in range(self.rounds)))
        return np.stack(ss), np.stack(tt)

    @property
    def row_bytes(self) -> int:
        return self.V * (2 if self.dtype == BF16 else 4)


WORKLOADS = {
    "C1": Workload("C1", 0, 1, 5, 32000, FP32, 20, False, False, "cycle"),
    "C2": Workload("C2", 1, 1, 8, 128256, BF16, 512, True, False, "uniform"),
    "C3": Workload("C3", 2, 32, 8, 128256, BF16, 256, False, True, "uniform"),
    "C4": Workload("C4", 3, 128, 16, 151936, BF16, 128, False, False, "peaked_mixture"),
    "C5": Workload("C5", 4, 256, 16, 128256, BF16, 1024, True, False, "drift"),
}


# ----------------------------------------------------------------------------- device generator

class GpuSynth:
    """Device-side generator for one workload: tables and parameters live in HBM."""

    def __init__(self, wl: Workload, device: str = "cuda:0"):
        import torch
        self.torch = torch
        self.wl = wl
        self.lib = _gpu()
        self.device = torch.device(device)
        self.gauss = torch.from_numpy(gauss_table()).to(self.device)
        self.lnrank = torch.from_numpy(lnrank_table(wl.seed, wl.V)).to(self.device)
        s, t = wl.all_params()
        self.s = torch.from_numpy(s).to(self.device)
        self.tau = torch.from_numpy(t).to(self.device)
        self.round_dev = torch.zeros(1, dtype=torch.int32, device=self.device)

    def _stream(self):
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def rows(self, kind: int, round_: int, out, k0: int, K: int, seq_stride: int,
             row_stride: int, use_round_dev: bool = False, B: Optional[int] = None) -> None:
        wl = self.wl
        rc = self.lib.synth_rows_gpu(
            kind, wl.seed, round_, self.round_dev.data_ptr() if use_round_dev else None,
            wl.B if B is None else B, K, k0, self.s.data_ptr(), self.tau.data_ptr(),
            wl.B * (wl.K + 1), wl.K + 1, wl.V, self.gauss.data_ptr(), self.lnrank.data_ptr(),
            wl.dtype, out.data_ptr(), seq_stride, row_stride, self._stream())
        if rc != 0:
            raise RuntimeError(f"synth_rows_gpu failed with CUDA error {rc}")

    def draft_rows(self, round_: int, out, use_round_dev: bool = False) -> None:
        """out: [B, K, V] draft logits of a round."""
        wl = self.wl
        self.rows(0, round_, out, 0, wl.K, wl.K * wl.V, wl.V, use_round_dev)

    def target_rows(self, round_: int, out, use_round_dev: bool = False) -> None:
        """out: [B, K+1, V] target logits of a round."""
        wl = self.wl
        self.rows(1, round_, out, 0, wl.K + 1, (wl.K + 1) * wl.V, wl.V, use_round_dev)

    def uniforms(self, substream: int, round_: int, out, use_round_dev: bool = False) -> None:
        """out: [B, n] float32 uniforms of a round."""
        B, n = out.shape
        rc = self.lib.synth_uniforms_gpu(
            self.wl.seed, substream, round_,
            self.round_dev.data_ptr() if use_round_dev else None, B, n, out.data_ptr(),
            self._stream())
        if rc != 0:
            raise RuntimeError(f"synth_uniforms_gpu failed with CUDA error {rc}")

    def round_uniforms(self, round_: int, out: dict, use_round_dev: bool = False) -> None:
        """Device twin of round_uniforms_cpu: fills out['draft'|'target'|'accept'|
        'vanilla_accept'|'resample'] (float32 tensors of the shapes given there)."""
        K = self.wl.K
        self.uniforms(U_DRAFT, round_, out["draft"], use_round_dev)
        self.uniforms(U_TARGET, round_, out["target"], use_round_dev)
        out["target"][:, :K].copy_(out["draft"])
        self.uniforms(U_ACCEPT, round_, out["accept"], use_round_dev)
        self.uniforms(U_VANILLA_ACCEPT, round_, out["vanilla_accept"], use_round_dev)
        self.uniforms(U_RESAMPLE, round_, out["resample"].view(-1, 1), use_round_dev)

    def new_round_uniforms(self) -> dict:
        t, B, K = self.torch, self.wl.B, self.wl.K
        f = dict(dtype=t.float32, device=self.device)
        return dict(draft=t.empty((B, K), **f), target=t.empty((B, K + 1), **f),
                    accept=t.empty((B, K), **f), vanilla_accept=t.empty((B, K), **f),
                    resample=t.empty(B, **f))

    def advance_round(self, inc: int = 1) -> None:
        rc = self.lib.synth_counter_add_gpu(self.round_dev.data_ptr(), inc, self._stream())
        if rc != 0:
            raise RuntimeError(f"synth_counter_add_gpu failed with CUDA error {rc}")


def host_round(wl: Workload, round_: int, b_list=None):
    """Host rows of one round for the sequences in b_list (default: all).

    Returns (draft [n,K,V], target [n,K+1,V]) as uint16 bf16 bits or float32.
    """
    if b_list is None:
        b_list = np.arange(wl.B)
    b_list = np.asarray(b_list, dtype=np.int32)
    s, t = wl.params(round_)
    n, K = len(b_list), wl.K
    bd = np.repeat(b_list, K)
    kd = np.tile(np.arange(K, dtype=np.int32), n)
    d = rows_cpu(0, wl.seed, round_, bd, kd, s[bd, kd], None, wl.V, wl.dtype).reshape(n, K, wl.V)
    bt = np.repeat(b_list, K + 1)
    kt = np.tile(np.arange(K + 1, dtype=np.int32), n)
    tg = rows_cpu(1, wl.seed, round_, bt, kt, s[bt, kt], t[bt, kt], wl.V, wl.dtype)
    return d, tg.reshape(n, K + 1, wl.V)
