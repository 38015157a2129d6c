"""ctypes front end of the float64 CPU oracle (``adasd_oracle.c``).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU-baseline leg
may import this; the product package never does.  The arithmetic lives in the C file,
one function per definition of the paper; this module only marshals numpy arrays and
keeps the three lists of Algorithm 1 for one sequence.
"""
from __future__ import annotations

import ctypes as C
import functools
import math
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libadasd_oracle.so")
_SRC = os.path.join(_HERE, "adasd_oracle.c")

BF16, FP32, F64 = 0, 1, 2
LN2 = math.log(2.0)


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-fno-fast-math", "-o", _SO, _SRC, "-lm"])
    return _SO


_D, _I, _P = C.c_double, C.c_int32, C.c_void_p


@functools.lru_cache(maxsize=None)
def lib():
    L = C.CDLL(build())
    L.oracle_widen.argtypes = [_P, _I, C.c_int64, _P]
    L.oracle_widen.restype = None
    L.oracle_softmax.argtypes = [_P, _I, _P]
    L.oracle_softmax.restype = _D
    for name in ("oracle_entropy",):
        getattr(L, name).argtypes = [_P, _I]
        getattr(L, name).restype = _D
    for name in ("oracle_cross_entropy", "oracle_kl", "oracle_jsd", "oracle_jsd_entropy_form"):
        getattr(L, name).argtypes = [_P, _P, _I]
        getattr(L, name).restype = _D
    L.oracle_js_distance.argtypes = [_D]
    L.oracle_js_distance.restype = _D
    L.oracle_js_distance_rows.argtypes = [_P, _P, _I, _P]
    L.oracle_js_distance_rows.restype = _D
    L.oracle_inv_cdf.argtypes = [_P, _I, _D, _P]
    L.oracle_inv_cdf.restype = _I
    L.oracle_sample_std.argtypes = [_P, _I]
    L.oracle_sample_std.restype = _D
    L.oracle_kde_bandwidth.argtypes = [_P, _I, _I]
    L.oracle_kde_bandwidth.restype = _D
    L.oracle_kde.argtypes = [_P, _I, _D, _I]
    L.oracle_kde.restype = _D
    L.oracle_accept_prob.argtypes = [_P, _I, _P, _I, _D, _I, _I]
    L.oracle_accept_prob.restype = _D
    L.oracle_draft_step.argtypes = [_P, _I, _I, _D, _D, _P, _P, _P, _P, _P]
    L.oracle_draft_step.restype = None
    L.oracle_verify_round.argtypes = [_P, _P, _I, _I, C.c_int64, C.c_int64, _I, _P, _P, _P,
                                      _P, _P, _P, _P, _P, _P, _P, _I, _I, _I, _I,
                                      _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P]
    L.oracle_verify_round.restype = None
    L.oracle_vanilla_round.argtypes = [_P, _P, _I, _I, C.c_int64, C.c_int64, _I, _P, _P, _D,
                                       _P, _P, _P, _P]
    L.oracle_vanilla_round.restype = None
    L.oracle_argmax.argtypes = [_P, _I, _I]
    L.oracle_argmax.restype = _I
    L.oracle_greedy_round.argtypes = [_P, _I, _I, C.c_int64, _I, _P, _P, _P, _P]
    L.oracle_greedy_round.restype = None
    L.oracle_gen_only_update.argtypes = [_P, _P, _P, _P, _I, _I]
    L.oracle_gen_only_update.restype = None
    L.oracle_warp_logits.argtypes = [_P, _I, _D, _I, _D, _D, _P, _P, _P]
    L.oracle_warp_logits.restype = None
    return L


def set_threads(n: int) -> None:
    """OpenMP threads the CALLING thread's oracle calls use from now on (the verify round
    runs its positions in parallel); lets a harness run several sequences side by side."""
    L = lib()
    L.omp_set_num_threads.argtypes = [C.c_int]
    L.omp_set_num_threads.restype = None
    L.omp_set_num_threads(max(1, int(n)))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _raw(z: np.ndarray):
    """(contiguous array, dtype code) for bf16-bit (uint16) or float32 logits, or for float64
    rows that `warp` returned."""
    z = np.ascontiguousarray(z)
    if z.dtype == np.uint16:
        return z, BF16
    if z.dtype == np.float32:
        return z, FP32
    if z.dtype == np.float64:
        return z, F64
    raise TypeError("logits must be uint16 (bf16 bits), float32 or float64 (warped rows)")


# ----------------------------------------------------------------------------- definitions

def widen(z: np.ndarray) -> np.ndarray:
    z, dt = _raw(z)
    out = np.empty(z.shape, dtype=np.float64)
    lib().oracle_widen(z.ctypes.data, dt, z.size, out.ctypes.data)
    return out


def warp(z: np.ndarray, temperature: float = 1.0, top_k: int = 0, top_p: float = 1.0,
         band: Optional[float] = None) -> tuple:
    """Adjusted distribution of Sec. 2.1.1 as logits (float64, -inf where a token is cut), for
    one row or a stack of rows; also the smallest top-p decision margin over the rows and, if
    `band` is given, the largest mass any row has within `band` of a top-p decision."""
    zz = widen(z) if z.dtype != np.float64 else np.ascontiguousarray(z)
    V = zz.shape[-1]
    flat = zz.reshape(-1, V)
    out = np.empty_like(flat)
    margin, band_mass = math.inf, 0.0
    for r in range(flat.shape[0]):
        m, bm = _D(0.0), _D(0.0)
        lib().oracle_warp_logits(flat[r].ctypes.data, V, float(temperature), int(top_k), float(top_p),
                                 float(band or 0.0), out[r].ctypes.data, C.byref(m), C.byref(bm))
        margin = min(margin, m.value)
        band_mass = max(band_mass, bm.value)
    if band is not None:
        return out.reshape(zz.shape), margin, band_mass
    return out.reshape(zz.shape), margin


def softmax(z) -> tuple:
    """(p, lse) of one float64 logit row."""
    z = _f64(z)
    p = np.empty_like(z)
    lse = lib().oracle_softmax(z.ctypes.data, z.size, p.ctypes.data)
    return p, lse


def entropy(p) -> float:
    p = _f64(p)
    return lib().oracle_entropy(p.ctypes.data, p.size)


def cross_entropy(p, q) -> float:
    p, q = _f64(p), _f64(q)
    return lib().oracle_cross_entropy(p.ctypes.data, q.ctypes.data, p.size)


def kl(p, q) -> float:
    p, q = _f64(p), _f64(q)
    return lib().oracle_kl(p.ctypes.data, q.ctypes.data, p.size)


def jsd(p, q) -> float:
    p, q = _f64(p), _f64(q)
    return lib().oracle_jsd(p.ctypes.data, q.ctypes.data, p.size)


def jsd_entropy_form(p, q) -> float:
    p, q = _f64(p), _f64(q)
    return lib().oracle_jsd_entropy_form(p.ctypes.data, q.ctypes.data, p.size)


def js_distance(jsd_nats: float) -> float:
    return lib().oracle_js_distance(jsd_nats)


def js_distance_rows(p, q) -> tuple:
    """(d, D_JS in nats) of two distributions, with the exact ends of Sec. 4.4."""
    p, q = _f64(p), _f64(q)
    j = C.c_double(0.0)
    d = lib().oracle_js_distance_rows(p.ctypes.data, q.ctypes.data, p.size, C.byref(j))
    return d, j.value


def inv_cdf(p, u: float) -> tuple:
    """(token, margin)."""
    p = _f64(p)
    m = C.c_double(0.0)
    v = lib().oracle_inv_cdf(p.ctypes.data, p.size, float(u), C.byref(m))
    return v, m.value


def sample_std(x) -> float:
    x = _f64(x)
    return lib().oracle_sample_std(x.ctypes.data, x.size)


def kde_bandwidth(x, rule: int = 0) -> float:
    x = _f64(x)
    return lib().oracle_kde_bandwidth(x.ctypes.data, x.size, rule)


def kde(x_list, x: float, rule: int = 0) -> float:
    x_list = _f64(x_list)
    return lib().oracle_kde(x_list.ctypes.data, x_list.size, float(x), rule)


def accept_prob(LA, LR, d: float, min_samples: int = 2, rule: int = 0) -> float:
    LA, LR = _f64(LA), _f64(LR)
    return lib().oracle_accept_prob(LA.ctypes.data, LA.size, LR.ctypes.data, LR.size, float(d),
                                    min_samples, rule)


# ----------------------------------------------------------------------------- Algorithm 1 state

class SequenceState:
    """L_E^R, L_D^A, L_D^R and T_G of one sequence (Alg. 1, initialisation)."""

    def __init__(self, capacity: int = 1 << 15, min_samples: int = 2, bw_rule: int = 0,
                 reject_rule: int = 0):
        self.cap = capacity
        self.LE = np.zeros(capacity, dtype=np.float64)
        self.LA = np.zeros(capacity, dtype=np.float64)
        self.LR = np.zeros(capacity, dtype=np.float64)
        self.nE = C.c_int32(0)
        self.nA = C.c_int32(0)
        self.nR = C.c_int32(0)
        self.T_G = C.c_double(0.0)
        self.min_samples = min_samples
        self.bw_rule = bw_rule
        self.reject_rule = reject_rule

    def lists(self):
        return (self.LE[: self.nE.value].copy(), self.LA[: self.nA.value].copy(),
                self.LR[: self.nR.value].copy())

    def accept_prob(self, d: float, extra_accepted=()) -> float:
        """P(A|d) on the lists as they stand, optionally with more accepted distances."""
        LA = np.concatenate([self.LA[: self.nA.value], np.asarray(extra_accepted, dtype=np.float64)])
        return accept_prob(LA, self.LR[: self.nR.value], d, self.min_samples, self.bw_rule)


def draft_step(z_row: np.ndarray, u: float, T_G: float) -> dict:
    """One draft step (Alg. 1 generation loop body) on a raw logit row."""
    z, dt = _raw(z_row)
    H, lse, mg = C.c_double(), C.c_double(), C.c_double()
    tok, stop = C.c_int32(), C.c_int32()
    lib().oracle_draft_step(z.ctypes.data, dt, z.size, float(u), float(T_G), C.byref(H),
                            C.byref(lse), C.byref(tok), C.byref(mg), C.byref(stop))
    return dict(H=H.value, lse=lse.value, token=tok.value, margin=mg.value, stop=bool(stop.value))


def verify_round(state: SequenceState, zd: np.ndarray, zt: np.ndarray, x, u_target, u_accept,
                 K_t: Optional[int] = None, update: bool = True) -> dict:
    """Verification + update of one round (Alg. 1, steps 2 and 3) for one sequence.

    zd: [>=K_t, V] draft rows, zt: [>=K_t+1, V] target rows (raw bf16 bits or fp32).
    """
    zd, dt = _raw(zd)
    zt, dt2 = _raw(zt)
    assert dt == dt2
    V = zt.shape[-1]
    if K_t is None:
        K_t = zd.shape[0]
    assert zt.shape[0] >= K_t + 1 and (K_t == 0 or zd.shape[0] >= K_t)
    assert state.nA.value + K_t <= state.cap and state.nE.value + 1 <= state.cap
    x = np.ascontiguousarray(x, dtype=np.int32)
    ut = np.ascontiguousarray(u_target, dtype=np.float32)
    ua = np.ascontiguousarray(u_accept, dtype=np.float32)
    K1 = K_t + 1
    out = {k: np.full(K_t, np.nan) for k in ("H_d", "lse_d", "jsd", "dist", "p_acc")}
    out.update({k: np.full(K1, np.nan) for k in ("H_t", "lse_t", "y_margin")})
    out["y"] = np.zeros(K1, dtype=np.int32)
    al, nt, rj = C.c_int32(), C.c_int32(), C.c_int32()
    lib().oracle_verify_round(
        zd.ctypes.data, zt.ctypes.data, dt, V, V, V, K_t, x.ctypes.data, ut.ctypes.data,
        ua.ctypes.data, state.LE.ctypes.data, C.byref(state.nE), state.LA.ctypes.data,
        C.byref(state.nA), state.LR.ctypes.data, C.byref(state.nR), C.byref(state.T_G),
        state.min_samples, state.bw_rule, state.reject_rule, 1 if update else 0,
        out["H_d"].ctypes.data, out["H_t"].ctypes.data, out["lse_d"].ctypes.data,
        out["lse_t"].ctypes.data, out["jsd"].ctypes.data, out["dist"].ctypes.data,
        out["p_acc"].ctypes.data, out["y"].ctypes.data, out["y_margin"].ctypes.data,
        C.byref(al), C.byref(nt), C.byref(rj))
    out.update(accept_len=al.value, next_token=nt.value, rejected=bool(rj.value), K_t=K_t)
    return out


def vanilla_round(zd: np.ndarray, zt: np.ndarray, x, u_accept, u_resample: float) -> dict:
    """Vanilla speculative sampling over a fixed window (Sec. 2.1.3)."""
    zd, dt = _raw(zd)
    zt, dt2 = _raw(zt)
    assert dt == dt2
    K, V = zd.shape[0], zt.shape[-1]
    assert zt.shape[0] >= K + 1
    x = np.ascontiguousarray(x, dtype=np.int32)
    ua = np.ascontiguousarray(u_accept, dtype=np.float32)
    alpha = np.full(K, np.nan)
    al, nt, mg = C.c_int32(), C.c_int32(), C.c_double()
    lib().oracle_vanilla_round(zd.ctypes.data, zt.ctypes.data, dt, V, V, V, K, x.ctypes.data,
                               ua.ctypes.data, float(u_resample), alpha.ctypes.data,
                               C.byref(al), C.byref(nt), C.byref(mg))
    return dict(alpha=alpha, accept_len=al.value, next_token=nt.value, margin=mg.value)


def argmax(z_row: np.ndarray) -> int:
    """Most probable token of a raw logit row; lowest index among equal maxima."""
    z, dt = _raw(z_row)
    return lib().oracle_argmax(z.ctypes.data, dt, z.size)


def greedy_round(zt: np.ndarray, x) -> dict:
    """Greedy verification (Sec. 2.1.3) of the candidates x against target rows zt [>=K+1, V]."""
    zt, dt = _raw(zt)
    x = np.ascontiguousarray(x, dtype=np.int32)
    K, V = x.size, zt.shape[-1]
    assert zt.shape[0] >= K + 1
    am = np.zeros(K + 1, dtype=np.int32)
    al, nt = C.c_int32(), C.c_int32()
    lib().oracle_greedy_round(zt.ctypes.data, dt, V, V, K, x.ctypes.data, am.ctypes.data, C.byref(al),
                              C.byref(nt))
    return dict(argmax=am, accept_len=al.value, next_token=nt.value)


def gen_only_update(state: SequenceState, H_d, K_t: int, accept_len: int) -> None:
    """Gen-Only feedback (Sec. 5): the rejected candidate's entropy joins L_E^R, T_G = mean."""
    H = _f64(H_d)
    lib().oracle_gen_only_update(state.LE.ctypes.data, C.byref(state.nE), C.byref(state.T_G),
                                 H.ctypes.data, int(K_t), int(accept_len))
