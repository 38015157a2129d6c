"""ctypes binding of ``include/adasd.h``: same names, argument marshalling only.

The raw functions (``adasd_verify`` ...) take device addresses as Python ints and
return the library's status code.  :class:`Context` wraps them for torch tensors
(``tensor.data_ptr()``, the current CUDA stream) and raises :class:`AdasdError` on a
non-zero code.  Nothing here computes anything.
"""
from __future__ import annotations

import ctypes as C
import functools
import os
from typing import Optional

from .build import LIB, build

ADASD_BF16, ADASD_FP32 = 0, 1
ADASD_FUSE_UPDATE = 1
ADASD_KMAX_LIMIT = 32
STATUS_CAPACITY, STATUS_TIMEOUT, STATUS_NAN = 1, 2, 4
ERR_NULL, ERR_ALIGN, ERR_SHAPE, ERR_DTYPE, ERR_CAPACITY, ERR_CUDA, ERR_DEVICE = -1, -2, -3, -4, -5, -7, -9


class AdasdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {adasd_strerror(code)} ({code})")


class AdasdConfig(C.Structure):
    _fields_ = [("B", C.c_int32), ("V", C.c_int32), ("Kmax", C.c_int32), ("dtype", C.c_int32),
                ("list_capacity", C.c_int32), ("kde_bandwidth", C.c_int32),
                ("reject_rule", C.c_int32), ("min_kde_samples", C.c_int32),
                ("cluster_size", C.c_int32), ("device", C.c_int32)]


class RoundRecord(C.Structure):
    """Host struct of device array addresses (``adasd_round_record``)."""
    _fields_ = [(n, C.c_void_p) for n in ("H_d", "H_t", "lse_d", "lse_t", "jsd", "dist", "p_acc",
                                          "y", "draft_len", "accept_len", "rejected")]


def library_path() -> str:
    return LIB


@functools.lru_cache(maxsize=None)
def lib() -> C.CDLL:
    """Loads libadasd.so, building it first if the sources are newer.  Raises if it
    cannot be built or loaded: there is no fallback."""
    path = build()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build the CUDA library first")
    L = C.CDLL(path)
    P, I32, I64, U32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32
    sigs = {
        "adasd_create": [C.POINTER(P), C.POINTER(AdasdConfig)],
        "adasd_destroy": [P],
        "adasd_reset": [P, P, I32, P],
        "adasd_draft_entropy": [P, P, I64, P, P, P, P, P, P, P, P],
        "adasd_verify": [P, P, P, I64, I64, I64, I64, P, P, P, P, P, P, C.POINTER(RoundRecord),
                         U32, P],
        "adasd_update_thresholds": [P, C.POINTER(RoundRecord), P],
        "adasd_vanilla_verify": [P, P, P, I64, I64, I64, I64, P, P, P, P, P, P, P, P],
        "adasd_vanilla_verify_static": [I32, I32, I32, I32, P, P, I64, I64, I64, I64, P, P, P, P,
                                        P, P, P, P, P],
        "adasd_greedy_verify": [P, P, I64, I64, P, P, P, P, P, P],
        "adasd_gen_only_update": [P, P, P, P, P],
        "adasd_selftest_expired_wait": [P, P, I64, I32, P, P, P, P],
        "adasd_set_warpers": [P, C.c_float, I32, C.c_float],
        "adasd_get_thresholds": [P, P, P, P, P, P],
        "adasd_state_export": [P, I32, P, C.POINTER(C.c_size_t)],
        "adasd_state_import": [P, I32, P, C.c_size_t],
        "adasd_status": [P, C.POINTER(U32)],
    }
    for name, args in sigs.items():
        fn = getattr(L, name)
        fn.argtypes = args
        fn.restype = C.c_int
    L.adasd_strerror.argtypes = [C.c_int]
    L.adasd_strerror.restype = C.c_char_p
    return L


# ------------------------------------------------------------------ raw calls, same names

def adasd_strerror(code: int) -> str:
    return lib().adasd_strerror(code).decode()


def adasd_create(cfg: AdasdConfig):
    """Returns (code, ctx handle)."""
    h = C.c_void_p()
    rc = lib().adasd_create(C.byref(h), C.byref(cfg))
    return rc, h


def adasd_destroy(ctx) -> int:
    return lib().adasd_destroy(ctx)


def adasd_reset(ctx, seq_ids_dev, n, stream) -> int:
    return lib().adasd_reset(ctx, seq_ids_dev, n, stream)


def adasd_draft_entropy(ctx, logits_dev, row_stride, u_dev, active_inout_dev, H_out_dev,
                        lse_out_dev, token_out_dev, stop_out_dev, draft_len_inout_dev, stream) -> int:
    return lib().adasd_draft_entropy(ctx, logits_dev, row_stride, u_dev, active_inout_dev,
                                     H_out_dev, lse_out_dev, token_out_dev, stop_out_dev,
                                     draft_len_inout_dev, stream)


def adasd_verify(ctx, draft_logits_dev, target_logits_dev, d_seq_stride, d_row_stride,
                 t_seq_stride, t_row_stride, draft_tokens_dev, draft_len_dev, u_target_dev,
                 u_accept_dev, accept_len_dev, next_token_dev, record, flags, stream) -> int:
    return lib().adasd_verify(ctx, draft_logits_dev, target_logits_dev, d_seq_stride,
                              d_row_stride, t_seq_stride, t_row_stride, draft_tokens_dev,
                              draft_len_dev, u_target_dev, u_accept_dev, accept_len_dev,
                              next_token_dev, C.byref(record) if record is not None else None,
                              flags, stream)


def adasd_update_thresholds(ctx, record, stream) -> int:
    return lib().adasd_update_thresholds(ctx, C.byref(record) if record is not None else None,
                                         stream)


def adasd_vanilla_verify(ctx, draft_logits_dev, target_logits_dev, d_seq_stride, d_row_stride,
                         t_seq_stride, t_row_stride, draft_tokens_dev, draft_len_dev,
                         u_accept_dev, u_resample_dev, accept_len_dev, next_token_dev,
                         alpha_out_dev, stream) -> int:
    return lib().adasd_vanilla_verify(ctx, draft_logits_dev, target_logits_dev, d_seq_stride,
                                      d_row_stride, t_seq_stride, t_row_stride, draft_tokens_dev,
                                      draft_len_dev, u_accept_dev, u_resample_dev, accept_len_dev,
                                      next_token_dev, alpha_out_dev, stream)


def adasd_vanilla_verify_static(B, V, Kmax, dtype, draft_logits_dev, target_logits_dev,
                                d_seq_stride, d_row_stride, t_seq_stride, t_row_stride,
                                draft_tokens_dev, draft_len_dev, u_accept_dev, u_resample_dev,
                                accept_len_dev, next_token_dev, alpha_out_dev, status_out_dev,
                                stream) -> int:
    """Context-free vanilla verification whose scratch is a fixed array inside the library:
    for callers that may not allocate device memory.  Same arguments as the C function."""
    return lib().adasd_vanilla_verify_static(B, V, Kmax, dtype, draft_logits_dev,
                                             target_logits_dev, d_seq_stride, d_row_stride,
                                             t_seq_stride, t_row_stride, draft_tokens_dev,
                                             draft_len_dev, u_accept_dev, u_resample_dev,
                                             accept_len_dev, next_token_dev, alpha_out_dev,
                                             status_out_dev, stream)


def adasd_greedy_verify(ctx, target_logits_dev, t_seq_stride, t_row_stride, draft_tokens_dev,
                        draft_len_dev, accept_len_dev, next_token_dev, argmax_out_dev, stream) -> int:
    return lib().adasd_greedy_verify(ctx, target_logits_dev, t_seq_stride, t_row_stride, draft_tokens_dev,
                                     draft_len_dev, accept_len_dev, next_token_dev, argmax_out_dev, stream)


def adasd_gen_only_update(ctx, H_draft_dev, draft_len_dev, accept_len_dev, stream) -> int:
    return lib().adasd_gen_only_update(ctx, H_draft_dev, draft_len_dev, accept_len_dev, stream)


def adasd_set_warpers(ctx, temperature, top_k, top_p) -> int:
    return lib().adasd_set_warpers(ctx, temperature, top_k, top_p)


def adasd_selftest_expired_wait(ctx, logits_dev, row_stride, row, u_dev, H_out_dev, token_out_dev, stream) -> int:
    return lib().adasd_selftest_expired_wait(ctx, logits_dev, row_stride, row, u_dev, H_out_dev, token_out_dev,
                                             stream)


def adasd_get_thresholds(ctx, T_G_dev, nE_dev, nA_dev, nR_dev, stream) -> int:
    return lib().adasd_get_thresholds(ctx, T_G_dev, nE_dev, nA_dev, nR_dev, stream)


def adasd_state_export(ctx, seq: int, host_buf, bytes_inout) -> int:
    return lib().adasd_state_export(ctx, seq, host_buf, bytes_inout)


def adasd_state_import(ctx, seq: int, host_buf, nbytes: int) -> int:
    return lib().adasd_state_import(ctx, seq, host_buf, nbytes)


def adasd_status(ctx):
    """Returns (code, status bits); clears the sticky word."""
    s = C.c_uint32(0)
    rc = lib().adasd_status(ctx, C.byref(s))
    return rc, s.value


# ------------------------------------------------------------------ torch convenience

def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


class Context:
    """Owns one ``adasd_ctx``; methods take torch CUDA tensors and use the current stream."""

    def __init__(self, B: int, V: int, Kmax: int, dtype: int = ADASD_BF16,
                 list_capacity: int = 1 << 14, kde_bandwidth: int = 0, reject_rule: int = 0,
                 min_kde_samples: int = 2, cluster_size: int = 0, device: int = 0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the AdaSD library needs a CUDA device; there is no CPU path")
        self.torch = torch
        self.cfg = AdasdConfig(B, V, Kmax, dtype, list_capacity, kde_bandwidth, reject_rule,
                               min_kde_samples, cluster_size, device)
        self.device = torch.device("cuda", device)
        rc, self.handle = adasd_create(self.cfg)
        if rc != 0:
            self.handle = None
            raise AdasdError(rc, "adasd_create")
        self.B, self.V, self.Kmax = B, V, Kmax

    def close(self) -> None:
        if getattr(self, "handle", None):
            adasd_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _stream(self) -> int:
        return self.torch.cuda.current_stream(self.device).cuda_stream

    @staticmethod
    def _check(rc: int, where: str) -> None:
        if rc != 0:
            raise AdasdError(rc, where)

    def new_record(self) -> dict:
        """Device tensors for every field of a round record."""
        t, B, K = self.torch, self.B, self.Kmax
        f = dict(dtype=t.float32, device=self.device)
        i = dict(dtype=t.int32, device=self.device)
        return dict(H_d=t.full((B, K), float("nan"), **f), H_t=t.full((B, K + 1), float("nan"), **f),
                    lse_d=t.full((B, K), float("nan"), **f), lse_t=t.full((B, K + 1), float("nan"), **f),
                    jsd=t.full((B, K), float("nan"), **f), dist=t.full((B, K), float("nan"), **f),
                    p_acc=t.full((B, K), float("nan"), **f), y=t.full((B, K + 1), -2, **i),
                    draft_len=t.zeros(B, **i), accept_len=t.zeros(B, **i), rejected=t.zeros(B, **i))

    @staticmethod
    def record_struct(rec: Optional[dict]) -> Optional[RoundRecord]:
        if rec is None:
            return None
        return RoundRecord(**{k: (v.data_ptr() if v is not None else None) for k, v in rec.items()})

    def reset(self, seq_ids=None) -> None:
        n = self.B if seq_ids is None else seq_ids.numel()
        self._check(adasd_reset(self.handle, _ptr(seq_ids), n, self._stream()), "adasd_reset")

    def draft_entropy(self, logits, H_out, u=None, token_out=None, active=None, lse_out=None,
                      stop_out=None, draft_len=None, row_stride: Optional[int] = None) -> None:
        rs = logits.stride(0) if row_stride is None else row_stride
        self._check(adasd_draft_entropy(self.handle, logits.data_ptr(), rs, _ptr(u), _ptr(active),
                                        H_out.data_ptr(), _ptr(lse_out), _ptr(token_out),
                                        _ptr(stop_out), _ptr(draft_len), self._stream()),
                    "adasd_draft_entropy")

    def verify(self, draft_logits, target_logits, draft_tokens, u_target, u_accept, accept_len,
               next_token, draft_len=None, record: Optional[dict] = None,
               fuse_update: bool = True) -> None:
        rs = self.record_struct(record)
        self._check(adasd_verify(self.handle, draft_logits.data_ptr(), target_logits.data_ptr(),
                                 draft_logits.stride(0), draft_logits.stride(1),
                                 target_logits.stride(0), target_logits.stride(1),
                                 draft_tokens.data_ptr(), _ptr(draft_len), u_target.data_ptr(),
                                 u_accept.data_ptr(), accept_len.data_ptr(), next_token.data_ptr(),
                                 rs, ADASD_FUSE_UPDATE if fuse_update else 0, self._stream()),
                    "adasd_verify")

    def update_thresholds(self, record: dict) -> None:
        self._check(adasd_update_thresholds(self.handle, self.record_struct(record), self._stream()),
                    "adasd_update_thresholds")

    def vanilla_verify(self, draft_logits, target_logits, draft_tokens, u_accept, u_resample,
                       accept_len, next_token, draft_len=None, alpha_out=None) -> None:
        self._check(adasd_vanilla_verify(self.handle, draft_logits.data_ptr(),
                                         target_logits.data_ptr(), draft_logits.stride(0),
                                         draft_logits.stride(1), target_logits.stride(0),
                                         target_logits.stride(1), draft_tokens.data_ptr(),
                                         _ptr(draft_len), u_accept.data_ptr(), u_resample.data_ptr(),
                                         accept_len.data_ptr(), next_token.data_ptr(),
                                         _ptr(alpha_out), self._stream()), "adasd_vanilla_verify")

    def greedy_verify(self, target_logits, draft_tokens, accept_len, next_token, draft_len=None,
                      argmax_out=None) -> None:
        self._check(adasd_greedy_verify(self.handle, target_logits.data_ptr(), target_logits.stride(0),
                                        target_logits.stride(1), draft_tokens.data_ptr(), _ptr(draft_len),
                                        accept_len.data_ptr(), next_token.data_ptr(), _ptr(argmax_out),
                                        self._stream()), "adasd_greedy_verify")

    def gen_only_update(self, H_draft, accept_len, draft_len=None) -> None:
        self._check(adasd_gen_only_update(self.handle, H_draft.data_ptr(), _ptr(draft_len),
                                          accept_len.data_ptr(), self._stream()), "adasd_gen_only_update")

    def set_warpers(self, temperature: float = 1.0, top_k: int = 0, top_p: float = 1.0) -> None:
        self._check(adasd_set_warpers(self.handle, float(temperature), int(top_k), float(top_p)),
                    "adasd_set_warpers")

    def get_thresholds(self):
        """(T_G, nE, nA, nR) as new device tensors."""
        t = self.torch
        T = t.empty(self.B, dtype=t.float32, device=self.device)
        n = [t.empty(self.B, dtype=t.int32, device=self.device) for _ in range(3)]
        self._check(adasd_get_thresholds(self.handle, T.data_ptr(), n[0].data_ptr(), n[1].data_ptr(),
                                         n[2].data_ptr(), self._stream()), "adasd_get_thresholds")
        return T, n[0], n[1], n[2]

    def state_export(self, seq: int) -> dict:
        """Host copy of one sequence's state: dict(T_G, LE, LA, LR) with numpy arrays."""
        import numpy as np
        nbytes = C.c_size_t(0)
        self._check(adasd_state_export(self.handle, seq, None, C.byref(nbytes)), "adasd_state_export")
        buf = (C.c_char * nbytes.value)()
        self._check(adasd_state_export(self.handle, seq, buf, C.byref(nbytes)), "adasd_state_export")
        raw = bytes(buf)
        nE, nA, nR, _ = np.frombuffer(raw[:16], dtype=np.int32)
        T_G = float(np.frombuffer(raw[16:20], dtype=np.float32)[0])
        body = np.frombuffer(raw[24:], dtype=np.float32)
        return dict(T_G=T_G, LE=body[:nE].copy(), LA=body[nE:nE + nA].copy(),
                    LR=body[nE + nA:nE + nA + nR].copy())

    def state_import(self, seq: int, T_G: float, LE, LA, LR) -> None:
        import numpy as np
        LE, LA, LR = (np.ascontiguousarray(a, dtype=np.float32) for a in (LE, LA, LR))
        raw = (np.array([LE.size, LA.size, LR.size, 0], dtype=np.int32).tobytes() +
               np.array([T_G, 0.0], dtype=np.float32).tobytes() + LE.tobytes() + LA.tobytes() +
               LR.tobytes())
        self._check(adasd_state_import(self.handle, seq, raw, len(raw)), "adasd_state_import")

    def status(self) -> int:
        rc, bits = adasd_status(self.handle)
        self._check(rc, "adasd_status")
        return bits
