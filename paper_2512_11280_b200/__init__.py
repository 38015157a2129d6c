"""B200-native AdaSD hot path: thin Python binding over the C-ABI CUDA library.

Everything numerical runs in the CUDA kernels of ``libadasd.so``; this package only
marshals arguments (device pointers of torch tensors, strides, streams).  There is
no CPU fallback: importing works anywhere, but every call needs the built library
and a CUDA device and raises otherwise.
"""
from .binding import (ERR_ALIGN, ERR_CAPACITY, ERR_CUDA, ERR_DEVICE, ERR_DTYPE, ERR_NULL, ERR_SHAPE,
                      ADASD_BF16, ADASD_FP32, ADASD_FUSE_UPDATE, ADASD_KMAX_LIMIT, STATUS_CAPACITY,
                      STATUS_NAN, STATUS_TIMEOUT, AdasdConfig, AdasdError, Context, RoundRecord,
                      adasd_create, adasd_destroy, adasd_draft_entropy, adasd_gen_only_update, adasd_get_thresholds, adasd_greedy_verify,
                      adasd_reset, adasd_selftest_expired_wait, adasd_set_warpers, adasd_state_export, adasd_state_import, adasd_status,
                      adasd_strerror, adasd_update_thresholds, adasd_vanilla_verify, adasd_vanilla_verify_static, adasd_verify,
                      lib, library_path)
from .build import build

__all__ = [n for n in dir() if not n.startswith("_")]
