"""Thin ctypes binding of librobe.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/robe.h) and does
no arithmetic of the method itself.  torch is used for device memory and streams.  There
is no fallback: if the shared library is missing or does not load, importing this module
raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# ROBE_LIBRARY names another build of the same library to load instead (the index-check build
# librobe_debug.so); it is not a fallback: a name that does not exist fails below like the default.
LIB_PATH = os.environ.get("ROBE_LIBRARY") or os.path.join(_HERE, "librobe.so")

ROBE_OK = 0
ROBE_ERR_INVALID_ARG = -1
ROBE_ERR_NO_ARRAY = -2
ROBE_ERR_WORKSPACE = -3
ROBE_ERR_CUDA = -4
ROBE_ERR_UNSUPPORTED = -5

ROBE_F32 = 0
ROBE_BF16 = 1

ROBE_OPT_SIGN = 1
ROBE_OPT_BWD_MODE = 2
ROBE_OPT_VALIDATE = 3
ROBE_OPT_FWD_KERNEL = 4
ROBE_OPT_BWD_KERNEL = 5
ROBE_OPT_INDEX_TYPE = 6
ROBE_OPT_ARRAY_L2_KEEP = 8

ROBE_I64 = 0
ROBE_I32 = 1
ROBE_OPT_BAG_LAYOUT = 7
ROBE_BAGS_SAMPLE_MAJOR = 0
ROBE_BAGS_TABLE_MAJOR = 1

ROBE_BWD_ATOMIC = 0
ROBE_BWD_DETERMINISTIC = 1
ROBE_BWD_BINNED = 2

ROBE_STATIC_SCRATCH_BYTES = 32 << 20

ROBE_DBG_SELFTEST = 99

EXPORTS = [
    "robe_create", "robe_destroy", "robe_set_option", "robe_attach_array",
    "robe_get_hash_constants", "robe_forward", "robe_backward_workspace_bytes", "robe_backward",
    "robe_set_status_word", "robe_last_device_status", "robe_status_string",
    "robe_backward_deterministic_static", "robe_backward_adam",
    "robe_forward_keep", "robe_backward_kept", "robe_apply_sgd",
    "robe_debug_status", "robe_debug_selftest", "robe_backward_adagrad",
]

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2108_02191_b200.build` "
        "(there is no CPU or PyTorch fallback)")

_lib = C.CDLL(LIB_PATH)

_vp, _i64, _u64, _u32 = C.c_void_p, C.c_int64, C.c_uint64, C.c_uint32
_lib.robe_create.argtypes = [C.POINTER(_vp), _u64, _u32, _u32, _u32, _u64]
_lib.robe_destroy.argtypes = [_vp]
_lib.robe_set_option.argtypes = [_vp, C.c_int, _i64]
_lib.robe_attach_array.argtypes = [_vp, _vp, C.c_int]
_lib.robe_get_hash_constants.argtypes = [_vp, C.POINTER(_u64)]
_lib.robe_forward.argtypes = [_vp, _vp, _vp, _i64, _i64, _vp, _vp]
_lib.robe_forward_keep.argtypes = [_vp, _vp, _vp, _i64, _i64, _vp, _vp, C.c_size_t, _vp]
_lib.robe_backward_workspace_bytes.argtypes = [_vp, _i64, _i64]
_lib.robe_backward_workspace_bytes.restype = C.c_size_t
_lib.robe_backward.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _vp, C.c_float, _vp, C.c_size_t, _vp]
_lib.robe_backward_kept.argtypes = list(_lib.robe_backward.argtypes)
_lib.robe_backward_deterministic_static.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _vp, C.c_float, _vp]
_lib.robe_backward_adam.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _vp, _vp, C.c_float, C.c_float,
                                    C.c_float, C.c_float, _i64, _vp, C.c_size_t, _vp]
_lib.robe_apply_sgd.argtypes = [_vp, _vp, C.c_float, C.c_int, _vp]
_lib.robe_backward_adagrad.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _vp, C.c_float, C.c_float, _vp,
                                       C.c_size_t, _vp]
_lib.robe_debug_status.argtypes = [_vp]
_lib.robe_debug_selftest.argtypes = [_vp]
_lib.robe_set_status_word.argtypes = [_vp, _vp]
_lib.robe_last_device_status.argtypes = [_vp, _vp]
_lib.robe_status_string.argtypes = [C.c_int]
_lib.robe_status_string.restype = C.c_char_p
for _name in EXPORTS:
    if _name not in ("robe_backward_workspace_bytes", "robe_status_string"):
        getattr(_lib, _name).restype = C.c_int


class RobeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {robe_status_string(status)} ({status})")


def _check(status: int, where: str) -> None:
    if status != ROBE_OK:
        raise RobeError(status, where)


def _dev_ptr(t, dtype=None):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return t.data_ptr()


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ids_ptr(t):
    """Device pointer of an id tensor: int64, or int32 for a handle set to ROBE_I32 (the handle's
    option says which the library reads; nothing is converted here)."""
    if t.dtype not in (torch.int64, torch.int32):
        raise TypeError(f"indices must be int64 or int32, got {t.dtype}")
    return _dev_ptr(t)


def _state_index_type(h, indices) -> None:
    """Tells the handle which element type the id tensor of the coming call has (the C ABI
    states it through ROBE_OPT_INDEX_TYPE, a tensor carries it in its dtype)."""
    _check(_lib.robe_set_option(h, ROBE_OPT_INDEX_TYPE,
                                ROBE_I32 if indices.dtype == torch.int32 else ROBE_I64), "robe_set_option")


def robe_status_string(status: int) -> str:
    return _lib.robe_status_string(status).decode()


def robe_create(M: int, Z: int, d: int, num_tables: int, hash_seed: int):
    h = _vp()
    if not (0 <= M < 2**64 and 0 <= Z < 2**32 and 0 <= d < 2**32 and 0 <= num_tables < 2**32):
        raise RobeError(ROBE_ERR_INVALID_ARG, "robe_create")
    _check(_lib.robe_create(C.byref(h), M, Z, d, num_tables, hash_seed & (2**64 - 1)), "robe_create")
    return h


def robe_destroy(h) -> None:
    _check(_lib.robe_destroy(h), "robe_destroy")


def robe_set_option(h, key: int, value: int) -> None:
    _check(_lib.robe_set_option(h, key, value), "robe_set_option")


def robe_attach_array(h, array: torch.Tensor) -> None:
    if array.dtype == torch.float32:
        dt = ROBE_F32
    elif array.dtype == torch.bfloat16:
        dt = ROBE_BF16
    else:
        raise TypeError("array must be float32 or bfloat16")
    _check(_lib.robe_attach_array(h, _dev_ptr(array), dt), "robe_attach_array")


def robe_get_hash_constants(h):
    out = (_u64 * 9)()
    _check(_lib.robe_get_hash_constants(h, out), "robe_get_hash_constants")
    return [int(v) for v in out]


def robe_forward(h, indices, offsets, batch: int, out, stream=None) -> None:
    _state_index_type(h, indices)
    _check(_lib.robe_forward(h, _ids_ptr(indices), _dev_ptr(offsets, torch.int64),
                             batch, indices.numel(), _dev_ptr(out, torch.float32),
                             _stream_ptr(stream)), "robe_forward")


def robe_forward_keep(h, indices, offsets, batch: int, out, workspace, stream=None) -> None:
    """robe_forward that also leaves the block starts in `workspace` for robe_backward_kept."""
    _state_index_type(h, indices)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.robe_forward_keep(h, _ids_ptr(indices), _dev_ptr(offsets, torch.int64),
                                  batch, indices.numel(), _dev_ptr(out, torch.float32),
                                  _dev_ptr(workspace), ws_bytes, _stream_ptr(stream)), "robe_forward_keep")


def robe_backward_workspace_bytes(h, batch: int, nnz: int) -> int:
    return int(_lib.robe_backward_workspace_bytes(h, batch, nnz))


def robe_backward(h, grad_out, indices, offsets, batch: int, grad_array=None, lr: float = 0.0,
                  workspace=None, stream=None) -> None:
    _state_index_type(h, indices)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.robe_backward(h, _dev_ptr(grad_out, torch.float32), _ids_ptr(indices),
                              _dev_ptr(offsets, torch.int64), batch, indices.numel(),
                              _dev_ptr(grad_array, torch.float32), lr, _dev_ptr(workspace),
                              ws_bytes, _stream_ptr(stream)), "robe_backward")


def robe_backward_kept(h, grad_out, indices, offsets, batch: int, grad_array=None, lr: float = 0.0,
                       workspace=None, stream=None) -> None:
    """robe_backward on the block starts that robe_forward_keep left in `workspace`."""
    _state_index_type(h, indices)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.robe_backward_kept(h, _dev_ptr(grad_out, torch.float32), _ids_ptr(indices),
                                   _dev_ptr(offsets, torch.int64), batch, indices.numel(),
                                   _dev_ptr(grad_array, torch.float32), lr, _dev_ptr(workspace),
                                   ws_bytes, _stream_ptr(stream)), "robe_backward_kept")


def robe_backward_deterministic_static(h, grad_out, indices, offsets, batch: int, grad_array=None,
                                       lr: float = 0.0, stream=None) -> None:
    """Deterministic backward on the library's built-in scratch array, for callers that cannot
    allocate a workspace (include/robe.h has the limit and the sharing rules).  No tensor is
    created here: the arguments are passed through as they are."""
    _state_index_type(h, indices)
    _check(_lib.robe_backward_deterministic_static(
        h, _dev_ptr(grad_out, torch.float32), _ids_ptr(indices),
        _dev_ptr(offsets, torch.int64), batch, indices.numel(), _dev_ptr(grad_array, torch.float32),
        lr, _stream_ptr(stream)), "robe_backward_deterministic_static")


def robe_backward_adam(h, grad_out, indices, offsets, batch: int, m1, m2, lr: float, beta1: float,
                       beta2: float, eps: float, step: int, workspace, stream=None) -> None:
    _state_index_type(h, indices)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.robe_backward_adam(
        h, _dev_ptr(grad_out, torch.float32), _ids_ptr(indices), _dev_ptr(offsets, torch.int64), batch,
        indices.numel(), _dev_ptr(m1, torch.float32), _dev_ptr(m2, torch.float32), lr, beta1, beta2, eps,
        step, _dev_ptr(workspace), ws_bytes, _stream_ptr(stream)), "robe_backward_adam")


def robe_backward_adagrad(h, grad_out, indices, offsets, batch: int, sum_sq, lr: float, eps: float,
                          workspace, stream=None) -> None:
    _state_index_type(h, indices)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.robe_backward_adagrad(
        h, _dev_ptr(grad_out, torch.float32), _ids_ptr(indices), _dev_ptr(offsets, torch.int64), batch,
        indices.numel(), _dev_ptr(sum_sq, torch.float32), lr, eps, _dev_ptr(workspace), ws_bytes,
        _stream_ptr(stream)), "robe_backward_adagrad")


def robe_apply_sgd(h, grad_array, lr: float, zero_grad: bool = True, stream=None) -> None:
    """Dense SGD apply of the data-parallel step: array <- fma(-lr, grad_array, array)."""
    _check(_lib.robe_apply_sgd(h, _dev_ptr(grad_array, torch.float32), lr, 1 if zero_grad else 0,
                               _stream_ptr(stream)), "robe_apply_sgd")


def robe_debug_status(stream=None) -> int:
    """Index-check build only: the first recorded ROBE_DBG_* code (0 = none), cleared by the call;
    ROBE_ERR_UNSUPPORTED (-5) from the release library."""
    return int(_lib.robe_debug_status(_stream_ptr(stream)))


def robe_debug_selftest(stream=None) -> int:
    return int(_lib.robe_debug_selftest(_stream_ptr(stream)))


def robe_set_status_word(h, word) -> None:
    _check(_lib.robe_set_status_word(h, _dev_ptr(word, torch.int32)), "robe_set_status_word")


def robe_last_device_status(h, stream=None) -> int:
    return int(_lib.robe_last_device_status(h, _stream_ptr(stream)))


def raw():
    """The ctypes library object itself, for callers that drive the C ABI with raw addresses
    (the host-side argument tests do)."""
    return _lib
