"""ctypes front end of the CPU oracle (``robe_oracle.c``).

Test infrastructure only: the test-suite, the smoke check and the benchmark's
CPU-baseline leg import this module; the product package never does.  The
functions here marshal numpy arrays into the plain-C oracle and hold none of the
method's arithmetic themselves.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "robe_oracle.c")
_LIB = os.path.join(_HERE, "librobe_oracle.so")

F32 = 0
BF16 = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (FP contraction off so no FMA is formed)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        u64, i64, p = C.c_uint64, C.c_int64, C.c_void_p
        _lib.robe_oracle_hash_constants.argtypes = [u64, p]
        _lib.robe_oracle_num_threads.restype = C.c_int
        _lib.robe_oracle_h.argtypes = [p, u64, u64, u64, u64]
        _lib.robe_oracle_h.restype = u64
        _lib.robe_oracle_idx.argtypes = [p, u64, u64, u64, u64, u64, u64]
        _lib.robe_oracle_idx.restype = u64
        _lib.robe_oracle_g.argtypes = [p, u64, u64, u64]
        _lib.robe_oracle_g.restype = C.c_int
        _lib.robe_oracle_locate.argtypes = [p, u64, u64, u64, u64, u64, p]
        _lib.robe_oracle_forward.argtypes = [p, u64, u64, u64, u64, C.c_int, p, C.c_int, p, p, i64, i64, p]
        _lib.robe_oracle_forward_bags.argtypes = [p, u64, u64, u64, u64, C.c_int, p, C.c_int, p, p,
                                                  p, i64, i64, p]
        _lib.robe_oracle_backward_f64.argtypes = [p, u64, u64, u64, u64, C.c_int, p, p, p, i64,
                                                  i64, u64, u64, p, p]
        _lib.robe_oracle_backward_canonical.argtypes = [p, u64, u64, u64, u64, C.c_int, p, p, p,
                                                        i64, i64, u64, u64, p, p]
        _lib.robe_oracle_backward_canonical.restype = C.c_int
        _lib.robe_oracle_sgd_apply.argtypes = [p, p, p, u64, C.c_float]
        _lib.robe_oracle_accumulate.argtypes = [p, p, p, u64]
        _lib.robe_oracle_dense_sgd_apply.argtypes = [p, p, u64, C.c_float]
        _lib.robe_oracle_adam_apply.argtypes = [p, p, p, p, p, u64] + [C.c_float] * 6
        _lib.robe_oracle_adagrad_apply.argtypes = [p, p, p, p, u64, C.c_float, C.c_float]
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _i64(a):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.int64)
    return a


def num_threads() -> int:
    return int(lib().robe_oracle_num_threads())


def hash_constants(seed: int) -> np.ndarray:
    out = np.zeros(9, dtype=np.uint64)
    lib().robe_oracle_hash_constants(C.c_uint64(seed & (2**64 - 1)), _ptr(out))
    return out


class Oracle:
    """The ROBE-Z mapping for one (M, Z, d, T, constants, sign) setting."""

    def __init__(self, M, Z, d, num_tables, consts, sign=False, table_major=False):
        """table_major: bags are numbered e*B + n (per-table id lists laid end to end) and the
        outputs and gradients are [T, B, d]; default: bags n*T + e, [B, T, d]."""
        self.M, self.Z, self.d, self.T = int(M), int(Z), int(d), int(num_tables)
        self.k = np.ascontiguousarray(consts, dtype=np.uint64)
        assert self.k.shape == (9,)
        self.sign = 1 if sign else 0
        self.table_major = bool(table_major)

    def _per_table(self, batch) -> int:
        return int(batch) if self.table_major else 0

    # -- mapping -------------------------------------------------------------
    def h(self, e, x, c) -> int:
        return int(lib().robe_oracle_h(_ptr(self.k), self.M, e, x, c))

    def idx(self, e, x, i) -> int:
        return int(lib().robe_oracle_idx(_ptr(self.k), self.M, self.Z, self.d, e, x, i))

    def g(self, e, x, i) -> int:
        return int(lib().robe_oracle_g(_ptr(self.k), e, x, i))

    def locate(self, e, x) -> np.ndarray:
        out = np.zeros(self.d, dtype=np.uint64)
        lib().robe_oracle_locate(_ptr(self.k), self.M, self.Z, self.d, e, x, _ptr(out))
        return out

    # -- forward -------------------------------------------------------------
    @staticmethod
    def _array_args(array):
        if array.dtype == np.float32:
            return np.ascontiguousarray(array), F32
        if array.dtype == np.uint16:  # raw bf16 bit patterns
            return np.ascontiguousarray(array), BF16
        raise TypeError("array must be float32 or uint16 (bf16 bits)")

    def forward(self, array, indices, offsets, batch) -> np.ndarray:
        array, dt = self._array_args(array)
        assert array.shape[0] == self.M
        indices, offsets = _i64(indices), _i64(offsets)
        out = np.empty((batch * self.T, self.d), dtype=np.float32)
        lib().robe_oracle_forward(_ptr(self.k), self.M, self.Z, self.d, self.T, self.sign,
                                  _ptr(array), dt, _ptr(indices), _ptr(offsets), batch,
                                  self._per_table(batch), _ptr(out))
        return out.reshape((self.T, batch, self.d) if self.table_major else (batch, self.T, self.d))

    def forward_bags(self, array, indices, offsets, bags, batch=None) -> np.ndarray:
        assert batch is not None or not self.table_major, "table-major bags need the batch size"
        array, dt = self._array_args(array)
        assert array.shape[0] == self.M
        indices, offsets, bags = _i64(indices), _i64(offsets), _i64(bags)
        out = np.empty((len(bags), self.d), dtype=np.float32)
        lib().robe_oracle_forward_bags(_ptr(self.k), self.M, self.Z, self.d, self.T, self.sign,
                                       _ptr(array), dt, _ptr(indices), _ptr(offsets), _ptr(bags),
                                       len(bags), self._per_table(batch or 0), _ptr(out))
        return out

    # -- backward ------------------------------------------------------------
    def backward_f64(self, grad_out, indices, offsets, batch, j0=0, jn=None):
        jn = self.M - j0 if jn is None else jn
        grad_out = np.ascontiguousarray(grad_out, dtype=np.float32)
        indices, offsets = _i64(indices), _i64(offsets)
        delta = np.zeros(jn, dtype=np.float64)
        l1 = np.zeros(jn, dtype=np.float64)
        lib().robe_oracle_backward_f64(_ptr(self.k), self.M, self.Z, self.d, self.T, self.sign,
                                       _ptr(grad_out), _ptr(indices), _ptr(offsets), batch,
                                       self._per_table(batch), j0, jn, _ptr(delta), _ptr(l1))
        return delta, l1

    def backward_canonical(self, grad_out, indices, offsets, batch, j0=0, jn=None):
        jn = self.M - j0 if jn is None else jn
        grad_out = np.ascontiguousarray(grad_out, dtype=np.float32)
        indices, offsets = _i64(indices), _i64(offsets)
        delta = np.empty(jn, dtype=np.float32)
        touched = np.empty(jn, dtype=np.uint8)
        rc = lib().robe_oracle_backward_canonical(_ptr(self.k), self.M, self.Z, self.d, self.T,
                                                  self.sign, _ptr(grad_out), _ptr(indices),
                                                  _ptr(offsets), batch, self._per_table(batch), j0, jn,
                                                  _ptr(delta), _ptr(touched))
        if rc != 0:
            raise MemoryError("oracle could not allocate its key list")
        return delta, touched


def sgd_apply(array, delta, touched, lr) -> None:
    """In place: array[j] = fma(-lr, delta[j], array[j]) on touched slots."""
    assert array.dtype == np.float32 and delta.dtype == np.float32 and touched.dtype == np.uint8
    lib().robe_oracle_sgd_apply(_ptr(array), _ptr(delta), _ptr(touched), len(delta), C.c_float(lr))


def dense_sgd_apply(array, grad, lr) -> None:
    """In place: array[j] = fma(-lr, grad[j], array[j]) on every slot (data-parallel step)."""
    assert array.dtype == np.float32 and grad.dtype == np.float32 and len(array) == len(grad)
    lib().robe_oracle_dense_sgd_apply(_ptr(array), _ptr(grad), len(array), C.c_float(lr))


def accumulate(grad_array, delta, touched) -> None:
    """In place: grad_array[j] = grad_array[j] + delta[j] on touched slots."""
    assert grad_array.dtype == np.float32 and delta.dtype == np.float32
    lib().robe_oracle_accumulate(_ptr(grad_array), _ptr(delta), _ptr(touched), len(delta))


def adagrad_apply(array, sum_sq, delta, touched, lr, eps) -> None:
    """In place: one Adagrad step (one accumulator per slot) on the touched slots."""
    for a in (array, sum_sq, delta):
        assert a.dtype == np.float32
    lib().robe_oracle_adagrad_apply(_ptr(array), _ptr(sum_sq), _ptr(delta), _ptr(touched), len(delta),
                                    C.c_float(lr), C.c_float(eps))


def adam_bias(beta: float, step: int) -> np.float32:
    """1 - beta^t, from the fp32 value of beta, evaluated in double and rounded to fp32."""
    return np.float32(1.0 - float(np.float32(beta)) ** step)


def adam_apply(array, m1, m2, delta, touched, lr, beta1, beta2, eps, step) -> None:
    """In place: one lazy Adam step (update number `step`) on the touched slots."""
    for a in (array, m1, m2, delta):
        assert a.dtype == np.float32
    lib().robe_oracle_adam_apply(_ptr(array), _ptr(m1), _ptr(m2), _ptr(delta), _ptr(touched), len(delta),
                                 C.c_float(lr), C.c_float(beta1), C.c_float(beta2), C.c_float(eps),
                                 C.c_float(adam_bias(beta1, step)), C.c_float(adam_bias(beta2, step)))
