"""Shared helpers of the GPU parity tests: run the CUDA library through its C ABI binding and
the CPU oracle on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

import paper_2108_02191_b200 as robe
from oracle import robe_oracle as orc
from paper_2108_02191_b200 import synth


class Case:
    """One workload instantiated on the device, with its oracle twin."""

    def __init__(self, w: synth.RobeWorkload, batch=None, sign=False, variant=0, array=None,
                 ids=None, host_array=True, table_major=False):
        self.w = w
        self.B = w.batch if batch is None else batch
        self.T = w.num_tables
        self.dev = torch.device("cuda:0")
        if ids is None:
            ids = synth.make_ids(w, self.B, variant)
        if table_major:  # the same bags, numbered table by table
            ids = synth.to_table_major(ids[0], ids[1], self.B, self.T)
        self.indices_h, self.offsets_h = ids
        self.nbags = self.B * self.T
        self.indices = torch.from_numpy(self.indices_h).to(self.dev)
        self.offsets = None if self.offsets_h is None else torch.from_numpy(self.offsets_h).to(self.dev)
        self.array = synth.make_array(w, self.dev) if array is None else array.to(self.dev)
        self.array_h = synth.array_to_numpy(self.array) if host_array else None
        self.h = robe.robe_create(w.M, w.Z, w.d, w.num_tables, w.hash_seed)
        robe.robe_attach_array(self.h, self.array)
        self.table_major = table_major
        if table_major:
            robe.robe_set_option(self.h, robe.ROBE_OPT_BAG_LAYOUT, robe.ROBE_BAGS_TABLE_MAJOR)
        self.sign = sign
        if sign:
            robe.robe_set_option(self.h, robe.ROBE_OPT_SIGN, 1)
        k = np.array(robe.robe_get_hash_constants(self.h), dtype=np.uint64)
        # the oracle draws its own constants; the library's must be the same numbers
        np.testing.assert_array_equal(k, orc.hash_constants(w.hash_seed))
        self.oracle = orc.Oracle(w.M, w.Z, w.d, w.num_tables, orc.hash_constants(w.hash_seed), sign,
                                 table_major=table_major)

    def close(self):
        if self.h is not None:
            robe.robe_destroy(self.h)
            self.h = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # ---- GPU side -------------------------------------------------------------------
    def forward(self, kernel=0) -> torch.Tensor:
        robe.robe_set_option(self.h, robe.ROBE_OPT_FWD_KERNEL, kernel)
        out = torch.full((self.B, self.T, self.w.d), float("nan"), dtype=torch.float32, device=self.dev)
        robe.robe_forward(self.h, self.indices, self.offsets, self.B, out)
        torch.cuda.synchronize()
        return out

    def backward(self, grad_out: torch.Tensor, mode="atomic", sgd=False, lr=0.0, kernel=0,
                 grad_array=None):
        """Returns the dense gradient array (sgd=False) or None (sgd=True: array updated in place)."""
        robe.robe_set_option(self.h, robe.ROBE_OPT_BWD_MODE,
                             {"atomic": robe.ROBE_BWD_ATOMIC, "det": robe.ROBE_BWD_DETERMINISTIC,
                              "binned": robe.ROBE_BWD_BINNED}[mode])
        robe.robe_set_option(self.h, robe.ROBE_OPT_BWD_KERNEL, kernel)
        ws = None
        nbytes = robe.robe_backward_workspace_bytes(self.h, self.B, self.indices.numel())
        if nbytes:
            ws = torch.empty(nbytes, dtype=torch.uint8, device=self.dev)
        if sgd:
            robe.robe_backward(self.h, grad_out, self.indices, self.offsets, self.B, None, lr, ws)
            torch.cuda.synchronize()
            return None
        if grad_array is None:
            grad_array = torch.zeros(self.w.M, dtype=torch.float32, device=self.dev)
        robe.robe_backward(self.h, grad_out, self.indices, self.offsets, self.B, grad_array, 0.0, ws)
        torch.cuda.synchronize()
        return grad_array

    def step_sharing_keys(self, grad_out: torch.Tensor, mode, sgd=False, lr=0.0, fwd_kernel=0):
        """robe_forward_keep then robe_backward_kept on the same workspace: (out, dense gradient
        or None)."""
        robe.robe_set_option(self.h, robe.ROBE_OPT_BWD_MODE,
                             {"atomic": robe.ROBE_BWD_ATOMIC, "det": robe.ROBE_BWD_DETERMINISTIC,
                              "binned": robe.ROBE_BWD_BINNED}[mode])
        robe.robe_set_option(self.h, robe.ROBE_OPT_FWD_KERNEL, fwd_kernel)
        robe.robe_set_option(self.h, robe.ROBE_OPT_BWD_KERNEL, 0)
        ws = None
        nbytes = robe.robe_backward_workspace_bytes(self.h, self.B, self.indices.numel())
        if nbytes:  # stale contents from an earlier call must not matter
            ws = torch.full((nbytes,), 0xA5, dtype=torch.uint8, device=self.dev)
        out = torch.full((self.B, self.T, self.w.d), float("nan"), dtype=torch.float32, device=self.dev)
        robe.robe_forward_keep(self.h, self.indices, self.offsets, self.B, out, ws)
        grad_array = None if sgd else torch.zeros(self.w.M, dtype=torch.float32, device=self.dev)
        robe.robe_backward_kept(self.h, grad_out, self.indices, self.offsets, self.B, grad_array, lr, ws)
        torch.cuda.synchronize()
        return out, grad_array

    # ---- oracle side ----------------------------------------------------------------
    def oracle_forward(self):
        return self.oracle.forward(self.array_h, self.indices_h, self.offsets_h, self.B)

    def oracle_forward_bags(self, bags):
        return self.oracle.forward_bags(self.array_h, self.indices_h, self.offsets_h, bags, batch=self.B)


def assert_bits_equal(a: np.ndarray, b: np.ndarray, what=""):
    a = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    b = np.ascontiguousarray(b, dtype=np.float32).view(np.uint32)
    if not np.array_equal(a, b):
        bad = np.flatnonzero(a.reshape(-1) != b.reshape(-1))
        raise AssertionError(f"{what}: {len(bad)} of {a.size} elements differ in bits; first at flat "
                             f"index {bad[0]}: {a.reshape(-1)[bad[0]]:#x} vs {b.reshape(-1)[bad[0]]:#x}")


def assert_within_l1(got: np.ndarray, delta64: np.ndarray, l1: np.ndarray, scale=1.0, what=""):
    """Tolerance of the atomic backward: |got - ref| <= 1e-5 * scale * L1 mass per slot (exactly equal
    where no gradient landed)."""
    err = np.abs(got.astype(np.float64) - delta64)
    tol = 1e-5 * scale * l1
    bad = np.flatnonzero(err > tol)
    if len(bad):
        j = bad[np.argmax(err[bad] / np.maximum(tol[bad], 1e-300))]
        raise AssertionError(f"{what}: {len(bad)} slots out of tolerance; worst slot {j}: "
                             f"err {err[j]:.3e} tol {tol[j]:.3e}")
    mask = l1 > 0
    return float(np.max(err[mask] / l1[mask])) if mask.any() else 0.0
