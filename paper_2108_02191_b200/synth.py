"""Seeded synthetic inputs with the shapes of the paper's workloads.

This module only *generates data*: vocabulary sizes, ids, bag lengths, array
initial values and output gradients.  It holds none of the method's arithmetic
(no hashing, no gather, no scatter) and is the one module that both the CUDA
path's tests/benchmark and the CPU oracle's tests draw their inputs from.

The five workloads mirror the paper's experiments in shape only (Section 5: 26
categorical tables, embedding size 128 for the terabyte model and 16 for the
Kaggle models, batch sizes of the 16K class, a 100 MB array); the records of
those datasets are not used or reproduced.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class RobeWorkload:
    name: str
    num_tables: int
    vocab_rule: str            # "list", "loguniform" (3 .. 4e7) or "const"
    vocab_arg: Tuple[int, ...]  # the list, or (value,) for "const"
    d: int
    Z: int
    M: int
    batch: int
    array_init: str            # "normal0.01" or "uniform0.01"
    array_dtype: str           # "f32" or "bf16"
    id_dist: str               # "uniform" or "zipf1.05"
    bag_rule: Optional[Tuple[int, int, int]]  # None = one-hot, else (poisson mean, min, max)
    hash_seed: int
    data_seed: int

    def with_(self, **kw) -> "RobeWorkload":
        return replace(self, **kw)


def workload(n: int, **overrides) -> RobeWorkload:
    """The n-th workload (1..5).  Workloads 3 and 5 are families: pass Z=..., M=...,
    array_dtype=... to pick a member."""
    base = {
        1: RobeWorkload("cfg1_tiny", 4, "list", (1000, 500, 2000, 100), 16, 4, 4096, 256,
                        "normal0.01", "f32", "uniform", None, 0x0B0E + 1, 1234 + 1),
        2: RobeWorkload("cfg2_dlrm_infer", 26, "loguniform", (), 128, 32, 25_000_000, 65536,
                        "uniform0.01", "f32", "zipf1.05", None, 0x0B0E + 2, 1234 + 2),
        3: RobeWorkload("cfg3_dlrm_train", 26, "loguniform", (), 128, 128, 25_000_000, 32768,
                        "uniform0.01", "f32", "zipf1.05", None, 0x0B0E + 3, 1234 + 2),
        4: RobeWorkload("cfg4_multihot", 26, "const", (1_000_000,), 64, 16, 250_000_000, 16384,
                        "uniform0.01", "f32", "uniform", (20, 1, 80), 0x0B0E + 4, 1234 + 4),
        5: RobeWorkload("cfg5_sweep", 26, "const", (10_000_000,), 128, 32, 25_000_000, 131072,
                        "uniform0.01", "f32", "uniform", None, 0x0B0E + 5, 1234 + 5),
    }[n]
    return base.with_(**overrides) if overrides else base


def vocab_sizes(w: RobeWorkload) -> np.ndarray:
    if w.vocab_rule == "list":
        v = np.array(w.vocab_arg, dtype=np.int64)
    elif w.vocab_rule == "const":
        v = np.full(w.num_tables, w.vocab_arg[0], dtype=np.int64)
    elif w.vocab_rule == "loguniform":
        rng = np.random.default_rng([w.data_seed, 11])
        v = np.floor(np.exp(rng.uniform(np.log(3.0), np.log(4.0e7), w.num_tables))).astype(np.int64)
    else:
        raise ValueError(w.vocab_rule)
    assert v.shape == (w.num_tables,)
    return v


def _zipf_ranks(rng, vocab: int, n: int, s: float) -> np.ndarray:
    """n draws of a rank in [0, vocab) with P(rank r) proportional to (r+1)^-s."""
    cdf = np.cumsum(np.arange(1, vocab + 1, dtype=np.float64) ** (-s))
    u = rng.random(n) * cdf[-1]
    return np.minimum(np.searchsorted(cdf, u, side="right"), vocab - 1).astype(np.int64)


def make_ids(w: RobeWorkload, batch: Optional[int] = None, variant: int = 0):
    """Returns (indices int64 [nnz], offsets int64 [batch*T+1] or None).

    Bags are sample-major: bag k = n*T + e belongs to table e = k mod T.
    ``variant`` picks an independent batch from the same distribution."""
    B = w.batch if batch is None else batch
    T = w.num_tables
    vocab = vocab_sizes(w)
    rng = np.random.default_rng([w.data_seed, 23, variant])
    if w.bag_rule is None:
        lengths = None
        per_table = np.full(T, B, dtype=np.int64)
    else:
        mean, lo, hi = w.bag_rule
        lengths = np.clip(rng.poisson(mean, size=B * T), lo, hi).astype(np.int64)
        per_table = lengths.reshape(B, T).sum(axis=0)
    # ids are drawn table by table, then placed sample-major
    if lengths is None:
        ids = np.empty((B, T), dtype=np.int64)
        for e in range(T):
            if w.id_dist == "uniform":
                ids[:, e] = rng.integers(0, vocab[e], size=B)
            else:
                ids[:, e] = _zipf_ranks(rng, int(vocab[e]), B, 1.05)
        return ids.reshape(-1), None
    offsets = np.zeros(B * T + 1, dtype=np.int64)
    np.cumsum(lengths, out=offsets[1:])
    nnz = int(offsets[-1])
    table_of = np.repeat(np.tile(np.arange(T, dtype=np.int64), B), lengths)
    indices = np.empty(nnz, dtype=np.int64)
    for e in range(T):
        sel = np.nonzero(table_of == e)[0]
        assert len(sel) == per_table[e]
        if w.id_dist == "uniform":
            indices[sel] = rng.integers(0, vocab[e], size=len(sel))
        else:
            indices[sel] = _zipf_ranks(rng, int(vocab[e]), len(sel), 1.05)
    return indices, offsets


def make_grad_out(w: RobeWorkload, batch: Optional[int] = None, variant: int = 0) -> np.ndarray:
    """Output gradient ~N(0,1), fp32 [batch, T, d]."""
    B = w.batch if batch is None else batch
    rng = np.random.default_rng([w.data_seed, 37, variant])
    return rng.standard_normal((B, w.num_tables, w.d), dtype=np.float32)


# -- array values: a counter-based generator, so a 10 GB array can be filled on the
# -- device chunk by chunk while the host evaluates the very same values pointwise.

_GOLD = 0x9E3779B97F4A7C15
_MUL1 = 0xBF58476D1CE4E5B9
_MUL2 = 0x94D049BB133111EB


def _s64(v: int) -> int:
    v &= (1 << 64) - 1
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(z: torch.Tensor, k: int) -> torch.Tensor:
    return (z >> k) & ((1 << (64 - k)) - 1)


def _mix64(z: torch.Tensor) -> torch.Tensor:
    """SplitMix64 finaliser on int64 tensors (two's-complement wrap-around)."""
    z = (z ^ _lsr(z, 30)) * _s64(_MUL1)
    z = (z ^ _lsr(z, 27)) * _s64(_MUL2)
    return z ^ _lsr(z, 31)


def array_values_at(w: RobeWorkload, j: torch.Tensor) -> torch.Tensor:
    """fp32 initial value of array slot j (int64 tensor, any device).

    uniform0.01: 24 random bits centred and scaled into [-0.01, 0.01) with one
    multiply, so CPU and GPU produce identical bits.  normal0.01: sum of twelve
    16-bit uniforms (Irwin-Hall), variance-matched to N(0, 0.01), also one multiply."""
    key = _s64(w.data_seed * _GOLD + 0x5151)
    z = _mix64((j + 1) * _s64(_GOLD) + key)
    if w.array_init == "uniform0.01":
        u = _lsr(z, 40) - (1 << 23)
        return u.to(torch.float32) * (0.01 / float(1 << 23))
    if w.array_init == "normal0.01":
        z2 = _mix64(z + _s64(_GOLD))
        z3 = _mix64(z2 + _s64(_GOLD))
        total = torch.zeros_like(z)
        for zz in (z, z2, z3):
            for sh in (0, 16, 32, 48):
                total = total + (_lsr(zz, sh) & 0xFFFF)
        centred = total - 6 * 65536 + 6  # mean of the sum of 12 draws of {0..65535} is 6*65535
        return centred.to(torch.float32) * (0.01 / 65536.0)
    raise ValueError(w.array_init)


def to_table_major(indices: np.ndarray, offsets: Optional[np.ndarray], batch: int, num_tables: int):
    """The ids of make_ids with the bags renumbered table by table (bag e*B + n instead of
    n*T + e): the per-table id lists laid end to end.  Returns (indices, offsets)."""
    old_of_new = (np.arange(batch, dtype=np.int64)[None, :] * num_tables
                  + np.arange(num_tables, dtype=np.int64)[:, None]).reshape(-1)
    if offsets is None:
        return np.ascontiguousarray(indices[old_of_new]), None
    lengths = np.diff(offsets)[old_of_new]
    new_offsets = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    starts = offsets[:-1][old_of_new]
    # position of every id of the new order in the old one
    src = np.repeat(starts - new_offsets[:-1], lengths) + np.arange(int(new_offsets[-1]), dtype=np.int64)
    return np.ascontiguousarray(indices[src]), new_offsets


def make_array(w: RobeWorkload, device="cpu", chunk: int = 1 << 25) -> torch.Tensor:
    """The full array [M] on ``device``: fp32, or bf16 (round-to-nearest-even of the fp32 value)."""
    dtype = torch.float32 if w.array_dtype == "f32" else torch.bfloat16
    out = torch.empty(w.M, dtype=dtype, device=device)
    for lo in range(0, w.M, chunk):
        hi = min(w.M, lo + chunk)
        j = torch.arange(lo, hi, dtype=torch.int64, device=device)
        out[lo:hi] = array_values_at(w, j).to(dtype)
    return out


def array_to_numpy(a: torch.Tensor) -> np.ndarray:
    """Host view the oracle accepts: float32, or the raw bf16 bit patterns as uint16."""
    a = a.detach().cpu().contiguous()
    if a.dtype == torch.bfloat16:
        return a.view(torch.int16).numpy().view(np.uint16)
    return a.numpy()
