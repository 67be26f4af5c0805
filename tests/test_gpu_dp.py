"""Data-parallel step on the GPU: robe_apply_sgd against the oracle's dense apply, and the step
backward -> all-reduce (NCCL, one rank) -> apply against the fused SGD step and the oracle."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist

import paper_2108_02191_b200 as robe
from oracle import robe_oracle as orc
from paper_2108_02191_b200 import dp, synth
from robe_testlib import Case, assert_bits_equal, assert_within_l1

pytestmark = pytest.mark.gpu


def _small(**kw):
    base = dict(name="dp", num_tables=3, vocab_rule="list", vocab_arg=(50, 7, 1000), d=16, Z=4, M=1000,
                batch=333, array_init="normal0.01", array_dtype="f32", id_dist="uniform", bag_rule=None,
                hash_seed=77, data_seed=5)
    base.update(kw)
    return synth.RobeWorkload(**base)


@pytest.mark.parametrize("M", [1, 3, 4, 5, 1000, 4099, 1_000_003, 8 * 1024 * 1024 + 2])
def test_apply_sgd_matches_oracle(M):
    w = _small(M=M, d=1, Z=1)
    with Case(w, batch=2) as c:
        rng = np.random.default_rng(M)
        g_h = rng.standard_normal(M).astype(np.float32)
        g_h[::7] = 0.0
        for zero in (False, True):
            before = c.array.cpu().numpy().copy()
            g_d = torch.from_numpy(g_h).to(c.dev)
            robe.robe_apply_sgd(c.h, g_d, 0.37, zero)
            torch.cuda.synchronize()
            want = before.copy()
            orc.dense_sgd_apply(want, g_h, 0.37)
            assert_bits_equal(c.array.cpu().numpy(), want, f"dense apply M={M} zero={zero}")
            if zero:
                assert not g_d.any() and not torch.signbit(g_d).any()
            else:
                assert_bits_equal(g_d.cpu().numpy(), g_h, "gradient left as it was")


def test_apply_sgd_argument_errors():
    with Case(_small()) as c:
        g = torch.zeros(c.w.M + 1, device=c.dev)
        with pytest.raises(robe.RobeError) as ei:
            robe.robe_apply_sgd(c.h, g[1:], 0.1)  # 4 bytes off a 16-byte boundary
        assert ei.value.status == robe.ROBE_ERR_INVALID_ARG
    with Case(_small(array_dtype="bf16")) as c:
        with pytest.raises(robe.RobeError) as ei:
            robe.robe_apply_sgd(c.h, torch.zeros(c.w.M, device=c.dev), 0.1)
        assert ei.value.status == robe.ROBE_ERR_INVALID_ARG


@pytest.fixture
def nccl_one_rank():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda:0"))
    try:
        yield
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("bags", [None, (3, 0, 9)])
def test_dp_step_equals_fused_step_on_one_rank(nccl_one_rank, bags):
    # deterministic mode: bit for bit the fused step; atomic mode: within the atomic bound of the oracle
    for w in (_small(bag_rule=bags), _small(d=64, Z=16, M=300_007, batch=1500, bag_rule=bags,
                                             vocab_arg=(10**6, 10**6, 50_000))):
        with Case(w) as fused, Case(w) as stepd:
            g_h = np.random.default_rng(3).standard_normal((fused.B, fused.T, w.d)).astype(np.float32)
            g_d = torch.from_numpy(g_h).to(fused.dev)
            before = fused.array_h.copy()
            fused.backward(g_d, "det", sgd=True, lr=0.25)
            robe.robe_set_option(stepd.h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_DETERMINISTIC)
            ws = torch.empty(robe.robe_backward_workspace_bytes(stepd.h, stepd.B, stepd.indices.numel()),
                             dtype=torch.uint8, device=stepd.dev)
            ga = torch.zeros(w.M, device=stepd.dev)
            for _ in range(2):  # two steps: the gradient buffer comes back zeroed
                dp.robe_dp_step(stepd.h, g_d, stepd.indices, stepd.offsets, stepd.B, ga, 0.25, ws)
            fused.backward(g_d, "det", sgd=True, lr=0.25)
            torch.cuda.synchronize()
            assert_bits_equal(stepd.array.cpu().numpy(), fused.array.cpu().numpy(), "dp step, deterministic")
            assert not ga.any()
            assert dp.replicas_identical(stepd.array)
            # against the oracle: canonical gradient, dense apply (first step only)
            can, touched = fused.oracle.backward_canonical(g_h, fused.indices_h, fused.offsets_h, fused.B)
            want = before.copy()
            orc.dense_sgd_apply(want, np.where(touched == 1, can, np.float32(0)).astype(np.float32), 0.25)
        with Case(w) as one:
            robe.robe_set_option(one.h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_DETERMINISTIC)
            ga = torch.zeros(w.M, device=one.dev)
            dp.robe_dp_step(one.h, g_d, one.indices, one.offsets, one.B, ga, 0.25, ws)
            torch.cuda.synchronize()
            assert_bits_equal(one.array.cpu().numpy(), want, "dp step vs oracle")
        with Case(w) as atom:
            d64, l1 = atom.oracle.backward_f64(g_h, atom.indices_h, atom.offsets_h, atom.B)
            robe.robe_set_option(atom.h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_ATOMIC)
            ga = torch.zeros(w.M, device=atom.dev)
            dp.robe_dp_step(atom.h, g_d, atom.indices, atom.offsets, atom.B, ga, 0.25, None)
            torch.cuda.synchronize()
            assert_within_l1(atom.array.cpu().numpy(), before.astype(np.float64) - 0.25 * d64,
                             0.25 * l1 + np.abs(before), what="dp step, atomic")
