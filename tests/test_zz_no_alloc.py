"""robe_backward_deterministic_static: the deterministic backward for callers that cannot hand
the library a workspace (a process whose memory pool owns the whole device, or an operator that
is given input and output buffers only).  Its scratch is an array inside the library image, so
it allocates nothing; the checks here are that it gives the same bits as robe_backward with a
caller-provided workspace and as the CPU oracle's canonical-order gradient, on two calls in a
row that leave different stale contents behind, that the device's free memory does not move
across the calls, and that a call too large for the fixed array is refused.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test."""
import gc

import numpy as np
import pytest
import torch

import paper_2108_02191_b200 as robe
from paper_2108_02191_b200 import synth
from robe_testlib import Case, assert_bits_equal

pytestmark = pytest.mark.gpu


def _workload(**kw):
    base = dict(name="noalloc", num_tables=5, vocab_rule="list", vocab_arg=(50, 7, 1000, 3, 20000),
                d=48, Z=8, M=20011, batch=700, array_init="normal0.01", array_dtype="f32",
                id_dist="uniform", bag_rule=(4, 0, 11), hash_seed=91, data_seed=8)
    base.update(kw)
    return synth.RobeWorkload(**base)


def _grad(c, seed):
    g = np.random.default_rng(seed).standard_normal((c.B, c.T, c.w.d), dtype=np.float32)
    return torch.from_numpy(g).to(c.dev)


def _reference_dense(c, g_d):
    """robe_backward, deterministic mode, workspace allocated by the caller."""
    return c.backward(g_d, "det").cpu().numpy()


def _oracle_dense(c, g_d):
    """The CPU oracle's canonical-order fp32 gradient of the same inputs."""
    can, _ = c.oracle.backward_canonical(g_d.cpu().numpy(), c.indices_h, c.offsets_h, c.B)
    return can


def _static_dense(c, g_d):
    ga = torch.zeros(c.w.M, dtype=torch.float32, device=c.dev)
    robe.robe_backward_deterministic_static(c.h, g_d, c.indices, c.offsets, c.B, ga, 0.0)
    torch.cuda.synchronize()
    return ga.cpu().numpy()


def test_two_calls_in_a_row_match_the_workspace_variant():
    # first a pooled call with many blocks, then a smaller one-hot call with another shape: the
    # second call finds the first one's keys, values, counters and bag numbers in the array
    big = _workload()
    small = _workload(d=16, Z=16, M=997, batch=90, bag_rule=None, num_tables=3, vocab_arg=(9, 400, 2))
    with Case(big) as c1, Case(small) as c2:
        g1, g2 = _grad(c1, 1), _grad(c2, 2)
        want1, want2 = _reference_dense(c1, g1), _reference_dense(c2, g2)
        # a first call so that the module holding the fixed array and the cached symbol address
        # are loaded; what is measured below is the steady state
        _static_dense(c2, g2)
        ga1 = torch.zeros(c1.w.M, dtype=torch.float32, device=c1.dev)
        ga2 = torch.zeros(c2.w.M, dtype=torch.float32, device=c2.dev)
        gc.collect()  # tensors of earlier tests that only the collector frees would move the figures
        torch.cuda.synchronize()
        pool_before = torch.cuda.memory_allocated()
        free_before = torch.cuda.mem_get_info()[0]  # cudaMemGetInfo: sees every allocation on the device
        robe.robe_backward_deterministic_static(c1.h, g1, c1.indices, c1.offsets, c1.B, ga1, 0.0)
        robe.robe_backward_deterministic_static(c2.h, g2, c2.indices, c2.offsets, c2.B, ga2, 0.0)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before   # no cudaMalloc inside the library
        assert torch.cuda.memory_allocated() == pool_before   # and nothing taken from torch's pool
        got1, got2 = ga1.cpu().numpy(), ga2.cpu().numpy()
        assert_bits_equal(got1, want1, "static scratch, first call")
        assert_bits_equal(got2, want2, "static scratch, second call")
        assert_bits_equal(got1, _oracle_dense(c1, g1), "static scratch, first call, against the oracle")
        assert_bits_equal(got2, _oracle_dense(c2, g2), "static scratch, second call, against the oracle")
        # and once more in the other order, with the sign hash on
        robe.robe_set_option(c1.h, robe.ROBE_OPT_SIGN, 1)
        want1s = _reference_dense(c1, g1)
        assert_bits_equal(_static_dense(c2, g2), want2, "static scratch, third call")
        assert_bits_equal(_static_dense(c1, g1), want1s, "static scratch, fourth call (sign)")
        c1.oracle.sign = 1
        assert_bits_equal(want1s, _oracle_dense(c1, g1), "sign on, against the oracle")


def test_fused_sgd_matches_the_workspace_variant():
    w = _workload()
    with Case(w) as ref, Case(w) as sta:
        g = _grad(ref, 3)
        from oracle import robe_oracle as orc
        can, touched = ref.oracle.backward_canonical(g.cpu().numpy(), ref.indices_h, ref.offsets_h, ref.B)
        want = ref.array_h.copy()
        orc.sgd_apply(want, can, touched, 0.25)
        ref.backward(g, "det", sgd=True, lr=0.25)
        robe.robe_backward_deterministic_static(sta.h, g, sta.indices, sta.offsets, sta.B, None, 0.25)
        torch.cuda.synchronize()
        assert_bits_equal(sta.array.cpu().numpy(), ref.array.cpu().numpy(), "static scratch SGD step 1")
        assert_bits_equal(sta.array.cpu().numpy(), want, "static scratch SGD step 1, against the oracle")
        ref.backward(g, "det", sgd=True, lr=0.25)
        robe.robe_backward_deterministic_static(sta.h, g, sta.indices, sta.offsets, sta.B, None, 0.25)
        torch.cuda.synchronize()
        assert_bits_equal(sta.array.cpu().numpy(), ref.array.cpu().numpy(), "static scratch SGD step 2")


def test_largest_and_too_large_calls():
    # one-hot, Z = d: one block per id
    w = _workload(d=32, Z=32, M=100003, bag_rule=None, num_tables=4, vocab_arg=(100, 10**6, 5, 77))
    with Case(w, batch=8) as c:
        robe.robe_set_option(c.h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_DETERMINISTIC)
        limit = robe.ROBE_STATIC_SCRATCH_BYTES
        need = lambda b: robe.robe_backward_workspace_bytes(c.h, b, b * c.T)
        lo, hi = 1, 1 << 22  # the largest batch whose workspace fits, by bisection
        assert need(lo) <= limit < need(hi)
        while hi - lo > 1:
            mid = (lo + hi) // 2
            lo, hi = (mid, hi) if need(mid) <= limit else (lo, mid)
        fits, too_big = lo, lo + 64
        assert need(fits) <= limit < need(too_big)
    with Case(w, batch=too_big) as c:
        g = torch.zeros(c.B, c.T, w.d, device=c.dev)
        ga = torch.zeros(w.M, device=c.dev)
        with pytest.raises(robe.RobeError) as ei:
            robe.robe_backward_deterministic_static(c.h, g, c.indices, None, c.B, ga, 0.0)
        assert ei.value.status == robe.ROBE_ERR_WORKSPACE
        assert not ga.any()  # nothing was launched
    with Case(w, batch=fits) as c:  # close to the limit: the whole array is in use
        g = _grad(c, 4)
        assert_bits_equal(_static_dense(c, g), _reference_dense(c, g), "static scratch at its limit")
