"""Parity of the CUDA library (called through its C ABI binding) with the CPU oracle.

Bars: forward bit-exact; atomic backward within 1e-5 of the per-slot L1 gradient mass;
deterministic backward bit-exact with the oracle's canonical-order fp32 gradient."""
import numpy as np
import pytest
import torch

import paper_2108_02191_b200 as robe
from oracle import robe_oracle as orc
from paper_2108_02191_b200 import synth
from robe_testlib import Case, assert_bits_equal, assert_within_l1

pytestmark = pytest.mark.gpu

FWD_KERNELS = [0, 1, 2]  # automatic, direct, staged


def small(**kw):
    """A small workload that still spans several CTAs and a ragged tail."""
    base = dict(name="small", num_tables=3, vocab_rule="list", vocab_arg=(50, 7, 1000), d=16, Z=4,
                M=1000, batch=333, array_init="normal0.01", array_dtype="f32", id_dist="uniform",
                bag_rule=None, hash_seed=77, data_seed=5)
    base.update(kw)
    return synth.RobeWorkload(**base)


# ---------------------------------------------------------------------------------------
# forward
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("sign", [False, True])
@pytest.mark.parametrize("kernel", FWD_KERNELS)
def test_cfg1_forward(kernel, sign):
    with Case(synth.workload(1), sign=sign) as c:
        assert_bits_equal(c.forward(kernel).cpu().numpy(), c.oracle_forward(), "cfg1 forward")


SHAPES = [
    # (d, Z, M) - powers of two, ragged, Z not dividing d, tiny arrays that wrap all the time
    (16, 4, 1000), (16, 16, 17), (16, 4, 17), (16, 1, 16), (1, 1, 1), (1, 1, 5), (2, 2, 3),
    (128, 1, 4099), (128, 2, 4099), (128, 8, 4099), (128, 32, 129), (128, 128, 128),
    (128, 128, 100003), (64, 16, 70), (100, 32, 1013), (96, 64, 1013), (33, 1, 64), (7, 2, 9),
    (12, 5, 64), (48, 3, 49), (130, 2, 1000), (200, 64, 777), (256, 1, 513), (37, 37, 37),
    # Z > d: rows clubbed into one block (R = Z/d = 4, 3, 4 with constant wrapping, 2, 2, 4, 2)
    (16, 64, 1000), (16, 48, 1000), (8, 32, 33), (64, 128, 5000), (128, 256, 100003), (1, 4, 7),
    (160, 320, 999),
]


@pytest.mark.parametrize("bags", [None, (3, 0, 9)])
@pytest.mark.parametrize("d,Z,M", SHAPES)
def test_forward_shapes(d, Z, M, bags):
    w = small(d=d, Z=Z, M=M, bag_rule=bags, batch=97)
    for sign in (False, True):
        with Case(w, sign=sign) as c:
            want = c.oracle_forward()
            warp_ok = d <= 128
            lane_hashed_ok = warp_ok and Z <= d and not sign  # kernel 4: every lane hashes its own chunks
            for kernel in ([0, 1, 2] if warp_ok else [0, 1]) + ([4] if lane_hashed_ok else []):
                assert_bits_equal(c.forward(kernel).cpu().numpy(), want, f"d={d} Z={Z} M={M} k={kernel}")
            if not warp_ok:
                with pytest.raises(robe.RobeError):
                    c.forward(2)
            if not lane_hashed_ok:
                with pytest.raises(robe.RobeError):
                    c.forward(4)


# The kernel with 16-byte loads (ROBE_OPT_FWD_KERNEL = 3): fp32 array, d, Z and M multiples of
# four, sign off.  Shapes: every lanes-per-id count (d/4 = 1 .. 32, powers of two and not), blocks
# of one vector and of many, arrays so short that every batch wraps, rows clubbed into one block.
VEC_SHAPES = [(16, 4, 1000), (16, 4, 20), (16, 16, 16), (64, 16, 68), (64, 16, 250_000), (128, 32, 132),
              (128, 128, 128), (128, 128, 100_004), (128, 4, 4096), (32, 8, 36), (96, 32, 100), (100, 20, 1000),
              (12, 4, 64), (8, 8, 8), (4, 4, 4), (48, 12, 52), (16, 64, 1000), (64, 128, 5000), (128, 8, 262_144)]


@pytest.mark.parametrize("bags", [None, (3, 0, 9), (20, 1, 80)])
@pytest.mark.parametrize("d,Z,M", VEC_SHAPES)
def test_forward_vector_kernel(d, Z, M, bags):
    w = small(d=d, Z=Z, M=M, bag_rule=bags, batch=97)
    with Case(w) as c:
        want = c.oracle_forward()
        assert_bits_equal(c.forward(3).cpu().numpy(), want, f"vector kernel d={d} Z={Z} M={M}")
        # int32 ids and the forward that keeps its block starts go through the same kernel
        g_h, g_d = _grad(c, 4)
        can, _ = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
        robe.robe_set_option(c.h, robe.ROBE_OPT_FWD_KERNEL, 3)
        out, det = c.step_sharing_keys(g_d, "det", fwd_kernel=3)
        assert_bits_equal(out.cpu().numpy(), want, "vector kernel that keeps")
        assert_bits_equal(det.cpu().numpy(), can, "deterministic on the vector kernel's kept starts")
        c.indices = c.indices.to(torch.int32)
        assert_bits_equal(c.forward(3).cpu().numpy(), want, "vector kernel, int32 ids")


def test_forward_vector_kernel_refuses_what_it_cannot_do():
    for kw in (dict(d=16, Z=4, M=1001), dict(d=16, Z=2, M=1000), dict(d=18, Z=6, M=1000),
               dict(d=16, Z=4, M=1000, array_dtype="bf16"), dict(d=256, Z=4, M=1000)):
        with Case(small(**kw)) as c:
            with pytest.raises(robe.RobeError):
                c.forward(3)
    with Case(small(), sign=True) as c:
        with pytest.raises(robe.RobeError):
            c.forward(3)


def test_two_handles_of_different_dimension_share_one_array():
    # Section 3.1, multiple embedding tables: tables of different embedding size live in the same array.
    # One handle per dimension, both attached to the same device array; a fused SGD step through one
    # handle is what the other one reads afterwards.
    wa = small(d=16, Z=4, M=5003, hash_seed=11)
    wb = small(d=48, Z=16, M=5003, hash_seed=12, num_tables=2, vocab_arg=(300, 9), bag_rule=(3, 0, 9))
    with Case(wa) as a, Case(wb, array=a.array) as b:
        assert b.array.data_ptr() == a.array.data_ptr()
        assert_bits_equal(a.forward().cpu().numpy(), a.oracle_forward(), "handle A")
        assert_bits_equal(b.forward().cpu().numpy(), b.oracle_forward(), "handle B")
        g_h, g_d = _grad(a, 9)
        can, touched = a.oracle.backward_canonical(g_h, a.indices_h, a.offsets_h, a.B)
        a.backward(g_d, "det", sgd=True, lr=0.5)
        orc.sgd_apply(b.array_h, can, touched, 0.5)   # the oracle twin of the shared array
        assert_bits_equal(b.array.cpu().numpy(), b.array_h, "shared array after A's step")
        assert_bits_equal(b.forward().cpu().numpy(), b.oracle_forward(), "handle B reads A's update")


def test_forward_bf16_array():
    w = small(array_dtype="bf16", d=64, Z=16, M=5000, bag_rule=(4, 0, 12))
    with Case(w) as c:
        want = c.oracle_forward()
        for kernel in FWD_KERNELS + [4]:
            assert_bits_equal(c.forward(kernel).cpu().numpy(), want, "bf16")
    for Z in (1, 2):  # short blocks take the lane-hashed kernel by themselves
        with Case(small(array_dtype="bf16", d=96, Z=Z, M=5003, bag_rule=(4, 0, 12))) as c:
            assert_bits_equal(c.forward().cpu().numpy(), c.oracle_forward(), "bf16, short blocks")


@pytest.mark.parametrize("bags", [None, (3, 0, 9)])
def test_int32_indices(bags):
    # the same ids as int32: identical bits out of every kernel
    for w in (synth.workload(1).with_(bag_rule=bags), small(d=128, Z=32, M=4099, bag_rule=bags, batch=97),
              small(d=16, Z=64, M=1000, bag_rule=bags, batch=97)):
        for sign in (False, True):
            with Case(w, sign=sign) as c:
                want = c.oracle_forward()
                g_h, g_d = _grad(c, 7)
                delta64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B)
                can, _ = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
                c.indices = c.indices.to(torch.int32)
                for kernel in FWD_KERNELS:
                    assert_bits_equal(c.forward(kernel).cpu().numpy(), want, "int32 ids forward")
                for kernel in (1, 2):
                    assert_within_l1(c.backward(g_d, "atomic", kernel=kernel).cpu().numpy(), delta64, l1,
                                     what="int32 ids atomic")
                assert_bits_equal(c.backward(g_d, "det").cpu().numpy(), can, "int32 ids deterministic")


def test_forward_lane_hashed_kernel_many_tables_and_large_ids():
    # more tables than the kernel keeps table terms for in shared memory; ids beyond 2^32
    T = 700
    w = small(num_tables=T, vocab_arg=tuple([2**40 + 12345] * T), d=40, Z=1, M=3001, batch=9)
    with Case(w) as c:
        assert_bits_equal(c.forward(4).cpu().numpy(), c.oracle_forward(), "lane-hashed, 700 tables")
    w = small(num_tables=T, vocab_arg=tuple([2**40 + 12345] * T), d=40, Z=2, M=3001, batch=9, bag_rule=(3, 0, 70))
    with Case(w) as c:
        assert_bits_equal(c.forward(4).cpu().numpy(), c.oracle_forward(), "lane-hashed, 700 tables, bags")


def test_forward_empty_and_degenerate_inputs():
    w = small(bag_rule=(2, 0, 5))
    with Case(w, batch=4) as c:
        # all bags empty
        c.offsets = torch.zeros(c.nbags + 1, dtype=torch.int64, device=c.dev)
        c.indices = torch.zeros(0, dtype=torch.int64, device=c.dev)
        out = c.forward().cpu().numpy()
        assert np.all(out == 0) and not np.any(np.signbit(out))
    with Case(small(), batch=1) as c:
        assert_bits_equal(c.forward().cpu().numpy(), c.oracle_forward(), "batch 1")
    with Case(small()) as c:
        # batch 0 launches nothing and succeeds
        out = torch.empty(0, c.T, c.w.d, device=c.dev)
        robe.robe_forward(c.h, torch.zeros(0, dtype=torch.int64, device=c.dev), None, 0, out)


def test_forward_huge_ids_and_negative_zero():
    # ids up to 2^63-1 go through the full 128-bit product; -0.0 in the array must survive
    # (the first term initialises the sum: +0 + -0 would turn it into +0)
    w = small(d=8, Z=4, M=64, num_tables=1, vocab_arg=(10,), bag_rule=(2, 1, 3))
    ids = np.array([2**63 - 1, 2**62 + 12345, (1 << 61) - 1, 1 << 61, 5, 5, 2**40 + 1], dtype=np.int64)
    offsets = np.array([0, 1, 2, 3, 4, 6, 7], dtype=np.int64)
    arr = torch.full((64,), -0.0, dtype=torch.float32)
    with Case(w, batch=6, ids=(ids, offsets), array=arr) as c:
        got = c.forward().cpu().numpy()
        want = c.oracle_forward()
        assert_bits_equal(got, want, "huge ids / -0")
        assert np.all(np.signbit(got))


def test_forward_max_array_size():
    # M + d = 2^32: block starts near 2^32 must not overflow 32-bit slot arithmetic.  The array
    # (bf16, 8.6 GB) is filled on the device by the counter-based generator; the oracle side
    # evaluates the same generator only at the slots it needs.
    d, Z = 128, 128
    M = (1 << 32) - d
    w = synth.workload(5, M=M, Z=Z, array_dtype="bf16", batch=64)
    free, _ = torch.cuda.mem_get_info()
    if free < 12 * 2**30:
        pytest.skip("not enough free device memory")
    with Case(w, host_array=False) as c:
        got = c.forward().cpu().numpy().reshape(c.nbags, d)
        near_end = 0
        for bag in range(0, c.nbags, 7):
            slots = c.oracle.locate(bag % c.T, int(c.indices_h[bag])).astype(np.int64)
            near_end += int(slots.max() > (1 << 32) - 4 * d)
            want = synth.array_values_at(w, torch.from_numpy(slots)).to(torch.bfloat16).to(torch.float32)
            assert_bits_equal(got[bag], want.numpy(), "max M")
    # force blocks that wrap around the very end: solve B*x = v - D - A*e (mod P) for a start v
    # within d of M (Python integers; the library only hands out its constants)
    with Case(w.with_(batch=1), host_array=False) as c:
        P_, A_, B_, _, D_ = [int(v) for v in robe.robe_get_hash_constants(c.h)[:5]]
        starts = [M - 1, M - 5, M - d + 1, M - 64]
        found = [((v - D_) * pow(B_, -1, P_)) % P_ for v in starts]
        ids = np.zeros((len(found), c.T), dtype=np.int64)
        ids[:, 0] = found
        c.B, c.nbags = len(found), len(found) * c.T
        c.indices_h = ids.reshape(-1)
        c.indices = torch.from_numpy(c.indices_h).to(c.dev)
        got = c.forward().cpu().numpy()
        for r, (xx, v) in enumerate(zip(found, starts)):
            assert c.oracle.h(0, int(xx), 0) == v
            slots = c.oracle.locate(0, int(xx)).astype(np.int64)
            assert slots.max() == M - 1 and slots.min() == 0
            want = synth.array_values_at(w, torch.from_numpy(slots)).to(torch.bfloat16).to(torch.float32)
            assert_bits_equal(got[r, 0], want.numpy(), "wrap at 2^32")


# ---------------------------------------------------------------------------------------
# backward, small shapes: all modes
# ---------------------------------------------------------------------------------------

def _grad(c, seed=0, integer=False):
    rng = np.random.default_rng(seed)
    if integer:
        g = rng.integers(-4, 5, size=(c.B, c.T, c.w.d)).astype(np.float32)
    else:
        g = rng.standard_normal((c.B, c.T, c.w.d), dtype=np.float32)
    return g, torch.from_numpy(g).to(c.dev)


BWD_SHAPES = [
    (16, 4, 4096), (16, 16, 17), (16, 4, 17), (1, 1, 1), (2, 2, 3), (128, 1, 4099), (128, 8, 4099),
    (128, 32, 129), (128, 128, 128), (64, 16, 70), (100, 32, 1013), (12, 5, 64), (48, 3, 49),
    (130, 2, 1000), (200, 64, 777), (37, 37, 37), (16, 8, 5000),
    (16, 64, 1000), (16, 48, 1000), (8, 32, 33), (64, 128, 5000), (1, 4, 7), (160, 320, 999),
]


@pytest.mark.parametrize("bags", [None, (3, 0, 9)])
@pytest.mark.parametrize("d,Z,M", BWD_SHAPES)
def test_backward_shapes(d, Z, M, bags):
    w = small(d=d, Z=Z, M=M, bag_rule=bags, batch=61)
    for sign in (False, True):
        with Case(w, sign=sign) as c:
            g_h, g_d = _grad(c, 1)
            delta64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B)
            can, touched = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
            warp_ok = d <= 128
            lane_hashed_ok = warp_ok and Z <= d and not sign  # kernel 6: every lane hashes its own chunks
            for kernel in ([0, 1, 2] if warp_ok else [0, 1]) + ([6] if lane_hashed_ok else []):
                ga = c.backward(g_d, "atomic", kernel=kernel).cpu().numpy()
                assert_within_l1(ga, delta64, l1, what=f"atomic d={d} Z={Z} M={M} k={kernel}")
            if not lane_hashed_ok:
                with pytest.raises(robe.RobeError):
                    c.backward(g_d, "atomic", kernel=6)
            gb = c.backward(g_d, "binned").cpu().numpy()
            assert_within_l1(gb, delta64, l1, what=f"binned d={d} Z={Z} M={M}")
            det = c.backward(g_d, "det").cpu().numpy()
            assert_bits_equal(det, can, f"deterministic d={d} Z={Z} M={M} sign={sign}")
            # integer gradients: every order gives the same bits, so atomic == canonical == fp64
            gi_h, gi_d = _grad(c, 2, integer=True)
            di, _ = c.oracle.backward_f64(gi_h, c.indices_h, c.offsets_h, c.B)
            assert_bits_equal(c.backward(gi_d, "atomic").cpu().numpy(), di.astype(np.float32), "int atomic")
            assert_bits_equal(c.backward(gi_d, "det").cpu().numpy(), di.astype(np.float32), "int det")


# Atomic backward with 16-byte reductions (ROBE_OPT_BWD_KERNEL = 3) and with the duplicates of an
# id merged in the warp first (4): the forward vector kernel's shapes, uniform ids and ids so
# skewed that most rows of a batch repeat one id.
@pytest.mark.parametrize("bags", [None, (3, 0, 9), (20, 1, 80)])
@pytest.mark.parametrize("d,Z,M", VEC_SHAPES)
def test_backward_vector_kernels(d, Z, M, bags):
    for vocab, dist_ in (((50, 7, 1000), "uniform"), ((3, 2, 40), "zipf1.05")):
        w = small(d=d, Z=Z, M=M, bag_rule=bags, batch=131, vocab_arg=vocab, id_dist=dist_)
        with Case(w) as c:
            g_h, g_d = _grad(c, 6)
            delta64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B)
            gi_h, gi_d = _grad(c, 2, integer=True)
            di, _ = c.oracle.backward_f64(gi_h, c.indices_h, c.offsets_h, c.B)
            for kernel in (3, 4) + ((5,) if bags is None else ()):
                ga = c.backward(g_d, "atomic", kernel=kernel).cpu().numpy()
                assert_within_l1(ga, delta64, l1, what=f"vector atomic k={kernel} d={d} Z={Z} M={M} {dist_}")
                # integer gradients: exact whatever the order and the grouping
                assert_bits_equal(c.backward(gi_d, "atomic", kernel=kernel).cpu().numpy(),
                                  di.astype(np.float32), f"vector atomic k={kernel}, integer gradient")
            before = c.array_h.copy()
            c.backward(g_d, "atomic", sgd=True, lr=0.5, kernel=4)
            assert_within_l1(c.array.cpu().numpy(), before.astype(np.float64) - 0.5 * delta64,
                             0.5 * l1 + np.abs(before), what="vector atomic sgd")


# Kernel 5: one-hot rows taken table by table and the repeats of an id merged in the warp before
# the reduction; any (d, Z, M) the staged kernel takes, both bag numberings, batches that do not
# fill the last warp, ids so skewed that most rows of a batch repeat one id.
@pytest.mark.parametrize("table_major", [False, True])
@pytest.mark.parametrize("d,Z,M", [(16, 4, 4096), (128, 128, 1280), (128, 32, 129), (128, 1, 4099), (64, 16, 70),
                                   (100, 32, 1013), (12, 5, 64), (33, 1, 64), (16, 64, 1000), (1, 1, 1)])
def test_backward_merged_rows_kernel(d, Z, M, table_major):
    for vocab, dist_, batch in (((50, 7, 1000), "uniform", 131), ((3, 2, 40), "zipf1.05", 200), ((1, 1, 1), "uniform", 65)):
        w = small(d=d, Z=Z, M=M, batch=batch, vocab_arg=vocab, id_dist=dist_)
        with Case(w, table_major=table_major) as c:
            rng = np.random.default_rng(8)
            shape = (c.T, c.B, d) if table_major else (c.B, c.T, d)
            g_h = rng.standard_normal(shape).astype(np.float32)
            gi_h = rng.integers(-4, 5, size=shape).astype(np.float32)
            delta64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B)
            di, _ = c.oracle.backward_f64(gi_h, c.indices_h, c.offsets_h, c.B)
            ga = c.backward(torch.from_numpy(g_h).to(c.dev), "atomic", kernel=5).cpu().numpy()
            assert_within_l1(ga, delta64, l1, what=f"merged rows d={d} Z={Z} M={M} {dist_} tm={table_major}")
            assert_bits_equal(c.backward(torch.from_numpy(gi_h).to(c.dev), "atomic", kernel=5).cpu().numpy(),
                              di.astype(np.float32), "merged rows, integer gradient")
    with Case(small(d=d, Z=Z, M=M, bag_rule=(3, 0, 9))) as c:  # pooled input is refused
        _, g_d = _grad(c, 1)
        with pytest.raises(robe.RobeError):
            c.backward(g_d, "atomic", kernel=5)


@pytest.mark.parametrize("mode", ["atomic", "det"])
def test_cfg1_backward_dense_and_sgd(mode):
    for sign in (False, True):
        with Case(synth.workload(1), sign=sign) as c:
            g_h = synth.make_grad_out(c.w)
            g_d = torch.from_numpy(g_h).to(c.dev)
            delta64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B)
            can, touched = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
            ga = c.backward(g_d, mode).cpu().numpy()
            if mode == "atomic":
                assert_within_l1(ga, delta64, l1, what="cfg1 atomic")
            else:
                assert_bits_equal(ga, can, "cfg1 det")
            # accumulation into a non-zero gradient array
            pre = torch.from_numpy(np.random.default_rng(3).standard_normal(c.w.M).astype(np.float32))
            ga2 = c.backward(g_d, mode, grad_array=pre.to(c.dev).clone()).cpu().numpy()
            if mode == "det":
                want = pre.numpy().copy()
                orc.accumulate(want, can, touched)
                assert_bits_equal(ga2, want, "cfg1 det accumulate")
            else:
                assert_within_l1(ga2 - pre.numpy(), delta64, l1 + np.abs(pre.numpy()), what="cfg1 atomic acc")
            # fused SGD step
            lr = 0.5
            before = c.array_h.copy()
            c.backward(g_d, mode, sgd=True, lr=lr)
            after = c.array.cpu().numpy()
            if mode == "det":
                want = before.copy()
                orc.sgd_apply(want, can, touched, lr)
                assert_bits_equal(after, want, "cfg1 det sgd")
            else:
                assert_within_l1(after, before.astype(np.float64) - lr * delta64,
                                 lr * l1 + np.abs(before), what="cfg1 atomic sgd")
                assert_bits_equal(after[l1 == 0], before[l1 == 0], "untouched slots")


@pytest.mark.parametrize("bags", [None, (3, 0, 9)])
def test_backward_adam_matches_oracle_over_steps(bags):
    # three Adam steps in a row (array and moments carried over), bit for bit
    lr, b1, b2, eps = 0.05, 0.9, 0.999, 1e-8
    for w in (synth.workload(1).with_(bag_rule=bags), small(d=64, Z=16, M=70, bag_rule=bags, batch=200),
              small(d=16, Z=64, M=1000, bag_rule=bags, batch=97, vocab_arg=(3, 7, 1000))):
        with Case(w) as c:
            robe.robe_set_option(c.h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_DETERMINISTIC)
            ws = torch.empty(robe.robe_backward_workspace_bytes(c.h, c.B, c.indices.numel()),
                             dtype=torch.uint8, device=c.dev)
            m1_d = torch.zeros(w.M, device=c.dev)
            m2_d = torch.zeros(w.M, device=c.dev)
            arr, m1, m2 = c.array_h.copy(), np.zeros(w.M, np.float32), np.zeros(w.M, np.float32)
            for step in (1, 2, 3):
                g_h, g_d = _grad(c, 10 + step)
                can, touched = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
                orc.adam_apply(arr, m1, m2, can, touched, lr, b1, b2, eps, step)
                robe.robe_backward_adam(c.h, g_d, c.indices, c.offsets, c.B, m1_d, m2_d, lr, b1, b2, eps,
                                        step, ws)
                torch.cuda.synchronize()
                assert_bits_equal(c.array.cpu().numpy(), arr, f"adam array, step {step}")
                assert_bits_equal(m1_d.cpu().numpy(), m1, f"adam first moment, step {step}")
                assert_bits_equal(m2_d.cpu().numpy(), m2, f"adam second moment, step {step}")
            with pytest.raises(robe.RobeError):
                robe.robe_backward_adam(c.h, g_d, c.indices, c.offsets, c.B, m1_d, m2_d, lr, 1.0, b2, eps, 1, ws)
            with pytest.raises(robe.RobeError):
                robe.robe_backward_adam(c.h, g_d, c.indices, c.offsets, c.B, m1_d, m2_d, lr, b1, b2, eps, 0, ws)


@pytest.mark.parametrize("bags", [None, (3, 0, 9)])
def test_backward_adagrad_matches_oracle_over_steps(bags):
    # three Adagrad steps in a row (array and accumulators carried over), bit for bit; the dense
    # window apply, the position-tile apply and rows clubbed into one block
    lr, eps = 0.05, 1e-8
    for w in (synth.workload(1).with_(bag_rule=bags), small(d=64, Z=16, M=70, bag_rule=bags, batch=200),
              small(d=16, Z=64, M=1000, bag_rule=bags, batch=97, vocab_arg=(3, 7, 1000)),
              small(d=32, Z=8, M=300_007, bag_rule=bags, batch=40)):
        with Case(w) as c:
            robe.robe_set_option(c.h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_DETERMINISTIC)
            ws = torch.empty(robe.robe_backward_workspace_bytes(c.h, c.B, c.indices.numel()),
                             dtype=torch.uint8, device=c.dev)
            ssq_d = torch.zeros(w.M, device=c.dev)
            arr, ssq = c.array_h.copy(), np.zeros(w.M, np.float32)
            for step in (1, 2, 3):
                g_h, g_d = _grad(c, 30 + step)
                can, touched = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
                orc.adagrad_apply(arr, ssq, can, touched, lr, eps)
                robe.robe_backward_adagrad(c.h, g_d, c.indices, c.offsets, c.B, ssq_d, lr, eps, ws)
                torch.cuda.synchronize()
                assert_bits_equal(c.array.cpu().numpy(), arr, f"adagrad array, step {step}")
                assert_bits_equal(ssq_d.cpu().numpy(), ssq, f"adagrad accumulators, step {step}")
            with pytest.raises(robe.RobeError):
                robe.robe_backward_adagrad(c.h, g_d, c.indices, c.offsets, c.B, ssq_d, lr, -1.0, ws)
            with pytest.raises(robe.RobeError):
                robe.robe_backward_adagrad(c.h, g_d, c.indices, c.offsets, c.B, None, lr, eps, ws)


def test_deterministic_is_bit_reproducible_and_order_sensitive_case():
    # a hot id: thousands of terms on the same slots; five runs must give identical bits
    w = small(d=32, Z=8, M=300, batch=2000, vocab_arg=(2, 3, 1000))
    with Case(w) as c:
        g_h, g_d = _grad(c, 5)
        can, _ = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
        runs = [c.backward(g_d, "det").cpu().numpy() for _ in range(5)]
        for r in runs:
            assert_bits_equal(r, can, "hot id deterministic")


# Densely touched arrays take the slot-major kernel (one CTA per window of 256..2048 slots); the
# cases span its branches: windows of every length, a ragged last window, blocks that wrap, ids
# repeated so often that their windows go back to the position-tile and long-walk kernels while
# the rest stay, windows whose blocks need several chunks of shared memory, block lengths that
# are no power of two or no multiple of four, and a gradient buffer that is not 16-byte aligned.
WINDOW_CASES = [
    # d, Z, M, batch, tables/vocab, bags, id_dist
    dict(d=64, Z=16, M=300_007, batch=1500, vocab_arg=(10**6, 10**6, 50_000), bag_rule=(6, 0, 20)),
    dict(d=32, Z=32, M=2_100_003, batch=9000, vocab_arg=(10**6, 10**5, 10**6, 3000), num_tables=4),
    dict(d=32, Z=32, M=2_100_003, batch=9000, vocab_arg=(10**6, 10**5, 10**6, 3000), num_tables=4,
         id_dist="zipf1.05"),
    dict(d=128, Z=128, M=700_001, batch=3000, vocab_arg=(10**5, 40, 10**6), id_dist="zipf1.05"),
    dict(d=16, Z=16, M=4099, batch=6000, vocab_arg=(10**6, 10**6, 10**6)),
    dict(d=48, Z=12, M=100_003, batch=2500, vocab_arg=(10**6, 10**6, 10**6)),
    dict(d=48, Z=6, M=100_003, batch=2500, vocab_arg=(10**6, 10**6, 10**6)),
    dict(d=8, Z=1, M=50_021, batch=4000, vocab_arg=(10**6, 10**6, 10**6), id_dist="zipf1.05"),
    dict(d=64, Z=256, M=600_011, batch=5000, vocab_arg=(10**6, 10**6, 10**6)),
]


@pytest.mark.parametrize("case", WINDOW_CASES, ids=lambda k: f"d{k['d']}_Z{k['Z']}_M{k['M']}_{k.get('id_dist', 'uniform')}")
def test_deterministic_window_apply(case):
    w = small(**case)
    with Case(w) as c:
        nb = c.indices.numel() * ((w.d + min(w.Z, w.d) - 1) // min(w.Z, w.d))
        assert nb * min(w.Z, w.d) * 2 >= w.M, "the case must touch the array densely"
        g_h, g_d = _grad(c, 11)
        can, touched = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
        assert_bits_equal(c.backward(g_d, "det").cpu().numpy(), can, "window apply, dense gradient")
        # the same values from a buffer that starts 4 bytes off a 16-byte boundary
        shifted = torch.empty(g_d.numel() + 1, dtype=torch.float32, device=c.dev)[1:]
        shifted.copy_(g_d.reshape(-1))
        assert shifted.data_ptr() % 16 == 4
        assert_bits_equal(c.backward(shifted.view_as(g_d), "det").cpu().numpy(), can, "unaligned gradient")
        # fused SGD: untouched slots keep their bits
        before = c.array_h.copy()
        c.backward(g_d, "det", sgd=True, lr=0.125)
        want = before.copy()
        orc.sgd_apply(want, can, touched, 0.125)
        assert_bits_equal(c.array.cpu().numpy(), want, "window apply, SGD")


# robe_forward_keep + robe_backward_kept: one hash of every id per training step.  The pair must
# give what robe_forward and robe_backward give: the forward bit for bit, the deterministic
# backward bit for bit, the binned and atomic ones within the atomic bound.  Shapes: rows of every
# kernel class (up to 32, 64, 128 elements and longer, where the forward kernel keeps nothing),
# ragged last blocks, rows clubbed into one block, one-hot and pooled input with empty bags.
KEEP_SHAPES = [(16, 4, 4096), (64, 16, 70), (100, 32, 1013), (128, 128, 1280), (12, 5, 64), (48, 3, 49),
               (130, 2, 1000), (200, 64, 777), (16, 64, 1000), (1, 1, 1), (32, 32, 100_003)]


@pytest.mark.parametrize("bags", [None, (3, 0, 9)])
@pytest.mark.parametrize("d,Z,M", KEEP_SHAPES)
def test_step_sharing_block_starts(d, Z, M, bags):
    w = small(d=d, Z=Z, M=M, bag_rule=bags, batch=61)
    for sign in (False, True):
        with Case(w, sign=sign) as c:
            g_h, g_d = _grad(c, 21)
            want_out = c.oracle_forward()
            delta64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B)
            can, touched = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
            out, det = c.step_sharing_keys(g_d, "det")
            assert_bits_equal(out.cpu().numpy(), want_out, "forward that keeps")
            assert_bits_equal(det.cpu().numpy(), can, f"deterministic on kept starts d={d} Z={Z} sign={sign}")
            out, binned = c.step_sharing_keys(g_d, "binned")
            assert_bits_equal(out.cpu().numpy(), want_out, "forward that keeps")
            assert_within_l1(binned.cpu().numpy(), delta64, l1, what=f"binned on kept starts d={d} Z={Z}")
            out, atomic = c.step_sharing_keys(g_d, "atomic")  # nothing to keep: plain calls
            assert_within_l1(atomic.cpu().numpy(), delta64, l1, what="atomic through the keep calls")
            # fused SGD through the pair
            before = c.array_h.copy()
            c.step_sharing_keys(g_d, "det", sgd=True, lr=0.25)
            want = before.copy()
            orc.sgd_apply(want, can, touched, 0.25)
            assert_bits_equal(c.array.cpu().numpy(), want, "SGD on kept starts")


def test_step_sharing_block_starts_int32_ids_and_workspace_check():
    w = small(d=64, Z=16, M=50_021, bag_rule=(4, 0, 12), batch=300)
    with Case(w) as c:
        g_h, g_d = _grad(c, 22)
        can, _ = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
        c.indices = c.indices.to(torch.int32)
        _, det = c.step_sharing_keys(g_d, "det")
        assert_bits_equal(det.cpu().numpy(), can, "kept starts, int32 ids")
        out = torch.empty(c.B, c.T, w.d, device=c.dev)
        small_ws = torch.empty(256, dtype=torch.uint8, device=c.dev)
        with pytest.raises(robe.RobeError) as ei:
            robe.robe_forward_keep(c.h, c.indices, c.offsets, c.B, out, small_ws)
        assert ei.value.status == robe.ROBE_ERR_WORKSPACE
        with pytest.raises(robe.RobeError) as ei:
            robe.robe_forward_keep(c.h, c.indices, c.offsets, c.B, out, None)
        assert ei.value.status == robe.ROBE_ERR_WORKSPACE


# Table-major bags (bag e*B + n: the per-table id lists laid end to end; out and grad_out are
# [T, B, d]).  Every kernel takes the table of a bag from the same helper, so each kernel family
# is run once: both forward kernels, the atomic, binned and deterministic backward (window and
# position-tile apply), the step that shares block starts, Adam; one-hot and pooled input.
@pytest.mark.parametrize("bags", [None, (3, 0, 9)])
@pytest.mark.parametrize("d,Z,M,batch", [(16, 4, 4096, 61), (64, 16, 300_007, 700), (130, 2, 1000, 33),
                                         (128, 128, 1280, 1), (16, 64, 1000, 50), (32, 8, 2_000_003, 90)])
def test_table_major_bags(d, Z, M, batch, bags):
    w = small(d=d, Z=Z, M=M, bag_rule=bags, batch=batch)
    for sign in (False, True):
        with Case(w, sign=sign, table_major=True) as c, Case(w, sign=sign) as ref:
            want = c.oracle_forward()  # [T, B, d]
            for kernel in ([0, 1, 2] if d <= 128 else [0, 1]):
                assert_bits_equal(c.forward(kernel).cpu().numpy().reshape(want.shape), want,
                                  f"table-major forward k={kernel} d={d} Z={Z}")
            # the same rows as the default numbering gives, at other places (not through the oracle)
            rows_ref = ref.forward().cpu().numpy().reshape(c.B, c.T, d).transpose(1, 0, 2)
            assert_bits_equal(c.forward().cpu().numpy().reshape(c.T, c.B, d), rows_ref, "rows renumbered")
            g_h = np.random.default_rng(31).standard_normal((c.T, c.B, d)).astype(np.float32)
            g_d = torch.from_numpy(g_h).to(c.dev)
            delta64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B)
            can, touched = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
            assert_within_l1(c.backward(g_d, "atomic").cpu().numpy(), delta64, l1, what="table-major atomic")
            assert_within_l1(c.backward(g_d, "binned").cpu().numpy(), delta64, l1, what="table-major binned")
            assert_bits_equal(c.backward(g_d, "det").cpu().numpy(), can, f"table-major det d={d} Z={Z} sign={sign}")
            out, detk = c.step_sharing_keys(g_d, "det")
            assert_bits_equal(out.cpu().numpy().reshape(want.shape), want, "table-major forward that keeps")
            assert_bits_equal(detk.cpu().numpy(), can, "table-major det on kept starts")
            before = c.array_h.copy()
            c.backward(g_d, "det", sgd=True, lr=0.5)
            wanted = before.copy()
            orc.sgd_apply(wanted, can, touched, 0.5)
            assert_bits_equal(c.array.cpu().numpy(), wanted, "table-major det SGD")


def test_backward_empty_inputs():
    w = small(bag_rule=(2, 0, 5))
    with Case(w, batch=4) as c:
        c.offsets = torch.zeros(c.nbags + 1, dtype=torch.int64, device=c.dev)
        c.indices = torch.zeros(0, dtype=torch.int64, device=c.dev)
        _, g_d = _grad(c, 0)
        for mode in ("atomic", "det"):
            ga = c.backward(g_d, mode).cpu().numpy()
            assert np.all(ga == 0)
        for mode in ("binned", "det"):  # and through the calls that share the block starts
            out, ga = c.step_sharing_keys(g_d, mode)
            assert not out.any() and not ga.any()


# ---------------------------------------------------------------------------------------
# the five workloads at full size (the launch configurations the benchmark times)
# ---------------------------------------------------------------------------------------

def _sample_bags(nbags, n, seed):
    rng = np.random.default_rng(seed)
    n = min(n, nbags)
    picks = rng.choice(nbags, size=n, replace=False)
    picks[:4] = [0, 1, nbags - 2, nbags - 1][:len(picks[:4])]
    return np.sort(picks).astype(np.int64)


def _check_forward_sampled(c, nsample=20000, kernel=0):
    got = c.forward(kernel).reshape(c.nbags, c.w.d)
    bags = _sample_bags(c.nbags, nsample, 1)
    want = c.oracle_forward_bags(bags)
    assert_bits_equal(got[torch.from_numpy(bags).to(c.dev)].cpu().numpy(), want, c.w.name + " forward")
    return got


def test_cfg2_forward_full_size():
    with Case(synth.workload(2)) as c:
        got = c.forward()
        # the whole output, not a sample: the oracle needs a few seconds for 1.7M rows
        want = c.oracle_forward()
        assert_bits_equal(got.cpu().numpy(), want, "cfg2 forward (all rows)")
        assert_bits_equal(c.forward(3).cpu().numpy(), want, "cfg2 forward, 16-byte loads (all rows)")


@pytest.mark.parametrize("Z", [1, 128])
def test_cfg3_forward_backward_full_size(Z):
    w = synth.workload(3, Z=Z)
    with Case(w) as c:
        _check_forward_sampled(c)
        g_h = synth.make_grad_out(w)
        g_d = torch.from_numpy(g_h).to(c.dev)
        delta64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B)
        ga = c.backward(g_d, "atomic").cpu().numpy()
        assert_within_l1(ga, delta64, l1, what=f"cfg3 Z={Z} atomic")
        for kernel in ((3, 4, 5) if Z == 128 else (5,)):
            gv = c.backward(g_d, "atomic", kernel=kernel).cpu().numpy()
            assert_within_l1(gv, delta64, l1, what=f"cfg3 Z={Z} atomic, kernel {kernel}")
        det = c.backward(g_d, "det").cpu().numpy()
        assert_within_l1(det, delta64, l1, what=f"cfg3 Z={Z} det vs fp64")
        assert_bits_equal(c.backward(g_d, "det").cpu().numpy(), det, "cfg3 det repeat")
        # the same step with the forward's block starts: same bits (window, position-tile and
        # long-walk kernels all take part at this size)
        _, detk = c.step_sharing_keys(g_d, "det")
        assert_bits_equal(detk.cpu().numpy(), det, "cfg3 det on kept starts")
        del detk
        if Z == 128:
            can, touched = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
            assert_bits_equal(det, can, "cfg3 Z=128 det vs canonical")
            before = c.array_h.copy()
            c.backward(g_d, "det", sgd=True, lr=1.0)
            want = before.copy()
            orc.sgd_apply(want, can, touched, 1.0)
            assert_bits_equal(c.array.cpu().numpy(), want, "cfg3 det sgd")
        else:
            before = c.array_h.copy()
            c.backward(g_d, "atomic", sgd=True, lr=1.0)
            assert_within_l1(c.array.cpu().numpy(), before.astype(np.float64) - delta64,
                             l1 + np.abs(before), what="cfg3 atomic sgd")


def test_cfg3_z1_deterministic_vs_canonical_reduced_batch():
    # the canonical oracle sorts every block on one core; 2048 samples x 26 x 128 blocks is its size
    w = synth.workload(3, Z=1)
    with Case(w, batch=2048) as c:
        g_h = synth.make_grad_out(w, 2048)
        g_d = torch.from_numpy(g_h).to(c.dev)
        can, _ = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
        assert_bits_equal(c.backward(g_d, "det").cpu().numpy(), can, "cfg3 Z=1 det")


def test_cfg4_forward_backward_full_size():
    w = synth.workload(4)
    with Case(w) as c:
        _check_forward_sampled(c)
        _check_forward_sampled(c, kernel=3)
        g_h = synth.make_grad_out(w)
        g_d = torch.from_numpy(g_h).to(c.dev)
        delta64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B)
        ga = c.backward(g_d, "atomic").cpu().numpy()
        assert_within_l1(ga, delta64, l1, what="cfg4 atomic")
        gv = c.backward(g_d, "atomic", kernel=3).cpu().numpy()
        assert_within_l1(gv, delta64, l1, what="cfg4 atomic, 16-byte reductions")
        del gv
        gb = c.backward(g_d, "binned").cpu().numpy()
        assert_within_l1(gb, delta64, l1, what="cfg4 binned")
        before = c.array_h.copy()
        c.backward(g_d, "binned", sgd=True, lr=0.5)
        assert_within_l1(c.array.cpu().numpy(), before.astype(np.float64) - 0.5 * delta64,
                         0.5 * l1 + np.abs(before), what="cfg4 binned sgd")
        c.array.copy_(torch.from_numpy(before))
        # the step as the benchmark runs it: the forward keeps its block starts for the binned backward
        out, gk = c.step_sharing_keys(g_d, "binned")
        bags = _sample_bags(c.nbags, 20000, 2)
        assert_bits_equal(out.reshape(c.nbags, w.d)[torch.from_numpy(bags).to(c.dev)].cpu().numpy(),
                          c.oracle_forward_bags(bags), "cfg4 forward that keeps")
        assert_within_l1(gk.cpu().numpy(), delta64, l1, what="cfg4 binned on kept starts")
        del out, gk
        # gradient mass is conserved (holds at any size)
        lengths = np.diff(c.offsets_h)
        mass = float((lengths * g_h.astype(np.float64).reshape(c.nbags, -1).sum(axis=1)).sum())
        assert abs(float(ga.astype(np.float64).sum()) - mass) < 1e-6 * float(l1.sum())
        del delta64, l1
        det = c.backward(g_d, "det").cpu().numpy()
        can, _ = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B, j0=1_000_000, jn=3_000_000)
        assert_bits_equal(det[1_000_000:4_000_000], can, "cfg4 det window")
        can0, _ = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B, j0=0, jn=100_000)
        assert_bits_equal(det[:100_000], can0, "cfg4 det low slots")
        canl, _ = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B, j0=w.M - 100_000, jn=100_000)
        assert_bits_equal(det[w.M - 100_000:], canl, "cfg4 det high slots")
        _, detk = c.step_sharing_keys(g_d, "det")
        assert_bits_equal(detk.cpu().numpy(), det, "cfg4 det on kept starts")


# the sweep: every cell of {1 MB, 100 MB} x Z in {1, 2, 8, 32, 128}, and the bf16 array
@pytest.mark.parametrize("M,Z,dtype",
                         [(M, Z, "f32") for M in (262_144, 25_000_000) for Z in (1, 2, 8, 32, 128)]
                         + [(25_000_000, 32, "bf16")])
def test_cfg5_forward_full_size(M, Z, dtype):
    w = synth.workload(5, M=M, Z=Z, array_dtype=dtype)
    with Case(w) as c:
        _check_forward_sampled(c)


def _need_device_memory(gib):
    free, _ = torch.cuda.mem_get_info()
    if free < gib * 2**30:
        pytest.skip("not enough free device memory")


def _array_window(w, j0, jn):
    """fp32 values of array slots [j0, j0+jn) from the counter-based generator (host side)."""
    return synth.array_values_at(w, torch.arange(j0, j0 + jn, dtype=torch.int64)).numpy()


@pytest.mark.parametrize("Z", [1, 2, 8, 32, 128])
def test_cfg5_forward_10gb_array(Z):
    w = synth.workload(5, M=2_500_000_000, Z=Z)
    _need_device_memory(16)
    with Case(w, host_array=False) as c:
        got = c.forward().reshape(c.nbags, w.d)
        bags = _sample_bags(c.nbags, 3000, 2)
        rows = got[torch.from_numpy(bags).to(c.dev)].cpu().numpy()
        for r, bag in enumerate(bags):
            slots = c.oracle.locate(int(bag % c.T), int(c.indices_h[bag])).astype(np.int64)
            want = synth.array_values_at(w, torch.from_numpy(slots)).numpy()
            assert_bits_equal(rows[r], want, "cfg5 10 GB")


def test_cfg5_backward_full_size():
    w = synth.workload(5, M=25_000_000, Z=32)
    with Case(w) as c:
        g_h = synth.make_grad_out(w)
        g_d = torch.from_numpy(g_h).to(c.dev)
        delta64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B)
        ga = c.backward(g_d, "atomic").cpu().numpy()
        assert_within_l1(ga, delta64, l1, what="cfg5 atomic")
        det = c.backward(g_d, "det").cpu().numpy()
        can, _ = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
        assert_bits_equal(det, can, "cfg5 det")


@pytest.mark.parametrize("M,Z,dtype", [(262_144, 1, "f32"), (262_144, 32, "f32"), (25_000_000, 1, "f32"),
                                       (25_000_000, 128, "f32"), (25_000_000, 32, "bf16")])
def test_cfg5_backward_atomic_full_size(M, Z, dtype):
    # dense fp32 gradient (the only backward a bf16 array has); fp32 arrays also take the fused step
    w = synth.workload(5, M=M, Z=Z, array_dtype=dtype)
    with Case(w) as c:
        g_h = synth.make_grad_out(w)
        g_d = torch.from_numpy(g_h).to(c.dev)
        delta64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B)
        ga = c.backward(g_d, "atomic").cpu().numpy()
        assert_within_l1(ga, delta64, l1, what=f"cfg5 M={M} Z={Z} {dtype} atomic")
        assert abs(float(ga.astype(np.float64).sum()) - float(g_h.astype(np.float64).sum())) \
            < 1e-6 * float(l1.sum())  # mass: every id contributes its row once
        if dtype == "f32":
            before = c.array_h.copy()
            c.backward(g_d, "atomic", sgd=True, lr=0.5)
            assert_within_l1(c.array.cpu().numpy(), before.astype(np.float64) - 0.5 * delta64,
                             0.5 * l1 + np.abs(before), what=f"cfg5 M={M} Z={Z} atomic sgd")


def test_cfg5_1mb_z32_deterministic_full_size():
    # 4000 terms per slot: every window of the slot-major apply streams many chunks
    w = synth.workload(5, M=262_144, Z=32)
    with Case(w) as c:
        g_h = synth.make_grad_out(w)
        g_d = torch.from_numpy(g_h).to(c.dev)
        can, touched = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
        det = c.backward(g_d, "det").cpu().numpy()
        assert_bits_equal(det, can, "cfg5 1 MB Z=32 det")
        assert_bits_equal(c.backward(g_d, "det").cpu().numpy(), det, "repeat")
        before = c.array_h.copy()
        c.backward(g_d, "det", sgd=True, lr=0.01)
        want = before.copy()
        orc.sgd_apply(want, can, touched, 0.01)
        assert_bits_equal(c.array.cpu().numpy(), want, "cfg5 1 MB Z=32 det sgd")


@pytest.mark.parametrize("M,Z", [(25_000_000, 2), (262_144, 1)])
def test_cfg5_small_blocks_deterministic_reduced_batch(M, Z):
    # more than 8 blocks per id: the one-thread-per-block key kernel, and the most sort passes
    w = synth.workload(5, M=M, Z=Z)
    with Case(w, batch=4096) as c:
        g_h = synth.make_grad_out(w, 4096)
        g_d = torch.from_numpy(g_h).to(c.dev)
        can, _ = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
        assert_bits_equal(c.backward(g_d, "det").cpu().numpy(), can, f"cfg5 M={M} Z={Z} det")
        _, detk = c.step_sharing_keys(g_d, "det")
        assert_bits_equal(detk.cpu().numpy(), can, f"cfg5 M={M} Z={Z} det on kept starts")


WINDOWS_10G = [(0, 200_000), (1_234_567_890, 300_000), (2_500_000_000 - 150_000, 150_000)]


def test_cfg5_10gb_fused_sgd_atomic():
    # the cell whose dense gradient would cost a 10 GB memset per step: the SGD step is fused into
    # the scatter; slot windows at the start, in the middle and at the end of the array
    w = synth.workload(5, M=2_500_000_000, Z=32)
    _need_device_memory(16)
    with Case(w, host_array=False) as c:
        g_h = synth.make_grad_out(w)
        g_d = torch.from_numpy(g_h).to(c.dev)
        c.backward(g_d, "atomic", sgd=True, lr=0.5)
        for j0, jn in WINDOWS_10G:
            d64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B, j0=j0, jn=jn)
            before = _array_window(w, j0, jn)
            after = c.array[j0:j0 + jn].cpu().numpy()
            assert l1.max() > 0
            assert_within_l1(after, before.astype(np.float64) - 0.5 * d64, 0.5 * l1 + np.abs(before),
                             what=f"cfg5 10 GB fused SGD, window at {j0}")
            assert_bits_equal(after[l1 == 0], before[l1 == 0], "untouched slots")


@pytest.mark.parametrize("mode", ["binned", "det"])
def test_cfg5_10gb_z128_sorted_backward(mode):
    # binned (atomic accuracy) and deterministic (bit-exact) on the 10 GB array, fused SGD
    w = synth.workload(5, M=2_500_000_000, Z=128)
    _need_device_memory(20)
    with Case(w, host_array=False) as c:
        g_h = synth.make_grad_out(w)
        g_d = torch.from_numpy(g_h).to(c.dev)
        c.backward(g_d, mode, sgd=True, lr=0.5)
        for j0, jn in WINDOWS_10G:
            before = _array_window(w, j0, jn)
            after = c.array[j0:j0 + jn].cpu().numpy()
            if mode == "binned":
                d64, l1 = c.oracle.backward_f64(g_h, c.indices_h, c.offsets_h, c.B, j0=j0, jn=jn)
                assert_within_l1(after, before.astype(np.float64) - 0.5 * d64, 0.5 * l1 + np.abs(before),
                                 what=f"cfg5 10 GB binned, window at {j0}")
            else:
                can, touched = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B, j0=j0, jn=jn)
                want = before.copy()
                orc.sgd_apply(want, can, touched, 0.5)
                assert touched.any()
                assert_bits_equal(after, want, f"cfg5 10 GB deterministic, window at {j0}")


def test_cfg4_deterministic_whole_array_vs_canonical():
    # every one of the 250 M slots against the canonical-order oracle (one sort of 34 M blocks on a
    # host core), dense gradient and fused SGD
    w = synth.workload(4)
    with Case(w) as c:
        g_h = synth.make_grad_out(w)
        g_d = torch.from_numpy(g_h).to(c.dev)
        can, touched = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
        det = c.backward(g_d, "det").cpu().numpy()
        assert_bits_equal(det, can, "cfg4 det, whole array")
        del det
        before = c.array_h.copy()
        c.step_sharing_keys(g_d, "det", sgd=True, lr=0.5)
        orc.sgd_apply(before, can, touched, 0.5)
        assert_bits_equal(c.array.cpu().numpy(), before, "cfg4 det SGD on kept starts, whole array")


def test_cfg3_z1_deterministic_full_batch_vs_canonical():
    # Zipf ids, every element hashed on its own: 109 M blocks, the hottest id adds thousands of
    # terms to each of its 128 slots (long walks); the whole 25 M-slot array bit for bit
    w = synth.workload(3, Z=1)
    with Case(w) as c:
        g_h = synth.make_grad_out(w)
        g_d = torch.from_numpy(g_h).to(c.dev)
        can, _ = c.oracle.backward_canonical(g_h, c.indices_h, c.offsets_h, c.B)
        assert_bits_equal(c.backward(g_d, "det").cpu().numpy(), can, "cfg3 Z=1 det, full batch")


# ---------------------------------------------------------------------------------------
# validation mode and argument errors that need a device pointer
# ---------------------------------------------------------------------------------------

def test_validate_mode_reports_bad_inputs_without_faulting():
    w = small(bag_rule=(2, 0, 5))
    with Case(w, batch=8) as c:
        word = torch.zeros(1, dtype=torch.int32, device=c.dev)
        robe.robe_set_status_word(c.h, word)
        robe.robe_set_option(c.h, robe.ROBE_OPT_VALIDATE, 1)
        good = c.forward().cpu().numpy()
        assert robe.robe_last_device_status(c.h) == 0
        assert_bits_equal(good, c.oracle_forward(), "validated forward")
        bad = c.offsets.clone()
        bad[3] = bad[4] + 5  # not monotone
        keep = c.offsets
        c.offsets = bad
        out = c.forward()
        assert robe.robe_last_device_status(c.h) == 2
        assert torch.isnan(out).all()  # nothing was written
        c.offsets = keep
        word.zero_()
        neg = c.indices.clone()
        neg[0] = -5
        c.indices = neg
        c.forward()
        assert robe.robe_last_device_status(c.h) == 1


@pytest.mark.parametrize("mode", ["atomic", "binned", "det"])
def test_validate_mode_stops_every_backward_variant(mode):
    # a bad id under ROBE_OPT_VALIDATE: the status word says so and no kernel touches the target
    w = small(bag_rule=(2, 0, 5))
    with Case(w, batch=8) as c:
        word = torch.zeros(1, dtype=torch.int32, device=c.dev)
        robe.robe_set_status_word(c.h, word)
        robe.robe_set_option(c.h, robe.ROBE_OPT_VALIDATE, 1)
        _, g_d = _grad(c, 3)
        good = c.backward(g_d, mode).cpu().numpy()
        assert robe.robe_last_device_status(c.h) == 0 and np.any(good != 0)
        c.indices = c.indices.clone()
        c.indices[1] = -7
        ga = c.backward(g_d, mode).cpu().numpy()
        assert robe.robe_last_device_status(c.h) == 1
        assert not np.any(ga)


def test_argument_errors_on_device():
    with Case(small()) as c:
        out = torch.empty(c.B, c.T, c.w.d, device=c.dev)
        with pytest.raises(robe.RobeError) as ei:
            robe.robe_forward(c.h, c.indices[:-1], None, c.B, out)  # nnz != batch*T
        assert ei.value.status == robe.ROBE_ERR_INVALID_ARG
        robe.robe_set_option(c.h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_DETERMINISTIC)
        g = torch.zeros(c.B, c.T, c.w.d, device=c.dev)
        ga = torch.zeros(c.w.M, device=c.dev)
        with pytest.raises(robe.RobeError) as ei:
            robe.robe_backward(c.h, g, c.indices, None, c.B, ga, 0.0, None)
        assert ei.value.status == robe.ROBE_ERR_WORKSPACE
    w = small(array_dtype="bf16")
    with Case(w) as c:
        g = torch.zeros(c.B, c.T, c.w.d, device=c.dev)
        with pytest.raises(robe.RobeError) as ei:
            robe.robe_backward(c.h, g, c.indices, None, c.B, None, 0.1, None)  # SGD on bf16
        assert ei.value.status == robe.ROBE_ERR_INVALID_ARG
