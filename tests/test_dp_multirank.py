"""The data-parallel step (Section 1 of the paper: the compressed model is trained data-parallel,
the ranks exchange one gradient the size of the array) on two gloo ranks on the CPU.

What is checked, with the oracle standing in for the kernels: the batch is split by sample, every
rank scatter-adds its shard into a dense gradient, the all-reduced sum equals the gradient of the
unsharded batch, and after the dense apply both replicas hold the same bits.  The sharding helper
is the product's own (paper_2108_02191_b200.dp.shard_by_sample); no CUDA library is touched."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _workload(bags):
    from paper_2108_02191_b200 import synth
    return synth.RobeWorkload(name="dp", num_tables=3, vocab_rule="list", vocab_arg=(50, 7, 1000), d=16, Z=4,
                              M=1000, batch=41, array_init="normal0.01", array_dtype="f32",
                              id_dist="uniform", bag_rule=bags, hash_seed=77, data_seed=5)


def _worker(rank: int, world: int, port: int, out_dir: str, bags):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from oracle import robe_oracle as orc
    from paper_2108_02191_b200 import dp, synth

    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = _workload(bags)
        ids, offs = synth.make_ids(w)
        # integer gradients: every summation order gives the same bits, so the check is exact
        grad = np.random.default_rng(9).integers(-4, 5, size=(w.batch, w.num_tables, w.d)).astype(np.float32)
        my_ids, my_offs, n0, n1 = dp.shard_by_sample(ids, offs, w.batch, w.num_tables, rank, world)
        o = orc.Oracle(w.M, w.Z, w.d, w.num_tables, orc.hash_constants(w.hash_seed))
        d64, _ = o.backward_f64(grad[n0:n1], my_ids, my_offs, n1 - n0)
        g = torch.from_numpy(d64.astype(np.float32))
        dist.all_reduce(g, op=dist.ReduceOp.SUM)
        array = synth.array_to_numpy(synth.make_array(w, "cpu")).copy()
        orc.dense_sgd_apply(array, g.numpy(), 0.5)
        assert dp.replicas_identical(torch.from_numpy(array))
        np.save(os.path.join(out_dir, f"grad_{rank}.npy"), g.numpy())
        np.save(os.path.join(out_dir, f"array_{rank}.npy"), array)
        np.save(os.path.join(out_dir, f"shard_{rank}.npy"), np.array([n0, n1, len(my_ids)]))
        # a replica that drifted is noticed
        array[rank] += 1.0
        different = not dp.replicas_identical(torch.from_numpy(array))
        np.save(os.path.join(out_dir, f"drift_{rank}.npy"), np.array([different]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("bags", [None, (3, 0, 9)])
def test_two_ranks_sum_to_the_unsharded_gradient_and_stay_identical(tmp_path, bags):
    from oracle import robe_oracle as orc
    from paper_2108_02191_b200 import synth

    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path), bags), nprocs=world, join=True)
    w = _workload(bags)
    ids, offs = synth.make_ids(w)
    grad = np.random.default_rng(9).integers(-4, 5, size=(w.batch, w.num_tables, w.d)).astype(np.float32)
    o = orc.Oracle(w.M, w.Z, w.d, w.num_tables, orc.hash_constants(w.hash_seed))
    whole, _ = o.backward_f64(grad, ids, offs, w.batch)
    g0, g1 = np.load(tmp_path / "grad_0.npy"), np.load(tmp_path / "grad_1.npy")
    np.testing.assert_array_equal(g0, g1)
    np.testing.assert_array_equal(g0, whole.astype(np.float32))
    a0, a1 = np.load(tmp_path / "array_0.npy"), np.load(tmp_path / "array_1.npy")
    np.testing.assert_array_equal(a0.view(np.uint32), a1.view(np.uint32))
    want = synth.array_to_numpy(synth.make_array(w, "cpu")).copy()
    orc.dense_sgd_apply(want, whole.astype(np.float32), 0.5)
    np.testing.assert_array_equal(a0.view(np.uint32), want.view(np.uint32))
    s0, s1 = np.load(tmp_path / "shard_0.npy"), np.load(tmp_path / "shard_1.npy")
    assert (s0[0], s0[1], s1[0], s1[1]) == (0, 20, 20, 41) and s0[2] + s1[2] == len(ids)
    assert np.load(tmp_path / "drift_0.npy")[0] and np.load(tmp_path / "drift_1.npy")[0]


def test_shard_by_sample_covers_the_batch_once():
    from paper_2108_02191_b200 import dp, synth

    for bags in (None, (3, 0, 9)):
        w = _workload(bags)
        ids, offs = synth.make_ids(w)
        for world in (1, 2, 3, 5):
            parts = [dp.shard_by_sample(ids, offs, w.batch, w.num_tables, r, world) for r in range(world)]
            np.testing.assert_array_equal(np.concatenate([p[0] for p in parts]), ids)
            assert [p[2] for p in parts] == [r * w.batch // world for r in range(world)]
            assert parts[-1][3] == w.batch
            if offs is not None:
                for p in parts:
                    assert p[1][0] == 0 and p[1][-1] == len(p[0]) and len(p[1]) == (p[3] - p[2]) * w.num_tables + 1
                    np.testing.assert_array_equal(np.diff(p[1]),
                                                  np.diff(offs)[p[2] * w.num_tables:p[3] * w.num_tables])
