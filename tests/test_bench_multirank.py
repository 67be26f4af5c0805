"""Host logic of the benchmark's N > 1 path, run as two gloo ranks on the CPU: the ranks shard
the batch by sample (independent id batches, no data-path collective), every time is reduced with
MAX and the units of work with SUM, and the oracle-timing arm runs on rank 0 only."""
import os
import socket
import subprocess
import sys

import numpy as np
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


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    import bench
    from paper_2108_02191_b200 import synth

    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.workload(1)
        variants = bench.rank_batch_variants(rank, 4)
        ids = [synth.make_ids(w, 64, variant=v)[0] for v in variants]
        # per-rank figures: rank r is slower and sees more ids the higher r is
        times = [10.0 + rank, 3.0 - rank, 1.0 + 2 * rank, 5.0]
        units = [1000.0 * (rank + 1), 7.0]
        t, u = bench.aggregate_over_ranks(dist, torch.device("cpu"), times, units)
        np.save(os.path.join(out_dir, f"ids_{rank}.npy"), np.concatenate(ids))
        np.save(os.path.join(out_dir, f"agg_{rank}.npy"), np.array(t + u))
        with open(os.path.join(out_dir, f"variants_{rank}.txt"), "w") as f:
            f.write(" ".join(str(v) for v in variants))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_and_reduce(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    agg = [np.load(tmp_path / f"agg_{r}.npy") for r in range(world)]
    # every rank holds the same whole-job figures: times MAX over ranks, units SUM over ranks
    np.testing.assert_array_equal(agg[0], agg[1])
    np.testing.assert_array_equal(agg[0], [11.0, 3.0, 3.0, 5.0, 3000.0, 14.0])
    v0 = set(open(tmp_path / "variants_0.txt").read().split())
    v1 = set(open(tmp_path / "variants_1.txt").read().split())
    assert len(v0) == 4 and len(v1) == 4 and not (v0 & v1)
    ids0, ids1 = np.load(tmp_path / "ids_0.npy"), np.load(tmp_path / "ids_1.npy")
    assert ids0.shape == ids1.shape and not np.array_equal(ids0, ids1)  # different shards


def test_single_process_aggregate_is_identity():
    import bench
    t, u = bench.aggregate_over_ranks(None, torch.device("cpu"), [1.5, 2.5], [10])
    assert t == [1.5, 2.5] and u == [10.0]


def test_reference_arm_runs_on_rank_0_only():
    # a non-zero rank of the oracle-timing arm exits 0 without printing or computing anything
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
