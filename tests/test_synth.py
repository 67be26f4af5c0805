"""The seeded input generators: shapes, ranges, determinism, host/device agreement."""
import numpy as np
import torch

from paper_2108_02191_b200 import synth


def test_workloads_have_the_stated_shapes():
    w1 = synth.workload(1)
    assert (w1.num_tables, w1.d, w1.Z, w1.M, w1.batch) == (4, 16, 4, 4096, 256)
    assert list(synth.vocab_sizes(w1)) == [1000, 500, 2000, 100]
    w2 = synth.workload(2)
    v = synth.vocab_sizes(w2)
    assert len(v) == 26 and v.min() >= 3 and v.max() <= 4e7
    assert list(v) == list(synth.vocab_sizes(synth.workload(3)))  # "same tables as config 2"
    w4 = synth.workload(4)
    assert (w4.d, w4.Z, w4.M, w4.batch) == (64, 16, 250_000_000, 16384)
    w5 = synth.workload(5, M=262_144, Z=2)
    assert (w5.M, w5.Z, w5.batch) == (262_144, 2, 131072)


def test_ids_one_hot_and_bags():
    w = synth.workload(1)
    ids, offs = synth.make_ids(w)
    assert offs is None and ids.shape == (256 * 4,)
    v = synth.vocab_sizes(w)
    assert np.all(ids.reshape(256, 4) < v[None, :]) and ids.min() >= 0
    ids2, _ = synth.make_ids(w)
    assert np.array_equal(ids, ids2)
    ids3, _ = synth.make_ids(w, variant=1)
    assert not np.array_equal(ids, ids3)
    w4 = synth.workload(4)
    ids, offs = synth.make_ids(w4, batch=512)
    lens = np.diff(offs)
    assert offs[0] == 0 and offs[-1] == len(ids) and lens.min() >= 1 and lens.max() <= 80
    assert abs(lens.mean() - 20.0) < 0.5
    assert ids.min() >= 0 and ids.max() < 1_000_000


def test_zipf_ids_are_head_heavy():
    w = synth.workload(2)
    ids, _ = synth.make_ids(w, batch=4096)
    ids = ids.reshape(4096, 26)
    v = synth.vocab_sizes(w)
    big = int(np.argmax(v))
    top = np.mean(ids[:, big] == 0)
    assert 0.04 < top < 0.2   # 1/H(V, 1.05) is 0.08 .. 0.16 for large vocabularies


def test_array_generator_is_pointwise_and_bounded():
    w = synth.workload(2, M=100_000)
    a = synth.make_array(w, "cpu", chunk=4096)
    j = torch.tensor([0, 1, 4095, 4096, 99_999], dtype=torch.int64)
    assert torch.equal(a[j], synth.array_values_at(w, j))
    assert a.abs().max() <= 0.01 and abs(float(a.mean())) < 1e-4
    assert abs(float(a.std()) - 0.01 / np.sqrt(3)) < 2e-4
    w1 = synth.workload(1)
    n = synth.make_array(w1.with_(M=200_000), "cpu")
    assert abs(float(n.std()) - 0.01) < 3e-4 and abs(float(n.mean())) < 1e-4
    b = synth.make_array(w.with_(array_dtype="bf16"), "cpu")
    assert b.dtype == torch.bfloat16
    assert synth.array_to_numpy(b).dtype == np.uint16


def test_grad_out_is_standard_normal():
    w = synth.workload(1)
    g = synth.make_grad_out(w)
    assert g.shape == (256, 4, 16) and g.dtype == np.float32
    assert abs(g.mean()) < 0.03 and abs(g.std() - 1) < 0.03


def test_to_table_major_moves_whole_bags():
    w = synth.RobeWorkload("t", 3, "list", (50, 7, 1000), 8, 4, 1000, 5, "normal0.01", "f32", "uniform",
                           (3, 0, 6), 1, 2)
    ids, offs = synth.make_ids(w)
    ids_tm, offs_tm = synth.to_table_major(ids, offs, w.batch, w.num_tables)
    assert offs_tm[0] == 0 and offs_tm[-1] == len(ids) and len(offs_tm) == len(offs)
    for e in range(w.num_tables):
        for n in range(w.batch):
            old, new = n * w.num_tables + e, e * w.batch + n
            np.testing.assert_array_equal(ids_tm[offs_tm[new]:offs_tm[new + 1]], ids[offs[old]:offs[old + 1]])
    one, none = synth.to_table_major(np.arange(15), None, 5, 3)
    assert none is None
    np.testing.assert_array_equal(one.reshape(3, 5), np.arange(15).reshape(5, 3).T)
