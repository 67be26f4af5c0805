"""Host-side arithmetic of the benchmark: byte models and workload names (no GPU)."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402


def test_byte_models_of_the_multihot_workload():
    # 26 tables x 16384 samples, bags of 20 ids, d=64, Z=16, fp32: per id 8 B of index + 256 B of
    # array (useful) or 4 blocks x (1 + 15/8) sectors x 32 B = 368 B (sector model)
    w = bench.pick_workload("cfg4")
    nbags, nnz = 16384 * 26, 20 * 16384 * 26
    fwd, bwd = bench.algorithmic_bytes(w, nbags, nnz, True)
    rest = 8 * nnz + 8 * (nbags + 1) + 4 * 64 * nbags
    assert fwd == rest + 256 * nnz and bwd == rest + 512 * nnz
    m = bench.forward_byte_models(w, nbags, nnz, True)
    assert m["useful"] == fwd and m["l2_resident"] == rest
    assert m["sector"] == pytest.approx(rest + 368 * nnz)
    assert bench.algorithmic_bytes(w, nbags, nnz, True, id_bytes=4)[0] == fwd - 4 * nnz


def test_sector_model_follows_the_paper_fetch_table():
    # Table 1 restated for 32-byte sectors (8 fp32): Z=1 fetches a sector per element, large Z
    # approaches d/8 sectors plus one per block
    one = bench.forward_byte_models(bench.pick_workload("cfg5_10g_z1"), 10, 10, False)
    big = bench.forward_byte_models(bench.pick_workload("cfg5_10g_z128"), 10, 10, False)
    club = bench.forward_byte_models(bench.pick_workload("cfg5_10g_z512"), 10, 10, False)
    assert one["sector"] - one["l2_resident"] == 10 * 128 * 32
    assert big["sector"] - big["l2_resident"] == pytest.approx(10 * (1 + 127 / 8) * 32)
    assert club["sector"] == big["sector"]  # Z > d: one block of d elements per id


@pytest.mark.parametrize("name,M,Z,dtype", [
    ("cfg2", 25_000_000, 32, "f32"), ("cfg3_z1", 25_000_000, 1, "f32"), ("cfg4", 250_000_000, 16, "f32"),
    ("cfg5", 25_000_000, 32, "f32"), ("cfg5_1m_z8", 262_144, 8, "f32"),
    ("cfg5_10g_z128", 2_500_000_000, 128, "f32"), ("cfg5_100m_z32_bf16", 25_000_000, 32, "bf16"),
])
def test_workload_names(name, M, Z, dtype):
    w = bench.pick_workload(name)
    assert (w.M, w.Z, w.array_dtype) == (M, Z, dtype)
    with pytest.raises(ValueError):
        bench.pick_workload(name + "_x")
