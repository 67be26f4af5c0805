"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each one compares the oracle with something
that is not the oracle's own formula: a library routine the method reduces to for a special
choice of constants, a closed form, an invariant, a brute-force table built by a separately
written routine, or a hand-computed value stored under tests/golden/.
"""
import functools
import os

import numpy as np
import pytest

from oracle import robe_oracle as orc

P = (1 << 61) - 1
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def consts(Ah=1, Bh=1, Ch=1, Dh=0, Ag=1, Bg=1, Cg=1, Dg=0):
    return np.array([P, Ah, Bh, Ch, Dh, Ag, Bg, Cg, Dg], dtype=np.uint64)


def layout_consts(V, d, Z):
    """Constants that make h(e,x,c) the row-major position of chunk c of row x of table e in
    the flattened, concatenated parameter vector (appendix, 'ROBE-Z' procedure)."""
    return consts(Ah=V * d, Bh=d, Ch=Z, Dh=0)


# ---------------------------------------------------------------------------------------
# 1. hash arithmetic
# ---------------------------------------------------------------------------------------

def test_constants_ranges_and_determinism():
    # Section 3.2: A_h, B_h, C_h in {1..P-1}, D_h in {0..P-1}; same for the sign hash
    for seed in [0, 1, 0x0B0F, 2**63, 2**64 - 1]:
        k = [int(v) for v in orc.hash_constants(seed)]
        assert k[0] == P
        for idx in (1, 2, 3, 5, 6, 7):
            assert 1 <= k[idx] <= P - 1
        for idx in (4, 8):
            assert 0 <= k[idx] <= P - 1
        assert k == [int(v) for v in orc.hash_constants(seed)]
    assert list(orc.hash_constants(1)) != list(orc.hash_constants(2))
    assert len(set(int(v) for v in orc.hash_constants(7)[1:])) == 8


def test_mod_p_by_modular_inverse():
    # B * B^-1 = 1 (mod P): with A = C = D = 0 and m = P the hash of x = B^-1 must be 1.
    rng = np.random.default_rng(5)
    for _ in range(50):
        B = int(rng.integers(1, P))
        o = orc.Oracle(P, 1, 1, 1, consts(Ah=0, Bh=B, Ch=0, Dh=0))
        assert o.h(0, pow(B, P - 2, P), 0) == 1
        assert o.h(0, pow(B, -1, P) * 2 % P, 0) == 2


def test_mod_p_period_and_zero():
    # x and x + P hash alike; x = P contributes nothing, leaving D.
    k = orc.hash_constants(99)
    for m in (17, 4096, 25_000_000, 2_500_000_000):
        o = orc.Oracle(m, 1, 1, 3, k)
        for e, x, c in [(0, 0, 0), (2, 12345, 7), (1, 2**62, 100)]:
            assert o.h(e, x, c) == o.h(e, x + P, c)
        assert o.h(0, P, 0) == int(k[4]) % m
        assert o.h(0, 0, 0) == int(k[4]) % m


def test_hash_is_affine_mod_p():
    # with m = P nothing is lost in the second reduction: increments are the multipliers
    k = orc.hash_constants(3)
    o = orc.Oracle(P, 1, 1, 5, k)
    A, B, Cc = int(k[1]), int(k[2]), int(k[3])
    for e, x, c in [(0, 0, 0), (3, 999_999_937, 5), (1, 2**63 - 2, 126)]:
        h0 = o.h(e, x, c)
        assert (o.h(e + 1, x, c) - h0) % P == A
        assert (o.h(e, x + 1, c) - h0) % P == B
        assert (o.h(e, x, c + 1) - h0) % P == Cc


def test_hash_against_big_integers():
    # cross-check of the 128-bit C arithmetic with Python's unbounded integers
    rng = np.random.default_rng(11)
    k = orc.hash_constants(0x0B0F)
    kk = [int(v) for v in k]
    edge_x = [0, 1, P - 1, P, P + 1, 2**63 - 1, 2**32, 2**32 - 1]
    for m in (1, 2, 17, 4096, 262_144, 25_000_000, 2_500_000_000, 2**32 - 129):
        o = orc.Oracle(m, 1, 1, 26, k)
        xs = edge_x + [int(v) for v in rng.integers(0, 2**63 - 1, size=40)]
        for x in xs:
            for e, c in [(0, 0), (25, 127), (7, 3)]:
                want = ((kk[1] * e + kk[2] * x + kk[3] * c + kk[4]) % P) % m
                assert o.h(e, x, c) == want
                assert 0 <= want < m
                gwant = 2 * (((kk[5] * e + kk[6] * x + kk[7] * c + kk[8]) % P) % 2) - 1
                assert o.g(e, x, c) == gwant


# ---------------------------------------------------------------------------------------
# 2. the mapping reduces to plain table indexing for a layout-preserving hash
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("Z", [1, 2, 4, 8, 16])
def test_identity_sketch_is_table_lookup(Z):
    # h = row-major position of the chunk, m = n: forward must be theta.reshape(T,V,d)[e,x]
    T, V, d = 3, 50, 16
    n = T * V * d
    rng = np.random.default_rng(Z)
    theta = rng.standard_normal(n).astype(np.float32)
    o = orc.Oracle(n, Z, d, T, layout_consts(V, d, Z))
    ids = rng.integers(0, V, size=(20, T))
    out = o.forward(theta, ids.reshape(-1), None, 20)
    table = theta.reshape(T, V, d)
    want = np.stack([table[e, ids[:, e]] for e in range(T)], axis=1)
    np.testing.assert_array_equal(out, want)


@pytest.mark.parametrize("m", [97, 160, 1000])
def test_identity_sketch_wraps_like_take_mode_wrap(m):
    # same hash, array shorter than the parameter vector: slot = position mod m (circular array)
    T, V, d, Z = 2, 40, 16, 8
    rng = np.random.default_rng(m)
    arr = rng.standard_normal(m).astype(np.float32)
    o = orc.Oracle(m, Z, d, T, layout_consts(V, d, Z))
    ids = rng.integers(0, V, size=(30, T))
    out = o.forward(arr, ids.reshape(-1), None, 30)
    for nn in range(30):
        for e in range(T):
            flat = (e * V + ids[nn, e]) * d + np.arange(d)
            np.testing.assert_array_equal(out[nn, e], np.take(arr, flat, mode="wrap"))


def test_identity_sketch_backward_is_add_at():
    # backward of a table lookup is np.add.at on the flattened table
    T, V, d, Z = 3, 30, 8, 4
    n = T * V * d
    rng = np.random.default_rng(8)
    o = orc.Oracle(n, Z, d, T, layout_consts(V, d, Z))
    B = 64
    ids = rng.integers(0, V, size=(B, T))
    grad = rng.standard_normal((B, T, d)).astype(np.float32)
    delta, l1 = o.backward_f64(grad, ids.reshape(-1), None, B)
    want = np.zeros(n)
    pos = ((np.arange(T)[None, :] * V + ids) * d)[:, :, None] + np.arange(d)[None, None, :]
    np.add.at(want, pos.reshape(-1), grad.astype(np.float64).reshape(-1))
    np.testing.assert_allclose(delta, want, rtol=0, atol=1e-12)
    wl1 = np.zeros(n)
    np.add.at(wl1, pos.reshape(-1), np.abs(grad.astype(np.float64)).reshape(-1))
    np.testing.assert_allclose(l1, wl1, rtol=0, atol=1e-12)


# ---------------------------------------------------------------------------------------
# 3. brute-force location table from the parameter-vector procedure (appendix "ROBE-Z")
# ---------------------------------------------------------------------------------------

def brute_force_locations(kk, m, Z, d, vocab):
    """Flatten every table row-wise, concatenate, cut every embedding into chunks of Z, hash each
    chunk with (table, row, chunk number), lay the chunk down circularly.  Returns
    loc[e][x] = list of the d array slots.  Written with Python integers only."""
    loc = []
    for e, V in enumerate(vocab):
        rows = []
        for x in range(V):
            slots = [None] * d
            pos = 0
            chunk_no = 0
            while pos < d:
                start = ((kk[1] * e + kk[2] * x + kk[3] * chunk_no + kk[4]) % kk[0]) % m
                for within in range(min(Z, d - pos)):
                    slots[pos + within] = (start + within) % m
                pos += Z
                chunk_no += 1
            rows.append(slots)
        loc.append(rows)
    return loc


@pytest.mark.parametrize("m,Z,d", [(4096, 4, 16), (17, 16, 16), (17, 4, 16), (33, 8, 32), (64, 5, 12)])
def test_forward_equals_brute_force_table(m, Z, d):
    vocab = [1000, 500, 2000, 100] if m == 4096 else [40, 7, 19]
    T = len(vocab)
    k = orc.hash_constants(0x0B0E + 1)
    kk = [int(v) for v in k]
    loc = brute_force_locations(kk, m, Z, d, vocab)
    o = orc.Oracle(m, Z, d, T, k)
    arr = np.random.default_rng(1).standard_normal(m).astype(np.float32)
    # every (e, x) once: a batch with x running over the largest vocabulary
    Vmax = max(vocab)
    ids = np.stack([np.arange(Vmax) % V for V in vocab], axis=1)
    out = o.forward(arr, ids.reshape(-1), None, Vmax)
    for e, V in enumerate(vocab):
        for x in range(V):
            want = arr[np.array(loc[e][x])]
            np.testing.assert_array_equal(out[x, e], want)
            np.testing.assert_array_equal(o.locate(e, x), np.array(loc[e][x], dtype=np.uint64))
            # the per-element form of the mapping (Section 3.2, idx equation), element by element:
            # an in-chunk offset taken inside the hash argument would fail here for every Z > 1
            if x < 64:
                assert [o.idx(e, x, i) for i in range(d)] == loc[e][x]


def brute_force_locations_clubbed(kk, m, Z, d, vocab):
    """Z > d by the appendix's procedure taken literally: flatten the table row-wise into one
    vector of V*d parameters, cut THAT into chunks of Z (the last may be short), hash chunk number
    X of table e with (e, X, 0), lay it down circularly.  loc[e][x][i] = slot of flat position
    x*d + i.  Python integers only; no division of x by Z/d anywhere."""
    loc = []
    for e, V in enumerate(vocab):
        flat = [None] * (V * d)
        for X in range((V * d + Z - 1) // Z):
            start = ((kk[1] * e + kk[2] * X + kk[3] * 0 + kk[4]) % kk[0]) % m
            for within in range(min(Z, V * d - X * Z)):
                flat[X * Z + within] = (start + within) % m
        loc.append([flat[x * d:(x + 1) * d] for x in range(V)])
    return loc


@pytest.mark.parametrize("m,Z,d", [(4096, 64, 16), (101, 32, 16), (50, 48, 16), (97, 24, 8), (40, 36, 12)])
def test_z_above_d_equals_flattened_table_chunks(m, Z, d):
    # Section 3.2, last paragraph, with the appendix's parameter-vector construction
    vocab = [1000, 37, 5] if m == 4096 else [40, 7, 19]
    T = len(vocab)
    k = orc.hash_constants(0x0B0E + 9)
    loc = brute_force_locations_clubbed([int(v) for v in k], m, Z, d, vocab)
    o = orc.Oracle(m, Z, d, T, k)
    arr = np.random.default_rng(2).standard_normal(m).astype(np.float32)
    Vmax = max(vocab)
    ids = np.stack([np.arange(Vmax) % V for V in vocab], axis=1)
    out = o.forward(arr, ids.reshape(-1), None, Vmax)
    for e, V in enumerate(vocab):
        for x in range(V):
            np.testing.assert_array_equal(out[x, e], arr[np.array(loc[e][x])])
            np.testing.assert_array_equal(o.locate(e, x), np.array(loc[e][x], dtype=np.uint64))
            assert [o.idx(e, x, i) for i in range(d)] == loc[e][x]
    # rows of one chunk sit side by side (mod m): that is the point of Z > d
    R = Z // d
    a, b = o.locate(0, R * 3), o.locate(0, R * 3 + 1)
    assert (int(a[-1]) + 1) % m == int(b[0])


def test_z_above_d_backward_adjoint_mass_and_canonical():
    m, Z, d, T, B = 211, 32, 8, 3, 50
    k = orc.hash_constants(5)
    o = orc.Oracle(m, Z, d, T, k)
    rng = np.random.default_rng(3)
    ids = rng.integers(0, 30, size=B * T)
    arr = rng.standard_normal(m)
    g = rng.standard_normal((B, T, d)).astype(np.float32)
    out = o.forward(arr.astype(np.float32), ids, None, B).astype(np.float64)
    delta, l1 = o.backward_f64(g, ids, None, B)
    lhs = float((out * g).sum())
    rhs = float((arr.astype(np.float32).astype(np.float64) * delta).sum())
    assert abs(lhs - rhs) <= 1e-9 * (abs(lhs) + 1)
    assert abs(delta.sum() - g.astype(np.float64).sum()) < 1e-9 * l1.sum()
    gi = rng.integers(-3, 4, size=(B, T, d)).astype(np.float32)
    di, _ = o.backward_f64(gi, ids, None, B)
    can, touched = o.backward_canonical(gi, ids, None, B)
    np.testing.assert_array_equal(can, di.astype(np.float32))
    assert touched.sum() == (di != 0).sum() + ((di == 0) & (touched == 1)).sum()


def test_blocks_are_consecutive_and_collision_free():
    # Section 4.1 intuition: elements inside one block never collide; slots are consecutive mod m
    k = orc.hash_constants(21)
    for m, Z, d in [(17, 16, 16), (100, 8, 32), (4096, 4, 16)]:
        o = orc.Oracle(m, Z, d, 2, k)
        for x in range(200):
            s = o.locate(1, x).astype(np.int64)
            for c in range(d // Z):
                blk = s[c * Z:(c + 1) * Z]
                assert len(set(blk.tolist())) == Z
                assert np.all((blk - blk[0]) % m == np.arange(Z))
                assert blk[0] == o.h(1, x, c)


# ---------------------------------------------------------------------------------------
# 4. special cases named by the paper
# ---------------------------------------------------------------------------------------

def test_robe_d_is_a_random_offset_window():
    # Section 3.1: Z = d, the embedding is one circular window starting at h(e,x)
    m, d = 1000, 16
    k = orc.hash_constants(4)
    o = orc.Oracle(m, d, d, 3, k)
    arr = np.arange(m, dtype=np.float32)
    ids = np.arange(300).reshape(100, 3)
    out = o.forward(arr, ids.reshape(-1), None, 100)
    wrapped = 0
    for nn in range(100):
        for e in range(3):
            h = o.h(e, int(ids[nn, e]), 0)
            np.testing.assert_array_equal(out[nn, e], np.take(arr, np.arange(h, h + d), mode="wrap"))
            wrapped += h + d > m
    assert wrapped > 0


def test_robe_1_hashes_every_element():
    # Section 3.3: Z = 1, element i is fetched from h(e,x,i)
    m, d = 5000, 16
    k = orc.hash_constants(5)
    o = orc.Oracle(m, 1, d, 2, k)
    arr = np.random.default_rng(0).standard_normal(m).astype(np.float32)
    ids = np.arange(100).reshape(50, 2)
    out = o.forward(arr, ids.reshape(-1), None, 50)
    for nn in range(50):
        for e in range(2):
            want = [arr[o.h(e, int(ids[nn, e]), i)] for i in range(d)]
            np.testing.assert_array_equal(out[nn, e], np.array(want, dtype=np.float32))


def test_iota_array_reads_index_sequence():
    m, d, Z = 50, 12, 4
    o = orc.Oracle(m, Z, d, 1, orc.hash_constants(6))
    arr = np.arange(m, dtype=np.float32)
    out = o.forward(arr, np.array([7]), None, 1)[0, 0]
    for c in range(3):
        assert np.all((out[c * Z:(c + 1) * Z] - out[c * Z]) % m == np.arange(Z))


def test_table_1_fetch_bounds():
    # Table 1: max number of B-element lines touched by one embedding (no block wrapping)
    k = orc.hash_constants(77)
    m, D = 1 << 20, 128
    for Z, Bl in [(1, 8), (2, 8), (4, 8), (32, 8), (64, 16), (128, 8), (128, 32)]:
        o = orc.Oracle(m, Z, D, 1, k)
        if Z == 1:
            bound = D
        elif Z < Bl:
            bound = 2 * D // Z
        elif Z < D:
            bound = D // Bl + D // Z
        else:
            bound = D // Bl + 2
        worst = 0
        for x in range(300):
            s = o.locate(0, x).astype(np.int64)
            if any(s[c * Z] + Z > m for c in range(D // Z)):
                continue
            worst = max(worst, len(set((s // Bl).tolist())))
        assert worst <= bound
        if Z >= Bl:
            assert worst >= D // Bl  # and a contiguous read cannot do better than D/B


# ---------------------------------------------------------------------------------------
# 5. pooling and sign
# ---------------------------------------------------------------------------------------

def _setup(m=4096, Z=4, d=16, T=4, seed=0x0B0F, sign=False):
    k = orc.hash_constants(seed)
    o = orc.Oracle(m, Z, d, T, k, sign=sign)
    arr = (np.random.default_rng(3).standard_normal(m) * 0.01).astype(np.float32)
    return o, arr


def test_pooling_is_sequential_fp32_sum_of_one_hot_rows():
    o, arr = _setup()
    rng = np.random.default_rng(9)
    B, T = 6, o.T
    lengths = rng.integers(0, 7, size=B * T)
    lengths[3] = 0
    offsets = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    ids = rng.integers(0, 100, size=int(offsets[-1]))
    out = o.forward(arr, ids, offsets, B).reshape(B * T, o.d)
    for bag in range(B * T):
        e = bag % T
        rows = []
        for p in range(offsets[bag], offsets[bag + 1]):
            tmp = np.zeros(T, dtype=np.int64)
            tmp[e] = ids[p]
            rows.append(o.forward(arr, tmp, None, 1)[0, e])
        if not rows:
            assert np.all(out[bag] == 0) and not np.any(np.signbit(out[bag]))
            continue
        want = functools.reduce(lambda a, b: (a + b).astype(np.float32), rows)
        np.testing.assert_array_equal(out[bag], want)
        np.testing.assert_allclose(out[bag], np.sum(np.array(rows, dtype=np.float64), axis=0),
                                   rtol=1e-6, atol=1e-9)


def test_bag_of_twice_the_same_id_doubles():
    o, arr = _setup(T=1)
    one = o.forward(arr, np.array([42]), None, 1)[0, 0]
    two = o.forward(arr, np.array([42, 42]), np.array([0, 2]), 1)[0, 0]
    np.testing.assert_array_equal(two, 2 * one)


def test_sign_is_plus_minus_one_and_only_flips():
    o_off, arr = _setup(sign=False)
    o_on, _ = _setup(sign=True)
    ids = np.arange(400).reshape(100, 4)
    a = o_off.forward(arr, ids.reshape(-1), None, 100)
    b = o_on.forward(arr, ids.reshape(-1), None, 100)
    np.testing.assert_array_equal(np.abs(a), np.abs(b))
    signs = np.array([[[o_on.g(e, int(ids[n, e]), i) for i in range(16)] for e in range(4)]
                      for n in range(100)])
    assert set(np.unique(signs).tolist()) == {-1, 1}
    np.testing.assert_array_equal(b, a * signs.astype(np.float32))
    assert abs(signs.mean()) < 0.05  # 6400 fair coins: sigma = 0.0125
    assert not np.array_equal(a, b)


# ---------------------------------------------------------------------------------------
# 6. backward: transpose of forward, mass conservation, canonical order
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("sign", [False, True])
@pytest.mark.parametrize("bags", [False, True])
def test_adjoint_identity(sign, bags):
    # backward is the transpose of the forward gather (sketching-matrix view, Section 4):
    # <forward(M), G> == <M, backward(G)> in exact-ish arithmetic
    m, Z, d, T, B = 300, 4, 12, 3, 40
    k = orc.hash_constants(12)
    o = orc.Oracle(m, Z, d, T, k, sign=sign)
    rng = np.random.default_rng(2)
    # integer-valued data make both sides exact in fp32/fp64
    arr = rng.integers(-8, 9, size=m).astype(np.float32)
    G = rng.integers(-8, 9, size=(B, T, d)).astype(np.float32)
    if bags:
        lengths = rng.integers(0, 5, size=B * T)
        offsets = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
        ids = rng.integers(0, 60, size=int(offsets[-1]))
    else:
        offsets = None
        ids = rng.integers(0, 60, size=B * T)
    out = o.forward(arr, ids, offsets, B)
    delta, _ = o.backward_f64(G, ids, offsets, B)
    lhs = float(np.sum(out.astype(np.float64) * G.astype(np.float64)))
    rhs = float(np.sum(arr.astype(np.float64) * delta))
    assert lhs == rhs


def _renumber_table_major(ids, offsets, B, T):
    """The same bags numbered e*B + n instead of n*T + e: ids, offsets, and old bag of every new one."""
    old_of_new = np.array([n * T + e for e in range(T) for n in range(B)], dtype=np.int64)
    if offsets is None:
        return ids[old_of_new], None, old_of_new
    pieces = [ids[offsets[k]:offsets[k + 1]] for k in old_of_new]
    lengths = np.diff(offsets)[old_of_new]
    return (np.concatenate(pieces) if pieces else ids[:0],
            np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64), old_of_new)


@pytest.mark.parametrize("sign", [False, True])
@pytest.mark.parametrize("bags", [False, True])
def test_table_major_bags_are_the_same_bags_renumbered(sign, bags):
    # Numbering the bags table by table changes which row of the output a bag is, nothing else:
    # forward rows and (on integer data, where no order matters) gradient sums are those of the
    # default numbering.
    m, Z, d, T, B = 307, 4, 12, 3, 17
    k = orc.hash_constants(21)
    o = orc.Oracle(m, Z, d, T, k, sign=sign)
    otm = orc.Oracle(m, Z, d, T, k, sign=sign, table_major=True)
    rng = np.random.default_rng(5)
    arr = (rng.standard_normal(m) * 0.01).astype(np.float32)
    G = rng.integers(-8, 9, size=(B, T, d)).astype(np.float32)
    if bags:
        lengths = rng.integers(0, 5, size=B * T)
        offsets = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
        ids = rng.integers(0, 60, size=int(offsets[-1]))
    else:
        offsets, ids = None, rng.integers(0, 60, size=B * T)
    ids_tm, offs_tm, old_of_new = _renumber_table_major(ids, offsets, B, T)
    want = o.forward(arr, ids, offsets, B).reshape(B * T, d)[old_of_new]
    got = otm.forward(arr, ids_tm, offs_tm, B)
    assert got.shape == (T, B, d)
    np.testing.assert_array_equal(got.reshape(B * T, d).view(np.uint32), want.view(np.uint32))
    some = np.array([0, 5, B, B * T - 1], dtype=np.int64)
    np.testing.assert_array_equal(otm.forward_bags(arr, ids_tm, offs_tm, some, batch=B).view(np.uint32),
                                  want[some].view(np.uint32))
    G_tm = G.reshape(B * T, d)[old_of_new].reshape(T, B, d)
    d_sm, l1_sm = o.backward_f64(G, ids, offsets, B)
    d_tm, l1_tm = otm.backward_f64(G_tm, ids_tm, offs_tm, B)
    np.testing.assert_array_equal(d_tm, d_sm)
    np.testing.assert_array_equal(l1_tm, l1_sm)
    can, touched = otm.backward_canonical(G_tm, ids_tm, offs_tm, B)
    np.testing.assert_array_equal(can.astype(np.float64), d_sm)
    assert not np.any(~touched.astype(bool) & (l1_sm > 0))  # every slot that got mass is marked
    np.testing.assert_array_equal(touched, o.backward_canonical(G, ids, offsets, B)[1])


def test_table_major_canonical_order_follows_the_position_in_that_numbering():
    # Four one-element embeddings on ONE slot: with A_h = B_h = 1 the ids 5 of table 0 and 4 of
    # table 1 hash alike.  Equal block starts are added in the order of their position in the id
    # array, which the bag numbering fixes.  Gradients (n, e): (0,0) 1e8, (0,1) 1, (1,0) -1e8,
    # (1,1) 1; in fp32 1e8 + 1 = 1e8.
    #   default numbering, positions (0,0) (0,1) (1,0) (1,1): ((1e8 + 1) - 1e8) + 1 = 1
    #   table by table,    positions (0,0) (1,0) (0,1) (1,1): ((1e8 - 1e8) + 1) + 1 = 2
    m, T, B = 97, 2, 2
    kk = consts()
    G = np.array([[[1e8], [1.0]], [[-1e8], [1.0]]], dtype=np.float32)  # [B, T, 1]
    ids = np.array([5, 4, 5, 4], dtype=np.int64)                       # (n, e) = (0,0) (0,1) (1,0) (1,1)
    o = orc.Oracle(m, 1, 1, T, kk)
    slot = o.idx(0, 5, 0)
    assert slot == o.idx(1, 4, 0)
    can, _ = o.backward_canonical(G, ids, None, B)
    assert can[slot] == np.float32(1.0)
    otm = orc.Oracle(m, 1, 1, T, kk, table_major=True)
    ids_tm, _, old_of_new = _renumber_table_major(ids, None, B, T)
    G_tm = G.reshape(B * T, 1)[old_of_new].reshape(T, B, 1)
    can_tm, _ = otm.backward_canonical(G_tm, ids_tm, None, B)
    assert can_tm[slot] == np.float32(2.0)


def test_gradient_mass_is_conserved():
    m, Z, d, T, B = 500, 8, 16, 2, 30
    o = orc.Oracle(m, Z, d, T, orc.hash_constants(13))
    rng = np.random.default_rng(4)
    lengths = rng.integers(0, 6, size=B * T)
    offsets = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    ids = rng.integers(0, 1000, size=int(offsets[-1]))
    G = rng.standard_normal((B, T, d)).astype(np.float32)
    delta, l1 = o.backward_f64(G, ids, offsets, B)
    G64 = G.astype(np.float64).reshape(B * T, d)
    np.testing.assert_allclose(delta.sum(), (lengths * G64.sum(axis=1)).sum(), rtol=1e-12)
    np.testing.assert_allclose(l1.sum(), (lengths * np.abs(G64).sum(axis=1)).sum(), rtol=1e-12)


def test_window_restriction_matches_full():
    m, Z, d, T, B = 257, 4, 8, 2, 50
    o = orc.Oracle(m, Z, d, T, orc.hash_constants(14))
    rng = np.random.default_rng(6)
    ids = rng.integers(0, 100, size=B * T)
    G = rng.standard_normal((B, T, d)).astype(np.float32)
    full, l1 = o.backward_f64(G, ids, None, B)
    part, pl1 = o.backward_f64(G, ids, None, B, j0=100, jn=57)
    np.testing.assert_array_equal(part, full[100:157])
    np.testing.assert_array_equal(pl1, l1[100:157])
    cf, tf = o.backward_canonical(G, ids, None, B)
    cp, tp = o.backward_canonical(G, ids, None, B, j0=100, jn=57)
    np.testing.assert_array_equal(cp, cf[100:157])
    np.testing.assert_array_equal(tp, tf[100:157])


def test_canonical_equals_f64_on_integer_gradients():
    # small integers add exactly in fp32, so every summation order gives the same bits
    m, Z, d, T, B = 64, 4, 8, 2, 200
    o = orc.Oracle(m, Z, d, T, orc.hash_constants(15), sign=True)
    rng = np.random.default_rng(7)
    ids = rng.integers(0, 30, size=B * T)
    G = rng.integers(-4, 5, size=(B, T, d)).astype(np.float32)
    delta64, l1 = o.backward_f64(G, ids, None, B)
    can, touched = o.backward_canonical(G, ids, None, B)
    np.testing.assert_array_equal(can.astype(np.float64), delta64)
    np.testing.assert_array_equal(touched.astype(bool), l1 > 0)


def test_canonical_close_to_f64_on_real_gradients():
    m, Z, d, T, B = 128, 4, 16, 2, 300
    o = orc.Oracle(m, Z, d, T, orc.hash_constants(16))
    rng = np.random.default_rng(17)
    ids = rng.integers(0, 50, size=B * T)
    G = rng.standard_normal((B, T, d)).astype(np.float32)
    delta64, l1 = o.backward_f64(G, ids, None, B)
    can, _ = o.backward_canonical(G, ids, None, B)
    nterms = B * T * d / m * 4
    assert np.all(np.abs(can - delta64) <= nterms * 2.0 ** -24 * l1 + 1e-30)


def _golden_cases():
    cases = []
    with open(os.path.join(GOLDEN, "canonical_order.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, Z, d, m, starts, rows, slot, want = [t.strip() for t in line.split("|")]
            cases.append((name, int(Z), int(d), int(m), [int(s) for s in starts.split(",")],
                          [[float(v) for v in r.split(",")] for r in rows.split(";")],
                          int(slot), float(want)))
    return cases


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: c[0])
def test_canonical_order_golden(case):
    # B = 1, A = C = D = 0 make the block start equal to the id itself
    name, Z, d, m, starts, rows, slot, want = case
    o = orc.Oracle(m, Z, d, 1, consts(Ah=0, Bh=1, Ch=0, Dh=0))
    ids = np.array(starts, dtype=np.int64)
    G = np.array(rows, dtype=np.float32).reshape(len(starts), 1, d)
    can, touched = o.backward_canonical(G, ids, None, len(starts))
    assert touched[slot] == 1
    assert can[slot] == np.float32(want)
    # repeated runs give the same bits
    can2, _ = o.backward_canonical(G, ids, None, len(starts))
    np.testing.assert_array_equal(can, can2)


def test_sgd_apply_and_accumulate():
    arr = np.array([1.0, 2.0, 3.0, -0.0], dtype=np.float32)
    delta = np.array([0.5, 0.25, 7.0, 0.0], dtype=np.float32)
    touched = np.array([1, 0, 1, 0], dtype=np.uint8)
    a = arr.copy()
    orc.sgd_apply(a, delta, touched, 2.0)
    np.testing.assert_array_equal(a, np.array([0.0, 2.0, -11.0, -0.0], dtype=np.float32))
    assert np.signbit(a[3])
    g = np.array([1.0, 1.0, 1.0, 1.0], dtype=np.float32)
    orc.accumulate(g, delta, touched)
    np.testing.assert_array_equal(g, np.array([1.5, 1.0, 8.0, 1.0], dtype=np.float32))


def test_adagrad_apply_hand_computed_and_torch():
    # Adagrad (Duchi et al.): s <- s + g^2, theta <- theta - lr g / (sqrt(s) + eps).  Powers of two make
    # the first step exact: g = eps = 2^-3, s = 2^-6, sqrt(s) + eps = 2^-2, update 1/2, theta = 1 - lr/2;
    # second step with the same g: s = 2^-5, no longer exact, closed form to rounding.
    g = np.float32(0.125)
    arr = np.array([1.0, 1.0, -3.0], np.float32)
    ssq = np.zeros(3, np.float32)
    delta = np.array([g, -g, 0.5], np.float32)
    touched = np.array([1, 1, 0], np.uint8)
    orc.adagrad_apply(arr, ssq, delta, touched, 0.25, float(g))
    np.testing.assert_array_equal(arr, np.array([0.875, 1.125, -3.0], np.float32))
    np.testing.assert_array_equal(ssq, np.array([g * g, g * g, 0.0], np.float32))
    orc.adagrad_apply(arr, ssq, delta, touched, 0.25, float(g))
    want = 0.875 - 0.25 * 0.125 / (np.sqrt(2.0 ** -5) + 0.125)
    assert abs(float(arr[0]) - want) < 1e-7 and arr[2] == -3.0 and ssq[2] == 0.0
    # a library routine: torch.optim.Adagrad (no decay), all slots touched, several steps
    import torch
    rng = np.random.default_rng(12)
    n, lr, eps = 1000, 0.05, 1e-10
    arr = rng.standard_normal(n).astype(np.float32)
    ssq = np.zeros(n, np.float32)
    p_ = torch.nn.Parameter(torch.from_numpy(arr.copy()))
    opt = torch.optim.Adagrad([p_], lr=lr, eps=eps)
    ones = np.ones(n, np.uint8)
    for _ in range(5):
        gr = rng.standard_normal(n).astype(np.float32)
        orc.adagrad_apply(arr, ssq, gr, ones, lr, eps)
        p_.grad = torch.from_numpy(gr.copy())
        opt.step()
        np.testing.assert_allclose(arr, p_.detach().numpy(), rtol=0, atol=5e-7)


def test_dense_sgd_apply_hand_values_and_agreement_with_the_fused_step():
    # data-parallel step: every slot gets fma(-lr, g, M); hand values (exact in fp32)
    arr = np.array([1.0, 2.0, 3.0, -0.0, 0.5], dtype=np.float32)
    g = np.array([0.5, 0.0, 7.0, 0.0, -0.25], dtype=np.float32)
    a = arr.copy()
    orc.dense_sgd_apply(a, g, 2.0)
    np.testing.assert_array_equal(a, np.array([0.0, 2.0, -11.0, -0.0, 1.0], dtype=np.float32))
    # one rounding, not two: 1 + 2^-24 * (1 + 2^-23) is 1 + 2^-23 under fma, 1 under mul-then-add
    one = np.array([1.0], np.float32)
    tiny = np.array([-(2.0 ** -24) * (1 + 2.0 ** -23)], np.float32)
    orc.dense_sgd_apply(one, tiny, 1.0)
    assert one[0] == np.float32(1.0 + 2.0 ** -23)
    # on touched slots it is the fused step; on untouched slots (gradient +0) it changes no bit
    rng = np.random.default_rng(4)
    arr = rng.standard_normal(500).astype(np.float32)
    delta = rng.standard_normal(500).astype(np.float32)
    touched = (rng.random(500) < 0.6).astype(np.uint8)
    fused, dense = arr.copy(), arr.copy()
    orc.sgd_apply(fused, delta, touched, 0.3)
    orc.dense_sgd_apply(dense, np.where(touched == 1, delta, np.float32(0.0)).astype(np.float32), 0.3)
    np.testing.assert_array_equal(fused.view(np.uint32), dense.view(np.uint32))


# ---------------------------------------------------------------------------------------
# 7. Theorem 1: the sketch's inner-product estimator is unbiased with the printed variance
# ---------------------------------------------------------------------------------------

def test_adam_apply_matches_torch_adam_and_closed_form():
    # all slots touched: the lazy step is the textbook one, so torch.optim.Adam (a library routine,
    # fp32) must agree to rounding over several steps; and step 1 has the closed form
    # M - lr g / (|g| + eps) whatever the betas are
    import torch
    rng = np.random.default_rng(11)
    n, lr, b1, b2, eps = 1000, 0.01, 0.9, 0.999, 1e-8
    arr = rng.standard_normal(n).astype(np.float32)
    m1, m2 = np.zeros(n, np.float32), np.zeros(n, np.float32)
    p = torch.nn.Parameter(torch.from_numpy(arr.copy()))
    opt = torch.optim.Adam([p], lr=lr, betas=(b1, b2), eps=eps)
    ones = np.ones(n, np.uint8)
    first = None
    for t in range(1, 6):
        g = rng.standard_normal(n).astype(np.float32)
        if t == 1:
            first = arr.astype(np.float64) - lr * g / (np.abs(g.astype(np.float64)) + eps)
        orc.adam_apply(arr, m1, m2, g, ones, lr, b1, b2, eps, t)
        if t == 1:
            np.testing.assert_allclose(arr, first, rtol=0, atol=2e-7)
        p.grad = torch.from_numpy(g.copy())
        opt.step()
        np.testing.assert_allclose(arr, p.detach().numpy(), rtol=0, atol=5e-7)
    # lazy: an untouched slot keeps array and moments bit for bit
    before = (arr.copy(), m1.copy(), m2.copy())
    touched = np.zeros(n, np.uint8)
    touched[::3] = 1
    orc.adam_apply(arr, m1, m2, rng.standard_normal(n).astype(np.float32), touched, lr, b1, b2, eps, 6)
    for now, was in zip((arr, m1, m2), before):
        np.testing.assert_array_equal(now[touched == 0], was[touched == 0])
        assert np.all(now[touched == 1] != was[touched == 1])


def test_adam_step_hand_computed_eps_sits_outside_the_square_root():
    # Kingma & Ba, Algorithm 1: theta <- theta - lr * mhat / (sqrt(vhat) + eps).  With powers of two
    # every operation is exact, so the step has one value that can be worked out by hand:
    #   g = eps = 2^-10, beta1 = 1/2, beta2 = 3/4, step 1, moments 0
    #   m1 = g/2, mhat = m1 / (1 - 1/2) = g;  m2 = g^2/4, vhat = m2 / (1 - 3/4) = g^2
    #   sqrt(vhat) + eps = 2g  ->  update = 1/2  ->  theta = 1 - lr/2
    # (eps inside the root would give g / sqrt(g^2 + eps) = 0.0312..., eps dropped would give 1)
    g = np.float32(2.0 ** -10)
    arr = np.array([1.0, 1.0, -3.0], np.float32)
    m1, m2 = np.zeros(3, np.float32), np.zeros(3, np.float32)
    delta = np.array([g, -g, 0.0], np.float32)
    orc.adam_apply(arr, m1, m2, delta, np.ones(3, np.uint8), 0.25, 0.5, 0.75, float(g), 1)
    np.testing.assert_array_equal(arr, np.array([0.875, 1.125, -3.0], np.float32))
    np.testing.assert_array_equal(m1, np.array([g / 2, -g / 2, 0.0], np.float32))
    np.testing.assert_array_equal(m2, np.array([g * g / 4, g * g / 4, 0.0], np.float32))
    # step 2, zero gradient on slot 0 (touched), slots 1 and 2 untouched: no longer exact in fp32,
    # but the closed form below fixes the move to rounding
    before = arr.copy()
    orc.adam_apply(arr, m1, m2, np.zeros(3, np.float32), np.array([1, 0, 0], np.uint8), 0.25, 0.5, 0.75,
                   float(g), 2)
    # mhat = g/3; vhat = (3/16 g^2)/(7/16) = 3/7 g^2; update = (1/3)/(sqrt(3/7) + 1)
    want = 0.25 * (1.0 / 3.0) / (np.sqrt(3.0 / 7.0) + 1.0)
    assert abs(float(before[0]) - float(arr[0]) - want) < 1e-7
    assert arr[1] == before[1] and arr[2] == before[2]


def test_theorem_1_mean_and_variance_monte_carlo():
    # parameter vector of n = V*d entries (one table), sketched into m slots with the sign hash on.
    # Theorem 1: E = <x,y>,  V = (1/m) * sum over i,j in different blocks of (x_i^2 y_j^2 + x_i y_i x_j y_j)
    V, d, Z, m = 6, 8, 4, 16
    n = V * d
    rng = np.random.default_rng(123)
    xv = rng.standard_normal(n)
    yv = rng.standard_normal(n)
    blk = np.arange(n) // Z
    diff = blk[:, None] != blk[None, :]
    var_thm = (np.sum(np.outer(xv ** 2, yv ** 2)[diff]) + np.sum(np.outer(xv * yv, xv * yv)[diff])) / m
    ids = np.arange(V, dtype=np.int64)
    Gx = xv.astype(np.float32).reshape(V, 1, d)
    Gy = yv.astype(np.float32).reshape(V, 1, d)
    x32, y32 = Gx.astype(np.float64).reshape(-1), Gy.astype(np.float64).reshape(-1)
    est = []
    for seed in range(3000):
        o = orc.Oracle(m, Z, d, 1, orc.hash_constants(1000 + seed), sign=True)
        xh, _ = o.backward_f64(Gx, ids, None, V)   # the projection S^T x
        yh, _ = o.backward_f64(Gy, ids, None, V)
        est.append(float(xh @ yh))
    est = np.array(est)
    true_ip = float(x32 @ y32)
    se = np.sqrt(var_thm / len(est))
    assert abs(est.mean() - true_ip) < 5 * se
    assert abs(est.var() / var_thm - 1.0) < 0.2
