"""Mobile data chunks and the elastic policies (Sec. 3, Sec. 4.4, Sec. 4.5, Sec. 5.3): the oracle's rules against
hand-worked cases and their defining properties, and the library's host functions against the oracle, bit for bit."""
import numpy as np
import pytest

import oracle
from oracle import chunks as och


def test_cut_hand_example():
    # entries per coordinate 3, 1, 4, 0, 2 -> bytes 32, 16, 40, 8, 24; chunks of at most 56 bytes
    indptr = np.array([0, 3, 4, 8, 8, 10], np.int64)
    assert och.cut(5, 56, indptr).tolist() == [0, 2, 4, 5]       # 32+16 | 40+8 | 24
    assert och.cut(5, 8, indptr).tolist() == [0, 1, 2, 3, 4, 5]  # a chunk holds at least one coordinate
    assert och.cut(5, 10**9, indptr).tolist() == [0, 5]
    assert och.cut(7, 3 * (4 * 10 + 8), dense_dim=10).tolist() == [0, 3, 6, 7]


def test_assign_is_a_random_equal_deal():
    oracle.build()
    t = och.assign(103, 8, 5)
    cnt = np.bincount(t, minlength=8)
    assert cnt.tolist() == [13] * 7 + [12]
    assert (och.assign(103, 8, 5) == t).all() and (och.assign(103, 8, 6) != t).any()
    # the same rule as the coordinate-level partition: one chunk per coordinate reproduces it
    owner, _, _ = oracle.partition(103, 8, 5)
    assert (owner == t).all()


def test_scale_in_hand_example_and_properties():
    t = np.array([0, 3, 1, 2, 3, 0, 2, 3, 1], np.int32)
    # tasks 2 and 3 are freed; their chunks 1, 3, 4, 6, 7 go to 0, 1, 0, 1, 0
    assert och.scale_in(t, 4, 2).tolist() == [0, 0, 1, 1, 0, 0, 1, 0, 1]
    oracle.build()
    t = och.assign(500, 16, 1)
    u = och.scale_in(t, 16, 6)
    stay = t < 6
    assert (u[stay] == t[stay]).all() and u.max() == 5
    got = np.bincount(u[~stay], minlength=6)
    assert got.max() - got.min() <= 1
    assert (och.scale_in(t, 16, 16) == t).all()


def test_scale_out_properties():
    oracle.build()
    C, K0, K1 = 640, 4, 16
    t = och.assign(C, K0, 2)
    u = och.scale_out(t, K0, K1, 9)
    moved = u != t
    assert (u[moved] >= K0).all() and (u[~moved] < K0).all()
    for j in range(K0):  # every old task gives away floor(m_j * 12 / 16) of its chunks
        mj = int((t == j).sum())
        assert int((moved & (t == j)).sum()) == mj * (K1 - K0) // K1
    cnt = np.bincount(u, minlength=K1)
    assert cnt.min() >= 39 and cnt.max() <= 41
    # the new tasks hold chunks of every old task (this is what reshuffles the samples, Sec. 5.3)
    for k in range(K0, K1):
        assert set(t[u == k].tolist()) == set(range(K0))
    # the picks are random: not the lowest-numbered chunks of a task, and another seed picks others
    first = np.nonzero(t == 0)[0][: int((moved & (t == 0)).sum())]
    assert not moved[first].all()
    assert (och.scale_out(t, K0, K1, 10) != u).any()
    assert (och.scale_out(t, K0, K0, 9) == t).all()


def test_scale_out_tiny_by_hand():
    oracle.build()
    t = np.array([0, 0, 0, 0, 1, 1, 1, 1], np.int32)
    u = och.scale_out(t, 2, 4, 3)
    s = oracle.mix64(3 ^ och.SCALE_OUT_STREAM)
    # each old task gives floor(4 * 2 / 4) = 2 chunks: those with the two smallest keys, dealt to tasks 2, 3, 2, 3
    want = t.copy()
    turn = 0
    for j in (0, 1):
        mine = sorted(np.nonzero(t == j)[0].tolist(), key=lambda c: oracle.mix64(s ^ c))
        for c in mine[:2]:
            want[c] = 2 + turn % 2
            turn += 1
    assert (u == want).all() and np.bincount(u).tolist() == [2, 2, 2, 2]


def test_rebalance_moves_chunks_from_slow_to_fast_until_level():
    C, K = 64, 4
    ln = np.full(C, 100, np.int64)
    t = (np.arange(C) % K).astype(np.int32)
    speed = [1.0, 1.0, 1.0, 3.0]  # task 3 takes three times as long per sample
    moves = 0
    while True:
        t, moved = och.rebalance_step(t, ln, K, speed)
        if not moved:
            break
        moves += 1
        assert moves < 100
    samples = np.bincount(t, weights=ln, minlength=K)
    times = samples * np.array(speed)
    assert samples[3] < samples[:3].min()
    assert times.max() - times.min() <= 100 * 3.0  # within one chunk of the slow task
    # level already: nothing moves
    t2, moved = och.rebalance_step((np.arange(C) % K).astype(np.int32), ln, K, [1.0] * 4)
    assert not moved


def test_partition_from_chunks():
    off = np.array([0, 2, 3, 7, 8], np.int64)
    owner, part_off, members = och.partition_from_chunks(8, 2, off, [1, 0, 1, 0])
    assert owner.tolist() == [1, 1, 0, 1, 1, 1, 1, 0]
    assert part_off.tolist() == [0, 2, 8] and members.tolist() == [2, 7, 0, 1, 3, 4, 5, 6]
    with pytest.raises(ValueError):
        och.partition_from_chunks(8, 3, off, [1, 0, 1, 0])  # task 2 holds nothing
    with pytest.raises(ValueError):
        och.partition_from_chunks(9, 2, off, [1, 0, 1, 0])


def test_rounds_on_a_chunk_partition_keep_the_invariants():
    oracle.build()
    rng = np.random.default_rng(0)
    n, d = 300, 10
    X = rng.standard_normal((n, d))
    y = np.where(X @ rng.standard_normal(d) >= 0, 1.0, -1.0)
    o = oracle.CocoaOracle("hinge", "dense", n, d, X.astype(np.float32).reshape(-1), y.astype(np.float32), 1.0 / n, threads=2)
    off = och.cut(n, 7 * (4 * d + 8), dense_dim=d)
    task = och.assign(len(off) - 1, 8, 0)
    o.partition_chunks(8, 0, off, task)
    prev = o.duality_gap()["dual"]
    for r, (K, fn) in enumerate([(8, None), (3, "in"), (3, None), (6, "out")]):
        if fn == "in":
            task = och.scale_in(task, 8, 3)
            o.partition_chunks(3, 0, off, task)
        if fn == "out":
            task = och.scale_out(task, 3, 6, 4)
            o.partition_chunks(6, 0, off, task)
        assert sorted(o.members.tolist()) == list(range(n))
        o.cocoa_round(0, float(K))
        g = o.duality_gap()
        assert g["dual"] >= prev - 1e-13 and g["gap"] >= -1e-12
        prev = g["dual"]
        v2 = o.recompute_shared_vector()
        assert np.abs(v2 - o.v).max() <= 1e-12 * max(1.0, np.abs(v2).max())


# ------------------------------------------------------------------ the library's host functions against the oracle
def _lib():
    from paper_1909_04885_b200 import binding, build
    build.build()
    return binding


def test_library_chunk_functions_match_the_oracle_bit_for_bit():
    oracle.build()
    b = _lib()
    rng = np.random.default_rng(3)
    for n, bytes_ in ((1, 64), (50, 8), (5000, 4096), (5000, 300)):
        nnz = rng.poisson(6, n)
        nnz[rng.integers(0, n, max(1, n // 50))] = 400  # a few coordinates larger than a chunk
        indptr = np.concatenate([[0], np.cumsum(nnz)]).astype(np.int64)
        assert np.array_equal(b.chunks_cut(n, bytes_, indptr), och.cut(n, bytes_, indptr))
    assert np.array_equal(b.chunks_cut(1000, 1000, None, 28), och.cut(1000, 1000, None, 28))
    for C, K, seed in ((1, 1, 0), (17, 17, 1), (1000, 7, 2**63 + 5), (4097, 64, 3)):
        assert np.array_equal(b.chunks_assign(C, K, seed), och.assign(C, K, seed))
    t = och.assign(1500, 24, 4)
    for K_new in (24, 23, 5, 1):
        assert np.array_equal(b.chunks_scale_in(t, 24, K_new), och.scale_in(t, 24, K_new))
    t = och.assign(1500, 3, 5)
    for K_new, seed in ((3, 0), (4, 1), (16, 2), (100, 2**64 - 1)):
        assert np.array_equal(b.chunks_scale_out(t, 3, K_new, seed), och.scale_out(t, 3, K_new, seed))
    # rebalancing: the same sequence of moves until both stop
    off = och.cut(5000, 300, indptr)
    C = len(off) - 1
    K = 5
    speed = [1.0, 2.5, 1.0, 0.7, 1.2]
    to, tl = och.assign(C, K, 0), b.chunks_assign(C, K, 0)
    ln = np.diff(off)
    for it in range(10 * C):
        to, mo = och.rebalance_step(to, ln, K, speed)
        tl, ml = b.chunks_rebalance_step(tl, off, K, speed)
        assert mo == ml and np.array_equal(to, tl)
        if not mo:
            break
    assert it > 3 and not mo


def test_library_chunk_functions_refuse_bad_arguments():
    b = _lib()
    with pytest.raises(b.ChicleError):
        b.chunks_assign(4, 5, 0)
    with pytest.raises(b.ChicleError):
        b.chunks_scale_in(np.zeros(4, np.int32), 2, 3)
    with pytest.raises(b.ChicleError):
        b.chunks_scale_out(np.zeros(4, np.int32), 3, 2, 0)
    with pytest.raises(b.ChicleError):
        b.chunks_scale_out(np.array([0, 5], np.int32), 2, 4, 0)
    with pytest.raises(ValueError):
        b.chunks_cut(0, 64, np.zeros(1, np.int64))


# ------------------------------------------------------------------ on the GPU: partitions from placements, rounds
@pytest.mark.gpu
def test_chunk_partitions_and_elastic_rounds_match_the_oracle():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    b = _lib()
    from paper_1909_04885_b200 import datagen
    from parity_util import REL_TOL, gap_close, make_pair, rel_l2
    w = datagen.make("hinge_csr", 100)
    orc, glm = make_pair(w)
    try:
        off = b.chunks_cut(w.n_coord, 16384, w.indptr)
        assert np.array_equal(off, och.cut(w.n_coord, 16384, w.indptr))
        C = len(off) - 1
        task = b.chunks_assign(C, 16, 1)
        schedule = [(16, None), (16, None), (6, "in"), (6, None), (24, "out"), (24, "rebalance"), (24, None)]
        K_prev = 16
        for r, (K, move) in enumerate(schedule):
            if move == "in":
                task = b.chunks_scale_in(task, K_prev, K)
            elif move == "out":
                task = b.chunks_scale_out(task, K_prev, K, 7)
            elif move == "rebalance":
                speed = [1.0 + (k % 3) for k in range(K)]
                for _ in range(40):
                    task, moved = b.chunks_rebalance_step(task, off, K, speed)
                    assert moved
            K_prev = K
            orc.partition_chunks(K, 3, off, task)
            glm.partition_chunks(K, 3, off, task)
            assert np.array_equal(glm.get_partition(), orc.owner)
            for k in (0, K // 2, K - 1):
                n_k = int(orc.part_off[k + 1] - orc.part_off[k])
                assert np.array_equal(glm.get_permutation(r, k, n_k), orc.permutation(r, k))
            orc.cocoa_round(0, float(K))
            glm.cocoa_round(0, float(K))
            assert rel_l2(glm.get_alpha(), orc.state) <= REL_TOL and rel_l2(glm.get_v(), orc.v) <= REL_TOL
            ok, tol = gap_close(glm.duality_gap(), orc.duality_gap())
            assert ok
        # bad placements leave the handle as it was
        before = glm.get_partition().copy()
        for bad_off, bad_task in ((off[:-1], task[:-1]), (off, np.where(task == 3, 4, task)), (off, task + 1)):
            with pytest.raises(b.ChicleError) as e:
                glm.partition_chunks(24, 3, bad_off, bad_task)
            assert e.value.status == 1
        assert np.array_equal(before, glm.get_partition())
        glm.cocoa_round(0, 24.0)
    finally:
        glm.close()


@pytest.mark.gpu
def test_chunk_partition_dense_and_one_chunk_per_coordinate():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    b = _lib()
    from paper_1909_04885_b200 import datagen
    from parity_util import REL_TOL, make_pair, rel_l2
    w = datagen.make("hinge_dense", 64)
    orc, glm = make_pair(w)
    try:
        n = w.n_coord
        # one chunk per coordinate with the random deal is chicle_partition itself
        off = np.arange(n + 1, dtype=np.int64)
        glm.partition_chunks(5, 9, off, b.chunks_assign(n, 5, 9))
        a = glm.get_partition().copy()
        glm.partition(5, 9)
        assert np.array_equal(a, glm.get_partition())
        off = b.chunks_cut(n, 40 * (4 * w.n_cols + 8), None, w.n_cols)
        task = b.chunks_assign(len(off) - 1, 4, 2)
        for K, t in ((4, task), (2, b.chunks_scale_in(task, 4, 2))):
            orc.partition_chunks(K, 1, off, t)
            glm.partition_chunks(K, 1, off, t)
            assert np.array_equal(glm.get_partition(), orc.owner)
            orc.cocoa_round(0, float(K))
            glm.cocoa_round(0, float(K))
            assert rel_l2(glm.get_alpha(), orc.state) <= REL_TOL and rel_l2(glm.get_v(), orc.v) <= REL_TOL
    finally:
        glm.close()
