"""Mobile data chunks and the elastic policies (Sec. 3, Sec. 4.3, Sec. 4.5, Sec. 5.3): the oracle's rules against
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
