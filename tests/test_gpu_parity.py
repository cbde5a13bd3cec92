"""GPU parity: the library, called through its C ABI, against the CPU oracle on the same seeded inputs.
Integer results (partition, visiting orders) must be bit-exact; alpha, v and the gap within 1e-4 per round."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from paper_1909_04885_b200 import binding, datagen  # noqa: E402
from paper_1909_04885_b200.datagen import Phase, Workload  # noqa: E402

import oracle  # noqa: E402
from parity_util import check_partition, make_pair, rel_l2, run_parity, REL_TOL  # noqa: E402


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_1909_04885_b200 import build
    build.build()
    oracle.build()


def tiny_dense(n, d, seed=0, loss="hinge", K=3, lam=None, rounds=4):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n, d)).astype(np.float32)
    w = rng.standard_normal(d)
    y = np.where(X @ w + 0.3 * rng.standard_normal(n) >= 0, 1.0, -1.0).astype(np.float32)
    return Workload("tiny_dense", loss, "dense", n, d, X.reshape(-1), y, lam or 1.0 / n, rounds,
                    [Phase(0, K, seed, float(K))])


def tiny_csr(n, d, seed=0, loss="hinge", K=3, density=0.2, rounds=4, long_row=0, zero_rows=()):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n, d)).astype(np.float32)
    X[rng.random((n, d)) > density] = 0.0
    if long_row:
        X[1, :long_row] = rng.standard_normal(long_row).astype(np.float32) * 0.1 + 0.5
    for r in zero_rows:
        X[r] = 0.0
    w = rng.standard_normal(d)
    y = np.where(X @ w >= 0, 1.0, -1.0).astype(np.float32)
    indptr = np.zeros(n + 1, np.int64)
    indptr[1:] = np.cumsum((X != 0).sum(1))
    idx = np.nonzero(X)[1].astype(np.int32)
    vals = X[X != 0].astype(np.float32)
    return Workload("tiny_csr", loss, "csr", n, d, vals, y, 1.0 / n, rounds, [Phase(0, K, seed, float(K))], indptr, idx)


# ------------------------------------------------------------------ a1, a2: integers, bit-exact
@pytest.mark.parametrize("n,K,seed", [(10, 3, 0), (4096, 16, 1), (3 * 4096 + 17, 5, 2), (1000, 1, 3), (257, 257, 4),
                                      (70000, 300, 5), (200003, 64, 2**63 + 11)])
def test_partition_and_orders_bit_exact(n, K, seed):
    w = tiny_dense(n, 4, seed=1, K=K)
    w.phases = [Phase(0, K, seed, float(K))]
    orc, glm = make_pair(w)
    try:
        orc.partition(K, seed)
        glm.partition(K, seed)
        check_partition(orc, glm, perm_rounds=(0, 3, 2**20 + 1))
        # repartition with another K and seed (elastic K between rounds)
        K2 = max(1, K // 2)
        orc.partition(K2, seed + 1)
        glm.partition(K2, seed + 1)
        check_partition(orc, glm, perm_rounds=(1,))
    finally:
        glm.close()


# ------------------------------------------------------------------ the five configurations
def test_config1_hinge_dense_full():
    run_parity(datagen.make("hinge_dense", 1))


def test_config2_hinge_csr_scaled():
    run_parity(datagen.make("hinge_csr", 100))


def test_config3_logistic_dense_scaled():
    run_parity(datagen.make("logistic_dense", 100))


def test_config4_hinge_hashed_elastic_scaled():
    w = datagen.make("hinge_hashed", 1000)
    assert [p.K for p in w.phases] == [64, 16]
    run_parity(w)


def test_config5_ridge_csc_scaled():
    run_parity(datagen.make("ridge_csc", 100))


def test_config2_full_size_three_rounds():
    # the benchmark's workload and launch configuration, element by element against the oracle
    w = datagen.make("hinge_csr", 1)
    run_parity(w, rounds=3, check_perm=True, on_device=True)


def test_config3_full_size_two_rounds():
    w = datagen.make("logistic_dense", 1)
    run_parity(w, rounds=2, check_perm=False, on_device=True)


# ------------------------------------------------------------------ edge cases
@pytest.mark.parametrize("loss", ["hinge", "logistic"])
@pytest.mark.parametrize("d", [1, 7, 28, 100, 1000])
def test_dense_shapes(loss, d):
    run_parity(tiny_dense(500, d, seed=d, loss=loss, K=4))


@pytest.mark.parametrize("loss", ["hinge", "logistic"])
def test_csr_with_zero_rows_and_a_row_longer_than_a_slot(loss):
    run_parity(tiny_csr(300, 400, seed=7, loss=loss, K=4, density=0.05, long_row=300, zero_rows=(0, 17)))


def test_single_partition_and_one_coordinate_per_partition():
    run_parity(tiny_csr(64, 40, seed=3, K=1))
    run_parity(tiny_csr(64, 40, seed=3, K=64))
    run_parity(tiny_dense(50, 5, seed=3, K=50))


@pytest.mark.parametrize("H", [1, 10, 37, 60, 250])
def test_partial_and_multi_epoch_H(H):
    # n_k = 25: H below, equal-ish and several local epochs
    run_parity(tiny_dense(100, 6, seed=5, K=4), H=H)
    run_parity(tiny_csr(100, 30, seed=5, K=4), H=H)


def test_rounds_of_several_local_epochs(monkeypatch):
    # H beyond one local epoch: the look-ahead solver runs once per epoch; ragged last epoch, unequal partitions
    # (the small ones go round more often), all three losses; then the blocked solver's own multi-epoch walk
    w = datagen.make("hinge_csr", 100)
    n_k = w.n_coord // w.phases[0].K
    run_parity(w, rounds=3, H=2 * n_k + n_k // 3)
    run_parity(w, rounds=2, H=n_k + 1)
    run_parity(tiny_csr(400, 40, seed=8, K=3), H=700, sizes=[50, 300, 50])
    run_parity(tiny_dense(500, 28, seed=2, loss="logistic", K=4), H=300)
    w = datagen.make("ridge_csc", 100)
    w.phases = [Phase(0, 4, 1, 4.0)]
    run_parity(w, rounds=2, H=w.n_coord // 4 * 2 + 17)
    glm = binding.from_workload(tiny_csr(400, 40, seed=8, K=4))
    try:
        glm.partition(4, 0)
        st = glm.cocoa_round(250, 4.0, stats=True)
        assert st["solver_variant"] == 4 and st["steps"] == 1000
    finally:
        glm.close()
    monkeypatch.setenv("CHICLE_FORCE_VARIANT", "blocked")
    run_parity(tiny_csr(400, 40, seed=8, K=3), H=700, sizes=[50, 300, 50])


def test_rounds_cut_into_slices(monkeypatch):
    # long walks are cut into three slices whose prepare kernels run beside the chain kernels; forced here on walks the
    # oracle finishes in seconds (at least 8 blocks per partition): all losses, unequal partitions, step budgets with an
    # idle partition, several local epochs, and a walk too short to cut
    monkeypatch.setenv("CHICLE_LA_SLICES", "3")
    w = datagen.make("hinge_csr", 100)
    run_parity(w, rounds=4)
    n_k = w.n_coord // w.phases[0].K
    run_parity(w, rounds=2, H=2 * n_k + 300)
    K = w.phases[0].K
    sizes = [n_k + (256 if k % 2 else -256) for k in range(K)]
    run_parity(w, rounds=3, sizes=sizes, steps=lambda r: [0 if (k + r) % 7 == 0 else s - 20 * k for k, s in enumerate(sizes)])
    # a slice of more blocks than the prepare kernel's grid beside the chains has CTAs: its CTAs take several blocks each
    run_parity(datagen.make("hinge_csr", 10), rounds=2, check_perm=False)
    run_parity(datagen.make("hinge_dense", 4), rounds=3)
    run_parity(datagen.make("logistic_dense", 100), rounds=2)
    run_parity(datagen.make("hinge_hashed", 1000), rounds=2)
    w = datagen.make("ridge_csc", 100)
    run_parity(w, rounds=2)
    run_parity(tiny_csr(100, 30, seed=5, K=4))


def test_ridge_small_with_long_and_empty_columns():
    rng = np.random.default_rng(11)
    n, d = 300, 500
    X = rng.random((n, d)).astype(np.float32)
    X[rng.random((n, d)) > 0.1] = 0.0
    X[:, 3] = rng.random(n).astype(np.float32) + 0.1      # a column longer than a slot
    X[:, 9] = 0.0                                          # an empty column
    w = np.zeros(d)
    w[rng.choice(d, 20, replace=False)] = rng.standard_normal(20)
    y = (X @ w + 0.01 * rng.standard_normal(n)).astype(np.float32)
    XT = np.ascontiguousarray(X.T)
    indptr = np.zeros(d + 1, np.int64)
    indptr[1:] = np.cumsum((XT != 0).sum(1))
    wl = Workload("ridge_tiny", "ridge", "csc", n, d, XT[XT != 0].astype(np.float32), y, 1e-2, 6,
                  [Phase(0, 8, 0, 8.0)], indptr, np.nonzero(XT)[1].astype(np.int32))
    run_parity(wl)


def test_resync_mode_and_recomputed_shared_vector():
    w = datagen.make("hinge_csr", 200)
    run_parity(w, rounds=5, resync=True)
    orc, glm = make_pair(w)
    try:
        orc.partition(4, 1)
        glm.partition(4, 1)
        for _ in range(2):
            orc.cocoa_round(0, 4.0)
        glm.set_state(orc.state.astype(np.float32), None, orc.round)      # v rebuilt on the device
        assert rel_l2(glm.get_v(), orc.v) < 1e-5
        assert glm.info()["round"] == 2
        orc.cocoa_round(0, 4.0)
        glm.cocoa_round(0, 4.0)
        assert rel_l2(glm.get_alpha(), orc.state) < REL_TOL and rel_l2(glm.get_v(), orc.v) < REL_TOL
    finally:
        glm.close()


def test_state_survives_repartition_bit_for_bit():
    w = datagen.make("hinge_csr", 200)
    orc, glm = make_pair(w)
    try:
        glm.partition(8, 0)
        glm.cocoa_round(0, 8.0)
        a0, v0, g0 = glm.get_alpha(), glm.get_v(), glm.duality_gap()
        glm.partition(3, 5)
        assert np.array_equal(a0, glm.get_alpha()) and np.array_equal(v0, glm.get_v())
        assert glm.duality_gap() == g0 and glm.info()["round"] == 1
    finally:
        glm.close()


def test_device_resident_inputs_and_plain_cuda_allocator_give_the_same_bits():
    w = datagen.make("hinge_csr", 200)
    res = []
    for kw in ({}, {"on_device": True}, {"torch_allocator": False}):
        glm = binding.from_workload(w, **kw)
        glm.partition(4, 0)
        for _ in range(3):
            glm.cocoa_round(0, 4.0)
        res.append((glm.get_alpha(), glm.get_v(), glm.duality_gap()["gap"]))
        glm.close()
    for r in res[1:]:
        assert np.array_equal(r[0], res[0][0]) and np.array_equal(r[1], res[0][1]) and r[2] == res[0][2]


# ------------------------------------------------------------------ partitions of unequal sizes
@pytest.mark.parametrize("sizes", [[1, 5000, 2499, 2500], [9000, 1000], [3, 3, 9990, 4]])
def test_unequal_partitions(sizes):
    # tasks that hold different numbers of samples: bit-exact partition map and visiting orders, alpha, v and the gap
    # within tolerance; a partition of one coordinate, and partitions whose last block of 32 steps is ragged
    w = datagen.make("hinge_csr", 100)
    w.phases = [Phase(0, len(sizes), 5, float(len(sizes)))]
    run_parity(w, rounds=4, sizes=sizes)


def test_unequal_partitions_dense_ridge_and_partial_H():
    run_parity(tiny_dense(500, 28, seed=2, loss="logistic", K=3), sizes=[100, 395, 5])
    w = datagen.make("ridge_csc", 100)
    K = 4
    n = w.n_coord
    w.phases = [Phase(0, K, 1, float(K))]
    run_parity(w, rounds=3, sizes=[n // 2, n // 4, n // 8, n - n // 2 - n // 4 - n // 8])
    # a step budget below the smallest partition (one look-ahead pass) and above it (several local epochs)
    run_parity(tiny_csr(100, 30, seed=5, K=4), H=10, sizes=[12, 40, 30, 18])
    run_parity(tiny_csr(100, 30, seed=5, K=4), H=30, sizes=[12, 40, 30, 18])


def test_step_budgets_per_partition(monkeypatch):
    # Sec. 3: every task gets the number of samples per iteration that suits its speed. Budgets that change from round
    # to round, ragged against the 32-step blocks, with partitions that sit a round out.
    sizes = [12, 40, 30, 18]
    table = [[12, 40, 30, 18], [5, 33, 0, 18], [0, 1, 30, 7], [0, 0, 0, 0], [12, 0, 0, 0]]
    w = tiny_csr(100, 30, seed=5, K=4)
    run_parity(w, rounds=5, sizes=sizes, steps=lambda r: table[r])
    w = datagen.make("hinge_csr", 100)
    K = w.phases[0].K
    n = w.n_coord
    base = np.diff(np.linspace(0, n, K + 1).astype(np.int64))
    budget = lambda r: [int(b) // (1 + (k + r) % 3) if (k + r) % 5 else 0 for k, b in enumerate(base)]
    run_parity(w, rounds=4, sizes=[int(b) for b in base], steps=budget)
    run_parity(tiny_dense(500, 28, seed=2, loss="logistic", K=3), sizes=[100, 395, 5], steps=lambda r: [100 - 33 * r, 64 + r, r])
    w = datagen.make("ridge_csc", 100)
    w.phases = [Phase(0, 4, 1, 4.0)]
    n = w.n_coord
    run_parity(w, rounds=3, steps=lambda r: [n // 4 - r, 31, 32 * r, n // 8])
    monkeypatch.setenv("CHICLE_FORCE_VARIANT", "blocked")
    run_parity(tiny_csr(100, 30, seed=5, K=4), rounds=5, sizes=sizes, steps=lambda r: table[r])


def test_step_budgets_equal_to_H_reproduce_the_round_and_bad_budgets_are_refused():
    w = tiny_csr(300, 40, seed=3, K=3)
    a, b = binding.from_workload(w), binding.from_workload(w)
    try:
        a.partition(3, 1)
        b.partition(3, 1)
        a.cocoa_round(37, 3.0)
        st = b.cocoa_round(0, 3.0, stats=True, steps=[37, 37, 37])
        assert st["steps"] == 111
        assert np.array_equal(a.get_alpha(), b.get_alpha()) and np.array_equal(a.get_v(), b.get_v())
        a.cocoa_round(0, 3.0)
        b.cocoa_round(0, 3.0, steps=[100, 100, 100])
        assert np.array_equal(a.get_alpha(), b.get_alpha()) and np.array_equal(a.get_v(), b.get_v())
        before = b.get_alpha().copy()
        for bad in ([101, 1, 1], [-1, 1, 1]):
            with pytest.raises(binding.ChicleError) as e:
                b.cocoa_round(0, 3.0, steps=bad)
            assert e.value.status == 1
        assert np.array_equal(before, b.get_alpha()) and b.info()["round"] == 2
    finally:
        a.close()
        b.close()


def test_partition_sizes_errors_and_equal_sizes():
    w = tiny_csr(60, 20, seed=1)
    glm = binding.from_workload(w)
    try:
        for bad in ([30, 31], [0, 60], [61, -1]):
            with pytest.raises(binding.ChicleError) as e:
                glm.partition(2, 0, bad)
            assert e.value.status == 1
        glm.partition(3, 7, [20, 20, 20])
        a = glm.get_partition().copy()
        glm.partition(3, 7)
        assert np.array_equal(a, glm.get_partition())
    finally:
        glm.close()


# ------------------------------------------------------------------ solver families
@pytest.mark.parametrize("variant", ["blocked"])
def test_older_solvers_still_match(variant, monkeypatch):
    # single-epoch rounds take the look-ahead solver by default; the blocked solver stays selectable
    monkeypatch.setenv("CHICLE_FORCE_VARIANT", variant)
    run_parity(datagen.make("hinge_csr", 100), rounds=4)
    run_parity(datagen.make("ridge_csc", 100), rounds=3)
    run_parity(tiny_dense(500, 28, seed=2, loss="logistic", K=4))


def test_lookahead_solver_is_the_default():
    for w, want in ((datagen.make("hinge_csr", 100), 4), (datagen.make("hinge_dense", 4), 5)):
        glm = binding.from_workload(w)
        try:
            glm.partition(w.phases[0].K, 0)
            assert glm.cocoa_round(0, float(w.phases[0].K), stats=True)["solver_variant"] == want
            assert glm.cocoa_round(5, float(w.phases[0].K), stats=True)["solver_variant"] == want
            n_k = w.n_coord // w.phases[0].K
            assert glm.cocoa_round(2 * n_k, float(w.phases[0].K), stats=True)["solver_variant"] == want  # once per local epoch
        finally:
            glm.close()


def test_lookahead_blocks_that_do_not_fit_are_walked_in_place():
    # rows longer than a staged row (128 entries), and blocks of long rows with hardly any id in common
    run_parity(tiny_csr(200, 3000, seed=9, K=2, density=0.03, long_row=500))
    rng = np.random.default_rng(4)
    n, d = 256, 40000
    indptr = np.arange(n + 1, dtype=np.int64) * 120
    idx = np.concatenate([np.sort(rng.choice(d, 120, replace=False)) for _ in range(n)]).astype(np.int32)
    vals = rng.standard_normal(n * 120).astype(np.float32) * 0.1
    y = np.where(rng.random(n) < 0.5, 1.0, -1.0).astype(np.float32)
    run_parity(Workload("wide_blocks", "hinge", "csr", n, d, vals, y, 1.0 / n, 3, [Phase(0, 2, 0, 2.0)], indptr, idx))


def test_gap_tile_that_does_not_fit_a_stage_is_read_in_place():
    # many short rows (so that the streamed gap kernel takes 128 coordinates per tile) and two neighbouring rows of
    # 3 000 entries each: their tile has more non-zeros than a stage of the ring holds; some empty rows as well
    rng = np.random.default_rng(21)
    n, d = 1500, 4000
    X = rng.standard_normal((n, d)).astype(np.float32) * 0.1
    X[rng.random((n, d)) > 0.005] = 0.0
    for r in (700, 701):
        X[r, :3000] = rng.standard_normal(3000).astype(np.float32) * 0.02 + 0.01
    X[10:14] = 0.0
    w = rng.standard_normal(d)
    y = np.where(X @ w >= 0, 1.0, -1.0).astype(np.float32)
    indptr = np.zeros(n + 1, np.int64)
    indptr[1:] = np.cumsum((X != 0).sum(1))
    wl = Workload("gap_overflow", "hinge", "csr", n, d, X[X != 0].astype(np.float32), y, 1.0 / n, 3, [Phase(0, 4, 0, 4.0)],
                  indptr, np.nonzero(X)[1].astype(np.int32))
    run_parity(wl)


@pytest.mark.parametrize("name,scale,slices", [("hinge_csr", 100, None), ("ridge_csc", 100, None), ("hinge_dense", 1, None),
                                               ("logistic_dense", 100, None), ("hinge_hashed", 1000, "3")])
def test_lookahead_runs_are_bit_reproducible(name, scale, slices, monkeypatch):
    # the skewed variant (part of the model in shared memory, split over a cluster), the flat one (every id goes through
    # reductions on the update rows in global memory), the dense one, and a round cut into slices
    if slices:
        monkeypatch.setenv("CHICLE_LA_SLICES", slices)
    w = datagen.make(name, scale)
    ph = w.phases[0]
    res = []
    for _ in range(2):
        glm = binding.from_workload(w)
        try:
            glm.partition(ph.K, ph.seed)
            for _ in range(3):
                glm.cocoa_round(0, ph.sigma_prime)
            res.append((glm.get_alpha().copy(), glm.get_v().copy(), glm.duality_gap()["gap"]))
        finally:
            glm.close()
    assert np.array_equal(res[0][0], res[1][0]) and np.array_equal(res[0][1], res[1][1]) and res[0][2] == res[1][2]


@pytest.mark.parametrize("depth,overlap,cluster", [("1", "0", "1"), ("1", "1", "2"), ("2", "0", "4"), ("2", "1", "8")])
def test_lookahead_depths_overlap_modes_and_cluster_sizes(depth, overlap, cluster, monkeypatch):
    # dot products one or two blocks ahead of the recurrence, prepare kernels beside the chain kernels or alternating
    # with them, 1 to 8 CTAs per partition: every combination walks the same order and must match the oracle
    monkeypatch.setenv("CHICLE_LA_DEPTH", depth)
    monkeypatch.setenv("CHICLE_LA_OVERLAP", overlap)
    monkeypatch.setenv("CHICLE_LA_CLUSTER", cluster)
    monkeypatch.setenv("CHICLE_LA_SLICES", "3")
    run_parity(datagen.make("hinge_csr", 100), rounds=3)
    run_parity(datagen.make("ridge_csc", 100), rounds=2)
    run_parity(tiny_dense(700, 28, seed=2, loss="logistic", K=3), rounds=3)
    run_parity(tiny_csr(200, 3000, seed=9, K=2, density=0.03, long_row=500), rounds=3)   # blocks walked in place


@pytest.mark.parametrize("cluster", ["1", "2"])
def test_ids_beyond_the_shared_memory_part_across_slices(cluster, monkeypatch):
    # 25 000 or 50 000 features against some 21 600 model entries per CTA in shared memory: the rest of the local model
    # lives in the partition's row of the update workspace, as the model itself between the launches of a round
    monkeypatch.setenv("CHICLE_LA_CLUSTER", cluster)
    monkeypatch.setenv("CHICLE_LA_SLICES", "3")
    run_parity(datagen.make("hinge_csr", 4 if cluster == "1" else 2), rounds=2)


def test_more_partitions_than_the_prepare_kernel_stages_block_bases_for():
    # up to 259 partitions the prepare kernel searches a shared-memory copy of the block bases; beyond, global memory
    run_parity(tiny_csr(3000, 60, seed=4, K=300, density=0.1), rounds=2)
    run_parity(tiny_csr(3000, 60, seed=4, K=259, density=0.1), rounds=2)


def test_warp_per_coordinate_gap_kernel_on_sparse_data(monkeypatch):
    # sparse data take the streamed gap kernel by default; the warp-per-coordinate kernel stays selectable
    monkeypatch.setenv("CHICLE_FORCE_VARIANT", "gapwarp")
    run_parity(datagen.make("hinge_csr", 100), rounds=2)
    run_parity(datagen.make("ridge_csc", 100), rounds=2)


def test_a_missing_record_ends_in_a_timeout_status_and_the_handle_stays_usable(monkeypatch):
    # Failure detection without a fault: one block's records are left unpublished (a host-side test aid), so the chain
    # kernel finds nothing to copy, sets the status word with no copy in flight, every wait in the cluster runs out
    # within its bound, all roles return, and the call reports the timeout. The handle then takes a new partition
    # and runs on.
    w = datagen.make("hinge_csr", 200)
    ph = w.phases[0]
    orc, glm = make_pair(w)
    try:
        glm.partition(ph.K, ph.seed)
        monkeypatch.setenv("CHICLE_TEST_DROP_RECORD", "3")
        with pytest.raises(binding.ChicleError) as e:
            glm.cocoa_round(0, ph.sigma_prime)
            glm.duality_gap()     # (the status word is read by the next synchronising call)
        assert e.value.status == binding.ERR_TIMEOUT
        monkeypatch.delenv("CHICLE_TEST_DROP_RECORD")
        # the state is whatever the aborted round left: start again from the oracle's
        glm.set_state(orc.state.astype(np.float32), orc.v.astype(np.float32), 0)
        orc.partition(ph.K, ph.seed)
        glm.partition(ph.K, ph.seed)
        orc.cocoa_round(0, ph.sigma_prime)
        glm.cocoa_round(0, ph.sigma_prime)
        assert rel_l2(glm.get_alpha(), orc.state) <= 1e-4 and rel_l2(glm.get_v(), orc.v) <= 1e-4
    finally:
        glm.close()


def test_allocator_that_returns_null_gives_oom(monkeypatch):
    # host-side fault injection: the allocator callback starts returning NULL
    w = tiny_csr(300, 40, seed=3, K=3)
    glm = binding.from_workload(w)
    try:
        glm.partition(3, 0)
        glm.cocoa_round(0, 3.0)
        glm.fail_allocations(True)
        with pytest.raises(binding.ChicleError) as e:
            glm.partition(5, 1)          # needs a new K x d update workspace
        assert e.value.status == binding.ERR_OOM
        glm.fail_allocations(False)
        with pytest.raises(binding.ChicleError) as e:
            glm.cocoa_round(0, 3.0)      # documented: the failed call released the old workspace, the handle has no partition
        assert e.value.status == binding.ERR_BAD_STATE
        glm.partition(5, 1)
        glm.cocoa_round(0, 5.0)
        assert glm.duality_gap()["gap"] >= 0
    finally:
        glm.close()


def test_round_stats():
    w = datagen.make("hinge_csr", 100)
    glm = binding.from_workload(w)
    try:
        glm.partition(16, 0)
        st = glm.cocoa_round(0, 16.0, stats=True)
        assert st["steps"] == w.n_rows and st["ms_total"] > 0 and st["ms_local"] > 0
        st = glm.cocoa_round(7, 16.0, stats=True)
        assert st["steps"] == 7 * 16
    finally:
        glm.close()


# ------------------------------------------------------------------ error behaviour
def test_errors():
    w = tiny_csr(50, 20, seed=1)
    glm = binding.from_workload(w)
    try:
        with pytest.raises(binding.ChicleError) as e:
            glm.cocoa_round(0, 1.0)
        assert e.value.status == 2                                   # BAD_STATE: no partition yet
        for K in (0, -1, 51):
            with pytest.raises(binding.ChicleError) as e:
                glm.partition(K, 0)
            assert e.value.status == 1
        glm.partition(2, 0)
        for H, sp in ((-1, 1.0), (0, 0.0), (0, -2.0), (0, float("nan"))):
            with pytest.raises(binding.ChicleError) as e:
                glm.cocoa_round(H, sp)
            assert e.value.status == 1
        with pytest.raises(binding.ChicleError):
            glm.get_permutation(0, 2, 25)
        with pytest.raises(binding.ChicleError):
            glm.get_permutation(0, 0, 24)
        out = np.empty(49, np.float32)
        with pytest.raises(binding.ChicleError):
            glm._get(glm._lib.chicle_get_alpha, 49, out)
        glm.cocoa_round(0, 2.0)                                      # the handle is still usable
        assert glm.info()["round"] == 1
    finally:
        glm.close()
    bad = tiny_csr(50, 20, seed=1)
    bad.values = bad.values.copy()
    bad.values[3] = np.nan
    with pytest.raises(binding.ChicleError) as e:
        binding.from_workload(bad)
    assert e.value.status == 6
    bad = tiny_csr(50, 20, seed=1)
    bad.labels = bad.labels.copy()
    bad.labels[4] = 0.5
    with pytest.raises(binding.ChicleError) as e:
        binding.from_workload(bad)
    assert e.value.status == 1
    bad = tiny_csr(50, 20, seed=1)
    bad.indices = bad.indices.copy()
    bad.indices[2] = 20
    with pytest.raises(binding.ChicleError) as e:
        binding.from_workload(bad)
    assert e.value.status == 1
    bad = tiny_csr(50, 20, seed=1)
    bad.loss = "ridge"
    with pytest.raises(binding.ChicleError) as e:
        binding.from_workload(bad)
    assert e.value.status == 5
