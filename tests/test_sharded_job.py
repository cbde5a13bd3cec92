"""The job spread over ranks (partitions k mod G on rank g, one exchange of summed updates per round; Sec. 4.2 and
the Appendix's example application), host side: who owns what, what is exchanged, in which order. Run as gloo ranks on
CPU with the oracle doing the arithmetic of each rank; the result must be the single-rank oracle's."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1909_04885_b200 import sharded  # noqa: E402


class OracleBackend:
    """One rank's arithmetic done by the CPU oracle (fp64): the methods `sharded.ShardedGlm` asks of a backend."""

    def __init__(self, orc):
        self.orc = orc

    def partition(self, K, seed):
        self.orc.partition(K, seed)

    def partition_sizes(self):
        return np.diff(self.orc.part_off).astype(np.int64)

    def round_delta(self, budgets, sigma_prime):
        before = self.orc.v.copy()
        self.orc.cocoa_round(0, sigma_prime, steps=budgets)
        delta = self.orc.v - before
        self.orc.v[:] = before
        return torch.from_numpy(delta)

    def apply_deltas(self, stacked):
        for g in range(stacked.shape[0]):      # rank order
            self.orc.v += stacked[g].numpy()

    def export_state_of(self, keep):
        keep = np.asarray(keep, bool)
        return torch.from_numpy(np.where(keep[self.orc.owner], self.orc.state, 0.0))

    def import_state(self, state):
        self.orc.state[:] = state.numpy()

    def duality_gap(self):
        return self.orc.duality_gap()

    def sync(self):
        pass


def _tiny(loss):
    rng = np.random.default_rng(5)
    n, d = 240, 30
    X = rng.standard_normal((n, d)).astype(np.float32)
    X[rng.random((n, d)) > 0.3] = 0.0
    X[:, 0] = 1.0
    indptr = np.zeros(n + 1, np.int64)
    if loss == "ridge":
        Xc = X.T.copy()                            # coordinates are the columns
        indptr = np.zeros(d + 1, np.int64)
        indptr[1:] = np.cumsum((Xc != 0).sum(1))
        y = (X @ rng.standard_normal(d)).astype(np.float32)
        return dict(loss="ridge", fmt="csc", n_rows=n, n_cols=d, values=Xc[Xc != 0], labels=y, lam=1e-2, indptr=indptr,
                    indices=np.nonzero(Xc)[1].astype(np.int32))
    indptr[1:] = np.cumsum((X != 0).sum(1))
    y = np.where(X @ rng.standard_normal(d) >= 0, 1.0, -1.0).astype(np.float32)
    return dict(loss=loss, fmt="csr", n_rows=n, n_cols=d, values=X[X != 0], labels=y, lam=1.0 / n, indptr=indptr,
                indices=np.nonzero(X)[1].astype(np.int32))


SCHEDULE = [(6, 11), (6, 11), (6, 11), (4, 12), (4, 12)]   # (K, seed) per round: a repartition before round 3


def _run(job, budgets_of=None):
    gaps, K_now = [], None
    for r, (K, seed) in enumerate(SCHEDULE):
        if (K, seed) != K_now:
            job.partition(K, seed)
            K_now = (K, seed)
        job.cocoa_round(0, float(K), steps=None if budgets_of is None else budgets_of(r, job.sizes))
        gaps.append(job.duality_gap()["gap"])
    return gaps


def _budgets(r, sizes):
    return [0 if (k + r) % 5 == 0 else int(s) - (k % 3) for k, s in enumerate(sizes)]


def _worker(rank, world, port, loss, out):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        orc = oracle.CocoaOracle(**_tiny(loss))
        job = sharded.ShardedGlm(OracleBackend(orc), sharded.Comm(dist))
        gaps = _run(job, _budgets if loss == "hinge" else None)
        job.sync_state()
        out[rank] = (orc.state.copy(), orc.v.copy(), gaps)
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("loss", ["hinge", "logistic", "ridge"])
def test_two_ranks_equal_the_single_rank_oracle(loss):
    import oracle
    oracle.build()
    world = 2
    port = 23000 + (os.getpid() * 7 + len(loss)) % 4000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, loss, out), nprocs=world, join=True)
        res = dict(out)
    # the single-rank reference: the plain oracle, no sharding code involved
    ref = oracle.CocoaOracle(**_tiny(loss))
    gaps, K_now = [], None
    for r, (K, seed) in enumerate(SCHEDULE):
        if (K, seed) != K_now:
            ref.partition(K, seed)
            K_now = (K, seed)
        sizes = np.diff(ref.part_off)
        ref.cocoa_round(0, float(K), steps=_budgets(r, sizes) if loss == "hinge" else None)
        gaps.append(ref.duality_gap()["gap"])
    for rank in range(world):
        state, v, g = res[rank]
        # a coordinate is stepped by exactly one rank with the single-rank arithmetic; only the order in which the
        # partitions' updates are added to v differs (per rank first, then over ranks): rounding-level differences in
        # fp64, which the later rounds' steps inherit
        assert np.allclose(state, ref.state, rtol=0, atol=1e-12)
        assert np.allclose(v, ref.v, rtol=0, atol=1e-12 * max(1.0, np.abs(ref.v).max()))
        assert np.allclose(g, gaps, rtol=1e-9, atol=1e-13)
    assert np.array_equal(res[0][1], res[1][1])     # the replicas of v: the same bits on both ranks


def test_ownership_and_budgets():
    assert sharded.owned_partitions(5, 1, 2).tolist() == [0, 1, 0, 1, 0]
    assert sum(sharded.owned_partitions(7, g, 3) for g in range(3)).tolist() == [1] * 7   # every partition has one owner
    sizes = [10, 11, 12, 13]
    assert sharded.shard_budgets(sizes, 0, 2).tolist() == [10, 0, 12, 0]
    assert sharded.shard_budgets(sizes, 1, 2, H=7).tolist() == [0, 7, 0, 7]
    assert sharded.shard_budgets(sizes, 1, 4, steps=[1, 2, 3, 4]).tolist() == [0, 2, 0, 0]
    assert sharded.shard_budgets(sizes, 0, 8).tolist() == [10, 0, 0, 0]                    # more ranks than partitions
    with pytest.raises(ValueError):
        sharded.shard_budgets(sizes, 0, 2, H=11)
    with pytest.raises(ValueError):
        sharded.owned_partitions(4, 2, 2)


def test_one_rank_without_a_process_group_is_the_plain_job():
    import oracle
    oracle.build()
    orc = oracle.CocoaOracle(**_tiny("hinge"))
    gaps = _run(sharded.ShardedGlm(OracleBackend(orc)))
    ref = oracle.CocoaOracle(**_tiny("hinge"))
    want, K_now = [], None
    for K, seed in SCHEDULE:
        if (K, seed) != K_now:
            ref.partition(K, seed)
            K_now = (K, seed)
        ref.cocoa_round(0, float(K))
        want.append(ref.duality_gap()["gap"])
    assert np.allclose(orc.state, ref.state, rtol=0, atol=1e-12)
    assert np.allclose(gaps, want, rtol=1e-9, atol=1e-13)
