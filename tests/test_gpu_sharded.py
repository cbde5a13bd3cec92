"""The calls behind a job spread over several GPUs, on one GPU: two handles over the same data stand for two ranks and
are driven one after the other (no kernel waits for another rank); the exchange that a collective would do is done by
hand. Against the single-rank CPU oracle."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from paper_1909_04885_b200 import binding, datagen, sharded  # noqa: E402

import oracle  # noqa: E402
from parity_util import MAX_TOL, REL_TOL, gap_close, make_pair, max_err, rel_l2  # noqa: E402


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_1909_04885_b200 import build
    build.build()
    oracle.build()


def _close(glm, orc, what):
    a, v = glm.get_alpha(), glm.get_v()
    assert rel_l2(a, orc.state) <= REL_TOL and max_err(a, orc.state) <= MAX_TOL, what + ": alpha"
    assert rel_l2(v, orc.v) <= REL_TOL and max_err(v, orc.v) <= MAX_TOL, what + ": v"
    ok, tol = gap_close(glm.duality_gap(), orc.duality_gap())
    assert ok, what + ": gap"


@pytest.mark.parametrize("name,scale", [("hinge_csr", 100), ("logistic_dense", 1000), ("ridge_csc", 100)])
def test_two_ranks_on_one_gpu_match_the_single_rank_oracle(name, scale):
    import torch
    w = datagen.make(name, scale)
    world = 2
    orc, g0 = make_pair(w)
    ranks = [g0, binding.from_workload(w)]
    dev = torch.device("cuda", 0)
    try:
        schedule = [(w.phases[0].K, 3), (w.phases[0].K, 3), (max(2, w.phases[0].K // 2), 4), (max(2, w.phases[0].K // 2), 4)]
        now = None
        for r, (K, seed) in enumerate(schedule):
            if (K, seed) != now:
                if now is not None:
                    # ownership is about to change: every rank needs the whole per-coordinate state first
                    parts = []
                    for g, glm in enumerate(ranks):
                        out = torch.empty(glm.n_coord, dtype=torch.float32, device=dev)
                        glm.export_state_of(sharded.owned_partitions(now[0], g, world), out)
                        parts.append(out)
                    torch.cuda.synchronize()
                    whole = parts[0] + parts[1]
                    for glm in ranks:
                        glm.import_state(whole)
                    torch.cuda.synchronize()
                orc.partition(K, seed)
                for glm in ranks:
                    glm.partition(K, seed)
                sizes = np.bincount(ranks[0].get_partition(), minlength=K)
                assert np.array_equal(sizes, np.diff(orc.part_off))
                now = (K, seed)
            orc.cocoa_round(0, float(K))
            deltas = torch.empty((world, ranks[0].dim), dtype=torch.float32, device=dev)
            for g, glm in enumerate(ranks):
                glm.cocoa_round_delta(sharded.shard_budgets(sizes, g, world), float(K), deltas[g])
            torch.cuda.synchronize()
            for glm in ranks:
                glm.apply_deltas(deltas)
            torch.cuda.synchronize()
            v0, v1 = ranks[0].get_v(), ranks[1].get_v()
            assert np.array_equal(v0, v1), "the replicas of v must hold the same bits"
            assert rel_l2(v0, orc.v) <= REL_TOL and max_err(v0, orc.v) <= MAX_TOL, "round %d: v" % r
            # a rank's alpha is current for the coordinates it owns
            for g, glm in enumerate(ranks):
                mine = sharded.owned_partitions(K, g, world)[orc.owner] != 0
                a = glm.get_alpha()
                assert max_err(a[mine], orc.state[mine]) <= MAX_TOL, "round %d: alpha of rank %d" % (r, g)
        # the whole state on both ranks, then the gap from either replica
        parts = []
        for g, glm in enumerate(ranks):
            out = torch.empty(glm.n_coord, dtype=torch.float32, device=dev)
            glm.export_state_of(sharded.owned_partitions(now[0], g, world), out)
            parts.append(out)
        torch.cuda.synchronize()
        whole = parts[0] + parts[1]
        for glm in ranks:
            glm.import_state(whole)
        torch.cuda.synchronize()
        for g, glm in enumerate(ranks):
            _close(glm, orc, "rank %d at the end" % g)
    finally:
        for glm in ranks:
            glm.close()


def test_the_sharded_job_on_one_rank_and_bad_arguments():
    import torch
    w = datagen.make("hinge_csr", 100)
    orc, glm = make_pair(w)
    try:
        job = sharded.ShardedGlm(sharded.GlmBackend(glm))
        K = w.phases[0].K
        for r in range(3):
            if r == 0:
                orc.partition(K, 9)
                job.partition(K, 9)
            orc.cocoa_round(0, float(K))
            job.cocoa_round(0, float(K))
            ok, tol = gap_close(job.duality_gap(), orc.duality_gap())
            assert ok
        _close(glm, orc, "one rank")
        short = torch.empty(glm.dim - 1, dtype=torch.float32, device="cuda")
        for call in (lambda: glm.cocoa_round_delta(job.sizes, float(K), short), lambda: glm.apply_deltas(short),
                     lambda: glm.import_state(short)):
            with pytest.raises(binding.ChicleError) as e:
                call()
            assert e.value.status == binding.ERR_INVALID_ARG
        before = glm.get_v().copy()
        assert np.array_equal(before, glm.get_v())     # nothing was enqueued by the refused calls
    finally:
        glm.close()
