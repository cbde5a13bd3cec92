"""The paper's qualitative claims about data parallelism, checked on the synthetic stand-in for its large sparse
workload (Sec. 1, Fig. 1b: more tasks need more epochs to converge; Sec. 2.2 and Sec. 5.3: starting with many
tasks and scaling in speeds convergence up relative to staying wide). No dataset of the paper is used: the inputs are
the seeded `hinge_hashed` workload at reduced size. The CPU test runs the oracle, the GPU test the library."""
import numpy as np
import pytest

from paper_1909_04885_b200 import datagen

import oracle

THRESHOLD = 1e-2


def rounds_to(gaps, threshold=THRESHOLD):
    return next((i + 1 for i, g in enumerate(gaps) if g < threshold), None)


def run(solver_factory, w, schedule, rounds):
    """schedule: list of (first_round, K, seed); sigma' = K. Returns the gap after every round."""
    s = solver_factory(w)
    gaps = []
    try:
        for r in range(rounds):
            for start, K, seed in schedule:
                if r == start:
                    s.partition(K, seed)
                    sigma = float(K)
            s.cocoa_round(0, sigma)
            gaps.append(s.duality_gap()["gap"])
    finally:
        if hasattr(s, "close"):
            s.close()
    return gaps


def check_claims(factory, w, wide, narrow, rounds):
    mid = int(round((narrow * wide) ** 0.5))
    static = {K: run(factory, w, [(0, K, 0)], rounds) for K in (narrow, mid, wide)}
    ks = sorted(static)
    need = [rounds_to(static[K]) for K in ks]
    # more tasks, more epochs (an epoch is a round here: H = one local epoch)
    assert all(n is not None for n in need[:-1]), need
    for a, b in zip(need, need[1:]):
        assert b is None or a < b, (ks, need)
    final = [static[K][-1] for K in ks]
    assert final == sorted(final), (ks, final)
    # wide for the first rounds, then scaled in: ends below the run that stayed wide, above the one that was narrow
    elastic = run(factory, w, [(0, wide, 0), (rounds // 3, narrow, 1)], rounds)
    assert static[narrow][-1] < elastic[-1] < static[wide][-1], (static[narrow][-1], elastic[-1], static[wide][-1])
    # the gap never goes negative and the rounds right after the scale-in gain more than the wide run's did
    assert min(min(g) for g in static.values()) >= 0.0 and min(elastic) >= 0.0
    cut = rounds // 3
    assert elastic[cut + 2] < static[wide][cut + 2]
    return ks, need, final, elastic[-1]


def test_more_tasks_need_more_epochs_oracle():
    oracle.build()
    w = datagen.make("hinge_hashed", 1000)

    def factory(w):
        return oracle.CocoaOracle(w.loss, w.fmt, w.n_rows, w.n_cols, w.values, w.labels, w.lam, w.indptr, w.indices, threads=4)

    ks, need, final, el = check_claims(factory, w, wide=64, narrow=4, rounds=30)
    print("oracle: K", ks, "rounds to gap %g" % THRESHOLD, need, "final gaps", final, "elastic", el)


@pytest.mark.gpu
def test_more_tasks_need_more_epochs_library():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_1909_04885_b200 import binding, build
    build.build()
    w = datagen.make("hinge_hashed", 100)

    def factory(w):
        return binding.from_workload(w, on_device=True)

    ks, need, final, el = check_claims(factory, w, wide=64, narrow=16, rounds=30)
    print("library: K", ks, "rounds to gap %g" % THRESHOLD, need, "final gaps", final, "elastic", el)
