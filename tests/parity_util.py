"""Round-by-round comparison of the GPU library with the CPU oracle on one workload."""
import os

import numpy as np

import oracle
from paper_1909_04885_b200 import binding

REL_TOL = 1e-4          # relative L2 tolerance on alpha and v per round (fp32 library vs fp64 oracle)
MAX_TOL = 1e-5          # largest error of a single entry of alpha or v, relative to max(1, largest entry): an L2 norm
                        # alone would let a handful of wrong coordinates through (measured: below 1e-6)


def max_err(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return np.abs(a - b).max() / max(1.0, np.abs(b).max())


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    den = np.linalg.norm(b)
    return np.linalg.norm(a - b) / den if den > 0 else np.linalg.norm(a - b)


def gap_close(g_gpu, g_or):
    tol = REL_TOL * max(g_or["gap"], 1e-3 * abs(g_or["primal"]))
    return abs(g_gpu["gap"] - g_or["gap"]) <= tol, tol


def make_pair(w, threads=None, **kw):
    threads = threads or min(os.cpu_count() or 1, 16)
    orc = oracle.CocoaOracle(w.loss, w.fmt, w.n_rows, w.n_cols, w.values, w.labels, w.lam, w.indptr, w.indices,
                             threads=threads)
    glm = binding.from_workload(w, **kw)
    return orc, glm


def check_partition(orc, glm, perm_rounds=(0,)):
    owner = glm.get_partition()
    assert np.array_equal(owner, orc.owner), "partition map differs"
    for r in perm_rounds:
        for k in sorted({0, orc.K // 2, orc.K - 1}):
            n_k = int(orc.part_off[k + 1] - orc.part_off[k])
            got = glm.get_permutation(r, k, n_k)
            assert np.array_equal(got, orc.permutation(r, k)), "visiting order differs (round %d, k %d)" % (r, k)


def run_parity(w, rounds=None, H=None, check_perm=True, resync=False, sizes=None, steps=None, **kw):
    """``steps``: a function of the round that returns the K step budgets of that round (instead of H).
    Free-running comparison (both sides evolve on their own) unless ``resync``: then the library's state is
    reset to the oracle's before every round, which isolates one round's error."""
    orc, glm = make_pair(w, **kw)
    rounds = w.rounds if rounds is None else rounds
    H = w.H if H is None else H
    worst = {"alpha": 0.0, "v": 0.0}
    try:
        g0, o0 = glm.duality_gap(), orc.duality_gap()
        ok, tol = gap_close(g0, o0)
        assert ok, "initial gap %r vs %r" % (g0, o0)
        for r in range(rounds):
            ph = w.phase_at(r)
            if r == 0 or r == ph.start:
                orc.partition(ph.K, ph.seed, sizes)
                glm.partition(ph.K, ph.seed, sizes)
                if check_perm:
                    check_partition(orc, glm, perm_rounds=(r,))
            if resync and r > 0:
                glm.set_state(orc.state.astype(np.float32), orc.v.astype(np.float32), orc.round)
            if steps is not None:
                orc.cocoa_round(0, ph.sigma_prime, steps=steps(r))
                glm.cocoa_round(0, ph.sigma_prime, steps=steps(r))
            else:
                orc.cocoa_round(H, ph.sigma_prime)
                glm.cocoa_round(H, ph.sigma_prime)
            a_gpu, v_gpu = glm.get_alpha(), glm.get_v()
            ea, ev = rel_l2(a_gpu, orc.state), rel_l2(v_gpu, orc.v)
            worst["alpha"], worst["v"] = max(worst["alpha"], ea), max(worst["v"], ev)
            assert ea <= REL_TOL, "round %d: alpha rel err %.3e" % (r, ea)
            assert ev <= REL_TOL, "round %d: v rel err %.3e" % (r, ev)
            ma, mv = max_err(a_gpu, orc.state), max_err(v_gpu, orc.v)
            worst["alpha_max"], worst["v_max"] = max(worst.get("alpha_max", 0.0), ma), max(worst.get("v_max", 0.0), mv)
            assert ma <= MAX_TOL, "round %d: largest alpha error %.3e" % (r, ma)
            assert mv <= MAX_TOL, "round %d: largest v error %.3e" % (r, mv)
            gg, go = glm.duality_gap(), orc.duality_gap()
            ok, tol = gap_close(gg, go)
            assert ok, "round %d: gap %.9e vs %.9e (tol %.2e)" % (r, gg["gap"], go["gap"], tol)
            assert abs(gg["primal"] - go["primal"]) <= REL_TOL * abs(go["primal"]) + 1e-12
        assert glm.info()["round"] == orc.round
    finally:
        glm.close()
    return worst
