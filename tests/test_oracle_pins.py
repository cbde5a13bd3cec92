"""Pins for the CPU oracle: each test ties a part of it to a fact that does not come from the oracle
itself (published constants, closed forms, brute force, textbook special cases, invariants)."""
import itertools
import math

import numpy as np
import pytest

import oracle
from oracle import CocoaOracle

M64 = (1 << 64) - 1
GAMMA = 0x9E3779B97F4A7C15
PERM_STREAM = 0xD1B54A32D192ED03


def py_mix64(x):
    z = (x + GAMMA) & M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


# ---------------------------------------------------------------- integers (a1, a2)

def test_mix64_matches_published_splitmix64_stream():
    # First outputs of SplitMix64 seeded with 0 (Steele/Lea/Flood; the values quoted with the public-domain
    # reference generator): output j is the mixer applied to state j*GAMMA.
    published = [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F, 0xF88BB8A8724C81EC]
    for j, want in enumerate(published):
        assert oracle.mix64((j * GAMMA) & M64) == want
        assert py_mix64((j * GAMMA) & M64) == want


def test_mix64_is_injective_on_a_sample():
    xs = list(range(5000)) + [M64 - i for i in range(5000)]
    assert len({oracle.mix64(x) for x in xs}) == len(xs)


@pytest.mark.parametrize("n,K,seed", [(10, 3, 0), (1000, 7, 1), (4096, 16, 12345), (17, 17, 5), (33, 1, 9)])
def test_partition_defining_properties(n, K, seed):
    owner, off, members = oracle.partition(n, K, seed)
    sizes = np.diff(off)
    assert off[0] == 0 and off[-1] == n
    assert sizes.max() - sizes.min() <= 1
    assert (sizes[: n % K] == n // K + 1).all() and (sizes[n % K:] == n // K).all()
    assert sorted(members.tolist()) == list(range(n))                      # disjoint and covering
    s = py_mix64(seed)
    keys = [py_mix64(s ^ i) for i in range(n)]
    for k in range(K):
        mk = members[off[k]:off[k + 1]]
        assert (np.diff(mk) > 0).all()                                      # ascending ids inside a partition
        assert (owner[mk] == k).all()
    # blocks of the key order: every key of partition k is below every key of partition k+1
    for k in range(K - 1):
        hi = max(keys[i] for i in members[off[k]:off[k + 1]])
        lo = min(keys[i] for i in members[off[k + 1]:off[k + 2]])
        assert hi < lo


@pytest.mark.parametrize("n,sizes,seed", [(10, [1, 6, 3], 0), (1000, [400, 1, 99, 500], 3), (64, [64], 5), (7, [1] * 7, 2)])
def test_partition_with_given_sizes(n, sizes, seed):
    K = len(sizes)
    owner, off, members = oracle.partition(n, K, seed, sizes)
    assert off.tolist() == [0] + np.cumsum(sizes).tolist()                  # the sizes asked for, in order
    assert sorted(members.tolist()) == list(range(n))                      # disjoint and covering
    s = py_mix64(seed)
    keys = [py_mix64(s ^ i) for i in range(n)]
    order = sorted(range(n), key=lambda i: keys[i])                        # the same random order as the equal split
    for k in range(K):
        mk = members[off[k]:off[k + 1]]
        assert (np.diff(mk) > 0).all() and (owner[mk] == k).all()
        assert sorted(order[off[k]:off[k + 1]]) == mk.tolist()              # consecutive blocks of that order
    # equal sizes give the equal split
    if n % K == 0:
        o2, off2, m2 = oracle.partition(n, K, seed, [n // K] * K)
        o1, off1, m1 = oracle.partition(n, K, seed)
        assert np.array_equal(o1, o2) and np.array_equal(off1, off2) and np.array_equal(m1, m2)


def test_partition_rejects_bad_sizes():
    for sizes in ([5, 6], [0, 10], [11, -1], [3, 3, 3]):
        with pytest.raises(ValueError):
            oracle.partition(10, len(sizes), 0, sizes)
    with pytest.raises(ValueError):
        oracle.partition(10, 3, 0, [5, 5])


def test_partition_rejects_bad_K():
    with pytest.raises(ValueError):
        oracle.partition(5, 6, 0)
    with pytest.raises(ValueError):
        oracle.partition(5, 0, 0)


@pytest.mark.parametrize("n,K,seed", [(10, 3, 0), (500, 4, 77)])
def test_permutation_defining_properties(n, K, seed):
    owner, off, members = oracle.partition(n, K, seed)
    seen = set()
    for rnd, epoch in [(0, 0), (1, 0), (0, 1), (7, 3)]:
        a = py_mix64(seed ^ PERM_STREAM)
        b = py_mix64(((rnd << 32) + epoch) & M64)
        for k in range(K):
            mk = members[off[k]:off[k + 1]]
            perm = oracle.permutation(mk, seed, rnd, epoch)
            assert sorted(perm.tolist()) == mk.tolist()                     # bijection on the members
            keys = [py_mix64(a ^ b ^ int(i)) for i in perm]
            assert all(x < y for x, y in zip(keys, keys[1:]))               # visiting order = ascending key
            seen.add((k, tuple(perm.tolist())))
    if n >= 100:
        assert len(seen) == 4 * K                                           # every (round, epoch) reshuffles


def test_partition_and_permutation_known_answers():
    # tests/golden/partition_n10_K3_seed0.txt is written by tests/golden/make_golden.py from the oracle;
    # here it is re-derived with Python integers from the published mixer.
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "partition_n10_K3_seed0.txt")
    rows = {}
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        name, vals = line.split(":")
        rows[name.strip()] = [int(t) for t in vals.split()]
    n, K, seed = 10, 3, 0
    s = py_mix64(seed)
    order = sorted(range(n), key=lambda i: (py_mix64(s ^ i), i))
    cuts = [0, 4, 7, 10]
    owner = [0] * n
    for k in range(K):
        for i in order[cuts[k]:cuts[k + 1]]:
            owner[i] = k
    assert rows["owner"] == owner
    o, off, members = oracle.partition(n, K, seed)
    assert o.tolist() == owner and off.tolist() == cuts
    a, b = py_mix64(seed ^ PERM_STREAM), py_mix64((2 << 32) + 1)
    for k in range(K):
        mk = sorted(order[cuts[k]:cuts[k + 1]])
        want = sorted(mk, key=lambda i: (py_mix64(a ^ b ^ i), i))
        assert rows["perm_r2_e1_k%d" % k] == want
        assert oracle.permutation(np.array(mk, np.int32), seed, 2, 1).tolist() == want


# ---------------------------------------------------------------- helpers

def dense_problem(n, d, seed, loss="hinge"):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n, d)).astype(np.float32)
    w = rng.standard_normal(d)
    if loss == "ridge":
        y = (X @ w + 0.1 * rng.standard_normal(n)).astype(np.float32)
    else:
        y = np.where(X @ w + 0.3 * rng.standard_normal(n) >= 0, 1.0, -1.0).astype(np.float32)
    return X, y


def to_csr(X):
    n, d = X.shape
    indptr = [0]
    idx, val = [], []
    for i in range(n):
        nz = np.nonzero(X[i])[0]
        idx += nz.tolist()
        val += X[i, nz].tolist()
        indptr.append(len(idx))
    return np.array(indptr, np.int64), np.array(idx, np.int32), np.array(val, np.float32)


def hinge_dual_value(X, y, lam, a):
    n = X.shape[0]
    w = (X.astype(np.float64) * (a * y)[:, None]).sum(0) / (lam * n)
    return a.sum() / n - 0.5 * lam * w @ w, w


# ---------------------------------------------------------------- P11: a case small enough to audit by hand

def test_hand_worked_d1_n3():
    # d = 1, x = (1, 2, -1), y = (+1, -1, +1), lambda = 0.5, n = 3 -> lambda n = 1.5; K = 1, sigma' = 1.
    # Start alpha = 0, v = 0.  The visiting order comes from the oracle; the arithmetic below is by hand.
    X = np.array([[1.0], [2.0], [-1.0]], np.float32)
    y = np.array([1.0, -1.0, 1.0], np.float32)
    lam, n = 0.5, 3
    o = CocoaOracle("hinge", "dense", 3, 1, X, y, lam)
    o.partition(1, 3)
    order = o.permutation(0, 0)
    v, a = 0.0, np.zeros(3)
    for i in order:
        x, s = float(X[i, 0]), float(X[i, 0]) ** 2
        m = y[i] * x * v / 1.5
        q = s / 1.5
        new = min(1.0, max(0.0, a[i] + (1.0 - m) / q))
        v += y[i] * (new - a[i]) * x
        a[i] = new
    o.cocoa_round(0, 1.0)
    assert np.allclose(o.state, a * y, atol=1e-15)
    assert abs(o.v[0] - v) < 1e-15
    # gap by hand: w = v / 1.5
    w = v / 1.5
    mu = y * X[:, 0] * w
    terms = np.maximum(0, 1 - mu) - a + a * mu
    P = np.maximum(0, 1 - mu).mean() + 0.25 * w * w
    g = o.duality_gap()
    assert abs(g["gap"] - terms.mean()) < 1e-15 and abs(g["primal"] - P) < 1e-15
    # one concrete number that no code above produces: first visited coordinate from alpha = 0 has m = 0,
    # so its new a is clip(1.5 / x^2) -> 1 for |x| = 1 and 0.375 for x = 2.
    first = order[0]
    a0 = 1.0 if abs(X[first, 0]) == 1 else 0.375
    o2 = CocoaOracle("hinge", "dense", 3, 1, X, y, lam)
    o2.partition(1, 3)
    o2.cocoa_round(1, 1.0)                      # a single coordinate step
    assert abs(abs(o2.state[first]) - a0) < 1e-15
    assert np.count_nonzero(o2.state) == 1


# ---------------------------------------------------------------- sigma' in the local model: K = 2, sigma' = 2 by hand

def test_hand_worked_K2_sigma2_n4():
    # n = 4, d = 2, lambda = 0.25 -> lambda n = 1; K = 2, sigma' = 2; rows are not orthogonal.
    #   x0 = (0.5, 1) y0 = +1 | x1 = (1, 1) y1 = +1 | x2 = (1, 0) y2 = +1 | x3 = (0, 2) y3 = -1
    # Partition and visiting orders re-derived here from the published mixer with Python integers.
    seed, n, K = 2, 4, 2
    s = py_mix64(seed)
    order = sorted(range(n), key=lambda i: py_mix64(s ^ i))
    parts = [sorted(order[:2]), sorted(order[2:])]
    a_, b_ = py_mix64(seed ^ PERM_STREAM), py_mix64(0)
    visits = [sorted(p, key=lambda i: py_mix64(a_ ^ b_ ^ i)) for p in parts]
    assert visits == [[2, 0], [3, 1]]                       # the numbers below are worked for these orders
    X = np.array([[0.5, 1.0], [1.0, 1.0], [1.0, 0.0], [0.0, 2.0]], np.float32)
    y = np.array([1.0, 1.0, 1.0, -1.0], np.float32)
    o = CocoaOracle("hinge", "dense", 4, 2, X, y, 0.25)
    o.partition(K, seed)
    o.cocoa_round(0, 2.0)
    # Task 0, from the round's v = 0. Coordinate 2: q = 2*1/1 = 2, m = 0, a = clip(1/2) = 0.5; the local model
    #   becomes sigma' * 0.5 * (1, 0) = (1, 0). Coordinate 0: |x|^2 = 1.25, q = 2.5, m = x0 . (1, 0) = 0.5,
    #   a = (1 - 0.5)/2.5 = 0.2.           (sigma' left out of the local model: m = 0.25, a = 0.3; doubled: m = 1, a = 0)
    # Task 1. Coordinate 3: |x|^2 = 4, q = 8, a = 1/8, alpha = -0.125; local model 2 * (-0.125) * (0, 2) = (0, -0.5).
    #   Coordinate 1: |x|^2 = 2, q = 4, m = (1, 1) . (0, -0.5) = -0.5, a = 1.5/4 = 0.375.
    # v = 0.5 (1, 0) + 0.2 (0.5, 1) - 0.125 (0, 2) + 0.375 (1, 1) = (0.975, 0.325): the updates are added, without sigma'.
    assert np.allclose(o.state, [0.2, 0.375, 0.5, -0.125], atol=1e-15)
    assert np.allclose(o.v, [0.975, 0.325], atol=1e-15)
    # gap by hand, w = v: margins y x.w = 0.8125, 1.3, 0.975, -0.65; hinge losses 0.1875, 0, 0.025, 1.65;
    # terms loss - a + a*margin = 0.15, 0.1125, 0.0125, 1.44375 -> gap 1.71875/4; P = 1.8625/4 + 0.125 * 1.05625
    g = o.duality_gap()
    assert abs(g["gap"] - 0.4296875) < 1e-15 and abs(g["primal"] - 0.59765625) < 1e-15


# ---------------------------------------------------------------- sigma' in the local model: every step maximises the
#                                                                  sigma'-subproblem of its task along its coordinate

def _subproblem_value(loss, X, y, lam, K, sigma_p, w, members, alpha0, dalpha):
    """The local objective of the CoCoA formulation with the updates added (the framework Sec. 2.2 "CoCoA" cites,
    sigma as in Sec. 5.1), written out from the accumulated change dalpha of one task's dual variables:
        -(1/n) sum_{i in task} conj_i(-(alpha_i + dalpha_i)) - (lambda/2K)|w|^2 - (1/n) w . A dalpha
        - (lambda sigma'/2) |A dalpha / (lambda n)|^2 ,        A dalpha = sum_i dalpha_i x_i.
    -inf outside the dual variables' domain."""
    n = X.shape[0]
    Ad = np.zeros(X.shape[1])
    conj = 0.0
    for i in members:
        a = y[i] * (alpha0[i] + dalpha[i])
        if a < 0.0 or a > 1.0:
            return -math.inf
        if loss == "hinge":
            conj += -a
        else:
            conj += (a * math.log(a) if a > 0 else 0.0) + ((1 - a) * math.log(1 - a) if a < 1 else 0.0)
        Ad += dalpha[i] * X[i].astype(np.float64)
    return -conj / n - lam / (2 * K) * (w @ w) - (w @ Ad) / n - 0.5 * lam * sigma_p * (Ad @ Ad) / (lam * n) ** 2


@pytest.mark.parametrize("loss", ["hinge", "logistic"])
@pytest.mark.parametrize("sigma_p", [2.0, 3.5])
def test_every_step_maximises_the_sigma_subproblem(loss, sigma_p):
    n, d, lam, K = 8, 3, 0.07, 2
    X, y = dense_problem(n, d, 41)                          # generic rows: no two are orthogonal
    assert np.abs(X.astype(np.float64) @ X.astype(np.float64).T).min() > 1e-3
    base = CocoaOracle(loss, "dense", n, d, X, y, lam)
    base.partition(K, 4)
    base.cocoa_round(0, sigma_p)                            # so that alpha and v are not zero at the round's start
    alpha0, v0 = base.state.copy(), base.v.copy()
    w = v0 / (lam * n)
    nk = int(np.diff(base.part_off).max())
    states = [alpha0]
    for t in range(1, nk + 1):                              # the round's first t steps of every task
        o = CocoaOracle(loss, "dense", n, d, X, y, lam)
        o.partition(K, 4)
        o.state, o.v, o.round = alpha0.copy(), v0.copy(), 1
        o.cocoa_round(t, sigma_p)
        states.append(o.state.copy())
    moved = 0
    for k in range(K):
        members = base.members[base.part_off[k]:base.part_off[k + 1]].tolist()
        order = base.permutation(1, k)
        for t in range(1, len(order) + 1):
            i = int(order[t - 1])
            before = states[t - 1] - alpha0                 # what the task's earlier steps of this round changed
            chosen = y[i] * states[t][i]

            def f(a_new):
                dal = before.copy()
                dal[i] = y[i] * a_new - alpha0[i]
                return _subproblem_value(loss, X, y, lam, K, sigma_p, w, members, alpha0, dal)

            if loss == "hinge":
                # along one coordinate the objective is exactly a parabola on [0, 1]: its vertex from three values
                f0, fh, f1 = f(0.0), f(0.5), f(1.0)
                curv, slope = 2 * (f0 - 2 * fh + f1), -3 * f0 + 4 * fh - f1
                best = min(1.0, max(0.0, -slope / (2 * curv)))
                assert abs(chosen - best) <= 1e-12
            else:
                lo, hi = 0.0, 1.0                           # golden section; the objective is strictly concave
                gr = (math.sqrt(5) - 1) / 2
                for _ in range(80):
                    c1, c2 = hi - gr * (hi - lo), lo + gr * (hi - lo)
                    if f(c1) < f(c2):
                        lo = c1
                    else:
                        hi = c2
                best = 0.5 * (lo + hi)
                assert abs(chosen - best) <= 1e-6           # (a maximum is located to about the root of the rounding)
            grid = np.linspace(0.0, 1.0, 2001)
            assert f(chosen) >= max(f(g) for g in grid) - 1e-13
            moved += abs(chosen - y[i] * states[t - 1][i]) > 1e-3
    assert moved >= n // 2                                  # the steps are real moves, not all clipped or at rest


# ---------------------------------------------------------------- P3: K = 1 is plain SDCA

@pytest.mark.parametrize("fmt", ["dense", "csr"])
def test_single_partition_round_is_textbook_sdca(fmt):
    n, d, lam = 60, 7, 0.05
    X, y = dense_problem(n, d, 3)
    if fmt == "csr":
        X[np.random.default_rng(0).random(X.shape) < 0.5] = 0.0
        ip, ix, vals = to_csr(X)
        o = CocoaOracle("hinge", "csr", n, d, vals, y, lam, ip, ix)
    else:
        o = CocoaOracle("hinge", "dense", n, d, X, y, lam)
    o.partition(1, 11)
    alpha = np.zeros(n)
    w = np.zeros(d)
    for rnd in range(3):
        order = o.permutation(rnd, 0)
        for i in order:                                    # SDCA for the hinge loss, primal-dual form
            xi = X[i].astype(np.float64)
            grad = 1.0 - y[i] * (xi @ w)
            a_old = alpha[i] * y[i]
            a_new = min(1.0, max(0.0, a_old + lam * n * grad / (xi @ xi))) if xi @ xi > 0 else 1.0
            alpha[i] = y[i] * a_new
            w += (a_new - a_old) * y[i] * xi / (lam * n)
        o.cocoa_round(0, 1.0)
        assert np.allclose(o.state, alpha, atol=1e-12)
        assert np.allclose(o.v / (lam * n), w, atol=1e-12)


# ---------------------------------------------------------------- P4: hinge dual against a brute-force QP

def brute_force_svm_dual(X, y, lam):
    """All 3^n assignments of {at 0, at 1, free}; a KKT point of the concave QP is a global maximiser."""
    n = X.shape[0]
    Z = X.astype(np.float64) * y[:, None]
    Q = Z @ Z.T
    best = None
    for pattern in itertools.product((0, 1, 2), repeat=n):
        pat = np.array(pattern)
        free = np.nonzero(pat == 2)[0]
        a = np.where(pat == 1, 1.0, 0.0)
        if free.size:
            rhs = lam * n - Q[np.ix_(free, np.arange(n))] @ a
            try:
                a[free] = np.linalg.solve(Q[np.ix_(free, free)], rhs)
            except np.linalg.LinAlgError:
                continue
            if (a[free] < -1e-12).any() or (a[free] > 1 + 1e-12).any():
                continue
        grad = lam * n - Q @ a                  # n * lam * n * dD/da
        if (grad[pat == 0] > 1e-10).any() or (grad[pat == 1] < -1e-10).any():
            continue
        val, _ = hinge_dual_value(X, y, lam, np.clip(a, 0, 1))
        if best is None or val > best[0]:
            best = (val, np.clip(a, 0, 1))
    return best


def test_hinge_reaches_brute_force_qp_optimum():
    n, d, lam = 7, 9, 0.1
    X, y = dense_problem(n, d, 21)
    d_star, a_star = brute_force_svm_dual(X, y, lam)
    _, w_star = hinge_dual_value(X, y, lam, a_star)
    for K, sp in [(1, 1.0), (2, 2.0), (3, 3.0)]:
        o = CocoaOracle("hinge", "dense", n, d, X, y, lam)
        o.partition(K, 4)
        for _ in range(4000):
            o.cocoa_round(0, sp)
            if o.duality_gap()["gap"] < 1e-12:
                break
        g = o.duality_gap()
        assert g["gap"] < 1e-10
        assert abs(g["dual"] - d_star) < 1e-9
        assert np.allclose(o.v / (lam * n), w_star, atol=1e-6)
        assert np.allclose(o.state * y, a_star, atol=1e-5)


def test_hinge_against_projected_gradient_n20():
    n, d, lam = 20, 24, 0.05
    X, y = dense_problem(n, d, 5)
    Z = X.astype(np.float64) * y[:, None]
    Q = Z @ Z.T / (lam * n * n)
    L = np.linalg.eigvalsh(Q).max()
    a = np.zeros(n)
    for _ in range(200000):
        a_new = np.clip(a + (1.0 / n - Q @ a) / L, 0, 1)
        if np.abs(a_new - a).max() < 1e-15:
            break
        a = a_new
    d_star, w_star = hinge_dual_value(X, y, lam, a)
    o = CocoaOracle("hinge", "dense", n, d, X, y, lam)
    o.partition(4, 0)
    for _ in range(5000):
        o.cocoa_round(0, 4.0)
        if o.duality_gap()["gap"] < 1e-12:
            break
    g = o.duality_gap()
    assert g["gap"] < 1e-10 and abs(g["dual"] - d_star) < 1e-9
    assert np.allclose(o.v / (lam * n), w_star, atol=1e-6)


# ---------------------------------------------------------------- P5: ridge against the normal equations

def to_csc(X):
    ip, ix, vals = to_csr(np.ascontiguousarray(X.T))
    return ip, ix, vals


@pytest.mark.parametrize("K", [1, 3])
def test_ridge_reaches_normal_equation_solution(K):
    n, d, lam = 40, 12, 0.03
    X, y = dense_problem(n, d, 8, "ridge")
    X[np.random.default_rng(1).random(X.shape) < 0.3] = 0.0
    Xd = X.astype(np.float64)
    w_star = np.linalg.solve(Xd.T @ Xd / n + lam * np.eye(d), Xd.T @ y.astype(np.float64) / n)
    ip, ix, vals = to_csc(X)
    o = CocoaOracle("ridge", "csc", n, d, vals, y, lam, ip, ix)
    o.partition(K, 2)
    for _ in range(3000):
        o.cocoa_round(0, float(K))
    g = o.duality_gap()
    p_star = ((Xd @ w_star - y) ** 2).sum() / (2 * n) + 0.5 * lam * w_star @ w_star
    assert np.allclose(o.state, w_star, atol=1e-10)
    assert np.allclose(o.v, Xd @ w_star, atol=1e-9)
    assert abs(g["primal"] - p_star) < 1e-12 and abs(g["gap"]) < 1e-12
    # away from the optimum the ridge gap is strictly positive and the dual stays below the optimum
    o2 = CocoaOracle("ridge", "csc", n, d, vals, y, lam, ip, ix)
    o2.partition(K, 2)
    g0 = o2.duality_gap()
    assert abs(g0["primal"] - (y.astype(np.float64) ** 2).sum() / (2 * n)) < 1e-12      # w = 0
    o2.cocoa_round(0, float(K))
    g1 = o2.duality_gap()
    assert g1["gap"] > 0 and g1["dual"] <= p_star + 1e-12 <= g1["primal"] + 2e-12


def test_ridge_single_step_is_exact_line_minimum():
    # K = 1, sigma' = 1: one coordinate step minimises P along that coordinate.
    n, d, lam = 15, 4, 0.2
    X, y = dense_problem(n, d, 13, "ridge")
    ip, ix, vals = to_csc(X)
    o = CocoaOracle("ridge", "csc", n, d, vals, y, lam, ip, ix)
    o.partition(1, 0)
    j = o.permutation(0, 0)[0]
    o.cocoa_round(1, 1.0)
    Xd, yd = X.astype(np.float64), y.astype(np.float64)
    want = (Xd[:, j] @ yd / n) / (Xd[:, j] @ Xd[:, j] / n + lam)
    assert abs(o.state[j] - want) < 1e-14 and np.count_nonzero(o.state) == 1


# ---------------------------------------------------------------- P6: logistic

def test_logistic_step_against_bisection():
    def sig(z):
        return 1 / (1 + math.exp(-z)) if z >= 0 else math.exp(z) / (1 + math.exp(z))

    rng = np.random.default_rng(0)
    for q in [0.0, 1e-3, 0.3, 1.0, 7.0, 81.0, 1e3, 1e5]:
        for _ in range(400):
            a = float(rng.choice([0.0, 1.0, rng.random(), 1e-8, 1 - 1e-8]))
            m = float(rng.choice([rng.uniform(-30, 30), rng.uniform(-2, 2)]))
            lo, hi = -2000.0, 2000.0
            for _ in range(300):
                mid = 0.5 * (lo + hi)
                if mid + m + q * (sig(mid) - a) > 0:
                    hi = mid
                else:
                    lo = mid
            got, resid = oracle.step_logistic(a, m, q)
            assert abs(got - sig(0.5 * (lo + hi))) < 1e-12
            assert abs(resid) <= 1e-9
            assert 0.0 <= got <= 1.0
    assert abs(oracle.step_logistic(0.3, 1.7, 0.0)[0] - sig(-1.7)) < 1e-15      # zero row
    # the regime of the workloads: a anywhere in (0, 1), margins of a few units, q over six decades (here Newton's
    # iteration from the middle of the bracket alternates between the two flat ends of the sigmoid)
    for _ in range(20000):
        q, a, m = float(10 ** rng.uniform(-3, 3)), float(rng.random()), float(3 * rng.standard_normal())
        lo, hi = q * a - m - q, q * a - m
        for _ in range(200):
            mid = 0.5 * (lo + hi)
            if mid + m + q * (sig(mid) - a) > 0:
                hi = mid
            else:
                lo = mid
        got, resid = oracle.step_logistic(a, m, q)
        assert abs(got - sig(0.5 * (lo + hi))) < 1e-12 and abs(resid) <= 1e-9


def test_logistic_converges_to_primal_minimiser():
    n, d, lam = 50, 3, 0.1
    X, y = dense_problem(n, d, 17)
    Xd = X.astype(np.float64)
    w = np.zeros(d)
    for _ in range(100):                                   # Newton on the primal objective
        mu = y * (Xd @ w)
        s = 1 / (1 + np.exp(mu))                           # sigmoid(-mu)
        grad = -(Xd * (y * s)[:, None]).mean(0) + lam * w
        H = (Xd.T * (s * (1 - s))) @ Xd / n + lam * np.eye(d)
        w -= np.linalg.solve(H, grad)
    o = CocoaOracle("logistic", "dense", n, d, X, y, lam)
    o.partition(2, 6)
    for _ in range(800):
        o.cocoa_round(0, 2.0)
    g = o.duality_gap()
    assert g["gap"] < 1e-12
    assert np.allclose(o.v / (lam * n), w, atol=1e-8)
    assert o.last_newton_resid < 1e-9
    p_star = np.log1p(np.exp(-y * (Xd @ w))).mean() + 0.5 * lam * w @ w
    assert abs(g["primal"] - p_star) < 1e-12 and abs(g["dual"] - p_star) < 1e-11


# ---------------------------------------------------------------- P7: orthogonal rows decouple

@pytest.mark.parametrize("K,sp", [(1, 1.0), (3, 1.0), (3, 3.0)])
def test_orthogonal_rows_closed_form(K, sp):
    n = d = 12
    rng = np.random.default_rng(2)
    scale = rng.uniform(0.05, 3.0, n)
    P = rng.permutation(n)
    X = np.zeros((n, d), np.float32)
    X[np.arange(n), P] = scale
    y = np.where(rng.random(n) < 0.5, 1.0, -1.0).astype(np.float32)
    lam = 0.02
    s = X.astype(np.float64)[np.arange(n), P] ** 2
    o = CocoaOracle("hinge", "dense", n, d, X, y, lam)
    o.partition(K, 1)
    a = np.zeros(n)
    for _ in range(3):
        m = a * s / (lam * n)                               # y x.v/(lam n) with v only from the same row
        a = np.clip(a + (1 - m) / (sp * s / (lam * n)), 0, 1)
        o.cocoa_round(0, sp)
        assert np.allclose(o.state * y, a, atol=1e-13)
    if sp == 1.0:
        assert np.allclose(a, np.clip(lam * n / s, 0, 1), atol=1e-13)      # exact optimum after one epoch
        assert o.duality_gap()["gap"] < 1e-14


# ---------------------------------------------------------------- P1, P2, P8, P9 on a mid-sized problem

@pytest.mark.parametrize("loss", ["hinge", "logistic"])
def test_gap_terms_consistency_ascent_and_repartition(loss):
    n, d, lam, K = 400, 30, 1.0 / 400, 4
    X, y = dense_problem(n, d, 31)
    X[np.random.default_rng(3).random(X.shape) < 0.6] = 0.0
    X[5] = 0.0                                              # a zero row
    ip, ix, vals = to_csr(X)
    o = CocoaOracle(loss, "csr", n, d, vals, y, lam, ip, ix, threads=2)
    o.partition(K, 0)
    g0 = o.duality_gap()
    assert abs(g0["gap"] - (1.0 if loss == "hinge" else math.log(2))) < 1e-12    # alpha = 0
    prev_dual, gaps = g0["dual"], []
    for r in range(25):
        if r == 12:
            before = (o.state.copy(), o.v.copy(), o.duality_gap())
            o.partition(2, 99)
            K = 2
            after = o.duality_gap()
            assert (o.state == before[0]).all() and (o.v == before[1]).all()
            assert after["gap"] == before[2]["gap"]
        o.cocoa_round(0, float(K))
        g = o.duality_gap(terms=True)
        assert g["terms"].min() >= -1e-12 and g["gap"] >= 0
        assert g["dual"] >= prev_dual - 1e-13
        prev_dual = g["dual"]
        v2 = o.recompute_shared_vector()
        assert np.abs(v2 - o.v).max() <= 1e-12 * max(1.0, np.abs(v2).max())
        gaps.append(g["gap"])
        assert g["primal"] >= g["dual"]
    assert gaps[-1] < 0.25 * gaps[0]
    assert abs(abs(o.state[5]) - (1.0 if loss == "hinge" else 0.5)) < 1e-12      # zero row: a' = 1 / sigmoid(0)


def test_unequal_partitions_keep_the_invariants():
    # tasks of very different sizes (one of a single coordinate): dual ascent for sigma' >= K, a non-negative gap
    # that shrinks, and v = X^T alpha after every round; repartitioning to equal sizes leaves the state alone
    n, d, lam, K = 300, 20, 1.0 / 300, 4
    X, y = dense_problem(n, d, 8)
    o = CocoaOracle("hinge", "dense", n, d, X, y, lam, threads=2)
    o.partition(K, 1, sizes=[200, 1, 59, 40])
    assert np.diff(o.part_off).tolist() == [200, 1, 59, 40]
    prev_dual, primals, duals = o.duality_gap()["dual"], [], []
    for r in range(20):
        if r == 10:
            before = (o.state.copy(), o.v.copy())
            o.partition(K, 2)
            assert (o.state == before[0]).all() and (o.v == before[1]).all()
        o.cocoa_round(0, float(K))
        g = o.duality_gap(terms=True)
        assert g["terms"].min() >= -1e-12 and g["dual"] >= prev_dual - 1e-13
        prev_dual = g["dual"]
        v2 = o.recompute_shared_vector()
        assert np.abs(v2 - o.v).max() <= 1e-12 * max(1.0, np.abs(v2).max())
        primals.append(g["primal"])
        duals.append(g["dual"])
    # weak duality across rounds: every primal value bounds every dual value, whichever round each comes from
    assert min(primals) >= max(duals) - 1e-13


def test_step_budgets_per_partition():
    # budgets equal to H reproduce the round with H; a budget of 0 leaves the partition's coordinates alone; the
    # invariants hold with ragged budgets
    n, d, K = 240, 12, 3
    X, y = dense_problem(n, d, 13)
    a = CocoaOracle("hinge", "dense", n, d, X, y, 1.0 / n, threads=2)
    b = CocoaOracle("hinge", "dense", n, d, X, y, 1.0 / n, threads=2)
    a.partition(K, 4)
    b.partition(K, 4)
    a.cocoa_round(50, 3.0)
    b.cocoa_round(0, 3.0, steps=[50, 50, 50])
    assert (a.state == b.state).all() and (a.v == b.v).all()
    a.cocoa_round(0, 3.0)
    b.cocoa_round(0, 3.0, steps=np.diff(b.part_off))
    assert (a.state == b.state).all() and (a.v == b.v).all()
    before = b.state.copy()
    prev = b.duality_gap()["dual"]
    b.cocoa_round(0, 3.0, steps=[80, 0, 7])
    idle = b.members[b.part_off[1]:b.part_off[2]]
    assert (b.state[idle] == before[idle]).all()
    busy0 = b.members[b.part_off[0]:b.part_off[1]]
    assert (b.state[busy0] != before[busy0]).any()
    assert np.count_nonzero(b.state[b.members[b.part_off[2]:]] != before[b.members[b.part_off[2]:]]) <= 7
    g = b.duality_gap(terms=True)
    assert g["dual"] >= prev - 1e-13 and g["terms"].min() >= -1e-12
    v2 = b.recompute_shared_vector()
    assert np.abs(v2 - b.v).max() <= 1e-12 * max(1.0, np.abs(v2).max())
    with pytest.raises(RuntimeError):
        b.cocoa_round(0, 3.0, steps=[1, -1, 1])


def test_result_is_independent_of_thread_count():
    n, d = 300, 10
    X, y = dense_problem(n, d, 4)
    res = []
    for th in (1, 4):
        o = CocoaOracle("hinge", "dense", n, d, X, y, 0.01, threads=th)
        o.partition(5, 2)
        for _ in range(3):
            o.cocoa_round(0, 5.0)
        res.append((o.state.copy(), o.v.copy()))
    assert (res[0][0] == res[1][0]).all() and (res[0][1] == res[1][1]).all()


def test_more_partitions_need_more_epochs():
    # Sec. 1 / Sec. 2.2: convergence per epoch degrades as the data parallelism K grows.
    n, d = 600, 20
    X, y = dense_problem(n, d, 9)
    gaps = {}
    for K in (1, 4, 16):
        o = CocoaOracle("hinge", "dense", n, d, X, y, 1.0 / n)
        o.partition(K, 0)
        for _ in range(10):
            o.cocoa_round(0, float(K))
        gaps[K] = o.duality_gap()["gap"]
    assert gaps[1] < gaps[4] < gaps[16]


def test_multi_epoch_H_and_partial_H():
    n, d = 50, 5
    X, y = dense_problem(n, d, 2)
    o = CocoaOracle("hinge", "dense", n, d, X, y, 0.05)
    o.partition(2, 0)
    o.cocoa_round(10, 2.0)                                  # 10 steps in each of the 2 partitions
    assert np.count_nonzero(o.state) <= 20
    touched = set(np.nonzero(o.state)[0].tolist())
    first = set(o.permutation(0, 0)[:10].tolist()) | set(o.permutation(0, 1)[:10].tolist())
    assert touched <= first
    o.cocoa_round(60, 2.0)                                  # more than one local epoch (n_k = 25)
    v2 = o.recompute_shared_vector()
    assert np.abs(v2 - o.v).max() < 1e-12
