"""Threshold assignment under a global sparsity budget (the one-choice-per-head problem of the
calibration section; last step of Algorithm 2): oracle pins, then the library's host-side exact
solver against the oracle.  No GPU involved: the solver runs on the host."""
import itertools

import numpy as np
import pytest

from oracle import heart_oracle as oracle


def tables(rs, M, K, monotone=True):
    """Measured-looking tables: sparsity rises and error rises as the threshold falls."""
    S = np.sort(rs.uniform(0.3, 0.95, (M, K)), axis=1)
    E = rs.uniform(0.0, 1.0, (M, K)) * rs.uniform(0.1, 3.0, (M, 1))
    return (np.sort(E, axis=1) if monotone else E), S


# ------------------------------------------------------------------ oracle pins
def test_oracle_hand_worked_two_heads():
    """Two heads, three candidates, worked by hand:
       head 0: (S, E) = (.1, 1) (.5, 2) (.9, 4);  head 1: (.2, 1) (.5, 3) (.8, 9).
       budget .30 -> need sum S >= .6: cheapest is (1, 0): .5 + .2 = .7, cost 3   [(0, 1) = .6 costs 4]
       budget .60 -> need 1.2: (2, 1) = 1.4, cost 7          [(1, 2) = 1.3 costs 11]
       budget .85 -> need 1.7: only (2, 2) = 1.7, cost 13;  budget .90 -> nothing reaches 1.8."""
    E = np.array([[1.0, 2, 4], [1, 3, 9]])
    S = np.array([[0.1, 0.5, 0.9], [0.2, 0.5, 0.8]])
    c, obj, ms = oracle.assign_thresholds(E, S, 0.30)
    assert c.tolist() == [1, 0] and obj == 3.0 and ms == pytest.approx(0.35)
    c, obj, ms = oracle.assign_thresholds(E, S, 0.60)
    assert c.tolist() == [2, 1] and obj == 7.0
    c, obj, ms = oracle.assign_thresholds(E, S, 0.85)
    assert c.tolist() == [2, 2] and obj == 13.0
    assert oracle.assign_thresholds(E, S, 0.90) is None


def test_oracle_forced_unconstrained_infeasible():
    rs = np.random.RandomState(1)
    E, S = tables(rs, 7, 1)
    c, obj, ms = oracle.assign_thresholds(E, S, S.mean() - 1e-9)  # K = 1: the only assignment
    assert c.tolist() == [0] * 7 and obj == pytest.approx(E.sum()) and ms == pytest.approx(S.mean())
    assert oracle.assign_thresholds(E, S, S.mean() + 1e-6) is None
    E, S = tables(rs, 8, 3, monotone=False)
    c, obj, _ = oracle.assign_thresholds(E, S, 0.0)               # no budget: each head's cheapest
    assert np.array_equal(c, E.argmin(axis=1)) and obj == pytest.approx(E.min(axis=1).sum())
    top = S.max(axis=1).mean()
    assert oracle.assign_thresholds(E, S, top + 1e-9) is None      # beyond the sparsest assignment
    c, _, ms = oracle.assign_thresholds(E, S, top - 1e-12)         # only the sparsest assignment fits
    assert np.array_equal(c, S.argmax(axis=1)) and ms == pytest.approx(top)


def test_oracle_monotone_in_the_budget_and_symmetric_closed_form():
    rs = np.random.RandomState(2)
    E, S = tables(rs, 7, 3)
    prev = -np.inf
    for smin in np.linspace(0.3, S.max(axis=1).mean(), 25):
        r = oracle.assign_thresholds(E, S, smin)
        assert r is not None and r[1] >= prev - 1e-15 and r[2] >= smin
        prev = r[1]
    # identical heads with candidates (S, E) = (.5, 1) (.75, 2): a budget of .5 + .25 m / M needs m upgrades
    M = 8
    E = np.tile([1.0, 2.0], (M, 1))
    S = np.tile([0.5, 0.75], (M, 1))
    for m in range(M + 1):
        c, obj, ms = oracle.assign_thresholds(E, S, 0.5 + 0.25 * m / M)
        assert c.sum() == m and obj == M + m


def test_oracle_against_an_independent_milp_solver():
    """scipy's MILP (HiGHS) on the same binary programme: equal optimal objective."""
    sopt = pytest.importorskip("scipy.optimize")
    rs = np.random.RandomState(3)
    for _ in range(25):
        M, K = int(rs.randint(2, 8)), int(rs.randint(2, 4))
        E, S = tables(rs, M, K, monotone=bool(rs.rand() < 0.5))
        smin = float(rs.uniform(S.min(axis=1).mean(), S.max(axis=1).mean()))
        A_one = np.zeros((M, M * K))
        for i in range(M):
            A_one[i, i * K:(i + 1) * K] = 1.0
        cons = [sopt.LinearConstraint(A_one, 1.0, 1.0), sopt.LinearConstraint(S.reshape(1, -1) / M, smin, np.inf)]
        res = sopt.milp(E.reshape(-1), constraints=cons, integrality=np.ones(M * K), bounds=sopt.Bounds(0, 1))
        got = oracle.assign_thresholds(E, S, smin)
        assert res.success and got is not None
        assert got[1] == pytest.approx(res.fun, rel=1e-9, abs=1e-12)


def test_oracle_brute_force_in_python_on_tiny_tables():
    rs = np.random.RandomState(4)
    for _ in range(20):
        M, K = int(rs.randint(1, 5)), int(rs.randint(1, 4))
        E, S = tables(rs, M, K, monotone=False)
        smin = float(rs.uniform(0.3, 0.9))
        best = None
        for ks in itertools.product(range(K), repeat=M):
            s = sum(S[i, k] for i, k in enumerate(ks)) / M
            e = sum(E[i, k] for i, k in enumerate(ks))
            if s >= smin and (best is None or e < best[0]):
                best = (e, ks)
        got = oracle.assign_thresholds(E, S, smin)
        assert (got is None) == (best is None)
        if best:
            assert got[0].tolist() == list(best[1])


# ------------------------------------------------------------------ the library's solver against the oracle
@pytest.fixture(scope="module")
def heart():
    from paper_2605_14513_b200 import heart as h

    h.lib()
    return h


def test_solver_equals_oracle_on_random_tables(heart):
    rs = np.random.RandomState(5)
    for _ in range(400):
        M, K = int(rs.randint(1, 10)), int(rs.randint(1, 5))
        E, S = tables(rs, M, K, monotone=bool(rs.rand() < 0.7))
        smin = float(rs.uniform(0.2, 1.0))
        got, ref = heart.heart_assign_thresholds(E, S, smin), oracle.assign_thresholds(E, S, smin)
        assert (got is None) == (ref is None), (M, K, smin)
        if ref is not None:
            # continuous random tables: the optimum is unique, so the choice vectors must coincide,
            # and both sides add the chosen entries left to right: sums equal to the last bit
            assert np.array_equal(got[0], ref[0]) and got[1] == ref[1] and got[2] == ref[2] and got[3]


def test_solver_on_ties_duplicates_and_edge_budgets(heart):
    # exactly tied optima: equal objective, feasible, proved
    E = np.array([[1.0, 2, 4], [1, 3, 9]])
    S = np.array([[0.1, 0.5, 0.9], [0.2, 0.5, 0.8]])
    got, ref = heart.heart_assign_thresholds(E, S, 0.5), oracle.assign_thresholds(E, S, 0.5)
    assert got[1] == ref[1] == 5.0 and got[2] >= 0.5 and got[3]
    assert heart.heart_assign_thresholds(E, S, 0.9) is None
    # identical heads: any m heads may take the upgrade
    M = 9
    E = np.tile([1.0, 2.0, 5.0], (M, 1))
    S = np.tile([0.5, 0.75, 0.875], (M, 1))
    for smin in (0.5, 0.6, 0.75, 0.8, 0.875):
        got, ref = heart.heart_assign_thresholds(E, S, smin), oracle.assign_thresholds(E, S, smin)
        assert got[1] == ref[1] and got[2] >= smin
    # duplicated and dominated candidates; a budget no assignment needs to work for
    E = np.array([[3.0, 1.0, 1.0, 2.0]] * 4)
    S = np.array([[0.9, 0.4, 0.4, 0.3]] * 4)
    got = heart.heart_assign_thresholds(E, S, -1.0)
    assert got[1] == 4.0 and set(got[0].tolist()) <= {1, 2}
    got, ref = heart.heart_assign_thresholds(E, S, 0.6), oracle.assign_thresholds(E, S, 0.6)
    assert got[1] == ref[1]
    # invalid arguments are refused
    import ctypes as C
    bad = np.array([[np.nan, 1.0]])
    out = np.empty(1, np.int32)
    rc = heart.lib().heart_assign_thresholds(bad.ctypes.data_as(C.c_void_p), bad.ctypes.data_as(C.c_void_p), 1, 2, 0.5,
                                             out.ctypes.data_as(C.c_void_p), None, None, None)
    assert rc == heart.ERR_INVALID


def test_solver_at_model_scale_against_milp(heart):
    """30 x 12 and 40 x 40 heads, three candidates: equal objective with scipy's MILP, solved to the end."""
    sopt = pytest.importorskip("scipy.optimize")
    sp = pytest.importorskip("scipy.sparse")
    rs = np.random.RandomState(6)
    for M in (360, 1600):
        K = 3
        E, S = tables(rs, M, K)
        smin = 0.9 * S.max(axis=1).mean() + 0.1 * S.min(axis=1).mean() if M == 360 else 0.7
        got = heart.heart_assign_thresholds(E, S, smin)
        assert got is not None and got[3] and got[2] >= smin
        assert got[1] == pytest.approx(sum(E[i, k] for i, k in enumerate(got[0])))
        rows = np.repeat(np.arange(M), K)
        A_one = sp.csr_matrix((np.ones(M * K), (rows, np.arange(M * K))), shape=(M, M * K))
        cons = [sopt.LinearConstraint(A_one, 1.0, 1.0), sopt.LinearConstraint(S.reshape(1, -1) / M, smin, np.inf)]
        res = sopt.milp(E.reshape(-1), constraints=cons, integrality=np.ones(M * K), bounds=sopt.Bounds(0, 1),
                        options={"mip_rel_gap": 0.0})
        assert res.success
        assert got[1] <= res.fun * (1 + 1e-9) + 1e-12  # never worse than the MILP solver's optimum
        assert got[1] >= res.fun * (1 - 1e-6)           # and no better than its (gap-tolerant) bound allows
