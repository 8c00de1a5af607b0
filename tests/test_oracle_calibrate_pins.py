"""Pins for the calibration-statistics oracle (Section 3.4): populations and bins recounted by another
route with library routines, the two-scalar fit against a library logistic regression and a closed
form, the monotone table against a library isotonic regression."""
import math
import os

import numpy as np
import pytest
from scipy.special import logit as sp_logit
from sklearn.isotonic import IsotonicRegression
from sklearn.linear_model import LogisticRegression

import oracle
from oracle import calibrate as cal
from helpers import tiny_problem, tiny_z_path, z_rows_for_tree

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")


def golden(name):
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line and line.split("=")[0].strip() == name:
            return float(line.split("=")[1])
    raise KeyError(name)


def verified_trees(T, rounds=12):
    V, D, r, K, N = 8, 3, 4, 3, 12
    o = oracle.Oracle(V, D, r, K, N)
    out = []
    for s in range(rounds):
        U, A, W = tiny_problem(500 + s, V, D, r, u_std=1.5)
        Zp = tiny_z_path(600 + s, U, A, W, D, sigma=0.7, anchor=2)
        tree = o.expand_tree(U, A, W, anchor_tok=2, theta=0.0, T=T, seed=s, req=0)
        ver = o.verify_tree(U, A, W, z_rows_for_tree(tree, Zp, V), 2, tree, T, s, 0, want_edge_stat=True)
        out.append((tree, ver))
    return D, out


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_populations_and_bins_recounted_by_another_route(T):
    D, rounds = verified_trees(T)
    lo, hi = -10.0, 10.0
    stats = cal.new_stats(D)
    for tree, ver in rounds:
        near = cal.accumulate(stats, D, lo, hi, tree["n"], tree["parent"], tree["depth"], tree["q0"],
                              ver["edge_stat"], ver["acc_len"], ver["acc_node"])
        assert near == 0
    # the other route: bins by a library search over the midpoints between knots, logit by a library
    # routine, and the ancestors-accepted population by walking up the parent pointers of every node
    knots = np.linspace(lo, hi, cal.KNOTS)
    mids = (knots[:-1] + knots[1:]) / 2
    want = np.zeros((2, D, cal.KNOTS, 2))
    total_edges = total_acc = 0
    for tree, ver in rounds:
        n = tree["n"]
        on_path = set(int(x) for x in ver["acc_node"][:ver["acc_len"]])
        for i in range(n):
            t = float(np.clip(sp_logit(min(tree["q0"][i], 1 - 1e-12)), -30, 30))
            j = int(np.searchsorted(mids, t))
            d = int(tree["depth"][i]) - 1
            anc, p = True, int(tree["parent"][i])
            while p >= 0:                                     # every strict ancestor was committed
                anc = anc and p in on_path
                p = int(tree["parent"][p])
            for pop in ((0, 1) if anc else (0,)):
                want[pop, d, j, 0] += 1
                want[pop, d, j, 1] += ver["edge_stat"][i]
        total_edges += n
        total_acc += ver["acc_len"]
    assert np.array_equal(stats[..., 0], want[..., 0].astype(np.int64))
    assert np.allclose(stats[..., 1] / cal.UNIT, want[..., 1], atol=1e-6)
    assert stats[0, ..., 0].sum() == total_edges
    assert (stats[1] <= stats[0]).all()
    if T == 0.0:
        # labels are 0/1 and the committed nodes are exactly the ancestors-accepted edges labelled 1
        assert stats[1, ..., 1].sum() == total_acc * (1 << 24)
        assert set(np.unique(stats[..., 1] % (1 << 24))) == {0}
    # the mean logit of a cell lies in the cell
    for cell in np.argwhere(stats[0, ..., 0] > 0):
        d, j = cell
        x = stats[0, d, j, 2] / cal.UNIT / stats[0, d, j, 0] - cal.X_SHIFT
        assert (j == 0 or x >= mids[j - 1] - 1e-6) and (j == cal.KNOTS - 1 or x <= mids[j] + 1e-6)


def test_two_scalar_fit_matches_a_library_logistic_regression():
    rng = np.random.default_rng(3)
    a0, b0 = golden("platt_a"), golden("platt_b")            # Eq. 3
    xs = np.linspace(-6, 6, 12)
    cells, X, y, w = [], [], [], []
    for x in xs:
        n = int(rng.integers(200, 2000))
        s = int(rng.binomial(n, 1 / (1 + math.exp(-(a0 * x + b0)))))
        cells.append((float(n), float(x), s / n))
        X += [[x], [x]]; y += [1, 0]; w += [s, n - s]
    a, b, it = cal.fit_platt(cells)
    lib = LogisticRegression(C=np.inf, tol=1e-12, max_iter=10000).fit(np.array(X), np.array(y), sample_weight=np.array(w))
    assert abs(a - lib.coef_[0, 0]) < 1e-5 and abs(b - lib.intercept_[0]) < 1e-5
    assert it < 30
    assert abs(a - a0) < 0.05 and abs(b - b0) < 0.08          # and it recovers the generating map


def test_two_scalar_fit_survives_cells_far_out_in_the_tails():
    # logits spread over the whole knot range with most of the mass in the tails: an unguarded Newton step
    # from a saturated start leaves for infinity; the guarded iteration lands on the library's optimum
    rng = np.random.default_rng(9)
    xs = np.linspace(-10, 10, 16)
    cells, X, y, w = [], [], [], []
    for x in xs:
        n = int(3000 * (0.1 + abs(x) / 10))
        s = int(rng.binomial(n, 1 / (1 + math.exp(-(1.4 * x + 0.8)))))
        cells.append((float(n), float(x), s / n))
        X += [[x], [x]]; y += [1, 0]; w += [s, n - s]
    a, b, it = cal.fit_platt(cells)
    lib = LogisticRegression(C=np.inf, tol=1e-12, max_iter=10000).fit(np.array(X), np.array(y), sample_weight=np.array(w))
    assert abs(a - lib.coef_[0, 0]) < 1e-4 and abs(b - lib.intercept_[0]) < 1e-4
    assert abs(a - 1.4) < 0.1 and it < 40


def test_two_scalar_fit_closed_form_with_two_logits():
    # with two distinct logits the likelihood is maximised by the line through the two empirical logits
    x1, x2, r1, r2 = -1.5, 2.0, 0.2, 0.85
    a, b, _ = cal.fit_platt([(1000.0, x1, r1), (400.0, x2, r2)])
    l1, l2 = math.log(r1 / (1 - r1)), math.log(r2 / (1 - r2))
    assert a == pytest.approx((l2 - l1) / (x2 - x1), abs=1e-10)
    assert b == pytest.approx(l1 - a * x1, abs=1e-10)


def test_cells_carry_mean_logit_and_mean_label():
    stats = cal.new_stats(2)
    stats[1, 0, 3] = (4, int(3 * cal.UNIT), int((4 * (-6.0 + cal.X_SHIFT)) * cal.UNIT))
    stats[1, 1, 9] = (2, int(1 * cal.UNIT), int((2 * (2.0 + cal.X_SHIFT)) * cal.UNIT))
    assert cal.cells_of(stats, 1) == [(4.0, -6.0, 0.75), (2.0, 2.0, 0.5)]
    assert cal.cells_of(stats, 0) == []


def test_monotone_table_matches_a_library_isotonic_regression():
    rng = np.random.default_rng(5)
    for trial in range(20):
        D = 3
        stats = cal.new_stats(D)
        for d in range(D):
            for j in range(cal.KNOTS):
                n = int(rng.integers(0, 60))
                if rng.random() < 0.25:
                    n = 0
                p = min(max(0.05 + 0.06 * j + rng.normal(0, 0.12), 0.0), 1.0)
                stats[1, d, j] = (n, int(rng.binomial(n, p)) << 24 if n else 0, 0)
        stats[1, 2] = 0                                       # a depth without data keeps the fallback row
        fallback = np.tile(np.linspace(0.1, 0.9, cal.KNOTS), (D, 1))
        min_count = 5
        table = cal.refit_table(stats, 1, min_count, fallback)
        assert np.array_equal(table[2], fallback[2])
        for d in range(2):
            have = [j for j in range(cal.KNOTS) if stats[1, d, j, 0] >= min_count]
            vals = [(stats[1, d, j, 1] / cal.UNIT + 1) / (stats[1, d, j, 0] + 2) for j in have]   # rule of succession
            wts = [stats[1, d, j, 0] for j in have]
            lib = IsotonicRegression(increasing=True, out_of_bounds="clip").fit(have, vals, sample_weight=wts)
            want = np.clip(lib.predict(np.arange(cal.KNOTS)), 1e-6, 1.0)   # linear between data knots, constant outside
            assert np.allclose(table[d], want, atol=1e-12)
            assert (np.diff(table[d]) >= -1e-15).all() and (table[d] > 0).all() and (table[d] <= 1).all()


def test_monotone_cells_keep_their_smoothed_frequencies():
    stats = cal.new_stats(1)
    rates = np.linspace(0.0, 1.0, cal.KNOTS)                  # the ends: all rejected, all accepted
    for j in range(cal.KNOTS):
        stats[0, 0, j] = (1000, int(round(rates[j] * 1000)) << 24, 0)
    table = cal.refit_table(stats, 0, 1, np.zeros((1, cal.KNOTS)) + 0.5)
    assert np.allclose(table[0], (np.round(rates * 1000) + 1) / 1002, atol=1e-12)
    assert table[0, 0] == pytest.approx(1 / 1002) and table[0, -1] == pytest.approx(1001 / 1002)
