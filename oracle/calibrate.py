"""Calibration statistics from verified trees and the refit of the edge-acceptance map -- TEST
INFRASTRUCTURE.

Plain numpy/Python restatement of Section 3.4: tree verification labels every materialised edge
(does the node match the target at its parent), the value function is fitted on the edges whose
ancestors were all accepted -- the population a path-survival product conditions on -- and the
fitted map is p_hat = sigmoid(a * logit q0 + b) (Eq. 3).  Only the tests, the smoke check and the
benchmark's CPU-baseline leg import this module; the product path never does.

Readings taken where the paper leaves the arithmetic open:
  * Statistics are kept as sums per (population, depth row, bin) so that rounds can be added up in any
    order: population 0 = every edge, 1 = ancestors-accepted edges; depth row = depth of the parent
    (the row of the per-depth table that priced the edge); bin = index of the nearest of the 16 knots
    that are uniform in logit(q0) on [lo, hi] (the knots of the per-depth table), the logit clamped to
    [-30, 30] as everywhere else.
  * Three sums per cell, integers so that the result does not depend on the order of addition:
    the count, the labels in units of 2^-24 and (logit + 32) in units of 2^-24.  The label of an edge is
    the per-edge statistic of verification: 1/0 "equals the parent's target arg-max" at T = 0, the
    first-stage acceptance probability min(1, p(x)/q_T(x)) at T > 0.
  * Two-scalar refit (Eq. 3): maximum likelihood of the logistic model over the cells of one population,
    each cell standing for `count` edges at its mean logit with its mean label (exact when the edges of
    a cell share one logit), pooled over depths; Newton's method from (a, b) = (0, 0) with 1e-12 added
    to the Hessian's diagonal and the step halved (at most 30 times) until the likelihood does not get
    worse -- the safeguards of the usual implementation of Platt scaling; a plain Newton step from a
    start where most cells are saturated overshoots --, at most 100 steps, stopped when both components
    move by less than 1e-12 or no step helps.
  * Table refit: knot value = (label sum + 1) / (count + 2) of its cell -- the rule-of-succession
    estimate, the smoothing Platt's method applies to its targets; it keeps a cell whose edges were all
    rejected away from 0, where log p_hat would be unbounded -- where the cell holds at least
    `min_count` edges; the values of a depth row are made non-decreasing by weighted
    pool-adjacent-violators (weights = counts); knots without data are filled by linear interpolation between their neighbours with data
    and held constant outside them; a depth row without any data keeps the row given as `fallback`;
    everything is clamped to [1e-6, 1] (the table format wants values in (0, 1]).
"""
from __future__ import annotations

import math

import numpy as np

KNOTS = 16
UNIT = float(1 << 24)
X_SHIFT = 32.0


def edge_logit(q0):
    """logit of the drafter's untempered probability of the edge's token, clamped like the expansion's."""
    q = float(q0)
    if q > 1.0 - 1e-12:
        q = 1.0 - 1e-12
    if q <= 0.0:
        return -30.0
    t = math.log(q) - math.log1p(-q)
    return max(-30.0, min(30.0, t))


def knot_bin(t, lo, hi):
    pos = (t - lo) / (hi - lo) * (KNOTS - 1)
    j = int(math.floor(pos + 0.5))
    return max(0, min(KNOTS - 1, j)), pos


def accumulate(stats, D, lo, hi, n, parent, depth, q0, edge_stat, acc_len, acc_node):
    """Add one request's edges to stats, an integer array [2][D][16][3] (Python ints or int64).
    Returns the number of edges whose bin decision sits within 1e-9 of a bin boundary."""
    accepted = set(int(acc_node[k]) for k in range(int(acc_len)))
    near = 0
    for i in range(int(n)):
        p = int(parent[i])
        # ancestors accepted: the parent is the root or lies on the committed path (whose nodes have
        # accepted ancestors by construction of the walk)
        anc = p < 0 or p in accepted
        t = edge_logit(q0[i])
        j, pos = knot_bin(t, lo, hi)
        if abs((pos + 0.5) - round(pos + 0.5)) < 1e-9:
            near += 1
        d = int(depth[i]) - 1
        y_units = int(np.rint(float(edge_stat[i]) * UNIT))
        x_units = int(np.rint((t + X_SHIFT) * UNIT))
        for pop in ((0, 1) if anc else (0,)):
            stats[pop][d][j][0] += 1
            stats[pop][d][j][1] += y_units
            stats[pop][d][j][2] += x_units
    return near


def new_stats(D):
    return np.zeros((2, D, KNOTS, 3), dtype=np.int64)


def neg_log_likelihood(cells, a, b):
    f = 0.0
    for n, x, y in cells:
        if n <= 0:
            continue
        z = a * x + b
        f += n * (max(z, 0.0) + math.log1p(math.exp(-abs(z))) - y * z)
    return f


def fit_platt(cells, max_iter=100, tol=1e-12):
    """Maximum-likelihood (a, b) of y ~ sigmoid(a x + b) over weighted cells [(count, mean x, mean y)].
    Returns (a, b, iterations)."""
    a, b = 0.0, 0.0
    f = neg_log_likelihood(cells, a, b)
    it = 0
    for it in range(1, max_iter + 1):
        ga = gb = haa = hab = hbb = 0.0
        for n, x, y in cells:
            if n <= 0:
                continue
            p = 1.0 / (1.0 + math.exp(-(a * x + b)))
            r = n * (y - p)
            w = n * p * (1.0 - p)
            ga += r * x; gb += r
            haa += w * x * x; hab += w * x; hbb += w
        haa += 1e-12; hbb += 1e-12
        det = haa * hbb - hab * hab
        if not (det > 1e-300):
            break
        da = (hbb * ga - hab * gb) / det
        db = (haa * gb - hab * ga) / det
        step, ok = 1.0, False
        for _ in range(30):                                   # halve the step until the likelihood does not get worse
            na, nb = a + step * da, b + step * db
            nf = neg_log_likelihood(cells, na, nb)
            if nf <= f:
                ok = True
                break
            step *= 0.5
        if not ok:
            break
        moved = max(abs(na - a), abs(nb - b))
        a, b, f = na, nb, nf
        if moved < tol:
            break
    return a, b, it


def cells_of(stats, pop):
    out = []
    for d in range(stats.shape[1]):
        for j in range(KNOTS):
            n, ys, xs = (int(v) for v in stats[pop][d][j])
            if n > 0:
                out.append((float(n), xs / UNIT / n - X_SHIFT, ys / UNIT / n))
    return out


def pav(values, weights):
    """Weighted pool-adjacent-violators: the non-decreasing sequence closest in weighted least squares."""
    blocks = []   # [mean, weight, length]
    for v, w in zip(values, weights):
        blocks.append([float(v), float(w), 1])
        while len(blocks) > 1 and blocks[-2][0] > blocks[-1][0]:
            m2, w2, l2 = blocks.pop()
            m1, w1, l1 = blocks.pop()
            blocks.append([(m1 * w1 + m2 * w2) / (w1 + w2), w1 + w2, l1 + l2])
    out = []
    for m, _, l in blocks:
        out.extend([m] * l)
    return out


def refit_table(stats, pop, min_count, fallback):
    """[D][16] table from the cells of one population; `fallback` [D][16] supplies rows without data."""
    D = stats.shape[1]
    table = np.array(fallback, dtype=np.float64).reshape(D, KNOTS).copy()
    for d in range(D):
        have = [j for j in range(KNOTS) if int(stats[pop][d][j][0]) >= max(int(min_count), 1)]
        if not have:
            continue
        vals = [(int(stats[pop][d][j][1]) / UNIT + 1.0) / (int(stats[pop][d][j][0]) + 2.0) for j in have]
        wts = [int(stats[pop][d][j][0]) for j in have]
        iso = pav(vals, wts)
        row = np.empty(KNOTS)
        for j in range(KNOTS):
            if j <= have[0]:
                row[j] = iso[0]
            elif j >= have[-1]:
                row[j] = iso[-1]
            else:
                k = max(i for i in range(len(have)) if have[i] <= j)
                if have[k] == j:
                    row[j] = iso[k]
                else:
                    f = (j - have[k]) / (have[k + 1] - have[k])
                    row[j] = iso[k] + f * (iso[k + 1] - iso[k])
        table[d] = np.clip(row, 1e-6, 1.0)
    return table
