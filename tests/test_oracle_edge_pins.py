"""More pins for the CPU oracle, each aimed at one branch that no other pin reaches with a value that
could tell a mistake from the right answer: the tempered first-stage edge statistic away from 1, the
dominant-token branch of logit q_0, and the near-tie flags that decide which requests a parity test
may skip.  Every expected value is recomputed here with numpy from the definitions."""
import math

import numpy as np
import pytest

import oracle
from helpers import np_logits, np_softmax, tiny_problem


# ----------------------------------------------------------------------------------------------
# Section 3.3: first-stage acceptance ratio min(1, p(x)/q_T(x)) of every materialised edge
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("T", [0.6, 1.0, 1.4])
def test_tempered_edge_statistic_equals_the_capped_probability_ratio(T):
    V, D, r, K, N = 40, 3, 5, 4, 30
    U, A, W = tiny_problem(910, V, D, r, u_std=1.8)
    o = oracle.Oracle(V, D, r, K, N)
    tree = o.expand_tree(U, A, W, 6, theta=0.0, T=T, seed=17, req=2)
    n = tree["n"]
    assert n >= 12
    # a target unrelated to the drafter: ratios land on both sides of 1
    Z = (np.random.RandomState(5).randn(n + 1, V) * 2.0).astype(np.float32)
    for i in range(0, n, 2):   # every other edge's token is one the target likes better than the drafter does
        Z[int(tree["parent"][i]) + 1, int(tree["tok"][i])] += 6.0
    res = o.verify_tree(U, A, W, Z, 6, tree, T, 17, 2, want_edge_stat=True)
    below = above = 0
    for i in range(n):
        par = int(tree["parent"][i])
        d = 0 if par < 0 else int(tree["depth"][par])
        x_par = 6 if par < 0 else int(tree["tok"][par])
        q = np_softmax(np_logits(U[d], A[x_par], W), T)
        p = np_softmax(Z[par + 1].astype(np.float64), T)
        x = int(tree["tok"][i])
        ratio = p[x] / q[x]
        want = min(1.0, ratio)
        assert abs(res["edge_stat"][i] - want) <= 1e-12 * max(1.0, want), (i, res["edge_stat"][i], want)
        below += ratio < 0.9
        above += ratio > 1.1
    # the pin only bites if both branches of the cap were taken with room to spare
    assert below >= 2 and above >= 2


def test_edge_statistic_uses_the_parents_row_and_the_parents_token():
    # a transposed operand (the child's own row or token instead of the parent's) would pass the test
    # above only by luck; here the two differ by construction in every edge below the root
    V, D, r, K, N = 12, 3, 3, 2, 10
    U, A, W = tiny_problem(77, V, D, r, u_std=1.0, bias_scale=3.0)
    o = oracle.Oracle(V, D, r, K, N)
    tree = o.expand_tree(U, A, W, 1, theta=0.0, T=1.0, seed=3, req=0)
    n = tree["n"]
    Z = (np.random.RandomState(9).randn(n + 1, V) * 1.5).astype(np.float32)
    res = o.verify_tree(U, A, W, Z, 1, tree, 1.0, 3, 0, want_edge_stat=True)
    deep = [i for i in range(n) if tree["parent"][i] >= 0]
    assert len(deep) >= 3
    wrong = 0
    for i in deep:
        par = int(tree["parent"][i])
        x = int(tree["tok"][i])
        q = np_softmax(np_logits(U[tree["depth"][par]], A[tree["tok"][par]], W))
        p = np_softmax(Z[par + 1].astype(np.float64))
        assert abs(res["edge_stat"][i] - min(1.0, p[x] / q[x])) < 1e-12
        q_wrong = np_softmax(np_logits(U[tree["depth"][i] - 1], A[x], W))
        wrong += abs(min(1.0, p[x] / q_wrong[x]) - res["edge_stat"][i]) > 1e-6
    assert wrong >= 2


# ----------------------------------------------------------------------------------------------
# Eq. 3 input: logit q_0 when one token holds more than half of the mass
# ----------------------------------------------------------------------------------------------
def test_survival_with_a_dominant_token_uses_the_cancellation_free_logit():
    V, D, r, K, N = 30, 2, 4, 3, 12
    U, A, W = tiny_problem(31, V, D, r, u_std=1.0)
    U = U.copy()
    U[0, 11] += 12.0     # q_0 of token 11 under the root is about 1 - 3e-4
    U[1, 4] += 25.0      # and this child is so dominant that 1 - q rounds badly in floating point
    o = oracle.Oracle(V, D, r, K, N)   # Platt, published constants
    tree = o.expand_tree(U, A, W, 2, theta=0.0, T=0.0, seed=1, req=0)
    n = tree["n"]
    seen_dominant = 0
    for i in range(n):
        par = int(tree["parent"][i])
        d = 0 if par < 0 else int(tree["depth"][par])
        x_par = 2 if par < 0 else int(tree["tok"][par])
        l = np_logits(U[d], A[x_par], W)
        x = int(tree["tok"][i])
        others = np.delete(l, x)
        m = others.max()
        t = l[x] - (m + math.log(np.exp(others - m).sum()))    # log q - log(1 - q) with no subtraction of near-equal numbers
        t = min(30.0, max(-30.0, t))
        log_phat = -math.log1p(math.exp(-(0.67 * t - 0.46)))
        parent_logS = 0.0 if par < 0 else tree["logS"][par]
        assert abs(tree["logS"][i] - (parent_logS + log_phat)) < 1e-11, (i, tree["logS"][i], parent_logS + log_phat)
        seen_dominant += np_softmax(l)[x] > 0.5
    assert seen_dominant >= 2   # the root's first child and a depth-2 child


# ----------------------------------------------------------------------------------------------
# Near-tie flags (they decide which requests a GPU parity test may exempt)
# ----------------------------------------------------------------------------------------------
def _two_level_problem(V=16, D=2, r=2):
    """Zero head, so logits are the base logits; distinct, widely spaced values."""
    U = np.zeros((D + 1, V), np.float32)
    for d in range(D + 1):
        U[d] = -1.5 * np.arange(V, dtype=np.float32)
    A = np.zeros((V, r), np.float32)
    W = np.zeros((r, V), np.float32)
    return U, A, W


def test_near_topk_flag_fires_for_a_gap_of_1e_6_and_not_for_1e_3():
    T = 0.0   # greedy children: the flag looks at logits (the sampling keys of T > 0 have the next test)
    V, D, r, K, N = 16, 2, 2, 2, 8
    o = oracle.Oracle(V, D, r, K, N)
    for rel, expect in ((1e-6, True), (1e-3, False)):
        U, A, W = _two_level_problem(V, D, r)
        U[0, 3] = 10.0
        U[0, 5] = np.float32(10.0 * (1.0 - rel))   # second candidate of the root, `rel` below the first
        assert U[0, 5] != U[0, 3]
        tree = o.expand_tree(U, A, W, 0, theta=0.0, T=T, seed=1, req=0)
        assert tree["tok"][0] == 3 and tree["tok"][1] == 5      # both are children: the gap decided their order
        assert bool(tree["flags"] & oracle.FLAG_NEAR_TOPK) == expect, (rel, tree["flags"])


def test_near_topk_flag_at_positive_temperature_follows_the_sampling_keys():
    # the keys of the two best draws are moved to a chosen distance by editing the logits they sit on
    V, D, r, K, N = 16, 1, 2, 2, 4
    o = oracle.Oracle(V, D, r, K, N)
    U, A, W = _two_level_problem(V, D, r)
    U[0] = 0.0
    s = o.score_parent(U[0], A[0], W, 1.0, 5, 0, 0)
    a, b = int(s["draw_tok"][0]), int(s["draw_tok"][1])
    ka, kb = float(s["draw_key"][0]), float(s["draw_key"][1])
    for rel, expect in ((1e-6, True), (1e-3, False)):
        U2 = U.copy()
        scale = max(1.0, abs(ka))
        U2[0, b] = np.float32((ka - kb) - rel * scale)   # lifts the second key to `rel` (relative) below the first
        t = o.expand_tree(U2, A, W, 0, theta=0.0, T=1.0, seed=5, req=0)
        s2 = o.score_parent(U2[0], A[0], W, 1.0, 5, 0, 0)
        assert list(s2["draw_tok"][:2]) == [a, b]
        gap = (s2["draw_key"][0] - s2["draw_key"][1]) / max(1.0, abs(s2["draw_key"][0]))
        assert (gap < oracle.TOPK_MARGIN) == expect, gap
        assert t["n"] >= 2 and bool(t["flags"] & oracle.FLAG_NEAR_TOPK) == expect, (rel, gap, t["flags"])


def test_near_theta_flag_fires_within_1e_4_of_the_price_in_log_space():
    V, D, r, K, N = 16, 2, 2, 2, 8
    o = oracle.Oracle(V, D, r, K, N)
    U, A, W = _two_level_problem(V, D, r)
    free = o.expand_tree(U, A, W, 0, theta=0.0, T=0.0, seed=1, req=0)
    keys = sorted({float(k) for k in free["logkey"][:free["n"]]}, reverse=True)
    assert len(keys) >= 3 and keys[0] - keys[1] > 1e-2 and keys[1] - keys[2] > 1e-2   # well separated slot keys
    k = keys[1]
    for delta, expect in ((5e-5, True), (-5e-5, True), (1e-3, False), (-1e-3, False)):
        t = o.expand_tree(U, A, W, 0, theta=math.exp(k - delta), T=0.0, seed=1, req=0)
        assert bool(t["flags"] & oracle.FLAG_NEAR_THETA) == expect, (delta, t["flags"])
        # the stop itself: a key at or above the price is admitted, one below it is not
        admitted = any(abs(float(x) - k) < 1e-12 for x in t["logkey"][:t["n"]])
        assert admitted == (delta > 0)


def test_near_cap_flag_fires_when_the_cap_cuts_between_two_close_keys():
    V, D, r, K = 16, 2, 2, 2
    for rel, expect in ((2e-6, True), (1e-2, False)):
        U, A, W = _two_level_problem(V, D, r)
        U[0, 3] = 10.0
        U[0, 5] = np.float32(10.0 * (1.0 - rel))
        U[1] -= 30.0   # children of the first node are far below the root's second slot
        U[1, 0] += 60.0   # ... in probability: one token takes the row, the best-unused bound of a child is ~1
        o = oracle.Oracle(V, D, r, K, Nmax=1)
        t = o.expand_tree(U, A, W, 0, theta=0.0, T=0.0, seed=1, req=0)
        assert t["n"] == 1 and t["tok"][0] == 3
        # what is left in the heap: the root's second slot (key close to the admitted one when rel is tiny)
        # and the child's first slot (key = child survival x ~1, just below the admitted key as well);
        # an independent recomputation of the two keys decides what the flag must say
        l0 = U[0].astype(np.float64)
        def log_phat(l, x):
            others = np.delete(l, x)
            m = others.max()
            tt = min(30.0, max(-30.0, l[x] - (m + math.log(np.exp(others - m).sum()))))
            return -math.log1p(math.exp(-(0.67 * tt - 0.46)))
        k_adm = log_phat(l0, 3)
        k_sib = log_phat(l0, 5)
        k_child = k_adm + log_phat(U[1].astype(np.float64), 0)
        rest = max(k_sib, k_child)
        want = (k_adm != rest) and (k_adm - rest) < 1e-4 * max(1.0, abs(rest))
        assert bool(t["flags"] & oracle.FLAG_NEAR_CAP) == want
        if rel == 1e-2:
            # make the far case a real test of "not flagged": drop the child's slot well below too
            U[1, 0] -= 60.0
            t2 = o.expand_tree(U, A, W, 0, theta=0.0, T=0.0, seed=1, req=0)
            assert not (t2["flags"] & oracle.FLAG_NEAR_CAP)
        else:
            assert want and expect


def test_near_accept_flag_follows_the_margin():
    # one edge, one accept test: the flag must be set exactly when |u - rho| is below the margin given
    V, D, r, K, N = 10, 1, 2, 1, 1
    U, A, W = tiny_problem(5, V, D, r)
    o = oracle.Oracle(V, D, r, K, N)
    tree = o.expand_tree(U, A, W, 0, theta=0.0, T=1.0, seed=8, req=3)
    assert tree["n"] == 1
    x = int(tree["tok"][0])
    u = oracle.u_accept(8, 3, 0, 0)
    q = np_softmax(np_logits(U[0], A[0], W))
    # a target whose probability at x is exactly what puts rho at a chosen distance from u
    for dist, margin, expect in ((3e-7, 1e-6, True), (3e-6, 1e-6, False), (3e-6, 1e-5, True), (3e-5, 1e-5, False)):
        rho = u + dist
        assert 0 < rho < 1
        px = rho * q[x]
        rest = (1.0 - px) / (V - 1)
        p = np.full(V, rest); p[x] = px
        Z = np.zeros((2, V), np.float32)
        Z[0] = np.log(p).astype(np.float32)
        res = o.verify_tree(U, A, W, Z, 0, tree, 1.0, 8, 3, accept_margin=margin)
        p32 = np_softmax(Z[0].astype(np.float64))
        d_true = abs(u - min(1.0, p32[x] / q[x]))
        if abs(d_true - margin) < 0.2 * margin:
            continue   # float32 rounding of the constructed logits moved the case onto the boundary
        assert bool(res["flags"] & oracle.FLAG_NEAR_ACCEPT) == (d_true < margin) == expect
