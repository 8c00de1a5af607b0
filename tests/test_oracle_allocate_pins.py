"""Pins for the budget-allocation oracle (Section 4, per-request budget allocation): each check
compares it with something other than itself -- a library sort of all candidates, exhaustive search
over every allocation of a tiny batch, the theta-stopped trees of the independent expansion oracle,
and the structural definition of a tree."""
import itertools
import math

import numpy as np
import pytest

import oracle
from oracle import allocate as alloc
from helpers import tiny_problem


def random_keys(rng, B, Nmax, tie_levels=0):
    """Per-request key sequences that never increase along the admission order, stored in a shuffled
    canonical order with the matching pop_rank."""
    n_nodes = rng.integers(0, Nmax + 1, size=B).astype(np.int32)
    logkey = np.zeros((B, Nmax), np.float32)
    pop = np.zeros((B, Nmax), np.int32)
    for b in range(B):
        n = int(n_nodes[b])
        if tie_levels:
            k = -np.sort(rng.integers(0, tie_levels, size=n)).astype(np.float32) * 0.25
        else:
            k = -np.sort(rng.random(n).astype(np.float32) * 6)
        perm = rng.permutation(n)
        for rank, i in enumerate(perm):
            logkey[b, i] = k[rank]
            pop[b, i] = rank
    return n_nodes, logkey, pop


@pytest.mark.parametrize("tie_levels", [0, 5])
def test_water_filling_equals_a_library_sort_of_all_candidates(tie_levels):
    rng = np.random.default_rng(7 + tie_levels)
    for trial in range(40):
        B, Nmax = int(rng.integers(1, 7)), int(rng.integers(1, 12))
        n_nodes, logkey, pop = random_keys(rng, B, Nmax, tie_levels)
        total = int(n_nodes.sum())
        for budget in {0, 1, total // 3, total // 2, max(total - 1, 0), total, total + 5}:
            keep, price = alloc.water_fill(n_nodes, logkey, pop, budget)
            cand = [(-float(logkey[b, i]), b, int(pop[b, i])) for b in range(B) for i in range(n_nodes[b])]
            cand.sort()                                       # key descending, request, admission order
            top = cand[:budget]
            want = np.bincount([b for _, b, _ in top], minlength=B)
            assert list(keep) == list(want)
            assert keep.sum() == min(budget, total)
            if top:
                assert price == -top[-1][0]
                for b in range(B):                            # the kept nodes are a prefix of the admission order
                    assert sorted(p for _, bb, p in top if bb == b) == list(range(keep[b]))
            else:
                assert price == float("-inf")


def test_water_filling_maximises_the_expected_accepted_length():
    # exhaustive search over every (N_1, N_2, N_3) with the same total: no allocation has a larger sum of
    # acceptance probabilities (a node's key at T = 0 is the probability that it is accepted)
    rng = np.random.default_rng(11)
    for trial in range(30):
        B, Nmax = 3, 5
        n_nodes, logkey, pop = random_keys(rng, B, Nmax)
        gains = []
        for b in range(B):
            g = np.zeros(n_nodes[b])
            for i in range(n_nodes[b]):
                g[pop[b, i]] = math.exp(logkey[b, i])
            gains.append(np.concatenate([[0.0], np.cumsum(g)]))
        total = int(n_nodes.sum())
        for budget in range(total + 1):
            keep, _ = alloc.water_fill(n_nodes, logkey, pop, budget)
            got = sum(gains[b][keep[b]] for b in range(B))
            best = max(sum(gains[b][c[b]] for b in range(B))
                       for c in itertools.product(*[range(n + 1) for n in n_nodes]) if sum(c) == budget)
            assert got >= best - 1e-12


@pytest.mark.parametrize("T", [0.0, 1.0])
@pytest.mark.parametrize("theta", [0.3, 0.1, 0.04])
def test_uniform_price_reduces_to_the_theta_rule(T, theta):
    # trees grown to the cap and then cut under a budget equal to the number of candidates priced
    # at or above theta are the trees the theta rule grows directly
    V, D, r, K, N = 60, 4, 5, 3, 24
    o = oracle.Oracle(V, D, r, K, N)
    full, stopped = [], []
    for b in range(5):
        U, A, W = tiny_problem(300 + b, V, D, r, u_std=2.5)
        full.append(o.expand_tree(U, A, W, anchor_tok=b, theta=0.0, T=T, seed=5, req=b))
        stopped.append(o.expand_tree(U, A, W, anchor_tok=b, theta=theta, T=T, seed=5, req=b))
    budget = sum(t["n"] for t in stopped)
    assert 0 < budget < sum(t["n"] for t in full)
    cut, keep, price = alloc.allocate(full, budget)
    assert price >= math.log(theta)
    for b in range(5):
        assert keep[b] == stopped[b]["n"] == cut[b]["n"]
        n = cut[b]["n"]
        for name in ("tok", "parent", "depth", "sib_rank", "pop_rank", "logS", "q0", "logqT", "logkey"):
            assert np.array_equal(np.asarray(cut[b][name])[:n], np.asarray(stopped[b][name])[:n]), name
        assert np.array_equal(cut[b]["node_hash"][:n + 1], stopped[b]["node_hash"][:n + 1])
        assert np.array_equal(cut[b]["mask"][:n], stopped[b]["mask"][:n])
        # every candidate left out is priced below theta unless the cap stopped the tree
        dropped = [full[b]["logkey"][i] for i in range(full[b]["n"]) if full[b]["pop_rank"][i] >= keep[b]]
        assert all(k < math.log(theta) for k in dropped) or n == N


def test_cut_tree_is_a_tree_with_complete_sibling_runs():
    V, D, r, K, N = 50, 5, 4, 4, 40
    o = oracle.Oracle(V, D, r, K, N)
    U, A, W = tiny_problem(77, V, D, r, u_std=2.0)
    tree = o.expand_tree(U, A, W, anchor_tok=3, theta=0.0, T=0.9, seed=9, req=2)
    assert tree["n"] == N
    for keep in (0, 1, 2, 7, 19, N - 1, N):
        t = alloc.trim_tree(tree, keep)
        n = t["n"]
        assert n == keep
        assert sorted(t["pop_rank"][:n]) == list(range(n))
        for i in range(n):
            p, d = int(t["parent"][i]), int(t["depth"][i])
            assert p < i and d == (1 if p < 0 else t["depth"][p] + 1)
            assert t["node_hash"][i + 1] == oracle.path_hash(int(t["node_hash"][p + 1]), int(t["tok"][i]))
            m = int(t["mask"][i, 0])
            assert m == ((int(t["mask"][p, 0]) if p >= 0 else 0) | (1 << i))
            assert bin(m).count("1") == d
            if i:
                a = (t["depth"][i - 1], t["parent"][i - 1], t["sib_rank"][i - 1])
                b = (t["depth"][i], t["parent"][i], t["sib_rank"][i])
                assert a < b                                   # canonical order survives the cut
        for v in range(-1, n):
            sibs = sorted(int(t["sib_rank"][i]) for i in range(n) if t["parent"][i] == v)
            assert sibs == list(range(len(sibs)))
        # the same root paths, token for token
        def path(tr, i):
            out = []
            while i >= 0:
                out.append(int(tr["tok"][i])); i = int(tr["parent"][i])
            return tuple(out)
        assert {path(t, i) for i in range(n)} == {path(tree, i) for i in range(N) if tree["pop_rank"][i] < keep}


def test_degenerate_budgets_and_empty_requests():
    n_nodes = np.array([0, 3, 0], np.int32)
    logkey = np.array([[0, 0, 0], [-0.1, -0.5, -0.2], [0, 0, 0]], np.float32)
    pop = np.array([[0, 0, 0], [0, 2, 1], [0, 0, 0]], np.int32)
    keep, price = alloc.water_fill(n_nodes, logkey, pop, 0)
    assert list(keep) == [0, 0, 0] and price == float("-inf")
    keep, price = alloc.water_fill(n_nodes, logkey, pop, 2)
    assert list(keep) == [0, 2, 0] and price == pytest.approx(-0.2)
    keep, price = alloc.water_fill(n_nodes, logkey, pop, 99)
    assert list(keep) == [0, 3, 0] and price == pytest.approx(-0.5)
