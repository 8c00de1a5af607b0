"""Pins for the flattened-tree attention inputs (Section 3.2 item 3): the allowed set of every row is
the reflexive-transitive closure of the parent relation, computed here with boolean matrix powers."""
import numpy as np

import oracle
from oracle import attention_inputs as att
from helpers import tiny_problem


def test_mask_is_the_closure_of_the_parent_relation_and_positions_are_depths():
    V, D, r, K, N = 40, 5, 4, 3, 30
    o = oracle.Oracle(V, D, r, K, N)
    for seed, theta in ((1, 0.0), (2, 0.02), (3, 0.3)):
        U, A, W = tiny_problem(700 + seed, V, D, r, u_std=2.0)
        t = o.expand_tree(U, A, W, anchor_tok=5, theta=theta, T=0.8, seed=seed, req=0)
        n = t["n"]
        flat, pos, m = att.attention_inputs(N, 5, 100, n, t["tok"], t["parent"], t["depth"])
        R = N + 1
        adj = np.eye(R, dtype=np.int64)                       # row -> its parent row (root = row 0)
        for i in range(n):
            adj[1 + i, 1 + int(t["parent"][i])] = 1           # parent -1 -> row 0
        closure = np.linalg.matrix_power(adj, D + 1) > 0
        assert np.array_equal(m == 0.0, closure)
        assert np.isneginf(m[m != 0.0]).all()
        for i in range(n):
            assert (m[1 + i] == 0.0).sum() == t["depth"][i] + 1   # root path: depth ancestors-or-self + the root
            assert pos[1 + i] == 100 + t["depth"][i] and flat[1 + i] == t["tok"][i]
            assert not (m[1 + i, n + 1:] == 0.0).any()        # no used row sees an unused column
        assert flat[0] == 5 and pos[0] == 100 and (flat[n + 1:] == -1).all() and (pos[n + 1:] == 0).all()
        # consistent with the bitmask the expansion emits
        for i in range(n):
            bits = int(t["mask"][i, 0])
            assert [j for j in range(N) if m[1 + i, 1 + j] == 0.0] == [j for j in range(N) if bits >> j & 1]
