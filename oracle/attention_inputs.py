"""Flattened-tree inputs of the target forward -- TEST INFRASTRUCTURE.

Plain restatement of Section 3.2, item 3: the tree is flattened for one target forward in which row i
attends to its root path only, and a node's position is its depth below the anchor.  Only the tests
and the smoke check import this module; the product path never does.

Layout taken (the paper fixes none): per request Nmax + 1 rows, row 0 = the anchor (root), row 1 + i =
node i in the tree's canonical order; token ids [Nmax+1] (anchor, then node tokens; -1 in unused rows);
position ids [Nmax+1] = base position + depth (0 in unused rows); additive mask [Nmax+1][Nmax+1] with 0
where row may attend column and -inf elsewhere.  An unused row attends to itself only, so that a
softmax over it stays defined; no used row attends to an unused column.
"""
from __future__ import annotations

import numpy as np


def attention_inputs(Nmax, anchor_tok, base_pos, n, tok, parent, depth):
    R = Nmax + 1
    flat = np.full(R, -1, np.int32)
    pos = np.zeros(R, np.int32)
    m = np.full((R, R), -np.inf, np.float32)
    flat[0] = anchor_tok
    pos[0] = base_pos
    m[0, 0] = 0.0
    for i in range(int(n)):
        flat[1 + i] = tok[i]
        pos[1 + i] = base_pos + int(depth[i])
        j = i
        while j >= 0:                      # the node itself and every ancestor
            m[1 + i, 1 + j] = 0.0
            j = int(parent[j])
        m[1 + i, 0] = 0.0                  # the root
    for i in range(int(n) + 1, R):
        m[i, i] = 0.0
    return flat, pos, m
