"""Per-request budget allocation under one node budget for the batch -- TEST INFRASTRUCTURE.

Plain Python/numpy restatement of the scheduler's second component (Section 4, item "per-request
budget allocation"): in each round the sizes N_i of the B trees are chosen to maximise the expected
number of accepted tokens under one total node budget, and greedy water-filling is enough because
every request's gain curve is concave.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg import this module; the product path never does, and nothing here is shared with it.

Reading taken (the paper gives one sentence, no pseudo-code):
  * A request's candidates come in its own best-first admission order (pop_rank), and the gain the
    allocator credits to a candidate is the key it was admitted under, exp(logkey): at T == 0 that
    is the node's calibrated path survival -- the probability that it is accepted, i.e. its share
    of the expected accepted length -- and at T > 0 it is the admissible bound of that survival that
    the expansion used before the token was drawn.  Using the admission key (never the realised
    survival of a drawn token) keeps the shaping policy independent of the drawn values, which is
    what the losslessness statement (Proposition 1) requires of it.
  * Keys never increase along a request's admission order (a child's key is its parent's survival
    times an estimate <= 1), which is the concavity the paper appeals to.
  * Water-filling: hand out the budget one node at a time, each time to the request whose next
    candidate has the largest key; equal keys go to the lowest request index.  It stops when the
    budget is spent or no candidate is left.
  * The price of the allocation is the key of the last node handed out (log domain); with the
    budget equal to the number of candidates whose key is >= theta it reproduces the theta rule.
A tree cut back to the first N_i nodes of its admission order is again a tree with complete sibling
runs, because a slot is created only when its parent, and its elder sibling, have been admitted.
"""
from __future__ import annotations

import numpy as np


def water_fill(n_nodes, logkey, pop_rank, budget):
    """Greedy water-filling.  n_nodes [B]; logkey, pop_rank [B][Nmax] in the trees' canonical node
    order.  Returns (keep [B] int, log_price float or -inf when nothing was handed out)."""
    B = len(n_nodes)
    # each request's keys in admission order
    by_pop = []
    for b in range(B):
        n = int(n_nodes[b])
        keys = [None] * n
        for i in range(n):
            keys[int(pop_rank[b][i])] = float(logkey[b][i])
        by_pop.append(keys)
    keep = [0] * B
    log_price = float("-inf")
    for _ in range(int(budget)):
        best = -1
        for b in range(B):
            if keep[b] < len(by_pop[b]):
                if best < 0 or by_pop[b][keep[b]] > by_pop[best][keep[best]]:
                    best = b
        if best < 0:
            break
        log_price = by_pop[best][keep[best]]
        keep[best] += 1
    return np.asarray(keep, np.int32), log_price


def ancestors(parent, i):
    out = []
    while i >= 0:
        out.append(i)
        i = int(parent[i])
    return out


def trim_tree(tree, keep):
    """The tree cut back to the `keep` nodes admitted first, renumbered in canonical order (the
    relative order of the surviving nodes does not change).  `tree` is a dict with n, tok, parent,
    depth, sib_rank, logS, q0, logqT, logkey, pop_rank [Nmax], node_hash [Nmax+1], optional
    node_lseT [Nmax+1], mask [Nmax][words]."""
    n = int(tree["n"])
    keep = int(keep)
    kept = [i for i in range(n) if int(tree["pop_rank"][i]) < keep]
    new_of = {old: new for new, old in enumerate(kept)}
    out = {"n": len(kept)}
    for name in ("tok", "depth", "sib_rank", "logS", "q0", "logqT", "logkey", "pop_rank"):
        a = np.zeros_like(np.asarray(tree[name]))
        for new, old in enumerate(kept):
            a[new] = tree[name][old]
        out[name] = a
    par = np.full_like(np.asarray(tree["parent"]), -1)
    for new, old in enumerate(kept):
        p = int(tree["parent"][old])
        par[new] = -1 if p < 0 else new_of[p]
    out["parent"] = par
    for name in ("node_hash", "node_lseT"):
        if tree.get(name) is None:
            continue
        src = np.asarray(tree[name])
        a = np.zeros_like(src)
        a[0] = src[0]
        for new, old in enumerate(kept):
            a[new + 1] = src[old + 1]
        out[name] = a
    mask = np.zeros_like(np.asarray(tree["mask"]))
    for new in range(len(kept)):
        for j in ancestors(par, new):
            mask[new][j // 64] |= np.uint64(1) << np.uint64(j % 64)
    out["mask"] = mask
    return out


def allocate(trees, budget):
    """Water-filling over a batch of oracle trees followed by the cut.  Returns (trimmed trees,
    keep [B], log_price)."""
    B = len(trees)
    Nmax = len(trees[0]["tok"])
    n_nodes = np.array([int(t["n"]) for t in trees], np.int32)
    logkey = np.zeros((B, Nmax), np.float64)
    pop = np.zeros((B, Nmax), np.int32)
    for b, t in enumerate(trees):
        logkey[b] = t["logkey"]
        pop[b] = t["pop_rank"]
    keep, log_price = water_fill(n_nodes, logkey, pop, budget)
    return [trim_tree(t, keep[b]) for b, t in enumerate(trees)], keep, log_price
