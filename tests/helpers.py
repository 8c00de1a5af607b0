"""Shared helpers for the tests: tiny seeded problems and independent numpy restatements used as pins."""
import math

import numpy as np
import torch

from paper_2609_22098_b200 import synth


def tiny_problem(seed, V=8, D=3, r=4, u_std=1.5, z_sigma=1.0, bias_scale=1.0):
    """Random fp32 inputs for a tiny vocabulary: U [D+1][V], A [V][r], W [r][V]."""
    U = (synth.normals(seed, 40, 0, (D + 1) * V).reshape(D + 1, V) * u_std).float().numpy()
    A = (synth.normals(seed, 41, 0, V * r).reshape(V, r) * bias_scale / math.sqrt(r)).float().numpy()
    W = (synth.normals(seed, 42, 0, r * V).reshape(r, V)).float().numpy()
    return U, A, W


def tiny_z_path(seed, U, A, W, D, sigma=1.0, anchor=0):
    """Target logits for every token path of length 0..D over a tiny vocabulary (row order: by
    length, then base-V value of the path)."""
    V = U.shape[1]
    rows = sum(V ** k for k in range(D + 1))
    noise = synth.normals(seed, 43, 0, rows * V).reshape(rows, V).numpy()
    Z = np.empty((rows, V), np.float32)
    idx = 0
    for k in range(D + 1):
        for p in range(V ** k):
            last = anchor if k == 0 else p % V
            base = U[k].astype(np.float64) + A[last].astype(np.float64) @ W.astype(np.float64)
            Z[idx] = (base + sigma * noise[idx]).astype(np.float32)
            idx += 1
    return Z


def path_row(path, V):
    off = sum(V ** k for k in range(len(path)))
    idx = 0
    for t in path:
        idx = idx * V + int(t)
    return off + idx


def node_path(tree, i):
    seq = []
    while i >= 0:
        seq.append(int(tree["tok"][i]))
        i = int(tree["parent"][i])
    return tuple(reversed(seq))


def z_rows_for_tree(tree, Z_path, V):
    n = int(tree["n"])
    rows = [Z_path[0]]
    for i in range(n):
        rows.append(Z_path[path_row(node_path(tree, i), V)])
    return np.stack(rows)


def np_logits(U_row, a_row, W):
    return U_row.astype(np.float64) + a_row.astype(np.float64) @ W.astype(np.float64)


def np_softmax(l, T=1.0):
    x = (l - l.max()) / T
    e = np.exp(x)
    return e / e.sum()


def sigmoid(x):
    return 1.0 / (1.0 + math.exp(-x))


def logit(q):
    return math.log(q) - math.log1p(-q)
