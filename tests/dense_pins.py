"""Dense, from-the-definition formulations used to pin the oracle (test-only code).

These build the full propagation matrix as a dense numpy array and use library matrix
products / torch autograd, i.e. they reach the same quantities by a different route
than the oracle's CSR loops.
"""
from __future__ import annotations

import numpy as np


def csr_from_edges(n, edges):
    nbr = [[] for _ in range(n)]
    for a, b in edges:
        nbr[a].append(b)
        nbr[b].append(a)
    rowptr = np.zeros(n + 1, dtype=np.int64)
    col = []
    for v in range(n):
        s = sorted(set(nbr[v]))
        col.extend(s)
        rowptr[v + 1] = len(col)
    return rowptr, np.asarray(col, dtype=np.int32)


def random_graph(rng, n, p):
    edges = [(i, j) for i in range(n) for j in range(i + 1, n) if rng.random() < p]
    return csr_from_edges(n, edges)


def dense_P(rowptr, col):
    """P = D~^{-1/2} (A + I) D~^{-1/2} as a dense float64 matrix."""
    n = rowptr.shape[0] - 1
    A = np.zeros((n, n))
    for v in range(n):
        A[v, col[rowptr[v]:rowptr[v + 1]]] = 1.0
    A = A + np.eye(n)
    dt = A.sum(1)
    return A / np.sqrt(np.outer(dt, dt))


def dense_gcn_forward(Pm, X, W, b):
    """H^(l) for l = 1..L: ReLU on hidden layers, none on the last."""
    H = np.asarray(X, dtype=np.float64)
    Hs, Zs = [], []
    L = len(W)
    for l in range(L):
        Z = Pm @ H @ np.asarray(W[l], dtype=np.float64) + np.asarray(b[l], dtype=np.float64)
        H = np.maximum(Z, 0.0) if l < L - 1 else Z
        Zs.append(Z)
        Hs.append(H)
    return Hs, Zs


def mean_ce(Z, y):
    Z = Z - Z.max(1, keepdims=True)
    lse = np.log(np.exp(Z).sum(1))
    return float(np.mean(lse - Z[np.arange(Z.shape[0]), y]))
