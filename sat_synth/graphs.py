"""Seeded synthetic graphs: stochastic block model and R-MAT, plus a BFS relabelling.

All graphs are returned as a symmetric CSR (rowptr int64 [n+1], col int32 [nnz]) of a
simple undirected graph: both directions of every edge are stored, columns are sorted
ascending inside each row, there are no self-loops and no duplicates.
"""
from __future__ import annotations

import numpy as np
import scipy.sparse as sp
from scipy.sparse.csgraph import breadth_first_order

from .tensors import stream_rng


def csr_from_undirected_pairs(n: int, lo: np.ndarray, hi: np.ndarray):
    """Symmetric CSR from unique unordered pairs (lo[i] != hi[i])."""
    lo = np.asarray(lo, dtype=np.int64)
    hi = np.asarray(hi, dtype=np.int64)
    keys = np.concatenate([lo * n + hi, hi * n + lo])
    keys.sort(kind="stable")
    rows = keys // n
    col = (keys - rows * n).astype(np.int32)
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(np.bincount(rows, minlength=n), out=rowptr[1:])
    return rowptr, col


def _pairs_from_csr(rowptr: np.ndarray, col: np.ndarray):
    n = rowptr.shape[0] - 1
    rows = np.repeat(np.arange(n, dtype=np.int64), np.diff(rowptr))
    keep = rows < col
    return rows[keep], col[keep].astype(np.int64)


def sbm_graph(seed: int, n: int, n_blocks: int, p_in: float, p_out: float):
    """Stochastic block model with `n_blocks` equal blocks of contiguous ids.

    Every unordered pair {i, j} is an edge independently with probability p_in (same
    block) or p_out (different blocks).  Returns (rowptr, col, block_of_node).
    """
    assert n % n_blocks == 0
    bs = n // n_blocks
    block = (np.arange(n) // bs).astype(np.int32)
    rng = stream_rng(seed, "sbm")
    lo_l, hi_l = [], []
    chunk = max(1, (1 << 22) // n)
    for r0 in range(0, n, chunk):
        r1 = min(n, r0 + chunk)
        u = rng.random((r1 - r0, n), dtype=np.float32)
        same = block[r0:r1, None] == block[None, :]
        thr = np.where(same, np.float32(p_in), np.float32(p_out))
        hit = u < thr
        ii, jj = np.nonzero(hit)
        ii = ii + r0
        keep = ii < jj
        lo_l.append(ii[keep])
        hi_l.append(jj[keep])
    lo = np.concatenate(lo_l)
    hi = np.concatenate(hi_l)
    rowptr, col = csr_from_undirected_pairs(n, lo, hi)
    return rowptr, col, block


def _rmat_endpoints(rng: np.random.Generator, scale: int, count: int, probs):
    """`count` directed R-MAT samples on a 2^scale x 2^scale grid."""
    a, b, c, _d = probs
    row = np.zeros(count, dtype=np.int64)
    colv = np.zeros(count, dtype=np.int64)
    for _level in range(scale):
        u = rng.random(count, dtype=np.float32)
        rbit = u >= np.float32(a + b)
        cbit = ((u >= np.float32(a)) & (u < np.float32(a + b))) | (u >= np.float32(a + b + c))
        row = (row << 1) | rbit
        colv = (colv << 1) | cbit
    return row, colv


def rmat_graph(seed: int, scale: int, n: int, probs=(0.57, 0.19, 0.19, 0.05), *,
               n_samples: int | None = None, n_unique_undirected: int | None = None,
               attach_isolated: bool = True, permute: bool = True):
    """R-MAT graph on `n` <= 2^scale nodes, symmetrised and de-duplicated.

    Exactly one of:
      n_samples            accept this many directed samples (endpoint >= n rejected),
                           then drop self-loops and duplicates;
      n_unique_undirected  keep sampling in rounds until at least this many distinct unordered
                           pairs exist; a surplus is dropped uniformly at random (seeded).
    attach_isolated: every node left without an edge gets one edge to a node drawn from
    the R-MAT row marginal, so the graph has no isolated node (the citation /
    co-purchase graphs this stands in for have none).
    permute: apply a seeded random relabelling so that ids carry no degree information.
    """
    assert (n_samples is None) != (n_unique_undirected is None)
    assert n <= (1 << scale)
    rng = stream_rng(seed, "rmat")

    def draw(count):
        r, c = _rmat_endpoints(rng, scale, count, probs)
        ok = (r < n) & (c < n)
        return r[ok], c[ok]

    if n_samples is not None:
        rs, cs, got = [], [], 0
        while got < n_samples:
            r, c = draw(int((n_samples - got) * 1.3) + 1024)
            take = min(r.shape[0], n_samples - got)
            rs.append(r[:take])
            cs.append(c[:take])
            got += take
        r = np.concatenate(rs)
        c = np.concatenate(cs)
        keep = r != c
        lo = np.minimum(r[keep], c[keep])
        hi = np.maximum(r[keep], c[keep])
        keys = np.unique(lo * n + hi)
    else:
        keys = np.empty(0, dtype=np.int64)
        while keys.shape[0] < n_unique_undirected:
            want = int((n_unique_undirected - keys.shape[0]) * 1.5) + (1 << 16)
            parts = [keys]
            while want > 0:                       # bounded chunks keep the temporaries small
                chunk = min(want, 1 << 25)
                r, c = draw(chunk)
                keep = r != c
                parts.append(np.minimum(r[keep], c[keep]) * n + np.maximum(r[keep], c[keep]))
                want -= chunk
            keys = np.unique(np.concatenate(parts))
        if keys.shape[0] > n_unique_undirected:   # drop the surplus uniformly at random (seeded)
            pick = rng.choice(keys.shape[0], size=n_unique_undirected, replace=False)
            pick.sort()
            keys = keys[pick]
    lo = keys // n
    hi = keys - lo * n

    if attach_isolated:
        deg = np.bincount(lo, minlength=n) + np.bincount(hi, minlength=n)
        iso = np.nonzero(deg == 0)[0]
        if iso.shape[0]:
            partner = np.full(iso.shape[0], -1, dtype=np.int64)
            todo = np.arange(iso.shape[0])
            while todo.shape[0]:
                r, _ = _rmat_endpoints(rng, scale, todo.shape[0], probs)
                good = (r < n) & (r != iso[todo])
                partner[todo[good]] = r[good]
                todo = todo[~good]
            k2 = np.minimum(iso, partner) * n + np.maximum(iso, partner)
            keys = np.union1d(keys, k2)
            lo = keys // n
            hi = keys - lo * n

    if permute:
        perm = stream_rng(seed, "rmat-perm").permutation(n).astype(np.int64)
        lo, hi = perm[lo], perm[hi]
    return csr_from_undirected_pairs(n, lo, hi)


def bfs_relabel(rowptr: np.ndarray, col: np.ndarray):
    """Relabel nodes by breadth-first visit order.

    The search starts at the highest-degree node (smallest id on ties) and visits
    neighbours in ascending id; nodes it cannot reach are appended in ascending id.
    Returns (rowptr, col, new_id_of_old_id).
    """
    n = rowptr.shape[0] - 1
    deg = np.diff(rowptr)
    start = int(np.argmax(deg))
    mat = sp.csr_matrix((np.ones(col.shape[0], dtype=np.int8), col, rowptr.astype(np.int64)), shape=(n, n))
    order = breadth_first_order(mat, i_start=start, directed=True, return_predecessors=False)
    seen = np.zeros(n, dtype=bool)
    seen[order] = True
    order = np.concatenate([order.astype(np.int64), np.nonzero(~seen)[0]])
    new_id = np.empty(n, dtype=np.int64)
    new_id[order] = np.arange(n, dtype=np.int64)
    lo, hi = _pairs_from_csr(rowptr, col)
    a, b = new_id[lo], new_id[hi]
    rp, c = csr_from_undirected_pairs(n, np.minimum(a, b), np.maximum(a, b))
    return rp, c, new_id.astype(np.int32)
