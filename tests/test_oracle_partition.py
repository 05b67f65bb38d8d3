"""Pins for the oracle's integer structures (partition lists, halo sets, cache slots)."""
import numpy as np
import pytest

from oracle import sat_ref as orc
from tests.dense_pins import csr_from_edges, random_graph


def _rows(rowptr, col):
    return [list(map(int, col[rowptr[i]:rowptr[i + 1]])) for i in range(rowptr.shape[0] - 1)]


def test_five_node_structures(five_node):
    g = five_node
    rowptr, col = csr_from_edges(5, g["edges"])
    dtil, dinv = orc.degrees(rowptr)
    assert dtil.tolist() == g["dtil"]
    np.testing.assert_allclose(dinv, 1.0 / np.sqrt(np.array(g["dtil"], dtype=np.float64)), rtol=1e-7)
    P = orc.build_partition(rowptr, col, np.array(g["part"], dtype=np.int32), 2)
    assert [x.tolist() for x in P.inner_gid] == g["inner"]
    assert [x.tolist() for x in P.halo_gid] == g["halo"]
    assert P.slot.tolist() == g["slot"] and P.n_slots == len(g["C"])
    assert [x.tolist() for x in P.halo_slot] == g["halo_slot"]
    assert [x.tolist() for x in P.push_local] == g["push_local"]
    assert [x.tolist() for x in P.push_slot] == g["push_slot"]
    for m in range(2):
        assert _rows(P.loc_rowptr[m], P.loc_col[m]) == g["loc_rows"][m]
        assert _rows(P.hrow_ptr[m], P.hrow_col[m]) == g["hrow"][m]


@pytest.mark.parametrize("seed,n,p,M", [(1, 23, 0.2, 3), (2, 40, 0.1, 5), (3, 17, 0.5, 4), (4, 30, 0.03, 2)])
def test_partition_brute_force(seed, n, p, M):
    """Every list against the set definitions, on graphs small enough for Python sets."""
    rng = np.random.default_rng(seed)
    rowptr, col = random_graph(rng, n, p)
    part = rng.integers(0, M, size=n).astype(np.int32)
    P = orc.build_partition(rowptr, col, part, M)
    nbr = [set(map(int, col[rowptr[v]:rowptr[v + 1]])) for v in range(n)]
    C = set()
    for m in range(M):
        V = [v for v in range(n) if part[v] == m]
        B = sorted({u for v in V for u in nbr[v] if part[u] != m})
        C |= set(B)
        assert P.inner_gid[m].tolist() == V
        assert P.halo_gid[m].tolist() == B
        assert not (set(V) & set(B))
        local = {v: i for i, v in enumerate(V)}
        local.update({u: len(V) + j for j, u in enumerate(B)})
        rows = _rows(P.loc_rowptr[m], P.loc_col[m])
        for i, v in enumerate(V):
            assert rows[i] == sorted(local[u] for u in (nbr[v] | {v}))
            assert i in rows[i]                                   # self-loop present
        hrows = _rows(P.hrow_ptr[m], P.hrow_col[m])
        for j, u in enumerate(B):
            assert hrows[j] == sorted(local[v] for v in nbr[u] if part[v] == m)
    Cs = sorted(C)
    # undirected graph: C is exactly the set of nodes touching a cut edge
    assert Cs == [v for v in range(n) if any(part[u] != part[v] for u in nbr[v])]
    assert P.n_slots == len(Cs)
    assert [int(P.slot[v]) for v in Cs] == list(range(len(Cs)))
    assert all(P.slot[v] == -1 for v in range(n) if v not in C)
    tot_push = 0
    for m in range(M):
        V = P.inner_gid[m]
        assert P.halo_slot[m].tolist() == [int(P.slot[u]) for u in P.halo_gid[m]]
        assert P.push_local[m].tolist() == [i for i, v in enumerate(V) if v in C]
        assert P.push_slot[m].tolist() == [int(P.slot[V[i]]) for i in P.push_local[m]]
        tot_push += len(P.push_local[m])
    assert tot_push == len(Cs)
    assert sum(int(p[-1]) for p in P.loc_rowptr) == col.shape[0] + n


def test_partition_invariants_on_tiny_workload():
    from sat_synth import make_workload
    wl = make_workload("tiny", with_dense=False)
    P = orc.build_partition(wl.rowptr, wl.col, wl.part_given, wl.M)
    assert sum(x.shape[0] for x in P.inner_gid) == wl.n
    assert np.array_equal(np.sort(np.concatenate(P.inner_gid)), np.arange(wl.n))
    assert sum(int(p[-1]) for p in P.loc_rowptr) == wl.nnz
    assert sum(x.shape[0] for x in P.push_local) == P.n_slots
    # inner neighbours of a halo node are themselves boundary nodes (lets the predictor
    # run from a boundary-only cache)
    for m in range(wl.M):
        assert np.all(P.slot[P.inner_gid[m][P.hrow_col[m]]] >= 0)


def test_contig_blocks():
    part = orc.contig_blocks(10, 3)
    assert part.tolist() == [0, 0, 0, 0, 1, 1, 1, 2, 2, 2]
    part = orc.contig_blocks(2_449_029, 32)
    assert part[0] == 0 and part[-1] == 31 and np.all(np.diff(part) >= 0)
    cnt = np.bincount(part)
    assert cnt.max() - cnt.min() <= 1


# ------------------------------------------------------------------------------------------
# breadth-first block partitioner
# ------------------------------------------------------------------------------------------
def test_bfs_blocks_five_node(five_node):
    """Hand-worked: from node 0 the queue visits 0, 1, then 1's unvisited neighbours 2, 3 in ascending id, then 4: the visit
    order is the id order, and two blocks of it are the example's partition (0, 0, 0, 1, 1)."""
    from tests.dense_pins import csr_from_edges
    rowptr, col = csr_from_edges(5, five_node["edges"])
    assert orc.bfs_rank(rowptr, col).tolist() == [0, 1, 2, 3, 4]
    assert orc.bfs_blocks(rowptr, col, 2).tolist() == five_node["part"]
    # a star seen from a leaf: 0 - 3, 3 - {1, 2, 4}: visit order 0, 3, 1, 2, 4
    rowptr, col = csr_from_edges(5, [[0, 3], [3, 1], [3, 2], [3, 4]])
    assert orc.bfs_rank(rowptr, col).tolist() == [0, 2, 3, 1, 4]


def _queue_bfs(rowptr, col):
    from collections import deque
    n = rowptr.shape[0] - 1
    rank = [-1] * n
    k = 0
    for s in range(n):
        if rank[s] >= 0:
            continue
        rank[s] = k
        k += 1
        q = deque([s])
        while q:
            u = q.popleft()
            for w in sorted(col[rowptr[u]:rowptr[u + 1]].tolist()):
                if rank[w] < 0:
                    rank[w] = k
                    k += 1
                    q.append(w)
    return rank


@pytest.mark.parametrize("seed,n,p", [(0, 40, 0.08), (1, 60, 0.02), (2, 25, 0.0), (3, 80, 0.05)])
def test_bfs_rank_against_a_queue_and_the_library_traversal(seed, n, p):
    """Random graphs, most of them disconnected (restarts at the smallest unvisited id): a deque written out in Python; on the
    component of node 0, scipy's breadth-first order (which also walks the sorted CSR rows); and the invariants of a
    breadth-first order (a bijection; every non-root node has a neighbour with a smaller rank inside its component)."""
    import scipy.sparse as sp
    from scipy.sparse.csgraph import breadth_first_order
    from tests.dense_pins import random_graph
    rng = np.random.default_rng(seed)
    rowptr, col = random_graph(rng, n, p)
    rank = orc.bfs_rank(rowptr, col)
    assert rank.tolist() == _queue_bfs(rowptr, col)
    assert sorted(rank.tolist()) == list(range(n))
    A = sp.csr_matrix((np.ones(col.shape[0], dtype=np.int8), col, rowptr), shape=(n, n))
    first = breadth_first_order(A, 0, directed=False, return_predecessors=False)
    assert rank[first].tolist() == list(range(first.shape[0]))
    part = orc.bfs_blocks(rowptr, col, 4)
    assert np.array_equal(part, (rank.astype(np.int64) * 4 // n).astype(np.int32))
    assert np.bincount(part, minlength=4).max() - np.bincount(part, minlength=4).min() <= 1
