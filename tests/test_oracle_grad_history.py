"""Pins for the oracle's gradient-side history (Appendix, back-propagation of SAT: the term P_out^T D^(t-1) W^T)."""
import numpy as np
import pytest

from oracle import sat_ref as orc
from tests.dense_pins import dense_P, random_graph
from tests.test_oracle_layers import _torch_dense_loss


def _case(seed, n=40, M=3, dims=(5, 7, 6, 4), tau=2):
    rng = np.random.default_rng(seed)
    rowptr, col = random_graph(rng, n, 0.15)
    dtil, _ = orc.degrees(rowptr)
    X = rng.standard_normal((n, dims[0])).astype(np.float32)
    L = len(dims) - 1
    W = [(rng.standard_normal((dims[i], dims[i + 1])) * 0.6).astype(np.float32) for i in range(L)]
    b = [(rng.standard_normal(dims[i + 1]) * 0.1).astype(np.float32) for i in range(L)]
    y = rng.integers(0, dims[-1], size=n).astype(np.int32)
    part = rng.integers(0, M, size=n).astype(np.int32)
    P = orc.build_partition(rowptr, col, part, M)
    return rowptr, col, dtil, X, W, b, y, P, list(dims), tau


@pytest.mark.parametrize("seed,dims", [(3, (5, 7, 4)), (4, (5, 7, 6, 4)), (5, (4, 6, 5, 5, 3))])
def test_frozen_weights_converge_to_the_full_graph_gradient(seed, dims):
    """With the weights frozen the historical embeddings become exact after L - 1 epochs (layer l after l epochs) and the
    gradient history after L - 1 more (the stale D equals the current D), so the partitioned epoch must then reproduce the
    gradient of the unpartitioned graph in EVERY layer; without the history only the last layer's is exact."""
    rowptr, col, dtil, X, W, b, y, P, dims, tau = _case(seed, dims=dims)
    L = len(dims) - 1
    loss, gW, gb = _torch_dense_loss(dense_P(rowptr, col), X, W, b, y, "ce")
    cache = orc.CacheRing(P.n_slots, dims[1:-1], tau)
    hist = orc.GradHistory(P.n_slots, dims[2:])
    for t in range(2 * L):
        res = orc.run_epoch(P, dtil, cache, X, y, W, b, None, "ce", grad_hist=hist)
    assert abs(res.loss - loss) < 1e-6
    for l in range(L):
        np.testing.assert_allclose(res.G_W[l], gW[l], atol=3e-6)
        np.testing.assert_allclose(res.G_b[l], gb[l], atol=3e-6)
    # the same run without the history: the lower layers stay off
    cache = orc.CacheRing(P.n_slots, dims[1:-1], tau)
    for t in range(2 * L):
        res0 = orc.run_epoch(P, dtil, cache, X, y, W, b, None, "ce")
    np.testing.assert_allclose(res0.G_W[L - 1], gW[L - 1], atol=3e-6)
    assert np.abs(res0.G_W[0] - gW[0]).max() > 1e-4


def test_first_epoch_has_no_stale_term_and_single_partition_none_at_all():
    rowptr, col, dtil, X, W, b, y, P, dims, tau = _case(7)
    cache0, cache1 = orc.CacheRing(P.n_slots, dims[1:-1], tau), orc.CacheRing(P.n_slots, dims[1:-1], tau)
    hist = orc.GradHistory(P.n_slots, dims[2:])
    a = orc.run_epoch(P, dtil, cache0, X, y, W, b, None, "ce")
    c = orc.run_epoch(P, dtil, cache1, X, y, W, b, None, "ce", grad_hist=hist)
    for l in range(len(W)):
        assert np.array_equal(a.G_W[l], c.G_W[l])          # nothing to read in the first epoch
    assert all(r is not None and np.abs(r).max() > 0 for r in hist.read)   # but the epoch left its history behind
    # one partition: no halo, no boundary, empty history
    P1 = orc.build_partition(rowptr, col, np.zeros(P.n, dtype=np.int32), 1)
    h1 = orc.GradHistory(P1.n_slots, dims[2:])
    assert P1.n_slots == 0
    cache = orc.CacheRing(0, dims[1:-1], tau)
    r1 = orc.run_epoch(P1, dtil, cache, X, y, W, b, None, "ce", grad_hist=h1)
    r2 = orc.run_epoch(P1, dtil, cache, X, y, W, b, None, "ce", grad_hist=h1)
    for l in range(len(W)):
        assert np.array_equal(r1.G_W[l], r2.G_W[l])


def test_history_rows_are_the_halo_gradients_summed_over_the_using_partitions():
    """Q^(j)[v] = sum over partitions q that hold v as a halo node of (P_out^(q)T D^(q, j))[v], checked against the dense
    statement: with P the full normalised adjacency, Q^(j)[v] = sum_{u ~ v, part(u) != part(v)} P[u, v] D[u]."""
    rowptr, col, dtil, X, W, b, y, P, dims, tau = _case(9)
    cache = orc.CacheRing(P.n_slots, dims[1:-1], tau)
    hist = orc.GradHistory(P.n_slots, dims[2:])
    res = orc.run_epoch(P, dtil, cache, X, y, W, b, None, "ce", grad_hist=hist)
    Pm = dense_P(rowptr, col)
    part = np.empty(P.n, dtype=np.int64)
    for m in range(P.M):
        part[P.inner_gid[m]] = m
    cross = Pm * (part[:, None] != part[None, :])
    L = len(W)
    for j in range(2, L + 1):
        D = np.zeros((P.n, dims[j]))
        for m in range(P.M):
            G = res.per_part[m]["G_L"] if j == L else res.per_part[m]["G_in"][j]      # gradient w.r.t. H^(j)
            Z = res.per_part[m]["Z"][j - 1]
            D[P.inner_gid[m]] = G if j == L else G * (Z > 0)
        want = cross.T @ D
        boundary = np.flatnonzero(P.slot >= 0)
        np.testing.assert_allclose(hist.read[j - 2][P.slot[boundary]], want[boundary], atol=2e-6)
