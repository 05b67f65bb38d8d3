"""Pins for the oracle's layer forward / backward / loss / epoch (CPU only)."""
import numpy as np
import pytest
import torch

from oracle import sat_ref as orc
from tests.dense_pins import csr_from_edges, dense_P, dense_gcn_forward, mean_ce, random_graph


def _five(g):
    rowptr, col = csr_from_edges(5, g["edges"])
    dtil, _ = orc.degrees(rowptr)
    X = np.array(g["X"], dtype=np.float32)
    W = [np.array(g["W1"], dtype=np.float32), np.array(g["W2"], dtype=np.float32)]
    b = [np.array(g["b1"], dtype=np.float32), np.array(g["b2"], dtype=np.float32)]
    y = np.array(g["labels"], dtype=np.int32)
    return rowptr, col, dtil, X, W, b, y


def test_five_node_full_graph_numbers(five_node):
    g = five_node
    rowptr, col, dtil, X, W, b, y = _five(g)
    P1 = orc.build_partition(rowptr, col, np.zeros(5, dtype=np.int32), 1)
    cache = orc.CacheRing(P1.n_slots, [2], 2)
    res = orc.run_epoch(P1, dtil, cache, X, y, W, b, None, "ce")
    rec = res.per_part[0]
    # P X is the aggregation of layer 1
    np.testing.assert_allclose(rec["AGG"][0], np.array(g["PX"]), atol=2e-6)
    np.testing.assert_allclose(rec["Z"][0], np.array(g["Z1"]), atol=2e-6)
    np.testing.assert_allclose(rec["Z"][1], np.array(g["Z2_exact"]), atol=2e-6)
    assert abs(res.loss - g["loss_full"]) < 2e-6
    np.testing.assert_allclose(res.G_W[1], np.array(g["G_W2"]), atol=2e-6)
    np.testing.assert_allclose(res.G_W[0], np.array(g["G_W1_full"]), atol=2e-6)
    np.testing.assert_allclose(res.G_b[0], np.array(g["G_b1_full"]), atol=2e-6)
    # the printed P entries
    Pm = dense_P(rowptr, col)
    for key, val in g["P_nonzeros"].items():
        i, j = map(int, key.split(","))
        assert abs(Pm[i, j] - val) < 1e-6 and abs(Pm[j, i] - val) < 1e-6


def test_five_node_first_sat_epoch(five_node):
    """Cache all zeros, identity predictor: halo input of layer 2 is zero."""
    g = five_node
    rowptr, col, dtil, X, W, b, y = _five(g)
    P = orc.build_partition(rowptr, col, np.array(g["part"], dtype=np.int32), 2)
    cache = orc.CacheRing(P.n_slots, [2], 2)
    res = orc.run_epoch(P, dtil, cache, X, y, W, b, None, "ce")
    Z2 = np.zeros((5, 2))
    for m in range(2):
        Z2[P.inner_gid[m]] = res.per_part[m]["Z"][1]
    np.testing.assert_allclose(Z2, np.array(g["Z2_first_epoch"]), atol=2e-6)
    # what was pushed is the newest snapshot after the commit
    H1 = np.maximum(np.array(g["Z1"]), 0.0)
    np.testing.assert_allclose(cache.newest(1), H1[np.array(g["C"])], atol=2e-6)
    assert cache.n_valid == 1


def test_five_node_exact_cache_halo_constant_gradient(five_node):
    """Exact halo values in the cache: forward equals the full graph, G_W2 too; G_W1 is
    the halo-as-constant value, and adding the halo gradient back restores the full one."""
    g = five_node
    rowptr, col, dtil, X, W, b, y = _five(g)
    P = orc.build_partition(rowptr, col, np.array(g["part"], dtype=np.int32), 2)
    H1 = np.maximum(np.array(g["Z1"]), 0.0).astype(np.float32)
    cache = orc.CacheRing(P.n_slots, [2], 2)
    cache.push(1, np.arange(3), H1[np.array(g["C"])])
    cache.commit()
    res = orc.run_epoch(P, dtil, cache, X, y, W, b, None, "ce", want_halo_grad=True)
    Z2 = np.zeros((5, 2))
    for m in range(2):
        Z2[P.inner_gid[m]] = res.per_part[m]["Z"][1]
    np.testing.assert_allclose(Z2, np.array(g["Z2_exact"]), atol=3e-6)
    np.testing.assert_allclose(res.G_W[1], np.array(g["G_W2"]), atol=2e-6)
    np.testing.assert_allclose(res.G_W[0], np.array(g["G_W1_halo_constant"]), atol=2e-6)
    # scatter the halo gradients of layer 2's input back to the owners and redo layer 1's G_W
    G1 = np.zeros((5, 2))
    for m in range(2):
        G1[P.inner_gid[m]] += res.per_part[m]["G_in"][1]
        G1[P.halo_gid[m]] += res.per_part[m]["G_halo"][1]
    Pm = dense_P(rowptr, col)
    D1 = G1 * (np.array(g["Z1"]) > 0)
    np.testing.assert_allclose((Pm @ X).T @ D1, np.array(g["G_W1_full"]), atol=3e-6)


@pytest.mark.parametrize("seed,n,p,M,dims", [(0, 48, 0.12, 4, [5, 7, 3]), (1, 64, 0.06, 3, [4, 6, 5, 3]), (2, 20, 0.4, 5, [3, 3])])
def test_dense_brute_force_and_partition_equivalence(seed, n, p, M, dims):
    """sigma(P X W + b) with a dense P equals (a) the oracle on the unpartitioned graph and
    (b) the oracle's partitioned layers when the halo input is exact (P = P_in + P_out)."""
    rng = np.random.default_rng(seed)
    rowptr, col = random_graph(rng, n, p)
    dtil, _ = orc.degrees(rowptr)
    X = rng.standard_normal((n, dims[0])).astype(np.float32)
    W = [rng.standard_normal((dims[i], dims[i + 1])).astype(np.float32) * 0.5 for i in range(len(dims) - 1)]
    b = [rng.standard_normal(dims[i + 1]).astype(np.float32) * 0.1 for i in range(len(dims) - 1)]
    Pm = dense_P(rowptr, col)
    Hs, Zs = dense_gcn_forward(Pm, X, W, b)
    part = rng.integers(0, M, size=n).astype(np.int32)
    P = orc.build_partition(rowptr, col, part, M)
    L = len(W)
    H_prev = X.astype(np.float64)
    for l in range(1, L + 1):
        H_l = np.zeros((n, dims[l]))
        for m in range(M):
            inner, halo = P.inner_gid[m], P.halo_gid[m]
            AGG, Z, H = orc.layer_fwd(P, m, dtil, H_prev[inner], H_prev[halo], W[l - 1], b[l - 1], 1 if l < L else 0)
            np.testing.assert_allclose(AGG, (Pm @ H_prev)[inner], atol=1e-5)
            np.testing.assert_allclose(Z, Zs[l - 1][inner], atol=1e-5)
            H_l[inner] = H
        np.testing.assert_allclose(H_l, Hs[l - 1], atol=1e-5)
        H_prev = Hs[l - 1].astype(np.float32).astype(np.float64)


def _torch_dense_loss(Pm, X, W, b, y, kind):
    Pm = torch.tensor(Pm, dtype=torch.float64)
    H = torch.tensor(X, dtype=torch.float64)
    Wt = [torch.tensor(w, dtype=torch.float64, requires_grad=True) for w in W]
    bt = [torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in b]
    for l in range(len(W)):
        Z = Pm @ H @ Wt[l] + bt[l]
        H = torch.relu(Z) if l < len(W) - 1 else Z
    if kind == "ce":
        loss = torch.nn.functional.cross_entropy(H, torch.tensor(y, dtype=torch.long))
    else:
        loss = torch.nn.functional.binary_cross_entropy_with_logits(H, torch.tensor(y, dtype=torch.float64))
    loss.backward()
    return float(loss), [w.grad.numpy() for w in Wt], [x.grad.numpy() for x in bt]


@pytest.mark.parametrize("kind", ["ce", "bce"])
def test_backward_matches_autograd_of_dense_formulation(kind):
    """Unpartitioned oracle epoch vs library autograd on the dense formulation (fp64)."""
    rng = np.random.default_rng(5)
    n, dims = 40, [6, 8, 7, 4]
    rowptr, col = random_graph(rng, n, 0.15)
    dtil, _ = orc.degrees(rowptr)
    X = rng.standard_normal((n, dims[0])).astype(np.float32)
    W = [(rng.standard_normal((dims[i], dims[i + 1])) * 0.6).astype(np.float32) for i in range(3)]
    b = [(rng.standard_normal(dims[i + 1]) * 0.2).astype(np.float32) for i in range(3)]
    y = rng.integers(0, dims[-1], size=n).astype(np.int32) if kind == "ce" else (rng.random((n, dims[-1])) < 0.3).astype(np.uint8)
    P1 = orc.build_partition(rowptr, col, np.zeros(n, dtype=np.int32), 1)
    cache = orc.CacheRing(0, [dims[1], dims[2]], 2)
    res = orc.run_epoch(P1, dtil, cache, X, y, W, b, None, kind)
    loss, gW, gb = _torch_dense_loss(dense_P(rowptr, col), X, W, b, y, kind)
    assert abs(res.loss - loss) < 1e-6
    for l in range(3):
        # layer outputs pass through fp32 between layers in the method; tolerance covers that
        np.testing.assert_allclose(res.G_W[l], gW[l], atol=2e-6)
        np.testing.assert_allclose(res.G_b[l], gb[l], atol=2e-6)


def test_partitioned_gradients_with_halo_gradient_equal_full_graph():
    """Layer-synchronous exact halo inputs + halo gradients scattered back to their owners
    reproduce the full-graph gradient of every layer; without them only the last layer's."""
    rng = np.random.default_rng(11)
    n, M, dims = 36, 3, [5, 6, 4]
    rowptr, col = random_graph(rng, n, 0.15)
    dtil, _ = orc.degrees(rowptr)
    X = rng.standard_normal((n, dims[0])).astype(np.float32)
    W = [(rng.standard_normal((dims[i], dims[i + 1])) * 0.6).astype(np.float32) for i in range(2)]
    b = [np.zeros(dims[i + 1], dtype=np.float32) for i in range(2)]
    y = rng.integers(0, dims[-1], size=n).astype(np.int32)
    part = rng.integers(0, M, size=n).astype(np.int32)
    P = orc.build_partition(rowptr, col, part, M)
    Pm = dense_P(rowptr, col)
    Hs, Zs = dense_gcn_forward(Pm, X, W, b)
    H1 = Hs[0].astype(np.float32)
    loss, gW, gb = _torch_dense_loss(Pm, X, W, b, y, "ce")
    GW = [np.zeros(w.shape) for w in W]
    Gb = [np.zeros(w.shape[1]) for w in W]
    G1 = np.zeros((n, dims[1]))
    saved = []
    for m in range(M):
        inner, halo = P.inner_gid[m], P.halo_gid[m]
        AGG1, Z1, H1m = orc.layer_fwd(P, m, dtil, X[inner], X[halo], W[0], b[0], 1)
        AGG2, Z2, H2m = orc.layer_fwd(P, m, dtil, H1[inner], H1[halo], W[1], b[1], 0)
        _, G = orc.loss_grad("ce", H2m, y[inner], 1.0 / n)
        gin, ghalo = orc.layer_bwd(P, m, dtil, G, None, AGG2, W[1], GW[1], Gb[1], want_in=True, want_halo=True)
        G1[inner] += gin
        G1[halo] += ghalo
        saved.append((AGG1, Z1))
    np.testing.assert_allclose(GW[1], gW[1], atol=2e-6)
    np.testing.assert_allclose(Gb[1], gb[1], atol=2e-6)
    for m in range(M):
        inner = P.inner_gid[m]
        AGG1, Z1 = saved[m]
        orc.layer_bwd(P, m, dtil, G1[inner].astype(np.float32), (Z1 > 0).astype(np.uint8), AGG1, W[0], GW[0], Gb[0],
                      want_in=False)
    np.testing.assert_allclose(GW[0], gW[0], atol=2e-6)
    np.testing.assert_allclose(Gb[0], gb[0], atol=2e-6)


def test_backward_finite_differences():
    """Central differences of the oracle's own epoch loss w.r.t. W (halo treated as constant:
    the cache is fixed, so the partitioned loss is a plain function of W)."""
    rng = np.random.default_rng(21)
    n, M, dims = 30, 3, [4, 5, 3]
    rowptr, col = random_graph(rng, n, 0.2)
    dtil, _ = orc.degrees(rowptr)
    X = rng.standard_normal((n, dims[0])).astype(np.float32)
    W = [(rng.standard_normal((dims[i], dims[i + 1])) * 0.7).astype(np.float32) for i in range(2)]
    b = [(rng.standard_normal(dims[i + 1]) * 0.3).astype(np.float32) for i in range(2)]
    y = rng.integers(0, dims[-1], size=n).astype(np.int32)
    part = rng.integers(0, M, size=n).astype(np.int32)
    P = orc.build_partition(rowptr, col, part, M)

    def fresh_cache():
        c = orc.CacheRing(P.n_slots, [dims[1]], 2)
        r = np.random.default_rng(3)
        c.push(1, np.arange(P.n_slots), np.abs(r.standard_normal((P.n_slots, dims[1]))).astype(np.float32))
        c.commit()
        return c

    res = orc.run_epoch(P, dtil, fresh_cache(), X, y, W, b, None, "ce")
    eps = 1e-3
    for l in range(2):
        for (i, j) in [(0, 0), (1, 2), (dims[l] - 1, dims[l + 1] - 1)]:
            Wp = [w.copy() for w in W]
            Wm = [w.copy() for w in W]
            Wp[l][i, j] += eps
            Wm[l][i, j] -= eps
            step = float(Wp[l][i, j]) - float(Wm[l][i, j])
            lp = orc.run_epoch(P, dtil, fresh_cache(), X, y, Wp, b, None, "ce").loss
            lm = orc.run_epoch(P, dtil, fresh_cache(), X, y, Wm, b, None, "ce").loss
            assert abs((lp - lm) / step - res.G_W[l][i, j]) < 2e-4
        bp = [x.copy() for x in b]
        bm = [x.copy() for x in b]
        bp[l][1] += eps
        bm[l][1] -= eps
        step = float(bp[l][1]) - float(bm[l][1])
        lp = orc.run_epoch(P, dtil, fresh_cache(), X, y, W, bp, None, "ce").loss
        lm = orc.run_epoch(P, dtil, fresh_cache(), X, y, W, bm, None, "ce").loss
        assert abs((lp - lm) / step - res.G_b[l][1]) < 2e-4


def test_loss_closed_forms():
    n, c = 7, 5
    Z = np.zeros((n, c), dtype=np.float32)
    y = np.arange(n, dtype=np.int32) % c
    val, G = orc.loss_grad("ce", Z, y, 1.0 / n)
    assert abs(val - np.log(c)) < 1e-12
    np.testing.assert_allclose(G.sum(1), 0.0, atol=1e-8)
    Y = (np.arange(n * c).reshape(n, c) % 3 == 0).astype(np.uint8)
    val, G = orc.loss_grad("bce", Z, Y, 1.0 / n)
    assert abs(val - np.log(2.0)) < 1e-12
    np.testing.assert_allclose(G, (0.5 - Y) / (n * c), atol=1e-9)
    # against the library losses on random logits
    rng = np.random.default_rng(0)
    Z = (rng.standard_normal((n, c)) * 3).astype(np.float32)
    val, G = orc.loss_grad("ce", Z, y, 1.0 / n)
    zt = torch.tensor(Z, dtype=torch.float64, requires_grad=True)
    lt = torch.nn.functional.cross_entropy(zt, torch.tensor(y, dtype=torch.long))
    lt.backward()
    assert abs(val - float(lt)) < 1e-9
    np.testing.assert_allclose(G, zt.grad.numpy(), atol=1e-8)
    assert abs(val - mean_ce(Z.astype(np.float64), y)) < 1e-9
    val, G = orc.loss_grad("bce", Z, Y, 1.0 / n)
    zt = torch.tensor(Z, dtype=torch.float64, requires_grad=True)
    lt = torch.nn.functional.binary_cross_entropy_with_logits(zt, torch.tensor(Y, dtype=torch.float64))
    lt.backward()
    assert abs(val - float(lt)) < 1e-9
    np.testing.assert_allclose(G, zt.grad.numpy(), atol=1e-8)


def test_epoch_is_partition_order_invariant():
    from sat_synth import make_workload
    wl = make_workload("tiny")
    dtil, _ = orc.degrees(wl.rowptr)
    P = orc.build_partition(wl.rowptr, wl.col, wl.part_given, wl.M)
    outs = []
    for order in ([0, 1, 2, 3], [3, 1, 0, 2]):
        cache = orc.CacheRing(P.n_slots, wl.dims[1:-1], wl.tau)
        for _ in range(3):
            res = orc.run_epoch(P, dtil, cache, wl.X, wl.labels, wl.W, wl.b, wl.pred, "ce", order=order)
        outs.append((res, cache))
    (r0, c0), (r1, c1) = outs
    assert np.array_equal(c0.buf[0], c1.buf[0]) and c0.write_idx == c1.write_idx
    for m in range(wl.M):
        assert np.array_equal(r0.per_part[m]["H"][-1], r1.per_part[m]["H"][-1])
    np.testing.assert_allclose(r0.G_W[0], r1.G_W[0], rtol=1e-12, atol=1e-15)
    assert abs(r0.loss - r1.loss) < 1e-12


def test_staleness_norm_closed_forms():
    """Eq. "staleness def": zero for identical embeddings, |c| sqrt(b_m d) for a constant offset, absolutely homogeneous,
    and equal to the library Frobenius norm of the explicitly gathered difference."""
    rng = np.random.default_rng(11)
    rowptr, col = random_graph(rng, 60, 0.12)
    part = rng.integers(0, 3, size=60).astype(np.int32)
    P = orc.build_partition(rowptr, col, part, 3)
    H = rng.normal(size=(60, 9)).astype(np.float32)
    for m in range(3):
        halo = P.halo_gid[m]
        assert orc.staleness(P, m, H, H[halo]) == 0.0
        used = (H[halo].astype(np.float64) + 0.25).astype(np.float32)
        want = np.linalg.norm(H[halo].astype(np.float64) - used.astype(np.float64), "fro")
        assert abs(orc.staleness(P, m, H, used) - want) <= 1e-12 * max(want, 1.0)
        other = rng.normal(size=(halo.shape[0], 9)).astype(np.float32)
        a = orc.staleness(P, m, H, other)
        assert abs(a - np.linalg.norm(H[halo].astype(np.float64) - other.astype(np.float64))) <= 1e-12 * max(a, 1.0)
        # constant offset on exactly representable values
        Hq = np.round(H * 8) / 8
        assert abs(orc.staleness(P, m, Hq, Hq[halo] + np.float32(0.5)) - 0.5 * np.sqrt(halo.shape[0] * 9)) <= 1e-12 * (1 + halo.shape[0])
        # a permutation of the halo rows changes the value unless the rows agree: the halo order matters
        if halo.shape[0] > 1:
            rolled = np.roll(H[halo], 1, axis=0)
            assert orc.staleness(P, m, H, rolled) > 0.0


def test_epoch_restricted_to_some_partitions_equals_the_full_epoch():
    """run_epoch(parts=...) computes the recurrent state only for the cache slots the selected partitions read; what it
    returns for them (predicted halo, every layer output, the gradients handed down, the state rows) must be the
    bits of the unrestricted epoch, and it must not commit the ring."""
    rng = np.random.default_rng(31)
    n, M, dims, tau, h = 60, 4, [6, 5, 7, 3], 3, 4
    rowptr, col = random_graph(rng, n, 0.1)
    dtil, _ = orc.degrees(rowptr)
    part = rng.integers(0, M, size=n).astype(np.int32)
    P = orc.build_partition(rowptr, col, part, M)
    X = rng.standard_normal((n, dims[0])).astype(np.float32)
    y = rng.integers(0, dims[-1], size=n).astype(np.int32)
    W = [rng.standard_normal((dims[i], dims[i + 1])).astype(np.float32) * 0.5 for i in range(3)]
    b = [rng.standard_normal(dims[i + 1]).astype(np.float32) * 0.1 for i in range(3)]
    pred = []
    for l in (1, 2):
        d = dims[l]
        pred.append(dict(Wx=rng.standard_normal((d, 4 * h)).astype(np.float32) * 0.4, Uh=rng.standard_normal((h, 4 * h)).astype(np.float32) * 0.4,
                         b=rng.standard_normal(4 * h).astype(np.float32) * 0.1, Wg=rng.standard_normal((h, d)).astype(np.float32) * 0.4,
                         bg=rng.standard_normal(d).astype(np.float32) * 0.1))

    def filled_ring():
        r = np.random.default_rng(77)
        c = orc.CacheRing(P.n_slots, dims[1:-1], tau)
        for _ in range(2):
            for l in (1, 2):
                c.push(l, np.arange(P.n_slots), r.standard_normal((P.n_slots, dims[l])).astype(np.float32))
            c.commit()
        return c

    full = orc.run_epoch(P, dtil, filled_ring(), X, y, W, b, pred, "ce")
    sel = [2, 0]
    ring = filled_ring()
    some = orc.run_epoch(P, dtil, ring, X, y, W, b, pred, "ce", parts=sel)
    assert ring.n_valid == 2 and ring.write_idx == 2          # not committed
    assert some.S_slots is not None and some.S_slots.shape[0] < P.n_slots
    for l in range(2):
        assert np.array_equal(some.S[l][some.S_slots], full.S[l][some.S_slots])
    for m in range(M):
        if m not in sel:
            assert some.per_part[m] is None
            continue
        for key in ("H", "halo", "Z", "AGG"):
            for got, want in zip(some.per_part[m][key], full.per_part[m][key]):
                assert np.array_equal(got, want), (m, key)
        for got, want in zip(some.per_part[m]["G_in"][1:], full.per_part[m]["G_in"][1:]):
            assert np.array_equal(got, want)
    # the gradients it returns are the sum over the selected partitions only
    only = [np.zeros_like(g) for g in full.G_W]
    for m in sel:
        one = orc.run_epoch(P, dtil, filled_ring(), X, y, W, b, pred, "ce", parts=[m])
        for l in range(3):
            only[l] += one.G_W[l]
    for l in range(3):
        np.testing.assert_allclose(some.G_W[l], only[l], rtol=1e-12, atol=1e-15)
