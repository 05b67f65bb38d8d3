"""Pins for the oracle's graph-attention layer (forward and backward) on partitioned graphs."""
import numpy as np
import pytest
import torch

from oracle import sat_ref as orc
from tests.dense_pins import csr_from_edges, random_graph


def _dense_gat(adj, H, W, a_src, a_dst, bias, act):
    """The layer written with a dense masked attention matrix in torch (float64): rows attend over adj[v] != 0."""
    Z = H @ W
    pre = (Z @ a_dst)[:, None] + (Z @ a_src)[None, :]
    e = torch.nn.functional.leaky_relu(pre, 0.2)
    e = e.masked_fill(~adj, float("-inf"))
    A = torch.softmax(e, dim=1)
    O = A @ Z + bias
    return torch.relu(O) if act else O


def _case(seed, n=30, M=3, d_in=5, d_out=4):
    rng = np.random.default_rng(seed)
    rowptr, col = random_graph(rng, n, 0.15)
    part = rng.integers(0, M, size=n).astype(np.int32)
    P = orc.build_partition(rowptr, col, part, M)
    H = rng.standard_normal((n, d_in))
    W = rng.standard_normal((d_in, d_out)) * 0.6
    a_src, a_dst = rng.standard_normal(d_out) * 0.7, rng.standard_normal(d_out) * 0.7
    bias = rng.standard_normal(d_out) * 0.2
    G = rng.standard_normal((n, d_out))
    adj = np.eye(n, dtype=bool)
    for v in range(n):
        adj[v, col[rowptr[v]:rowptr[v + 1]]] = True
    return rowptr, col, P, H, W, a_src, a_dst, bias, G, adj


@pytest.mark.parametrize("seed,act,M", [(1, 1, 3), (2, 0, 3), (3, 1, 1), (4, 1, 5)])
def test_forward_and_backward_against_autograd_of_the_dense_layer(seed, act, M):
    """With exact out-of-subgraph inputs the partitioned layer is the full-graph layer: outputs per partition equal the dense
    masked-softmax formulation, and the parameter gradients summed over the partitions equal autograd's (the inputs'
    gradient only receives the in-partition paths, so it is compared on a single partition)."""
    rowptr, col, P, H, W, a_src, a_dst, bias, G, adj = _case(seed, M=M)
    t = lambda a, g=False: torch.tensor(a, dtype=torch.float64, requires_grad=g)
    Ht, Wt, ast, adt, bt = t(H, True), t(W, True), t(a_src, True), t(a_dst, True), t(bias, True)
    out = _dense_gat(torch.tensor(adj), Ht, Wt, ast, adt, bt, act)
    (out * t(G)).sum().backward()
    gW, gas, gad, gb = np.zeros_like(W), np.zeros_like(a_src), np.zeros_like(a_dst), np.zeros_like(bias)
    for m in range(P.M):
        inner, halo = P.inner_gid[m], P.halo_gid[m]
        if inner.shape[0] == 0:
            continue
        f = orc.gat_fwd(P, m, H[inner], H[halo], W, a_src, a_dst, bias, act)
        np.testing.assert_allclose(f["H"], out.detach().numpy()[inner], atol=2e-6)
        # rows of alpha sum to one
        rows, _ = orc._gat_rows(P, m)
        s = np.zeros(inner.shape[0])
        np.add.at(s, rows, f["alpha"])
        np.testing.assert_allclose(s, 1.0, atol=1e-12)
        g = orc.gat_bwd(P, m, H[inner], H[halo], W, a_src, a_dst, f, G[inner], act)
        gW += g["W"]
        gas += g["a_src"]
        gad += g["a_dst"]
        gb += g["b"]
        if P.M == 1:
            np.testing.assert_allclose(g["H_in"], Ht.grad.numpy(), atol=1e-10)
    np.testing.assert_allclose(gW, Wt.grad.numpy(), atol=1e-10)
    np.testing.assert_allclose(gas, ast.grad.numpy(), atol=1e-10)
    np.testing.assert_allclose(gad, adt.grad.numpy(), atol=1e-10)
    np.testing.assert_allclose(gb, bt.grad.numpy(), atol=1e-10)


def test_input_gradient_by_finite_differences_with_constant_halo():
    """The gradient with respect to the inner rows with the halo rows held constant (the method's reading)."""
    rowptr, col, P, H, W, a_src, a_dst, bias, G, adj = _case(7, n=16, M=2, d_in=3, d_out=3)
    m = 0
    inner, halo = P.inner_gid[m], P.halo_gid[m]
    f = orc.gat_fwd(P, m, H[inner], H[halo], W, a_src, a_dst, bias, 1)
    g = orc.gat_bwd(P, m, H[inner], H[halo], W, a_src, a_dst, f, G[inner], 1)
    loss = lambda Hi: float(np.sum(np.maximum(orc.gat_fwd(P, m, Hi, H[halo], W, a_src, a_dst, bias, 1)["O"], 0) * G[inner]))
    eps = 1e-6
    fd = np.zeros_like(H[inner])
    for i in range(fd.shape[0]):
        for j in range(fd.shape[1]):
            Hp, Hm = H[inner].copy(), H[inner].copy()
            Hp[i, j] += eps
            Hm[i, j] -= eps
            fd[i, j] = (loss(Hp) - loss(Hm)) / (2 * eps)
    np.testing.assert_allclose(g["H_in"], fd, atol=1e-6)


def test_uniform_attention_closed_form():
    """a_src = a_dst = 0: every row attends uniformly, the layer is the row-mean of z over the closed neighbourhood."""
    rowptr, col, P, H, W, a_src, a_dst, bias, G, adj = _case(9, M=2)
    for m in range(P.M):
        inner, halo = P.inner_gid[m], P.halo_gid[m]
        f = orc.gat_fwd(P, m, H[inner], H[halo], W, np.zeros_like(a_src), np.zeros_like(a_dst), None, 0)
        want = np.stack([(H[adj[v]] @ W).mean(axis=0) for v in inner])
        np.testing.assert_allclose(f["O"], want, atol=1e-12)


# ------------------------------------------------------------------------------------------
# the epoch sequencing around the attention layers (run_epoch_gat): which cached layer feeds which layer, the push, the
# loss weighting, the hand-down of the gradient
# ------------------------------------------------------------------------------------------
def _epoch_case(seed, n, M, dims, p=0.14):
    rng = np.random.default_rng(seed)
    rowptr, col = random_graph(rng, n, p)
    part = rng.integers(0, M, size=n).astype(np.int32)
    P = orc.build_partition(rowptr, col, part, M)
    dtil, _ = orc.degrees(rowptr)
    X = rng.standard_normal((n, dims[0])).astype(np.float32)
    y = rng.integers(0, dims[-1], size=n).astype(np.int32)
    params = []
    for l in range(len(dims) - 1):
        params.append(dict(W=(rng.standard_normal((dims[l], dims[l + 1])) * 0.6).astype(np.float32),
                           a_src=(rng.standard_normal(dims[l + 1]) * 0.7).astype(np.float32),
                           a_dst=(rng.standard_normal(dims[l + 1]) * 0.7).astype(np.float32),
                           b=(rng.standard_normal(dims[l + 1]) * 0.2).astype(np.float32)))
    adj = np.eye(n, dtype=bool)
    for v in range(n):
        adj[v, col[rowptr[v]:rowptr[v + 1]]] = True
    return rowptr, col, P, dtil, X, y, params, adj


def _dense_model(adj, X, y, params):
    """The unpartitioned multi-layer attention network in torch (float64) with the mean cross-entropy loss; returns
    (loss, per-layer outputs, per-layer parameter gradients)."""
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64), requires_grad=True)
    tp = [{k: t(v) for k, v in p.items()} for p in params]
    H = torch.tensor(np.asarray(X, dtype=np.float64))
    outs = []
    L = len(params)
    for l, p in enumerate(tp):
        H = _dense_gat(torch.tensor(adj), H, p["W"], p["a_src"], p["a_dst"], p["b"], 1 if l < L - 1 else 0)
        outs.append(H)
    loss = torch.nn.functional.cross_entropy(H, torch.tensor(y, dtype=torch.long), reduction="mean")
    loss.backward()
    grads = [{k: v.grad.numpy() for k, v in p.items()} for p in tp]
    return float(loss.detach()), [o.detach().numpy() for o in outs], grads


@pytest.mark.parametrize("seed,dims", [(11, [5, 4, 6, 3]), (12, [4, 7, 3])])
def test_attention_epoch_on_one_partition_is_the_dense_network(seed, dims):
    """M = 1: no out-of-subgraph nodes, so the epoch is plain full-graph training — loss and every parameter gradient of
    every layer equal autograd's on the dense multi-layer model."""
    rowptr, col, P, dtil, X, y, params, adj = _epoch_case(seed, 26, 1, dims)
    cache = orc.CacheRing(P.n_slots, dims[1:-1], 2)
    res = orc.run_epoch_gat(P, dtil, cache, X, y, params, None, "ce")
    want_loss, outs, grads = _dense_model(adj, X, y, params)
    assert abs(res["loss"] - want_loss) <= 2e-6 * abs(want_loss)
    for l in range(len(params)):
        np.testing.assert_allclose(res["H"][0][l], outs[l], atol=5e-6)
        for k in ("W", "a_src", "a_dst", "b"):
            # the oracle rounds the activations it hands from layer to layer to fp32 (as the device path stores them)
            np.testing.assert_allclose(res["grads"][l][k], grads[l][k], atol=3e-6, err_msg=f"layer {l + 1} G_{k}")
    assert cache.n_valid == 1


@pytest.mark.parametrize("with_predictor", [False, True])
def test_attention_epoch_with_exact_cache_is_the_full_graph_forward(with_predictor):
    """M > 1 with the ring holding the exact embeddings of every cached layer (different widths per layer, so a wrong
    layer index cannot go unnoticed): every layer's output equals the dense full-graph network; the last layer's
    parameter gradients too (its inputs are exact and nothing below it is differentiated through the halo); what the
    epoch pushed is again the exact embedding of the boundary nodes.  With a predictor whose output weights are zero
    the prediction is the newest snapshot, so the same holds through the LSTM / graph-convolution path."""
    dims = [5, 4, 6, 3]
    rowptr, col, P, dtil, X, y, params, adj = _epoch_case(21, 30, 3, dims)
    want_loss, outs, grads = _dense_model(adj, X, y, params)
    Cn = np.nonzero(P.slot >= 0)[0]
    cache = orc.CacheRing(P.n_slots, dims[1:-1], 3)
    for l in range(1, len(dims) - 1):
        cache.push(l, P.slot[Cn], outs[l - 1][Cn].astype(np.float32))
    cache.commit()
    pred = None
    if with_predictor:
        rng = np.random.default_rng(5)
        pred = []
        for l in range(1, len(dims) - 1):
            d, h = dims[l], 4
            pred.append(dict(Wx=rng.standard_normal((d, 4 * h)).astype(np.float32), Uh=rng.standard_normal((h, 4 * h)).astype(np.float32),
                             b=rng.standard_normal(4 * h).astype(np.float32), Wg=np.zeros((h, d), dtype=np.float32),
                             bg=np.zeros(d, dtype=np.float32)))
    res = orc.run_epoch_gat(P, dtil, cache, X, y, params, pred, "ce")
    L = len(params)
    for l in range(L):
        got = np.zeros_like(outs[l])
        for m in range(P.M):
            got[P.inner_gid[m]] = res["H"][m][l]
        np.testing.assert_allclose(got, outs[l], atol=1e-5, err_msg=f"H^{l + 1}")
    assert abs(res["loss"] - want_loss) <= 1e-5 * abs(want_loss)
    for k in ("W", "a_src", "a_dst", "b"):
        np.testing.assert_allclose(res["grads"][L - 1][k], grads[L - 1][k], atol=1e-5, err_msg=f"last layer G_{k}")
    # the lower layers' gradients miss the paths through the halo copies, so they differ from the full graph's
    assert np.max(np.abs(res["grads"][0]["W"] - grads[0]["W"])) > 1e-4
    for l in range(1, L):
        np.testing.assert_allclose(cache.newest(l)[P.slot[Cn]], outs[l - 1][Cn], atol=1e-5)
    assert cache.n_valid == 2


def test_slope_override_of_the_backward():
    """gat_bwd(positive=...) replaces the LeakyReLU's sign decision entry by entry: the oracle's own decision gives the
    same bits, and flipping one entry changes the logit's gradient by exactly the ratio of the two slopes."""
    rowptr, col, P, H, W, a_src, a_dst, bias, G, adj = _case(13, M=2)
    m = 0
    inner, halo = P.inner_gid[m], P.halo_gid[m]
    f = orc.gat_fwd(P, m, H[inner], H[halo], W, a_src, a_dst, bias, 1)
    g0 = orc.gat_bwd(P, m, H[inner], H[halo], W, a_src, a_dst, f, G[inner], 1)
    g1 = orc.gat_bwd(P, m, H[inner], H[halo], W, a_src, a_dst, f, G[inner], 1, positive=f["pre"] > 0)
    for k in g0:
        assert np.array_equal(g0[k], g1[k])
    pos = f["pre"] > 0
    e = int(np.argmax(np.abs(f["pre"])))       # one entry, decided the other way
    flipped = pos.copy()
    flipped[e] = ~flipped[e]
    g2 = orc.gat_bwd(P, m, H[inner], H[halo], W, a_src, a_dst, f, G[inner], 1, positive=flipped)
    # only the path through that logit changes: G_a_dst changes by (new slope - old slope) * alpha (d_alpha - t) * z_v
    rows, cols = orc._gat_rows(P, m)
    Z, alpha = f["Z"], f["alpha"]
    D = G[inner] * (f["O"] > 0)
    d_alpha = np.sum(D[rows] * Z[cols], axis=1)
    t = np.zeros(inner.shape[0])
    np.add.at(t, rows, alpha * d_alpha)
    base = alpha[e] * (d_alpha[e] - t[rows[e]])
    delta = ((1.0 if flipped[e] else orc.GAT_SLOPE) - (1.0 if pos[e] else orc.GAT_SLOPE)) * base
    np.testing.assert_allclose(g2["a_dst"] - g0["a_dst"], delta * Z[rows[e]], atol=1e-12)
