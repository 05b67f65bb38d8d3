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
