"""Pins for the oracle's embedding-predictor objective and gradient (Eq. "predictor loss", Eq. "mini-batch training")."""
import numpy as np
import pytest

from oracle import sat_ref as orc
from tests.dense_pins import random_graph


def _case(seed, n=40, M=3, d=5, h=4, k=3, p=0.15):
    rng = np.random.default_rng(seed)
    rowptr, col = random_graph(rng, n, p)
    part = rng.integers(0, M, size=n).astype(np.int32)
    dtil, _ = orc.degrees(rowptr)
    P = orc.build_partition(rowptr, col, part, M)
    ns = P.n_slots
    snaps = [rng.standard_normal((ns, d)).astype(np.float32) for _ in range(k)]
    target = rng.standard_normal((ns, d)).astype(np.float32)
    par = dict(Wx=rng.standard_normal((d, 4 * h)) * 0.5, Uh=rng.standard_normal((h, 4 * h)) * 0.5,
               b=rng.standard_normal(4 * h) * 0.3, Wg=rng.standard_normal((h, d)) * 0.5, bg=rng.standard_normal(d) * 0.3)
    return P, dtil, snaps, target, par


def _loss_from_forward_oracle(P, dtil, snaps, target, par, row_weight=None):
    """The objective assembled from the forward functions of the C oracle (a different implementation of the LSTM and of
    the graph convolution than the one the gradient code uses)."""
    h, d = par["Wg"].shape
    S = orc.lstm_state(snaps, d, h, par["Wx"], par["Uh"], par["b"], P.n_slots)
    newest = snaps[-1] if snaps else None
    total = 0.0
    for m in range(P.M):
        nh = P.halo_gid[m].shape[0]
        if nh == 0:
            continue
        pred = orc.predict_halo(P, m, dtil, S, newest, par["Wg"], par["bg"]).astype(np.float64)
        w = np.full(nh, 1.0 / nh) if row_weight is None else row_weight[m]
        diff = pred - target[P.halo_slot[m]].astype(np.float64)
        total += float(np.sum(w * 0.5 * np.sum(diff * diff, axis=1))) / P.M
    return total


@pytest.mark.parametrize("seed,k", [(1, 1), (2, 3), (3, 4), (4, 0)])
def test_loss_matches_the_forward_functions(seed, k):
    P, dtil, snaps, target, par = _case(seed, k=k)
    par32 = {a: v.astype(np.float32) for a, v in par.items()}
    loss, _ = orc.pred_loss_grad(P, dtil, snaps, target, **par32)
    want = _loss_from_forward_oracle(P, dtil, snaps, target, par32)
    assert abs(loss - want) <= 2e-6 * max(1.0, abs(want))


@pytest.mark.parametrize("seed,k,h", [(5, 1, 3), (6, 2, 4), (7, 4, 5)])
def test_gradient_against_central_differences(seed, k, h):
    """Every entry of every parameter: (L(w + e) - L(w - e)) / 2e in float64."""
    P, dtil, snaps, target, par = _case(seed, n=30, d=4, h=h, k=k)
    loss, G = orc.pred_loss_grad(P, dtil, snaps, target, **par)
    eps = 1e-6
    for name in ("Wx", "Uh", "b", "Wg", "bg"):
        fd = np.zeros_like(par[name])
        it = np.nditer(par[name], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = par[name][idx]
            par[name][idx] = keep + eps
            lp, _ = orc.pred_loss_grad(P, dtil, snaps, target, **par)
            par[name][idx] = keep - eps
            lm, _ = orc.pred_loss_grad(P, dtil, snaps, target, **par)
            par[name][idx] = keep
            fd[idx] = (lp - lm) / (2 * eps)
        scale = max(np.abs(fd).max(), 1e-12)
        assert np.abs(G[name] - fd).max() <= 1e-6 * max(scale, 1.0), name
        if k == 1 and name == "Uh":
            assert np.all(G[name] == 0)      # one step from a zero state: the recurrent weights are not used
        elif name != "Uh" or k > 1:
            assert np.abs(G[name]).max() > 0


def test_zero_output_weights_closed_form():
    """Wg = 0: the prediction is newest + bg, so the LSTM parameters get no gradient, G_Wg = a^T E and
    G_bg = (1/M) sum_m mean_u (newest_u + bg - target_u)."""
    P, dtil, snaps, target, par = _case(11)
    par["Wg"][:] = 0
    loss, G = orc.pred_loss_grad(P, dtil, snaps, target, **par)
    assert np.all(G["Wx"] == 0) and np.all(G["Uh"] == 0) and np.all(G["b"] == 0)
    want = np.zeros_like(par["bg"])
    lsum = 0.0
    for m in range(P.M):
        hs = P.halo_slot[m]
        if hs.shape[0] == 0:
            continue
        diff = snaps[-1][hs].astype(np.float64) + par["bg"] - target[hs]
        want += diff.mean(axis=0) / P.M
        lsum += 0.5 * np.mean(np.sum(diff * diff, axis=1)) / P.M
    np.testing.assert_allclose(G["bg"], want, rtol=1e-12, atol=1e-14)
    assert abs(loss - lsum) < 1e-12


def test_perfect_prediction_has_zero_loss_and_gradient():
    P, dtil, snaps, _, par = _case(12)
    par["Wg"][:] = 0
    par["bg"][:] = 0
    loss, G = orc.pred_loss_grad(P, dtil, snaps, snaps[-1], **par)   # target = newest snapshot, prediction = newest
    assert loss == 0
    assert all(np.all(g == 0) for g in G.values())


def test_mini_batch_weights():
    """Weights 1/|batch| on a sampled batch and 0 elsewhere: the loss only sees the batch; the full-batch gradient is the
    average of the gradients of the batches of a partition of the halo rows into equal parts."""
    P, dtil, snaps, target, par = _case(13, n=60)
    rng = np.random.default_rng(0)
    batches = []
    for m in range(P.M):
        nh = P.halo_gid[m].shape[0]
        batches.append(rng.permutation(nh)[: max(1, nh // 3)])
    rw = []
    for m in range(P.M):
        w = np.zeros(P.halo_gid[m].shape[0])
        w[batches[m]] = 1.0 / batches[m].shape[0]
        rw.append(w)
    loss, G = orc.pred_loss_grad(P, dtil, snaps, target, row_weight=rw, **par)
    want = _loss_from_forward_oracle(P, dtil, snaps, target, {a: v.astype(np.float32) for a, v in par.items()}, rw)
    assert abs(loss - want) <= 1e-5 * max(1.0, abs(want))
    # changing the target outside the batch changes nothing
    t2 = target.copy()
    inside = np.zeros(P.n_slots, dtype=bool)
    for m in range(P.M):
        inside[P.halo_slot[m][batches[m]]] = True
    t2[~inside] += 3.0
    loss2, G2 = orc.pred_loss_grad(P, dtil, snaps, t2, row_weight=rw, **par)
    assert loss2 == loss and all(np.array_equal(G[a], G2[a]) for a in G)
    # linearity in the weights: two complementary halves average to the full batch
    halves = [[], []]
    for m in range(P.M):
        nh = P.halo_gid[m].shape[0]
        perm = rng.permutation(nh)
        for s, part in enumerate((perm[: nh // 2], perm[nh // 2:])):
            w = np.zeros(nh)
            w[part] = 1.0 / nh
            halves[s].append(w)
    la, Ga = orc.pred_loss_grad(P, dtil, snaps, target, row_weight=halves[0], **par)
    lb, Gb = orc.pred_loss_grad(P, dtil, snaps, target, row_weight=halves[1], **par)
    lf, Gf = orc.pred_loss_grad(P, dtil, snaps, target, **par)
    assert abs(la + lb - lf) < 1e-12
    for a in Gf:
        np.testing.assert_allclose(Ga[a] + Gb[a], Gf[a], rtol=1e-10, atol=1e-13)


def test_gradient_step_lowers_the_loss():
    """Algorithm 1's update omega <- omega - eta grad: a small step reduces the objective by about eta |grad|^2."""
    P, dtil, snaps, target, par = _case(14)
    loss, G = orc.pred_loss_grad(P, dtil, snaps, target, **par)
    eta = 1e-3
    g2 = sum(float(np.sum(g * g)) for g in G.values())
    stepped = {a: par[a] - eta * G[a] for a in par}
    loss2, _ = orc.pred_loss_grad(P, dtil, snaps, target, **stepped)
    assert loss2 < loss
    assert abs((loss - loss2) - eta * g2) <= 0.05 * eta * g2
