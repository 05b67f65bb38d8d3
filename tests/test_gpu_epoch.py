"""GPU vs oracle on whole SAT epochs (all partitions per launch, the configuration the benchmark times),
from identical state, for ring fill levels k = 0..tau and beyond; plus reproducibility, per-partition
equivalence and checkpoint / resume of the cache ring."""
import copy

import numpy as np
import pytest

from oracle import sat_ref as orc
from sat_synth import make_workload
from tests.gpu_util import assert_close, dev, dev2d, pred_to_device, relu_tie_masks

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import paper_2308_13466_b200.binding as binding
    return binding


def _setup(B, wl):
    import torch
    from paper_2308_13466_b200.epoch import SatEpoch
    part = wl.part_given if wl.part_given is not None else orc.contig_blocks(wl.n, wl.M)
    dtil, _ = orc.degrees(wl.rowptr)
    P = orc.build_partition(wl.rowptr, wl.col, part, wl.M)
    ep = SatEpoch(wl.rowptr, wl.col, wl.M, wl.dims, wl.tau, wl.loss, part_given=wl.part_given)
    perm = np.concatenate(P.inner_gid)
    ep.set_inputs(dev2d(wl.X), dev(wl.labels[perm]))
    return ep, P, dtil, perm


def _gather_H(res, P, l):
    return np.concatenate([res.per_part[m]["H"][l - 1] for m in range(P.M)])


@pytest.mark.parametrize("name,shrink,over,version", [
    ("tiny", 1, {}, 0), ("medium", 16, {}, 0),
    ("medium", 16, {"h": 256}, 0),     # wide predictor: 4h = 1024 gate columns, cell update as a kernel of its own
    # widths that are no multiple of a tile / k-block / 8, non-zero biases in the layers and the predictor; with and
    # without cached input projections (the oracle keeps no such state)
    ("odd", 1, {}, 0), ("odd", 1, {}, 3), ("odd", 1, {"h": 20}, 0), ("odd", 1, {"h": 20}, 3), ("odd", 1, {"h": 32}, 3),
    # GRU-GCN variant of the predictor
    ("tiny", 1, {"cell": "gru"}, 0), ("medium", 16, {"cell": "gru"}, 0), ("odd", 1, {"cell": "gru"}, 0), ("odd", 1, {"cell": "gru", "h": 20}, 5)])
def test_epochs_from_synchronised_state(B, name, shrink, over, version):
    import torch
    over = dict(over)
    cell = over.pop("cell", "lstm")
    wl = make_workload(name, shrink=shrink, **over)
    if cell == "gru":
        from sat_synth import as_gru
        wl.pred = as_gru(wl.pred)
    ep, P, dtil, perm = _setup(B, wl)
    try:
        cache = orc.CacheRing(P.n_slots, wl.dims[1:-1], wl.tau)
        W = [w.copy() for w in wl.W]
        b = [x.copy() for x in wl.b]
        preds = pred_to_device(wl.pred, B, version)
        for t in range(1, wl.tau + 3):
            Wd = [dev(w) for w in W]
            bd = [dev(x) for x in b]
            before = copy.deepcopy(cache)
            res = orc.run_epoch(P, dtil, cache, wl.X, wl.labels, W, b, wl.pred, wl.loss)
            ep.step(Wd, bd, preds)
            torch.cuda.synchronize()
            # ReLU ties: where |Z| is at rounding level the two sides may decide the sign differently; both are
            # correct, so the oracle's backward is redone with the CUDA path's decision on exactly those entries.
            H_gpu = [None] + [ep.H[l].cpu().numpy() for l in range(1, wl.L + 1)]
            masks, redo = relu_tie_masks(res, P, H_gpu, ep.inner_off, wl.L)
            if redo:
                cache = before
                res = orc.run_epoch(P, dtil, cache, wl.X, wl.labels, W, b, wl.pred, wl.loss, masks=masks)
            for l in range(1, wl.L + 1):
                assert_close(ep.H[l].cpu().numpy(), _gather_H(res, P, l), f"epoch {t} H^{l}")
            loss = float(ep.loss_sum.item())
            assert abs(loss - res.loss) <= 1e-5 * abs(res.loss), (loss, res.loss)
            for l in range(wl.L):
                assert_close(ep.gW[l].cpu().numpy(), res.G_W[l], f"epoch {t} G_W{l + 1}")
                assert_close(ep.gb[l].cpu().numpy(), res.G_b[l], f"epoch {t} G_b{l + 1}")
            assert B.sat_cache_state(ep.ctx) == (cache.write_idx, cache.n_valid)
            for l in range(1, wl.L):
                ring = B.sat_cache_export(ep.ctx, l, wl.tau, P.n_slots, wl.dims[l])
                newest = (cache.write_idx - 1) % (wl.tau + 1)
                assert_close(ring[newest], cache.buf[l - 1][newest], f"epoch {t} pushed snapshot of layer {l}")
                B.sat_cache_import(ep.ctx, l, cache.buf[l - 1])       # re-synchronise: errors do not compound
            # plain SGD on the oracle's gradient moves the weights between epochs
            W = [(w - 0.5 * g).astype(np.float32) for w, g in zip(W, res.G_W)]
            b = [(x - 0.5 * g).astype(np.float32) for x, g in zip(b, res.G_b)]
    finally:
        ep.close()


def test_per_partition_equals_batched_and_is_reproducible(B):
    import torch
    wl = make_workload("medium", shrink=16)
    Wd = [dev(w) for w in wl.W]
    bd = [dev(x) for x in wl.b]
    preds = pred_to_device(wl.pred, B)
    outs = []
    for mode in ("batched", "batched", "per-part", "per-part-reversed"):
        ep, P, dtil, perm = _setup(B, wl)
        try:
            for _ in range(3):
                if mode == "batched":
                    ep.step(Wd, bd, preds)
                else:
                    order = list(range(wl.M)) if mode == "per-part" else list(range(wl.M - 1, -1, -1))
                    ep.step_per_partition(Wd, bd, preds, order=order)
            torch.cuda.synchronize()
            outs.append(dict(H=[h.cpu().numpy().copy() for h in ep.H[1:]], gW=[g.cpu().numpy().copy() for g in ep.gW],
                             ring=[B.sat_cache_export(ep.ctx, l, wl.tau, P.n_slots, wl.dims[l]) for l in range(1, wl.L)],
                             loss=float(ep.loss_sum.item())))
        finally:
            ep.close()
    a, a2, p, pr = outs
    for l in range(wl.L):
        assert np.array_equal(a["H"][l], a2["H"][l]), "batched epoch is not bit-reproducible"
        assert np.array_equal(a["gW"][l], a2["gW"][l]), "batched gradients are not bit-reproducible"
        assert np.array_equal(a["H"][l], p["H"][l]), "per-partition calls differ from the batched launch"
        assert np.array_equal(p["H"][l], pr["H"][l]), "partition order changes the result"
        assert_close(p["gW"][l], a["gW"][l], "per-partition summed G_W vs batched", 1e-5)
    for r0, r1 in zip(a["ring"], p["ring"]):
        assert np.array_equal(r0, r1)
    assert abs(a["loss"] - p["loss"]) <= 1e-6 * abs(a["loss"])


def test_cache_checkpoint_resume(B):
    """export -> fresh context -> import -> next epoch is bit-identical."""
    import torch
    wl = make_workload("tiny")
    Wd = [dev(w) for w in wl.W]
    bd = [dev(x) for x in wl.b]
    preds = pred_to_device(wl.pred, B)
    ep, P, dtil, perm = _setup(B, wl)
    try:
        for _ in range(4):
            ep.step(Wd, bd, preds)
        rings = [B.sat_cache_export(ep.ctx, l, wl.tau, P.n_slots, wl.dims[l]) for l in range(1, wl.L)]
        state = B.sat_cache_state(ep.ctx)
        ep.step(Wd, bd, preds)
        torch.cuda.synchronize()
        want = [h.cpu().numpy().copy() for h in ep.H[1:]]
    finally:
        ep.close()
    ep2, _, _, _ = _setup(B, wl)
    try:
        for l, r in enumerate(rings, start=1):
            B.sat_cache_import(ep2.ctx, l, r)
        B.sat_cache_set_state(ep2.ctx, *state)
        ep2.step(Wd, bd, preds)
        torch.cuda.synchronize()
        for a, b_ in zip(want, [h.cpu().numpy() for h in ep2.H[1:]]):
            assert np.array_equal(a, b_)
    finally:
        ep2.close()


def test_cached_input_projections_over_a_wrapping_ring(B):
    """Predictor parameters with a version promise: the library keeps x Wx + b per cached snapshot and projects only new
    snapshots.  Free-running epochs (no re-synchronisation, fixed weights) until the ring has wrapped twice; the LSTM state,
    the layer outputs and the ring must still match the oracle running the same epochs, and the versioned and unversioned
    paths must agree."""
    import torch
    wl = make_workload("medium", shrink=16)
    Wd = [dev(w) for w in wl.W]
    bd = [dev(x) for x in wl.b]
    n_epochs = 2 * (wl.tau + 1) + 1
    outs = {}
    for version in (0, 9, "bump"):
        preds = pred_to_device(wl.pred, B, 9 if version == "bump" else version)
        ep, P, dtil, perm = _setup(B, wl)
        try:
            for t in range(n_epochs):
                if version == "bump" and t == wl.tau + 2:
                    # same values under a new version: the cached projections are dropped; the epochs that follow mix steps
                    # with a cached projection (new snapshots) and steps that contract over [x | s] (older snapshots)
                    for pp in preds:
                        pp.version = 10
                ep.step(Wd, bd, preds)
            torch.cuda.synchronize()
            # the LSTM state of the ring as the next epoch would see it (the commit dropped the one the epochs used)
            S = []
            for l in range(1, wl.L):
                halo0 = torch.empty((P.halo_gid[0].shape[0], wl.dims[l]), dtype=torch.float32, device="cuda")
                B.sat_predict(ep.ctx, l, 0, preds[l - 1], 0, halo0)
                S.append(B.sat_predict_state(ep.ctx, l, P.n_slots, wl.pred[l - 1]["h"]))
            outs[version] = dict(H=[h.cpu().numpy().copy() for h in ep.H[1:]], S=S,
                                 ring=[B.sat_cache_export(ep.ctx, l, wl.tau, P.n_slots, wl.dims[l]) for l in range(1, wl.L)],
                                 state=B.sat_cache_state(ep.ctx))
        finally:
            ep.close()
    cache = orc.CacheRing(P.n_slots, wl.dims[1:-1], wl.tau)
    for _ in range(n_epochs):
        res = orc.run_epoch(P, dtil, cache, wl.X, wl.labels, wl.W, wl.b, wl.pred, wl.loss, keep=False)
    for version in (0, 9, "bump"):
        o = outs[version]
        assert o["state"] == (cache.write_idx, cache.n_valid)
        for l in range(1, wl.L):
            pr = wl.pred[l - 1]
            S_want = orc.lstm_state(cache.snapshots(l), wl.dims[l], pr["h"], pr["Wx"], pr["Uh"], pr["b"], P.n_slots)
            assert_close(o["S"][l - 1], S_want, f"version {version}: LSTM state of layer {l} after {n_epochs} epochs")
            newest = (cache.write_idx - 1) % (wl.tau + 1)
            assert_close(o["ring"][l - 1][newest], cache.buf[l - 1][newest], f"version {version}: newest snapshot of layer {l}")
        for l in range(1, wl.L + 1):
            assert_close(o["H"][l - 1], _gather_H(res, P, l), f"version {version}: H^{l} after {n_epochs} epochs")


def test_staleness_of_historical_and_predicted_halos(B):
    """Eq. "staleness def" on a running ring: || H_out - H~_out || with the newest committed snapshot as H~ (what
    historical-embedding training would use) and with the predictor's output, per partition and summed, against the oracle
    on the same arrays."""
    import torch
    wl = make_workload("medium", shrink=16)
    Wd = [dev(w) for w in wl.W]
    bd = [dev(x) for x in wl.b]
    preds = pred_to_device(wl.pred, B, 2)
    ep, P, dtil, perm = _setup(B, wl)
    try:
        for _ in range(wl.tau + 1):
            ep.step(Wd, bd, preds, 0.01)
        nb = sum(h.shape[0] for h in P.halo_gid)
        used = {}
        for l in range(1, wl.L):     # what the next epoch will use for its halos, taken before that epoch runs
            hist = torch.empty((nb, wl.dims[l]), dtype=torch.float32, device="cuda")
            pred = torch.empty((nb, wl.dims[l]), dtype=torch.float32, device="cuda")
            B.sat_predict(ep.ctx, l, B.SAT_ALL_PARTS, None, 0, hist)
            B.sat_predict(ep.ctx, l, B.SAT_ALL_PARTS, preds[l - 1], 0, pred)
            used[l] = (hist, pred)
        ep.step(Wd, bd, preds, 0.01)
        torch.cuda.synchronize()
        sq = torch.zeros(1, dtype=torch.float64, device="cuda")
        off = np.concatenate([[0], np.cumsum([h.shape[0] for h in P.halo_gid])])
        for l in range(1, wl.L):
            H_pm = ep.H[l].cpu().numpy()
            H_gid = np.empty_like(H_pm)
            H_gid[perm] = H_pm
            for kind, u in zip(("historical", "predicted"), used[l]):
                u_host = u.cpu().numpy()
                total = 0.0
                for m in range(wl.M):
                    want = orc.staleness(P, m, H_gid, u_host[off[m]:off[m + 1]])
                    B.sat_staleness(ep.ctx, m, ep.H[l], u[off[m]:off[m + 1]], sq)
                    got = float(sq.item()) ** 0.5
                    assert abs(got - want) <= 1e-10 * max(want, 1e-30), (kind, l, m, got, want)
                    assert want > 0.0          # the weights moved: the history is stale
                    total += want * want
                B.sat_staleness(ep.ctx, B.SAT_ALL_PARTS, ep.H[l], u, sq)
                assert abs(float(sq.item()) - total) <= 1e-10 * total
        # identical embeddings: exactly zero
        pos = np.empty(wl.n, dtype=np.int64)
        pos[perm] = np.arange(wl.n)
        same = ep.H[1][torch.as_tensor(pos[P.halo_gid[0]], device="cuda")].contiguous()
        B.sat_staleness(ep.ctx, 0, ep.H[1], same, sq)
        assert float(sq.item()) == 0.0
    finally:
        ep.close()


@pytest.mark.parametrize("over,empty_part", [
    ({"dims": [50, 70, 38, 7], "h": 20}, False),     # cached widths that are no multiple of 4 (padded row strides)
    ({"tau": 1}, False),                               # a window of one snapshot
    ({"M": 5}, True),                                  # a partition without nodes
    ({"M": 2, "h": 4, "dims": [50, 6, 5, 3]}, False),  # widths below the tensor-core threshold everywhere
])
def test_odd_shapes_and_degenerate_partitions(B, over, empty_part):
    import torch
    wl = make_workload("odd", **over)
    if empty_part:
        rng = np.random.default_rng(3)
        wl.part_given = rng.choice(np.array([0, 1, 3, 4], dtype=np.int32), size=wl.n)     # nobody lands in partition 2
    ep, P, dtil, perm = _setup(B, wl)
    try:
        if empty_part:
            assert P.inner_gid[2].shape[0] == 0
        cache = orc.CacheRing(P.n_slots, wl.dims[1:-1], wl.tau)
        hist = orc.GradHistory(P.n_slots, wl.dims[2:])
        Wd = [dev(w) for w in wl.W]
        bd = [dev(x) for x in wl.b]
        for version, use_hist in ((0, False), (7, True)):
            preds = pred_to_device(wl.pred, B, version)
            for t in range(wl.tau + 2):
                before, hist_before = copy.deepcopy(cache), copy.deepcopy(hist)
                res = orc.run_epoch(P, dtil, cache, wl.X, wl.labels, wl.W, wl.b, wl.pred, wl.loss, grad_hist=hist if use_hist else None)
                ep.step(Wd, bd, preds, grad_history=use_hist)
                torch.cuda.synchronize()
                H_gpu = [None] + [ep.H[l].cpu().numpy() for l in range(1, wl.L + 1)]
                masks, redo = relu_tie_masks(res, P, H_gpu, ep.inner_off, wl.L)
                if redo:
                    cache, hist = before, hist_before
                    res = orc.run_epoch(P, dtil, cache, wl.X, wl.labels, wl.W, wl.b, wl.pred, wl.loss, masks=masks,
                                        grad_hist=hist if use_hist else None)
                for l in range(1, wl.L + 1):
                    assert_close(H_gpu[l], _gather_H(res, P, l), f"{over} epoch {t} H^{l}")
                for l in range(wl.L):
                    assert_close(ep.gW[l].cpu().numpy(), res.G_W[l], f"{over} epoch {t} G_W{l + 1}")
                    assert_close(ep.gb[l].cpu().numpy(), res.G_b[l], f"{over} epoch {t} G_b{l + 1}")
                for l in range(1, wl.L):
                    B.sat_cache_import(ep.ctx, l, cache.buf[l - 1])
                if use_hist:
                    for j in range(2, wl.L + 1):
                        B.sat_grad_history_write(ep.ctx, j, wl.dims[j], hist.read[j - 2])
            # the predictor gradient on the same shapes
            if version == 0:
                ep.loss_sum.zero_()
                ep._forward_backward(B.SAT_ALL_PARTS, Wd, bd, preds, 0, 0)
                write_idx, n_valid = B.sat_cache_state(ep.ctx)
                for l in range(1, wl.L):
                    ring = B.sat_cache_export(ep.ctx, l, wl.tau, P.n_slots, wl.dims[l])
                    snaps = [ring[(write_idx - 1 - a) % (wl.tau + 1)] for a in range(n_valid - 1, -1, -1)]
                    pr = wl.pred[l - 1]
                    want_loss, want = orc.pred_loss_grad(P, dtil, snaps, ring[write_idx], pr["Wx"], pr["Uh"], pr["b"], pr["Wg"], pr["bg"])
                    g = tuple(torch.full_like(x, float("nan")) for x in preds[l - 1]._keep)
                    loss = B.sat_pred_grad(ep.ctx, l, preds[l - 1], None, *g, want_loss=True)
                    assert abs(loss - want_loss) <= 1e-5 * abs(want_loss)
                    for a, x in zip(("Wx", "Uh", "b", "Wg", "bg"), g):
                        assert_close(x.cpu().numpy(), want[a], f"{over} predictor gradient layer {l}: G_{a}")
                for l in range(1, wl.L):
                    B.sat_cache_import(ep.ctx, l, cache.buf[l - 1])
                B.sat_cache_set_state(ep.ctx, cache.write_idx, cache.n_valid)
    finally:
        ep.close()
