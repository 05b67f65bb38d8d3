"""GPU vs oracle on the embedding predictor's objective and gradient (Eq. "predictor loss"), from identical ring contents."""
import numpy as np
import pytest

from oracle import sat_ref as orc
from sat_synth import make_workload
from tests.gpu_util import assert_close, dev, pred_to_device

pytestmark = pytest.mark.gpu

NAMES = ("Wx", "Uh", "b", "Wg", "bg")


@pytest.fixture(scope="module")
def B():
    import paper_2308_13466_b200.binding as binding
    return binding


def _setup(B, wl):
    from paper_2308_13466_b200.epoch import SatEpoch
    part = wl.part_given if wl.part_given is not None else orc.contig_blocks(wl.n, wl.M)
    dtil, _ = orc.degrees(wl.rowptr)
    P = orc.build_partition(wl.rowptr, wl.col, part, wl.M)
    ep = SatEpoch(wl.rowptr, wl.col, wl.M, wl.dims, wl.tau, wl.loss, part_given=wl.part_given)
    return ep, P, dtil


def _random_ring(rng, P, wl, n_valid, write_idx):
    """A ring with embedding-like contents (non-negative, a third of the entries zero) in every buffer."""
    cache = orc.CacheRing(P.n_slots, wl.dims[1:-1], wl.tau)
    for buf in cache.buf:
        x = rng.standard_normal(buf.shape).astype(np.float32) * 0.6
        buf[...] = np.where(x > -0.25, np.abs(x), 0.0)
    cache.write_idx, cache.n_valid = write_idx, n_valid
    return cache


def _grads(B, ep, l, p, rw=None):
    import torch
    g = tuple(torch.full_like(t, float("nan")) for t in p._keep)
    loss = B.sat_pred_grad(ep.ctx, l, p, rw, *g, want_loss=True)
    return loss, {a: t.cpu().numpy() for a, t in zip(NAMES, g)}


@pytest.mark.parametrize("name,shrink,over", [("tiny", 1, {}), ("medium", 16, {}), ("medium", 16, {"h": 256}),
                                              ("odd", 1, {}), ("odd", 1, {"h": 20}), ("odd", 1, {"h": 32})])
def test_gradient_for_every_fill_level(B, name, shrink, over):
    wl = make_workload(name, shrink=shrink, **over)
    ep, P, dtil = _setup(B, wl)
    rng = np.random.default_rng(5)
    try:
        preds = pred_to_device(wl.pred, B, 0)
        for n_valid, write_idx in [(0, 0), (1, 1), (2, 0), (wl.tau, wl.tau), (wl.tau, 1)]:
            if n_valid > wl.tau:
                continue
            cache = _random_ring(rng, P, wl, n_valid, write_idx)
            for l in range(1, wl.L):
                B.sat_cache_import(ep.ctx, l, cache.buf[l - 1])
            B.sat_cache_set_state(ep.ctx, write_idx, n_valid)
            for l in range(1, wl.L):
                pr = wl.pred[l - 1]
                want_loss, want = orc.pred_loss_grad(P, dtil, cache.snapshots(l), cache.buf[l - 1][write_idx], pr["Wx"], pr["Uh"], pr["b"],
                                                     pr["Wg"], pr["bg"])
                loss, got = _grads(B, ep, l, preds[l - 1])
                what = f"{name} layer {l} k={n_valid} write={write_idx}"
                assert abs(loss - want_loss) <= 1e-5 * abs(want_loss), (what, loss, want_loss)
                for a in NAMES:
                    if np.all(want[a] == 0):
                        assert np.all(got[a] == 0), f"{what}: G_{a} must be zero"
                    else:
                        assert_close(got[a], want[a], f"{what}: G_{a}")
    finally:
        ep.close()


def test_mini_batch_weights_and_reproducibility(B):
    import torch
    wl = make_workload("medium", shrink=16)
    ep, P, dtil = _setup(B, wl)
    rng = np.random.default_rng(9)
    try:
        preds = pred_to_device(wl.pred, B, 0)
        cache = _random_ring(rng, P, wl, wl.tau, 2)
        for l in range(1, wl.L):
            B.sat_cache_import(ep.ctx, l, cache.buf[l - 1])
        B.sat_cache_set_state(ep.ctx, 2, wl.tau)
        rw = []
        for m in range(P.M):
            nh = P.halo_gid[m].shape[0]
            w = np.zeros(nh)
            pick = rng.permutation(nh)[: max(1, nh // 4)]
            w[pick] = 1.0 / pick.shape[0]
            rw.append(w)
        rw_dev = dev(np.concatenate(rw).astype(np.float32))
        l = 1
        pr = wl.pred[0]
        want_loss, want = orc.pred_loss_grad(P, dtil, cache.snapshots(l), cache.buf[0][2], pr["Wx"], pr["Uh"], pr["b"], pr["Wg"], pr["bg"],
                                             row_weight=rw)
        loss, got = _grads(B, ep, l, preds[0], rw_dev)
        assert abs(loss - want_loss) <= 1e-5 * abs(want_loss)
        for a in NAMES:
            assert_close(got[a], want[a], f"mini-batch G_{a}")
        loss2, got2 = _grads(B, ep, l, preds[0], rw_dev)
        assert loss2 == loss and all(np.array_equal(got[a], got2[a]) for a in NAMES), "not bit-reproducible"
    finally:
        ep.close()


def test_update_inside_running_epochs(B):
    """Algorithm 1 with the predictor update switched on: epochs on real embeddings; in an update epoch the gradient is
    checked against the oracle on the ring exported from the device, the step lowers the objective, and the next epoch's
    prediction uses the new parameters."""
    import torch
    from tests.gpu_util import dev2d
    wl = make_workload("medium", shrink=16)
    ep, P, dtil = _setup(B, wl)
    perm = np.concatenate(P.inner_gid)
    ep.set_inputs(dev2d(wl.X), dev(wl.labels[perm]))
    try:
        Wd = [dev(w) for w in wl.W]
        bd = [dev(x) for x in wl.b]
        preds = pred_to_device(wl.pred, B, 1)
        for _ in range(wl.tau + 1):
            ep.step(Wd, bd, preds, 0.05)
        # an epoch by hand: forward + backward, then the update before the commit
        ep.loss_sum.zero_()
        ep._forward_backward(B.SAT_ALL_PARTS, Wd, bd, preds, 0, 0)
        write_idx, n_valid = B.sat_cache_state(ep.ctx)
        for l in range(1, wl.L):
            ring = B.sat_cache_export(ep.ctx, l, wl.tau, P.n_slots, wl.dims[l])
            snaps = [ring[(write_idx - 1 - a) % (wl.tau + 1)] for a in range(n_valid - 1, -1, -1)]
            par = {a: t.cpu().numpy() for a, t in zip(NAMES, preds[l - 1]._keep)}
            want_loss, want = orc.pred_loss_grad(P, dtil, snaps, ring[write_idx], **par)
            loss, got = _grads(B, ep, l, preds[l - 1])
            assert abs(loss - want_loss) <= 1e-5 * abs(want_loss)
            for a in NAMES:
                assert_close(got[a], want[a], f"running epoch, layer {l}: G_{a}")
        before = [p.version for p in preds]
        seen = ep.pred_update(preds, 0.05, max_steps=4, min_gain=1e-4)
        for l, losses in enumerate(seen, start=1):
            assert len(losses) >= 2 and losses[1] < losses[0], (l, losses)
        assert all(p.version > v for p, v in zip(preds, before))
        B.sat_cache_commit(ep.ctx)
        ep.step(Wd, bd, preds, 0.05, pred_lr=0.05)     # the next epochs run with the updated predictor
        ep.step(Wd, bd, preds, 0.05)
        torch.cuda.synchronize()
        assert np.isfinite(float(ep.loss_sum.item()))
    finally:
        ep.close()


def test_degenerate_cases_and_argument_errors(B):
    """One partition (no halo, no cached node): empty objective, zero gradients, history flag is a no-op.  Unsupported
    requests are refused with a status, not run."""
    import torch
    from tests.gpu_util import dev2d
    wl = make_workload("odd", M=1)
    ep, P, dtil = _setup(B, wl)
    try:
        assert P.n_slots == 0 and ep.nb == 0
        perm = np.concatenate(P.inner_gid)
        ep.set_inputs(dev2d(wl.X), dev(wl.labels[perm]))
        Wd = [dev(w) for w in wl.W]
        bd = [dev(x) for x in wl.b]
        preds = pred_to_device(wl.pred, B, 0)
        ep.step(Wd, bd, preds, grad_history=True)
        ep.loss_sum.zero_()
        ep._forward_backward(B.SAT_ALL_PARTS, Wd, bd, preds, 0, 0, True)
        loss, got = _grads(B, ep, 1, preds[0])
        assert loss == 0.0 and all(np.all(g == 0) for g in got.values())
        B.sat_cache_commit(ep.ctx)
        # the single-partition epoch equals the oracle's unpartitioned epoch
        res = orc.run_epoch(P, dtil, orc.CacheRing(0, wl.dims[1:-1], wl.tau), wl.X, wl.labels, wl.W, wl.b, None, wl.loss)
        torch.cuda.synchronize()
        for l in range(wl.L):
            assert_close(ep.gW[l].cpu().numpy(), res.G_W[l], f"single partition G_W{l + 1}")
    finally:
        ep.close()
    wl = make_workload("tiny")
    ep, P, dtil = _setup(B, wl)
    try:
        from sat_synth import as_gru
        gru = pred_to_device(as_gru(wl.pred), B, 0)
        g = tuple(torch.zeros_like(t) for t in gru[0]._keep)
        with pytest.raises(B.SatError) as e:
            B.sat_pred_grad(ep.ctx, 1, gru[0], None, *g)          # only the LSTM predictor is differentiated
        assert e.value.status == B.SAT_EINVAL
        lstm = pred_to_device(wl.pred, B, 0)
        g = tuple(torch.zeros_like(t) for t in lstm[0]._keep)
        with pytest.raises(B.SatError) as e:
            B.sat_pred_grad(ep.ctx, wl.L, lstm[0], None, *g)      # not a cached layer
        assert e.value.status == B.SAT_EINVAL
        with pytest.raises(B.SatError) as e:
            B.sat_grad_history_read(ep.ctx, 2, 0, P.n_slots, wl.dims[2])   # nothing committed yet
        assert e.value.status == B.SAT_ESTATE
        # a context stays usable after refused calls
        B.sat_pred_grad(ep.ctx, 1, lstm[0], None, *g)
        torch.cuda.synchronize()
        assert all(bool(torch.isfinite(t).all()) for t in g)
    finally:
        ep.close()
