"""Parity at full workload sizes, in the launch configuration bench.py times (all partitions per launch).

medium (the benchmark workload) always runs: whole epochs against the oracle.
dense / large / multilabel run at full size too (minutes of host time to generate 100 M+ edges in numpy; SAT_TEST_SHRINK=8
in the environment runs the same checks on the workloads shrunk 8x, for a quick look).  Those checks use what the oracle
can compute in seconds: partition structures of sampled partitions (bit-exact), predictor and layer outputs on sampled
rows with the oracle computing exactly the inputs those rows need, and whole sampled partitions forward and backward.
"""
import os

import numpy as np
import pytest

from oracle import sat_ref as orc
from sat_synth import embedding_table, make_workload, table_rows
import copy

from tests.gpu_util import TIE, assert_close, dev, dev2d, empty2d, pred_to_device, relu_tie_masks

pytestmark = pytest.mark.gpu
SHRINK = int(os.environ.get("SAT_TEST_SHRINK", "1"))


@pytest.fixture(scope="module")
def B():
    import paper_2308_13466_b200.binding as binding
    return binding


def test_medium_full_size_epochs(B):
    """The benchmark workload, batched launches, two epochs from an empty ring (k = 0, then k = 1)."""
    import torch
    from paper_2308_13466_b200.epoch import SatEpoch
    wl = make_workload("medium")
    part = orc.contig_blocks(wl.n, wl.M)
    dtil, _ = orc.degrees(wl.rowptr)
    P = orc.build_partition(wl.rowptr, wl.col, part, wl.M)
    ep = SatEpoch(wl.rowptr, wl.col, wl.M, wl.dims, wl.tau, wl.loss)
    try:
        # every integer structure, bit-exact
        gpart, gslot, n_slots = B.sat_slot_map(ep.ctx, wl.n)
        assert np.array_equal(gpart, part) and np.array_equal(gslot, P.slot) and n_slots == P.n_slots
        for m in range(wl.M):
            got = B.sat_part_lists(ep.ctx, m)
            for key, want in (("inner_gid", P.inner_gid[m]), ("halo_gid", P.halo_gid[m]), ("halo_slot", P.halo_slot[m]),
                              ("push_local", P.push_local[m]), ("push_slot", P.push_slot[m]), ("loc_rowptr", P.loc_rowptr[m]),
                              ("loc_col", P.loc_col[m]), ("hrow_ptr", P.hrow_ptr[m]), ("hrow_col", P.hrow_col[m])):
                assert np.array_equal(got[key], want), f"{key}[{m}]"
        perm = np.concatenate(P.inner_gid)
        ep.set_inputs(dev2d(wl.X), dev(wl.labels[perm]))
        Wd = [dev(w) for w in wl.W]
        bd = [dev(x) for x in wl.b]
        preds = pred_to_device(wl.pred, B)
        cache = orc.CacheRing(P.n_slots, wl.dims[1:-1], wl.tau)
        for t in (1, 2):
            before = copy.deepcopy(cache)
            res = orc.run_epoch(P, dtil, cache, wl.X, wl.labels, wl.W, wl.b, wl.pred, wl.loss, keep=True)
            ep.step(Wd, bd, preds)
            torch.cuda.synchronize()
            H_gpu = [None] + [ep.H[l].cpu().numpy() for l in range(1, wl.L + 1)]
            for l in range(1, wl.L + 1):
                want = np.concatenate([res.per_part[m]["H"][l - 1] for m in range(wl.M)])
                assert_close(H_gpu[l], want, f"epoch {t} H^{l}")
            assert abs(float(ep.loss_sum.item()) - res.loss) <= 1e-5 * abs(res.loss)
            # ReLU ties (|Z| at rounding level): among 87 M hidden activations some are decided differently by the two
            # sides; the oracle's backward is redone with the CUDA path's decision on exactly those entries
            masks, redo = relu_tie_masks(res, P, H_gpu, ep.inner_off, wl.L)
            if redo:
                del res
                cache = before
                res = orc.run_epoch(P, dtil, cache, wl.X, wl.labels, wl.W, wl.b, wl.pred, wl.loss, keep=False, masks=masks)
            for l in range(wl.L):
                assert_close(ep.gW[l].cpu().numpy(), res.G_W[l], f"epoch {t} G_W{l + 1}")
                assert_close(ep.gb[l].cpu().numpy(), res.G_b[l], f"epoch {t} G_b{l + 1}")
            for l in range(1, wl.L):
                ring = B.sat_cache_read(ep.ctx, l, 0, P.n_slots, wl.dims[l])
                assert_close(ring, cache.newest(l), f"epoch {t} newest snapshot of layer {l}")
                B.sat_cache_import(ep.ctx, l, cache.buf[l - 1])
            del res
    finally:
        ep.close()


def test_medium_full_size_predictor_gradient(B):
    """sat_pred_grad at the benchmark's size on a ring of real embeddings: tau epochs on the device fill the ring, the
    forward of one more epoch fills the write buffer; the oracle gets both through the export and computes the objective
    and the gradient of every predictor array in float64."""
    import torch
    from paper_2308_13466_b200.epoch import SatEpoch
    wl = make_workload("medium")
    part = orc.contig_blocks(wl.n, wl.M)
    dtil, _ = orc.degrees(wl.rowptr)
    P = orc.build_partition(wl.rowptr, wl.col, part, wl.M)
    ep = SatEpoch(wl.rowptr, wl.col, wl.M, wl.dims, wl.tau, wl.loss)
    try:
        perm = np.concatenate(P.inner_gid)
        ep.set_inputs(dev2d(wl.X), dev(wl.labels[perm]))
        Wd = [dev(w) for w in wl.W]
        bd = [dev(x) for x in wl.b]
        preds = pred_to_device(wl.pred, B, 1)
        for _ in range(wl.tau):
            ep.step(Wd, bd, preds, 0.05)
        ep.loss_sum.zero_()
        ep._forward_backward(B.SAT_ALL_PARTS, Wd, bd, preds, 0, 0)
        write_idx, n_valid = B.sat_cache_state(ep.ctx)
        assert n_valid == wl.tau
        names = ("Wx", "Uh", "b", "Wg", "bg")
        for l in range(1, wl.L):
            ring = B.sat_cache_export(ep.ctx, l, wl.tau, P.n_slots, wl.dims[l])
            snaps = [ring[(write_idx - 1 - a) % (wl.tau + 1)] for a in range(n_valid - 1, -1, -1)]
            pr = wl.pred[l - 1]
            want_loss, want = orc.pred_loss_grad(P, dtil, snaps, ring[write_idx], pr["Wx"], pr["Uh"], pr["b"], pr["Wg"], pr["bg"])
            g = tuple(torch.full_like(t, float("nan")) for t in preds[l - 1]._keep)
            loss = B.sat_pred_grad(ep.ctx, l, preds[l - 1], None, *g, want_loss=True)
            assert abs(loss - want_loss) <= 1e-5 * abs(want_loss), (l, loss, want_loss)
            for a, t in zip(names, g):
                assert_close(t.cpu().numpy(), want[a], f"full-size predictor gradient, layer {l}: G_{a}")
            del ring, snaps
    finally:
        ep.close()


def test_medium_full_size_gradient_history(B):
    """Two epochs with the gradient-side history at the benchmark's size, from an empty ring: the second one back-propagates
    with the stale term."""
    import torch
    from paper_2308_13466_b200.epoch import SatEpoch
    wl = make_workload("medium")
    part = orc.contig_blocks(wl.n, wl.M)
    dtil, _ = orc.degrees(wl.rowptr)
    P = orc.build_partition(wl.rowptr, wl.col, part, wl.M)
    ep = SatEpoch(wl.rowptr, wl.col, wl.M, wl.dims, wl.tau, wl.loss)
    try:
        perm = np.concatenate(P.inner_gid)
        ep.set_inputs(dev2d(wl.X), dev(wl.labels[perm]))
        Wd = [dev(w) for w in wl.W]
        bd = [dev(x) for x in wl.b]
        preds = pred_to_device(wl.pred, B)
        cache = orc.CacheRing(P.n_slots, wl.dims[1:-1], wl.tau)
        hist = orc.GradHistory(P.n_slots, wl.dims[2:])
        for t in (1, 2):
            before, hist_before = copy.deepcopy(cache), copy.deepcopy(hist)
            res = orc.run_epoch(P, dtil, cache, wl.X, wl.labels, wl.W, wl.b, wl.pred, wl.loss, keep=True, grad_hist=hist)
            ep.step(Wd, bd, preds, grad_history=True)
            torch.cuda.synchronize()
            H_gpu = [None] + [ep.H[l].cpu().numpy() for l in range(1, wl.L + 1)]
            masks, redo = relu_tie_masks(res, P, H_gpu, ep.inner_off, wl.L)
            if redo:
                del res
                cache, hist = before, hist_before
                res = orc.run_epoch(P, dtil, cache, wl.X, wl.labels, wl.W, wl.b, wl.pred, wl.loss, keep=False, masks=masks, grad_hist=hist)
            for l in range(wl.L):
                assert_close(ep.gW[l].cpu().numpy(), res.G_W[l], f"epoch {t} G_W{l + 1} with the gradient history")
                assert_close(ep.gb[l].cpu().numpy(), res.G_b[l], f"epoch {t} G_b{l + 1} with the gradient history")
            for j in range(2, wl.L + 1):
                got = B.sat_grad_history_read(ep.ctx, j, 0, P.n_slots, wl.dims[j])
                assert_close(got, hist.read[j - 2], f"epoch {t} history of layer {j}")
                B.sat_grad_history_write(ep.ctx, j, wl.dims[j], hist.read[j - 2])
            for l in range(1, wl.L):
                B.sat_cache_import(ep.ctx, l, cache.buf[l - 1])
            del res
    finally:
        ep.close()


def _compact_predictor_oracle(P, m, dtil, wl, layer, halo_rows, table, tau):
    """Oracle prediction for the given halo rows of partition m from a ring whose snapshot s holds, for node u,
    table_rows(table, u, salt(s, layer)): the recurrent state is computed only for the cache slots those rows read (the halo
    nodes themselves and their neighbours inside the partition), on compact arrays addressed through a renumbered slot map."""
    import copy
    halo_rows = np.asarray(halo_rows, dtype=np.int32)
    u = P.halo_gid[m][halo_rows]
    nb = [P.inner_gid[m][P.hrow_col[m][P.hrow_ptr[m][j]:P.hrow_ptr[m][j + 1]]] for j in halo_rows]
    gids = np.unique(np.concatenate([u] + nb))
    slot2 = np.full(P.n, -1, dtype=np.int32)
    slot2[gids] = np.arange(gids.shape[0], dtype=np.int32)
    snaps = [np.ascontiguousarray(table_rows(table, gids, _salt(s, layer))) for s in range(tau)]     # oldest first
    pr = wl.pred[layer - 1]
    h, d = pr["Wg"].shape
    S = orc.lstm_state(snaps, d, h, pr["Wx"], pr["Uh"], pr["b"], gids.shape[0])
    P2 = copy.copy(P)
    P2.slot = slot2
    out = orc.predict_halo(P2, m, dtil, S, snaps[-1], pr["Wg"], pr["bg"], rows_sel=halo_rows)
    return out[halo_rows]


def _salt(s: int, layer: int) -> int:
    return 1 + s + 100 * layer


@pytest.mark.parametrize("name", ["dense", "large", "multilabel"])
def test_big_workloads_full_size(B, name):
    """The three large configurations at their full size, all partitions per launch (the configuration bench.py times).
    What the oracle cannot compute whole in minutes it computes row by row, on the inputs those rows need:
      - integer structures of three partitions, bit-exact;
      - the ring is filled with tau seeded snapshots through the push call itself; sat_predict (LSTM over the window, graph
        convolution, skip connection) on sampled halo rows of those partitions, among them the row with the most neighbours;
      - one whole epoch with that full ring: sampled rows of H^1 and of H^2 (the latter through the predicted halo
        embeddings), the pushed rows;
      - per partition, every layer shape (first, hidden, classifier): sat_layer_fwd and sat_layer_bwd of the whole
        partition on seeded inputs: H, G_W, G_b, G_in, G_halo against the oracle."""
    import torch
    from paper_2308_13466_b200.epoch import SatEpoch
    wl = make_workload(name, shrink=SHRINK)
    rng = np.random.default_rng(1)
    part = orc.contig_blocks(wl.n, wl.M)
    dtil, dinv = orc.degrees(wl.rowptr)
    sample_parts = [0, wl.M // 2, wl.M - 1]
    P = orc.build_partition(wl.rowptr, wl.col, part, wl.M, only_parts=sample_parts)
    ep = SatEpoch(wl.rowptr, wl.col, wl.M, wl.dims, wl.tau, wl.loss)
    ctx = ep.ctx
    try:
        assert_close(B.sat_graph_dinv(ctx, wl.n), dinv, "dinv", 1e-6)
        gpart, gslot, n_slots = B.sat_slot_map(ctx, wl.n)
        assert np.array_equal(gpart, part) and np.array_equal(gslot, P.slot) and n_slots == P.n_slots
        tot = B.sat_part_sizes(ctx, B.SAT_ALL_PARTS)
        assert tot[0] == wl.n and tot[2] == wl.nnz and tot[3] == P.n_slots
        for m in sample_parts:
            got = B.sat_part_lists(ctx, m)
            for key, want in (("inner_gid", P.inner_gid[m]), ("halo_gid", P.halo_gid[m]), ("halo_slot", P.halo_slot[m]),
                              ("push_local", P.push_local[m]), ("push_slot", P.push_slot[m]), ("loc_rowptr", P.loc_rowptr[m]),
                              ("loc_col", P.loc_col[m]), ("hrow_ptr", P.hrow_ptr[m]), ("hrow_col", P.hrow_col[m])):
                assert np.array_equal(got[key], want), f"{key}[{m}]"
            del got
        print(f"{name}: n={wl.n} nnz={wl.nnz} |C|/n={P.n_slots / wl.n:.4f} halo rows={tot[1]} ({tot[1] / wl.n:.2f} n)")
        # partition-major order of all rows = concatenated inner lists; partitions are contiguous id blocks here
        perm = np.arange(wl.n)
        ep.set_inputs(dev2d(wl.X), dev(wl.labels[perm]))
        Wd = [dev(w) for w in wl.W]
        bd = [dev(x) for x in wl.b]
        preds = pred_to_device(wl.pred, B)
        # ---- fill the ring: snapshot s of cached layer l holds table_l[(u * 7919 + salt(s, l) * 104729) mod 8191] for node u ----
        tables = {l: embedding_table(wl.seed, wl.dims[l]) for l in range(1, wl.L)}
        ids = torch.arange(wl.n, device="cuda", dtype=torch.int64)
        for s in range(wl.tau):
            for l in range(1, wl.L):
                t_dev = dev(tables[l])
                rows = t_dev.index_select(0, (ids * 7919 + _salt(s, l) * 104729) % t_dev.shape[0])
                B.sat_cache_update(ctx, B.SAT_ALL_PARTS, l, rows)
                del rows, t_dev
            B.sat_cache_commit(ctx)
        assert B.sat_cache_state(ctx) == (wl.tau, wl.tau)
        # ---- sat_predict on sampled halo rows ----
        sel_halo = {}
        for i, m in enumerate(sample_parts):
            b_m = P.halo_gid[m].shape[0]
            hlen = np.diff(P.hrow_ptr[m])
            sel = np.unique(np.concatenate([rng.integers(0, b_m, size=24), [int(np.argmax(hlen))]])).astype(np.int32)
            sel_halo[m] = sel
            out = empty2d(b_m, wl.dims[1])
            B.sat_predict(ctx, 1, m, preds[0], 0 if i == 0 else 1, out)
            got = out[torch.from_numpy(sel.astype(np.int64)).cuda()].cpu().numpy()
            want = _compact_predictor_oracle(P, m, dtil, wl, 1, sel, tables[1], wl.tau)
            assert_close(got, want, f"{name} predicted halo rows of partition {m} (longest row: {int(hlen.max())} neighbours)")
            del out
        # ---- one epoch, all partitions per launch, ring full ----
        ep.step(Wd, bd, preds)
        torch.cuda.synchronize()
        assert B.sat_cache_state(ctx) == (0, wl.tau)
        for m in sample_parts:
            inner, halo = P.inner_gid[m], P.halo_gid[m]
            r0 = int(inner[0])
            n_m = inner.shape[0]
            # sampled rows, plus the longest row of the partition (cut into many SpMM chunks)
            rows_len = np.diff(P.loc_rowptr[m])
            sel = np.unique(np.concatenate([rng.integers(0, n_m, size=48), [int(np.argmax(rows_len))]])).astype(np.int32)
            _, _, H1o = orc.layer_fwd(P, m, dtil, wl.X[inner], wl.X[halo], wl.W[0], wl.b[0], 1, rows_sel=sel)
            H1g = ep.H[1][torch.from_numpy(r0 + sel.astype(np.int64)).cuda()].cpu().numpy()
            assert_close(H1g, H1o[sel], f"{name} H^1 sampled rows of partition {m}")
            # layer 2 on a few rows: the oracle computes H^1 for exactly the inner neighbours those rows read and the
            # predicted embeddings for exactly the halo neighbours they read
            sel2 = sel[:8]
            need = np.unique(np.concatenate([P.loc_col[m][P.loc_rowptr[m][r]:P.loc_rowptr[m][r + 1]] for r in sel2]))
            need_in = need[need < n_m].astype(np.int32)
            need_halo = (need[need >= n_m] - n_m).astype(np.int32)
            _, _, H1need = orc.layer_fwd(P, m, dtil, wl.X[inner], wl.X[halo], wl.W[0], wl.b[0], 1, rows_sel=need_in)
            halo2 = np.zeros((halo.shape[0], wl.dims[1]), dtype=np.float32)
            if need_halo.shape[0]:
                halo2[need_halo] = _compact_predictor_oracle(P, m, dtil, wl, 1, need_halo, tables[1], wl.tau)
            _, _, H2o = orc.layer_fwd(P, m, dtil, H1need, halo2, wl.W[1], wl.b[1], 1 if wl.L > 2 else 0, rows_sel=sel2)
            H2g = ep.H[2][torch.from_numpy(r0 + sel2.astype(np.int64)).cuda()].cpu().numpy()
            assert_close(H2g, H2o[sel2], f"{name} H^2 sampled rows of partition {m} ({need_halo.shape[0]} predicted halo rows)")
            del H1need, halo2
            # what was pushed is the boundary rows of H^1
            pushed = B.sat_cache_read(ctx, 1, 0, P.n_slots, wl.dims[1])[P.push_slot[m]]
            mine = ep.H[1][torch.from_numpy(r0 + P.push_local[m].astype(np.int64)).cuda()].cpu().numpy()
            assert np.array_equal(pushed, mine)
            del pushed, mine
        loss = float(ep.loss_sum.item())
        assert np.isfinite(loss) and loss > 0
        B.sat_sync_status(ctx)
        # ---- whole partitions, layer by layer, forward and backward on seeded inputs ----
        layers = sorted({1, 2, wl.L})
        for m in sample_parts[1:]:
            inner, halo = P.inner_gid[m], P.halo_gid[m]
            n_m, b_m = inner.shape[0], halo.shape[0]
            for l in layers:
                d_in, d_out = wl.dims[l - 1], wl.dims[l]
                act = 1 if l < wl.L else 0
                tin = embedding_table(wl.seed, d_in, tag="layer-input", signed=(l == 1))
                H_in = np.ascontiguousarray(table_rows(tin, inner, 7 + l))
                H_halo = np.ascontiguousarray(table_rows(tin, halo, 7 + l))
                G_out = (np.ascontiguousarray(table_rows(embedding_table(wl.seed, d_out, tag="upstream-gradient", signed=True), inner, 11 + l))
                         / np.float32(wl.n)).astype(np.float32)
                AGG, Z, Ho = orc.layer_fwd(P, m, dtil, H_in, H_halo, wl.W[l - 1], wl.b[l - 1], act)
                h_in, h_halo = dev2d(H_in), dev2d(H_halo)
                h_out = empty2d(n_m, d_out)
                B.sat_layer_fwd(ctx, m, l, h_in, h_halo, Wd[l - 1], bd[l - 1], B.SAT_ACT_RELU if act else B.SAT_ACT_NONE, h_out)
                Hg = h_out.cpu().numpy()
                assert_close(Hg, Ho, f"{name} partition {m} layer {l}: H")
                mask = None
                if act:
                    mask = Hg > 0
                    diff = mask != (Z > 0)
                    if diff.any():
                        assert np.all(np.abs(Z[diff]) <= TIE * float(np.sqrt(np.mean(Z * Z)))), f"ReLU mask differs away from zero ({m}, {l})"
                    mask = mask.astype(np.uint8)
                del Hg, Ho, Z
                GW, Gb = np.zeros(wl.W[l - 1].shape), np.zeros(d_out)
                gin_o, ghalo_o = orc.layer_bwd(P, m, dtil, G_out, mask, AGG, wl.W[l - 1], GW, Gb, want_in=True, want_halo=True)
                del AGG
                g_out = dev2d(G_out)
                gW, gb = torch.full_like(Wd[l - 1], float("nan")), torch.full_like(bd[l - 1], float("nan"))
                g_in = empty2d(n_m, d_in)
                B.sat_layer_bwd(ctx, m, l, g_out, Wd[l - 1], gW, gb, 0, g_in, None)       # the path the epoch takes
                assert_close(gW.cpu().numpy(), GW, f"{name} partition {m} layer {l}: G_W")
                assert_close(gb.cpu().numpy(), Gb, f"{name} partition {m} layer {l}: G_b")
                assert_close(g_in.cpu().numpy(), gin_o, f"{name} partition {m} layer {l}: G_in")
                g_halo = empty2d(b_m, d_in)
                g_in.fill_(float("nan"))
                B.sat_layer_bwd(ctx, m, l, g_out, Wd[l - 1], gW, gb, 0, g_in, g_halo)     # with the optional halo gradient
                assert_close(g_in.cpu().numpy(), gin_o, f"{name} partition {m} layer {l}: G_in (halo-gradient path)")
                assert_close(g_halo.cpu().numpy(), ghalo_o, f"{name} partition {m} layer {l}: G_halo")
                del h_in, h_halo, h_out, g_out, g_in, g_halo, gin_o, ghalo_o, H_in, H_halo, G_out
        B.sat_sync_status(ctx)
    finally:
        ep.close()
