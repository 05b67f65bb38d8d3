"""GPU vs oracle on the graph-attention layer (forward and backward), per partition and all partitions per launch."""
import numpy as np
import pytest

from oracle import sat_ref as orc
from sat_synth import make_workload
from tests.gpu_util import assert_close, dev, dev2d, empty2d

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import paper_2308_13466_b200.binding as binding
    return binding


def _setup(B, wl):
    from paper_2308_13466_b200.epoch import SatEpoch
    part = wl.part_given if wl.part_given is not None else orc.contig_blocks(wl.n, wl.M)
    P = orc.build_partition(wl.rowptr, wl.col, part, wl.M)
    ep = SatEpoch(wl.rowptr, wl.col, wl.M, wl.dims, wl.tau, wl.loss, part_given=wl.part_given)
    return ep, P


def _params(rng, d_in, d_out):
    W = (rng.standard_normal((d_in, d_out)) * (1.0 / np.sqrt(d_in))).astype(np.float32)
    a_src = (rng.standard_normal(d_out) * 0.3).astype(np.float32)
    a_dst = (rng.standard_normal(d_out) * 0.3).astype(np.float32)
    bias = (rng.standard_normal(d_out) * 0.1).astype(np.float32)
    return W, a_src, a_dst, bias


@pytest.mark.parametrize("name,shrink,d_in,d_out,act", [("tiny", 1, 32, 16, 1), ("odd", 1, 50, 70, 1), ("odd", 1, 38, 7, 0),
                                                        ("medium", 16, 128, 256, 1), ("medium", 16, 256, 40, 0)])
def test_layer_per_partition_and_batched(B, name, shrink, d_in, d_out, act):
    import torch
    wl = make_workload(name, shrink=shrink)
    ep, P = _setup(B, wl)
    rng = np.random.default_rng(17)
    try:
        W, a_src, a_dst, bias = _params(rng, d_in, d_out)
        X = np.abs(rng.standard_normal((wl.n, d_in))).astype(np.float32) * 0.7       # embedding-like inputs, global id order
        G = (rng.standard_normal((wl.n, d_out)) / wl.n).astype(np.float32)
        Wd, asd, add, bd = dev(W), dev(a_src), dev(a_dst), dev(bias)
        perm = np.concatenate(P.inner_gid)
        halo_all = np.concatenate(P.halo_gid)
        inner_off = np.concatenate([[0], np.cumsum([g.shape[0] for g in P.inner_gid])])
        halo_off = np.concatenate([[0], np.cumsum([g.shape[0] for g in P.halo_gid])])
        want = dict(W=np.zeros((d_in, d_out)), a_src=np.zeros(d_out), a_dst=np.zeros(d_out), b=np.zeros(d_out))
        # the oracle, partition by partition
        fw, bw = [], []
        for m in range(P.M):
            inner, halo = P.inner_gid[m], P.halo_gid[m]
            f = orc.gat_fwd(P, m, X[inner], X[halo], W, a_src, a_dst, bias, act)
            fw.append(f)
        # all partitions in one launch set
        h_in, h_halo = dev2d(X[perm]), dev2d(X[halo_all])
        g_out = dev2d(G[perm])
        h_out = empty2d(wl.n, d_out)
        B.sat_gat_fwd(ep.ctx, B.SAT_ALL_PARTS, 1, h_in, h_halo, Wd, asd, add, bd, B.SAT_ACT_RELU if act else B.SAT_ACT_NONE, h_out)
        torch.cuda.synchronize()
        H_gpu = h_out.cpu().numpy()
        assert_close(H_gpu, np.concatenate([f["H"] for f in fw]), f"{name} forward, all partitions")
        # ReLU ties decided as the device decided them
        for m in range(P.M):
            inner, halo = P.inner_gid[m], P.halo_gid[m]
            mask = None
            if act:
                mask = H_gpu[inner_off[m]:inner_off[m + 1]] > 0
                diff = mask != (fw[m]["O"] > 0)
                if diff.any():
                    rms = float(np.sqrt(np.mean(fw[m]["O"] ** 2)))
                    assert np.all(np.abs(fw[m]["O"][diff]) <= 1e-4 * rms)
            g = orc.gat_bwd(P, m, X[inner], X[halo], W, a_src, a_dst, fw[m], G[inner], act, mask=mask)
            bw.append(g)
            for k in want:
                want[k] += g[k]
        gW, gas, gad, gb = (torch.full((d_in, d_out), float("nan"), device="cuda"), torch.full((d_out,), float("nan"), device="cuda"),
                            torch.full((d_out,), float("nan"), device="cuda"), torch.full((d_out,), float("nan"), device="cuda"))
        g_in = empty2d(wl.n, d_in)
        B.sat_gat_bwd(ep.ctx, B.SAT_ALL_PARTS, 1, g_out, h_out, h_in, h_halo, Wd, asd, add, gW, gas, gad, gb, 0, g_in)
        torch.cuda.synchronize()
        assert_close(gW.cpu().numpy(), want["W"], f"{name} G_W")
        assert_close(gas.cpu().numpy(), want["a_src"], f"{name} G_a_src")
        assert_close(gad.cpu().numpy(), want["a_dst"], f"{name} G_a_dst")
        assert_close(gb.cpu().numpy(), want["b"], f"{name} G_b")
        assert_close(g_in.cpu().numpy(), np.concatenate([g["H_in"] for g in bw]), f"{name} G_in")
        # partition by partition, accumulating: the same outputs (forward bit-identical), the summed gradients close
        h_out2 = empty2d(wl.n, d_out)
        gW2, gas2, gad2, gb2 = (torch.zeros_like(gW), torch.zeros_like(gas), torch.zeros_like(gad), torch.zeros_like(gb))
        g_in2 = empty2d(wl.n, d_in)
        for m in range(P.M):
            r0, r1, q0, q1 = inner_off[m], inner_off[m + 1], halo_off[m], halo_off[m + 1]
            B.sat_gat_fwd(ep.ctx, m, 2, h_in[r0:r1], h_halo[q0:q1], Wd, asd, add, bd, B.SAT_ACT_RELU if act else B.SAT_ACT_NONE, h_out2[r0:r1])
        for m in range(P.M - 1, -1, -1):
            r0, r1, q0, q1 = inner_off[m], inner_off[m + 1], halo_off[m], halo_off[m + 1]
            B.sat_gat_bwd(ep.ctx, m, 2, g_out[r0:r1], h_out2[r0:r1], h_in[r0:r1], h_halo[q0:q1], Wd, asd, add, gW2, gas2, gad2, gb2,
                          1, g_in2[r0:r1])
        torch.cuda.synchronize()
        assert np.array_equal(h_out2.cpu().numpy(), H_gpu), "per-partition forward differs from the batched launch"
        assert np.array_equal(g_in2.cpu().numpy(), g_in.cpu().numpy())
        assert_close(gW2.cpu().numpy(), want["W"], f"{name} G_W, per partition")
        assert_close(gas2.cpu().numpy(), want["a_src"], f"{name} G_a_src, per partition")
        assert_close(gad2.cpu().numpy(), want["a_dst"], f"{name} G_a_dst, per partition")
        # backward without a forward is refused
        with pytest.raises(B.SatError) as e:
            B.sat_gat_bwd(ep.ctx, B.SAT_ALL_PARTS, 3, g_out, h_out, h_in, h_halo, Wd, asd, add, gW, gas, gad, gb, 0, g_in)
        assert e.value.status == B.SAT_ESTATE
    finally:
        ep.close()


@pytest.mark.parametrize("name,shrink", [("tiny", 1), ("odd", 1), ("medium", 16)])
def test_epochs_with_the_attention_backbone(B, name, shrink):
    """Whole SAT epochs with graph-attention layers (pull / predict, forward, push, loss, backward, commit) against the
    oracle, from synchronised state, for an empty, a filling and a full ring."""
    import copy
    import torch
    from tests.gpu_util import TIE, pred_to_device
    wl = make_workload(name, shrink=shrink)
    ep, P = _setup(B, wl)
    dtil, _ = orc.degrees(wl.rowptr)
    rng = np.random.default_rng(23)
    try:
        perm = np.concatenate(P.inner_gid)
        ep.set_inputs(dev2d(wl.X), dev(wl.labels[perm]))
        params = []
        for l in range(wl.L):
            W, a_src, a_dst, bias = _params(rng, wl.dims[l], wl.dims[l + 1])
            params.append(dict(W=W, a_src=a_src, a_dst=a_dst, b=bias))
        preds = pred_to_device(wl.pred, B, 0)
        cache = orc.CacheRing(P.n_slots, wl.dims[1:-1], wl.tau)
        inner_off = np.concatenate([[0], np.cumsum([g.shape[0] for g in P.inner_gid])])
        for t in range(wl.tau + 2):
            pd = [{k: dev(v) for k, v in p.items()} for p in params]
            before = copy.deepcopy(cache)
            res = orc.run_epoch_gat(P, dtil, cache, wl.X, wl.labels, params, wl.pred, wl.loss)
            ep.step_gat(pd, preds)
            torch.cuda.synchronize()
            H_gpu = [None] + [ep.H[l].cpu().numpy() for l in range(1, wl.L + 1)]
            # Ties.  A hidden output (ReLU) or an attention logit (LeakyReLU) that is zero up to rounding gets its sign decided
            # by the last bit on either side, and both decisions are correct results.  The device's decisions are read back
            # (H > 0 for the ReLU; the fp32 sum s_dst[v] + s_src[u] of the exported scores for the logits); every
            # disagreement with the oracle must lie inside the tie window, and the oracle's backward is then redone with the
            # device's decisions, so that the gradients are compared at the full tolerance in every epoch.
            masks, positive, redo = [], [], False
            scores = [None] + [B.sat_gat_scores(ep.ctx, l, wl.n, ep.nb) for l in range(1, wl.L + 1)]
            for m in range(P.M):
                mm, pp = [], []
                rows, cols = orc._gat_rows(P, m)
                for l in range(1, wl.L + 1):
                    s_in, s_dst, s_halo = scores[l]
                    # scores by local column id: the partition's inner rows, then its halo positions
                    s_loc = np.concatenate([s_in[inner_off[m]:inner_off[m + 1]], s_halo[ep.halo_off[m]:ep.halo_off[m + 1]]])
                    theirs_pos = (s_dst[inner_off[m] + rows] + s_loc[cols]) > 0          # the device's fp32 sum
                    pre = res["pre"][m][l - 1]
                    diff = theirs_pos != (pre > 0)
                    if diff.any():
                        assert np.all(np.abs(pre[diff]) <= TIE * float(np.sqrt(np.mean(pre * pre)))), f"LeakyReLU slope differs away from zero ({m}, {l})"
                        redo = True
                    pp.append(theirs_pos)
                    if l < wl.L:
                        O = res["O"][m][l - 1]
                        theirs = H_gpu[l][inner_off[m]:inner_off[m + 1]] > 0
                        diff = theirs != (O > 0)
                        if diff.any():
                            assert np.all(np.abs(O[diff]) <= TIE * float(np.sqrt(np.mean(O * O)))), f"ReLU mask differs away from zero ({m}, {l})"
                            redo = True
                        mm.append(theirs)
                masks.append(mm + [None])
                positive.append(pp)
            if redo:
                cache = before
                res = orc.run_epoch_gat(P, dtil, cache, wl.X, wl.labels, params, wl.pred, wl.loss, masks=masks, positive=positive)
            for l in range(1, wl.L + 1):
                assert_close(H_gpu[l], np.concatenate([res["H"][m][l - 1] for m in range(P.M)]), f"{name} epoch {t} H^{l}")
            assert abs(float(ep.loss_sum.item()) - res["loss"]) <= 1e-5 * abs(res["loss"])
            for l in range(wl.L):
                for k in ("W", "a_src", "a_dst", "b"):
                    assert_close(ep.gat_grads[l][k].cpu().numpy(), res["grads"][l][k], f"{name} epoch {t} layer {l + 1} G_{k}")
            for l in range(1, wl.L):
                B.sat_cache_import(ep.ctx, l, cache.buf[l - 1])
            params = [{k: (v - 0.5 * res["grads"][l][k]).astype(np.float32) for k, v in p.items()} for l, p in enumerate(params)]
    finally:
        ep.close()
