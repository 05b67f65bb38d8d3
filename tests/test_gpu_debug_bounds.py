"""The bounds-checking debug build of the library (libsat_b200_dbg.so) on the small cases.

compute-sanitizer is not available where this suite runs; its stand-in is a build of the same sources in which every index
the graph kernels load is checked against the matrix it addresses: an index outside raises a status bit and is replaced by
a valid one before use (no trap, no assert, nothing outside the matrix is touched).  A process loads one build of the library, so the
checks run in a child process with SAT_B200_DEBUG=1: whole epochs of the tiny workload against the oracle with a clean
status word, then one column id is overwritten with a value far outside, the layer forward must report it through
sat_sync_status (SAT_EDATA, once) and leave the context usable, and with the id restored the results are the regular ones.
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _child():
    import numpy as np
    import torch
    sys.path.insert(0, ROOT)
    import paper_2308_13466_b200.binding as B
    from paper_2308_13466_b200.build import lib_path
    from paper_2308_13466_b200.epoch import SatEpoch
    from oracle import sat_ref as orc
    from sat_synth import make_workload
    from tests.gpu_util import assert_close, dev, dev2d, empty2d, pred_to_device
    assert B._lib._name == lib_path(debug=True), B._lib._name
    wl = make_workload("tiny")
    dtil, _ = orc.degrees(wl.rowptr)
    P = orc.build_partition(wl.rowptr, wl.col, wl.part_given, wl.M)
    cache = orc.CacheRing(P.n_slots, wl.dims[1:-1], wl.tau)
    ep = SatEpoch(wl.rowptr, wl.col, wl.M, wl.dims, wl.tau, wl.loss, part_given=wl.part_given)
    try:
        if os.environ.get("SAT_TEST_EXPECT_BLOCKED"):
            assert B.sat_spmm_plan(ep.ctx, B.SAT_ALL_PARTS, wl.dims[1])[0] > 1
        perm = np.concatenate(P.inner_gid)
        ep.set_inputs(dev2d(wl.X), dev(wl.labels[perm]))
        W, b = [dev(w) for w in wl.W], [dev(x) for x in wl.b]
        preds = pred_to_device(wl.pred, B)
        for t in range(wl.tau + 1):                      # every ring fill level, all kernels of the epoch under the checks
            res = orc.run_epoch(P, dtil, cache, wl.X, wl.labels, wl.W, wl.b, wl.pred, wl.loss)
            ep.step(W, b, preds)
            B.sat_sync_status(ep.ctx)                    # clean: no index left its matrix
            assert_close(ep.H[wl.L].cpu().numpy(), np.concatenate([r["H"][-1] for r in res.per_part]), f"debug build, epoch {t}: logits")
            for l in range(wl.L):
                assert_close(ep.gW[l].cpu().numpy(), res.G_W[l], f"debug build, epoch {t}: G_W{l + 1}")
        # one column id far outside: reported, replaced, context usable
        m = 1
        inner, halo = P.inner_gid[m], P.halo_gid[m]
        h_in, h_halo = dev2d(wl.X[inner]), dev2d(wl.X[halo])
        good = empty2d(inner.shape[0], wl.dims[1])
        B.sat_layer_fwd(ep.ctx, m, 1, h_in, h_halo, W[0], b[0], B.SAT_ACT_RELU, good)
        B.sat_sync_status(ep.ctx)
        pos = int(sum(int(P.loc_rowptr[q][-1]) for q in range(m))) + 5           # an entry of partition m's local CSR
        old = B.sat_debug_poke_index(ep.ctx, 0, pos, wl.n + int(ep.nb) + 12345)
        bad = empty2d(inner.shape[0], wl.dims[1])
        B.sat_layer_fwd(ep.ctx, m, 1, h_in, h_halo, W[0], b[0], B.SAT_ACT_RELU, bad)
        try:
            B.sat_sync_status(ep.ctx)
            raise AssertionError("the out-of-range column id went unnoticed")
        except B.SatError as e:
            assert e.status == B.SAT_EDATA, e
        B.sat_sync_status(ep.ctx)                        # reported once
        assert bool(torch.isfinite(bad).all())
        B.sat_debug_poke_index(ep.ctx, 0, pos, old)
        again = empty2d(inner.shape[0], wl.dims[1])
        B.sat_layer_fwd(ep.ctx, m, 1, h_in, h_halo, W[0], b[0], B.SAT_ACT_RELU, again)
        B.sat_sync_status(ep.ctx)
        assert torch.equal(again, good)
    finally:
        ep.close()
    print("debug-bounds child ok")


@pytest.mark.parametrize("source_blocked", [False, True])
def test_bounds_checking_build_on_the_small_cases(source_blocked):
    """source_blocked: the forward aggregation walks its source-blocked work list (forced: blocks of a few hundred
    rows, every partition) instead of the row-by-row one, so that kernel's index checks run too."""
    from paper_2308_13466_b200.build import build
    build(debug=True)
    env = dict(os.environ, SAT_B200_DEBUG="1")
    if source_blocked:
        env["SAT_SPMM_SRC_BLOCK"] = "16384,16384,0"
        env["SAT_TEST_EXPECT_BLOCKED"] = "1"
    else:
        env.pop("SAT_SPMM_SRC_BLOCK", None)
    out = subprocess.run([sys.executable, os.path.abspath(__file__), "--child"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert out.returncode == 0 and "debug-bounds child ok" in out.stdout, out.stdout[-2000:] + out.stderr[-4000:]


def test_poke_is_refused_by_the_regular_build():
    import paper_2308_13466_b200.binding as B
    ctx = B.sat_create(0, 0)
    try:
        with pytest.raises(B.SatError) as ei:
            B.sat_debug_poke_index(ctx, 0, 0, 0)
        assert ei.value.status == B.SAT_ESTATE
    finally:
        B.sat_destroy(ctx)


if __name__ == "__main__" and "--child" in sys.argv:
    _child()
