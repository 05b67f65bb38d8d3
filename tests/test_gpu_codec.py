"""GPU vs oracle for the embedding codec (Supplement, "Data Compression for Historical Embedding Storage"): sizes, row
offsets and bytes bit-exact, decoded floats bit-exact, ragged shapes and extreme values, malformed input, and the
in-place requantisation of a ring snapshot."""
import numpy as np
import pytest

from oracle import sat_ref as orc
from sat_synth import make_workload
from tests.gpu_util import dev, dev2d, pred_to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import paper_2308_13466_b200.binding as binding
    return binding


@pytest.fixture(scope="module")
def ctx(B):
    c = B.sat_create(0, 0)
    yield c
    B.sat_destroy(c)


def _encode_gpu(B, ctx, x_dev, p):
    import torch
    rows = x_dev.shape[0]
    off = torch.zeros(rows + 1, dtype=torch.int64, device="cuda")
    total = B.sat_codec_plan(ctx, x_dev, p, off)
    out = torch.full((max(total, 1),), 255, dtype=torch.uint8, device="cuda")
    B.sat_codec_encode(ctx, x_dev, p, off, out)
    return out[:total], off, total


def _case(rng, rows, d, scale):
    x = (rng.normal(size=(rows, d)) * scale).astype(np.float32)
    if rows > 2:
        x[1] = 0.0                                        # all-zero row
        x[2, ::3] = np.maximum(x[2, ::3], 0)              # ReLU-like zeros inside a row
    return x


@pytest.mark.parametrize("rows,d,p,scale", [
    (1, 1, 0, 5.0), (33, 7, 2, 1.0), (1000, 40, 5, 1.0), (257, 256, 3, 2.0), (64, 300, 7, 0.5), (5, 1025, 1, 100.0),
    (300, 64, 0, 1e6), (17, 33, 7, 1e-4), (4096, 72, 4, 1.0)])
def test_bytes_offsets_and_floats_are_bit_exact(B, ctx, rows, d, p, scale):
    import torch
    rng = np.random.default_rng(rows * 131 + d)
    x = _case(rng, rows, d, scale)
    data_o, off_o = orc.codec_encode(x, p)
    xd = dev2d(x)                                         # padded leading dimension
    data_g, off_g, total = _encode_gpu(B, ctx, xd[:, :d], p)
    assert total == int(off_o[-1])
    assert np.array_equal(off_g.cpu().numpy(), off_o)
    assert np.array_equal(data_g.cpu().numpy(), data_o)
    back = torch.full_like(xd, float("nan"))
    B.sat_codec_decode(ctx, data_g, off_g, p, back[:, :d])
    B.sat_sync_status(ctx)
    want = orc.codec_decode(data_o, off_o, d, p)
    assert np.array_equal(back[:, :d].cpu().numpy(), want)
    if back.shape[1] > d:
        assert bool(torch.isnan(back[:, d:]).all()), "decode wrote outside the row"


def test_extreme_values_and_ties(B, ctx):
    import torch
    x = np.array([[0.5, -0.5, 1.5, -2.5, 0.0, -0.0, 3.4e30, -3.4e30, 1e-30, 2.0 ** 24, -(2.0 ** 24) - 2, 123456.789]],
                 dtype=np.float32)
    x[0, 6:8] = [9.0e10, -9.0e10]                         # 9e10 * 1e7 < 2^62: still inside the 64-bit range at p = 7
    for p in (0, 3, 7):
        data_o, off_o = orc.codec_encode(x, p)
        data_g, off_g, _ = _encode_gpu(B, ctx, dev2d(x)[:, :x.shape[1]], p)
        assert np.array_equal(data_g.cpu().numpy(), data_o), p
        back = torch.zeros((1, 12), dtype=torch.float32, device="cuda")
        B.sat_codec_decode(ctx, data_g, off_g, p, back)
        B.sat_sync_status(ctx)
        assert np.array_equal(back.cpu().numpy(), orc.codec_decode(data_o, off_o, 12, p))


def test_empty_and_capacity(B, ctx):
    import torch
    off = torch.zeros(1, dtype=torch.int64, device="cuda")
    x0 = torch.zeros((0, 8), dtype=torch.float32, device="cuda")
    assert B.sat_codec_plan(ctx, x0, 3, off) == 0
    x = dev2d(np.ones((4, 8), dtype=np.float32))[:, :8]
    off = torch.zeros(5, dtype=torch.int64, device="cuda")
    total = B.sat_codec_plan(ctx, x, 3, off)
    small = torch.zeros(total - 1, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SatError):
        B.sat_codec_encode(ctx, x, 3, off, small)
    with pytest.raises(B.SatError):
        B.sat_codec_plan(ctx, x, 8, off)                  # precision outside 0..7


def test_malformed_rows_raise_edata_and_leave_the_context_usable(B, ctx):
    import torch
    x = np.arange(12, dtype=np.float32).reshape(2, 6)
    data_g, off_g, total = _encode_gpu(B, ctx, dev2d(x)[:, :6], 1)
    back = torch.zeros((2, 6), dtype=torch.float32, device="cuda")
    bad = data_g.clone()
    bad[total - 1] = ord("_")                             # continuation bit on the last byte
    B.sat_codec_decode(ctx, bad, off_g, 1, back)
    with pytest.raises(B.SatError) as ei:
        B.sat_sync_status(ctx)
    assert ei.value.status == B.SAT_EDATA
    wrong_d = torch.zeros((2, 5), dtype=torch.float32, device="cuda")
    B.sat_codec_decode(ctx, data_g, off_g, 1, wrong_d)    # one value too many per row
    with pytest.raises(B.SatError):
        B.sat_sync_status(ctx)
    # an offset table that does not match the byte buffer (past its end, negative, descending): the rows are flagged
    # and skipped, nothing outside the buffer is read
    for r, val in ((2, total + 4096), (0, -8), (1, total + 1)):
        off_bad = off_g.clone()
        off_bad[r] = val
        B.sat_codec_decode(ctx, data_g, off_bad, 1, back)
        with pytest.raises(B.SatError) as ei:
            B.sat_sync_status(ctx)
        assert ei.value.status == B.SAT_EDATA
    B.sat_codec_decode(ctx, data_g, off_g, 1, back)       # and the context still works
    B.sat_sync_status(ctx)
    assert np.array_equal(back.cpu().numpy(), orc.codec_decode(data_g.cpu().numpy(), off_g.cpu().numpy(), 6, 1))


def test_requantised_ring_snapshot(B):
    """Snapshots of a running ring stored at three decimals: the ring holds exactly the oracle's encode + decode image,
    the reported size is the oracle's, and the next epoch (predictor reading the requantised history) matches the oracle
    run on the same history."""
    import torch
    from paper_2308_13466_b200.epoch import SatEpoch
    wl = make_workload("medium", shrink=16)
    part = orc.contig_blocks(wl.n, wl.M)
    dtil, _ = orc.degrees(wl.rowptr)
    P = orc.build_partition(wl.rowptr, wl.col, part, wl.M)
    ep = SatEpoch(wl.rowptr, wl.col, wl.M, wl.dims, wl.tau, wl.loss)
    try:
        perm = np.concatenate(P.inner_gid)
        ep.set_inputs(dev2d(wl.X), dev(wl.labels[perm]))
        Wd = [dev(w) for w in wl.W]
        bd = [dev(x) for x in wl.b]
        preds = pred_to_device(wl.pred, B, 4)
        cache = orc.CacheRing(P.n_slots, wl.dims[1:-1], wl.tau)
        for _ in range(3):
            orc.run_epoch(P, dtil, cache, wl.X, wl.labels, wl.W, wl.b, wl.pred, wl.loss, keep=False)
            ep.step(Wd, bd, preds)
        for l in range(1, wl.L):
            B.sat_cache_import(ep.ctx, l, cache.buf[l - 1])            # identical history on both sides
        for l in range(1, wl.L):
            for age in (1, 2):                                          # the older snapshots are the ones stored compressed
                idx = (cache.write_idx - 1 - age) % (wl.tau + 1)
                data, off = orc.codec_encode(cache.buf[l - 1][idx], 3)
                cache.buf[l - 1][idx] = orc.codec_decode(data, off, wl.dims[l], 3)
                size = B.sat_cache_requantise(ep.ctx, l, age, 3)
                assert size == int(off[-1])
                got = B.sat_cache_read(ep.ctx, l, age, P.n_slots, wl.dims[l])
                assert np.array_equal(got, cache.buf[l - 1][idx])
                assert size < 0.75 * 4 * P.n_slots * wl.dims[l]
        res = orc.run_epoch(P, dtil, cache, wl.X, wl.labels, wl.W, wl.b, wl.pred, wl.loss, keep=True)
        ep.step(Wd, bd, preds)
        torch.cuda.synchronize()
        from tests.gpu_util import assert_close
        for l in range(1, wl.L + 1):
            want = np.concatenate([res.per_part[m]["H"][l - 1] for m in range(wl.M)])
            assert_close(ep.H[l].cpu().numpy(), want, f"H^{l} after requantised history")
        with pytest.raises(B.SatError):
            B.sat_cache_requantise(ep.ctx, 1, wl.tau, 3)                # not a committed snapshot
    finally:
        ep.close()
