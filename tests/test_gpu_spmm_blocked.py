"""The source-blocked walk of the forward aggregation (`P_in H_in + P_out Hhat`; Appendix, forward of SAT).

By default only partitions whose source rows are several times the L2 are walked block by block, i.e. none of the small
test graphs (the full-size tests of the large and dense workloads run through it as the bench does).  Here the cut is
forced onto small graphs through SAT_SPMM_SRC_BLOCK (blocks of 64 to a few hundred source rows, every partition), and the
whole layer step is compared with the oracle as in the other layer tests; the all-partition launch must give the bits of
the per-partition calls, in every addressing mode of the layer's inputs; and the plan query must describe what runs.
"""
import numpy as np
import pytest

from sat_synth import make_workload
from tests import test_gpu_layers as TL
from tests.gpu_util import dev, dev2d, empty2d

pytestmark = pytest.mark.gpu

FORCED = "16384,16384,0"     # blocks of 16 KiB of source rows (at least 64 rows), every partition, runs of any length
GROUPED = "16384,16384,0,6"  # the same cut, rows of fewer than 6 entries per block walked in groups of blocks (len / 6 groups)


@pytest.fixture(scope="module")
def B():
    import paper_2308_13466_b200.binding as binding
    return binding


@pytest.mark.parametrize("name,shrink,parts,warm", [
    ("tiny", 1, [0, 1, 2, 3], 4),
    ("medium", 8, [0, 5], 2),
    ("dense", 64, [0, 9], 2),     # rows of thousands of entries: runs longer than one 256-entry chunk inside a block
    ("odd", 1, [0, 2], 2),        # ragged widths 50 / 72 / 40
])
@pytest.mark.parametrize("cut", [FORCED, GROUPED])
def test_every_call_with_the_blocked_walk(B, monkeypatch, name, shrink, parts, warm, cut):
    monkeypatch.setenv("SAT_SPMM_SRC_BLOCK", cut)
    wl = make_workload(name, shrink=shrink)
    case = TL.Case(B, wl, warm)
    try:
        for d in set(wl.dims[:-1]):
            n_blocks, n_items, n_partial = B.sat_spmm_plan(case.ctx, B.SAT_ALL_PARTS, d)
            assert n_blocks > 1 and n_partial > 0 and n_items >= wl.n, (d, n_blocks, n_items, n_partial)
        worst = TL._check_calls(B, case, parts)
        print(name, {k: f"{v:.2e}" for k, v in worst.items()})
    finally:
        case.close()


@pytest.mark.parametrize("name,shrink,given", [("medium", 16, False), ("odd", 1, True)])
def test_addressing_modes_with_the_blocked_walk(B, monkeypatch, name, shrink, given):
    """Gathered copies, out-of-subgraph rows by node id, all rows by node id: same bits, per partition and all at once."""
    monkeypatch.setenv("SAT_SPMM_SRC_BLOCK", FORCED)
    TL.test_rows_read_from_the_global_feature_matrix(B, name, shrink, given)


def test_blocked_and_plain_walks_agree_and_the_plan_says_which_ran(B, monkeypatch):
    wl = make_workload("medium", shrink=8)
    rng = np.random.default_rng(5)
    d, d_out = wl.dims[1], wl.dims[2]
    ctx = B.sat_create(0, 0)
    try:
        B.sat_graph_load(ctx, wl.rowptr, wl.col)
        B.sat_partition(ctx, wl.M, B.SAT_PART_CONTIG_BLOCKS)
        B.sat_cache_init(ctx, wl.dims[1:-1], wl.tau)
        n_halo = B.sat_part_sizes(ctx, B.SAT_ALL_PARTS)[1]
        h_in = dev2d(rng.standard_normal((wl.n, d)).astype(np.float32))
        h_halo = dev2d(rng.standard_normal((n_halo, d)).astype(np.float32))
        W, b = dev(wl.W[1]), dev(wl.b[1])
        monkeypatch.delenv("SAT_SPMM_SRC_BLOCK", raising=False)
        plain_plan = B.sat_spmm_plan(ctx, B.SAT_ALL_PARTS, d)
        assert plain_plan[0] == 1                       # a 20 k-node graph is nowhere near the L2: plain walk by default
        plain = empty2d(wl.n, d_out)
        B.sat_layer_fwd(ctx, B.SAT_ALL_PARTS, 2, h_in, h_halo, W, b, B.SAT_ACT_NONE, plain)
        monkeypatch.setenv("SAT_SPMM_SRC_BLOCK", "0")
        assert B.sat_spmm_plan(ctx, B.SAT_ALL_PARTS, d) == plain_plan
        monkeypatch.setenv("SAT_SPMM_SRC_BLOCK", FORCED)
        n_blocks, n_items, n_partial = B.sat_spmm_plan(ctx, B.SAT_ALL_PARTS, d)
        assert n_blocks > 4 and n_items > plain_plan[1] and n_partial > plain_plan[2]
        per_part = [B.sat_spmm_plan(ctx, m, d) for m in range(wl.M)]
        assert sum(p[1] for p in per_part) == n_items and sum(p[2] for p in per_part) == n_partial
        assert max(p[0] for p in per_part) == n_blocks
        blocked = empty2d(wl.n, d_out)
        B.sat_layer_fwd(ctx, B.SAT_ALL_PARTS, 2, h_in, h_halo, W, b, B.SAT_ACT_NONE, blocked)
        B.sat_sync_status(ctx)
        a, c = plain.cpu().numpy().astype(np.float64), blocked.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(a - c)) <= 2e-6 * np.max(np.abs(a))      # same sums, other grouping
        # a higher run-length threshold than any partition reaches: plain walk again, and the bits of the first call
        monkeypatch.setenv("SAT_SPMM_SRC_BLOCK", "16384,16384,100000")
        assert B.sat_spmm_plan(ctx, B.SAT_ALL_PARTS, d) == plain_plan
        again = empty2d(wl.n, d_out)
        B.sat_layer_fwd(ctx, B.SAT_ALL_PARTS, 2, h_in, h_halo, W, b, B.SAT_ACT_NONE, again)
        assert np.array_equal(again.cpu().numpy(), plain.cpu().numpy())
    finally:
        B.sat_destroy(ctx)


def B_items_forced(B, ctx, d, monkeypatch):
    """Work items of the all-partition launch with every row cut at every block (the environment is left on GROUPED)."""
    monkeypatch.setenv("SAT_SPMM_SRC_BLOCK", FORCED)
    n_items = B.sat_spmm_plan(ctx, B.SAT_ALL_PARTS, d)[1]
    monkeypatch.setenv("SAT_SPMM_SRC_BLOCK", GROUPED)
    return n_items


@pytest.mark.parametrize("kind", ["one_partition", "an_empty_partition", "random_assignment"])
def test_degenerate_partitionings_with_the_blocked_walk(B, monkeypatch, kind):
    """No halo rows at all (one partition: the blocks cut the inner rows alone), a partition without any node, and a random
    assignment (nearly every entry has a halo column): blocked and plain walks agree, and under the blocked walk the
    all-partition launch gives the bits of the per-partition calls."""
    wl = make_workload("odd")
    rng = np.random.default_rng(11)
    if kind == "one_partition":
        M, part = 1, np.zeros(wl.n, dtype=np.int32)
    elif kind == "an_empty_partition":
        M = 4
        part = rng.integers(0, 3, wl.n).astype(np.int32)
        part[part == 2] = 3                              # partition 2 owns nothing
    else:
        M, part = 5, rng.integers(0, 5, wl.n).astype(np.int32)
    d, d_out = wl.dims[1], wl.dims[2]
    ctx = B.sat_create(0, 0)
    try:
        B.sat_graph_load(ctx, wl.rowptr, wl.col)
        B.sat_partition(ctx, M, B.SAT_PART_GIVEN, part)
        B.sat_cache_init(ctx, wl.dims[1:-1], wl.tau)
        sizes = [B.sat_part_sizes(ctx, m) for m in range(M)]
        n_halo = sum(s[1] for s in sizes)
        if kind == "one_partition":
            assert n_halo == 0
        h_in = dev2d(rng.standard_normal((wl.n, d)).astype(np.float32))
        h_halo = dev2d(rng.standard_normal((max(n_halo, 1), d)).astype(np.float32))
        W, b = dev(wl.W[1]), dev(wl.b[1])

        def run(part_id, rows0, rows1, halo0, halo1):
            out = empty2d(rows1 - rows0, d_out)
            B.sat_layer_fwd(ctx, part_id, 2, h_in[rows0:rows1], h_halo[halo0:max(halo1, halo0 + 1)] if n_halo else h_halo,
                            W, b, B.SAT_ACT_RELU, out)
            return out.cpu().numpy()

        monkeypatch.setenv("SAT_SPMM_SRC_BLOCK", "0")
        plain = run(B.SAT_ALL_PARTS, 0, wl.n, 0, n_halo)
        monkeypatch.setenv("SAT_SPMM_SRC_BLOCK", FORCED)
        assert B.sat_spmm_plan(ctx, B.SAT_ALL_PARTS, d)[0] > 1
        blocked = run(B.SAT_ALL_PARTS, 0, wl.n, 0, n_halo)
        B.sat_sync_status(ctx)
        assert np.max(np.abs(plain.astype(np.float64) - blocked)) <= 2e-6 * np.max(np.abs(plain))
        monkeypatch.setenv("SAT_SPMM_SRC_BLOCK", GROUPED)          # fewer, longer runs for the short rows: same sums again
        plan_g = B.sat_spmm_plan(ctx, B.SAT_ALL_PARTS, d)
        assert plan_g[0] > 1 and plan_g[1] < B_items_forced(B, ctx, d, monkeypatch)
        grouped = run(B.SAT_ALL_PARTS, 0, wl.n, 0, n_halo)
        assert np.max(np.abs(plain.astype(np.float64) - grouped)) <= 2e-6 * np.max(np.abs(plain))
        monkeypatch.setenv("SAT_SPMM_SRC_BLOCK", FORCED)
        r0 = h0 = 0
        for m in range(M):
            n_m, b_m = sizes[m][0], sizes[m][1]
            if n_m:
                got = run(m, r0, r0 + n_m, h0, h0 + b_m)
                assert np.array_equal(got, blocked[r0:r0 + n_m]), f"partition {m} alone"
            else:
                assert B.sat_spmm_plan(ctx, m, d) == (1, 0, 0)
            r0 += n_m
            h0 += b_m
        B.sat_sync_status(ctx)
    finally:
        B.sat_destroy(ctx)


def test_plan_query_errors(B):
    wl = make_workload("tiny")
    ctx = B.sat_create(0, 0)
    try:
        B.sat_graph_load(ctx, wl.rowptr, wl.col)
        with pytest.raises(B.SatError) as ei:                 # no partition yet
            B.sat_spmm_plan(ctx, B.SAT_ALL_PARTS, 16)
        assert ei.value.status == B.SAT_ESTATE
        B.sat_partition(ctx, wl.M, B.SAT_PART_GIVEN, wl.part_given)
        for bad_part, bad_d in ((wl.M, 16), (-7, 16), (0, 0), (0, -4)):
            with pytest.raises(B.SatError) as ei:
                B.sat_spmm_plan(ctx, bad_part, bad_d)
            assert ei.value.status == B.SAT_EINVAL
        assert B.sat_spmm_plan(ctx, 0, 16)[0] == 1          # usable after the refusals
    finally:
        B.sat_destroy(ctx)
