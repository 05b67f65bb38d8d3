"""GPU vs oracle: graph load and partition structures, bit-exact (integer work)."""
import numpy as np
import pytest

from oracle import sat_ref as orc
from sat_synth import make_workload
from tests.dense_pins import csr_from_edges, random_graph
from tests.gpu_util import assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import paper_2308_13466_b200.binding as binding
    return binding


def _compare_partition(B, ctx, rowptr, col, part, M):
    n = rowptr.shape[0] - 1
    P = orc.build_partition(rowptr, col, part, M)
    gpart, gslot, n_slots = B.sat_slot_map(ctx, n)
    assert np.array_equal(gpart, part)
    assert n_slots == P.n_slots
    assert np.array_equal(gslot, P.slot)
    tot = B.sat_part_sizes(ctx, B.SAT_ALL_PARTS)
    assert tot[0] == n and tot[1] == sum(x.shape[0] for x in P.halo_gid)
    assert tot[2] == col.shape[0] + n and tot[3] == P.n_slots
    for m in range(M):
        got = B.sat_part_lists(ctx, m)
        assert np.array_equal(got["inner_gid"], P.inner_gid[m]), f"inner_gid[{m}]"
        assert np.array_equal(got["halo_gid"], P.halo_gid[m]), f"halo_gid[{m}]"
        assert np.array_equal(got["halo_slot"], P.halo_slot[m]), f"halo_slot[{m}]"
        assert np.array_equal(got["push_local"], P.push_local[m]), f"push_local[{m}]"
        assert np.array_equal(got["push_slot"], P.push_slot[m]), f"push_slot[{m}]"
        assert np.array_equal(got["loc_rowptr"], P.loc_rowptr[m]), f"loc_rowptr[{m}]"
        assert np.array_equal(got["loc_col"], P.loc_col[m]), f"loc_col[{m}]"
        assert np.array_equal(got["hrow_ptr"], P.hrow_ptr[m]), f"hrow_ptr[{m}]"
        assert np.array_equal(got["hrow_col"], P.hrow_col[m]), f"hrow_col[{m}]"
    return P


def test_five_node(B, five_node):
    g = five_node
    rowptr, col = csr_from_edges(5, g["edges"])
    ctx = B.sat_create(0, 0)
    try:
        B.sat_graph_load(ctx, rowptr, col)
        _, dinv = orc.degrees(rowptr)
        assert_close(B.sat_graph_dinv(ctx, 5), dinv, "dinv", 1e-6)
        part = np.array(g["part"], dtype=np.int32)
        B.sat_partition(ctx, 2, B.SAT_PART_GIVEN, part)
        _compare_partition(B, ctx, rowptr, col, part, 2)
    finally:
        B.sat_destroy(ctx)


@pytest.mark.parametrize("seed,n,p,M", [(1, 23, 0.2, 3), (2, 300, 0.02, 7), (3, 1000, 0.01, 33), (4, 64, 0.0, 4), (5, 257, 0.05, 1)])
def test_random_given_partitions(B, seed, n, p, M):
    """Random graphs with random (non-contiguous) partition assignments; includes an edgeless graph and M = 1."""
    rng = np.random.default_rng(seed)
    rowptr, col = random_graph(rng, n, p)
    part = rng.integers(0, M, size=n).astype(np.int32)
    ctx = B.sat_create(0, 0)
    try:
        B.sat_graph_load(ctx, rowptr, col)
        B.sat_partition(ctx, M, B.SAT_PART_GIVEN, part)
        _compare_partition(B, ctx, rowptr, col, part, M)
    finally:
        B.sat_destroy(ctx)


@pytest.mark.parametrize("name,shrink", [("tiny", 1), ("medium", 8), ("dense", 32), ("large", 64), ("multilabel", 16)])
def test_workload_partitions(B, name, shrink):
    """The five workloads (the R-MAT ones shrunk): contiguous-block / given partitions, power-law rows far longer
    than one SpMM chunk, empty and ragged cases."""
    wl = make_workload(name, shrink=shrink, with_dense=False)
    ctx = B.sat_create(0, 0)
    try:
        B.sat_graph_load(ctx, wl.rowptr, wl.col)
        dtil, dinv = orc.degrees(wl.rowptr)
        assert_close(B.sat_graph_dinv(ctx, wl.n), dinv, "dinv", 1e-6)
        if wl.part_given is not None:
            B.sat_partition(ctx, wl.M, B.SAT_PART_GIVEN, wl.part_given)
            part = wl.part_given
        else:
            B.sat_partition(ctx, wl.M, B.SAT_PART_CONTIG_BLOCKS)
            part = orc.contig_blocks(wl.n, wl.M)
        _compare_partition(B, ctx, wl.rowptr, wl.col, part, wl.M)
    finally:
        B.sat_destroy(ctx)


@pytest.mark.parametrize("case", ["five", "random-disconnected", "edgeless", "rmat"])
def test_bfs_block_partitioner(B, five_node, case):
    """SAT_PART_BFS_BLOCKS: breadth-first order inside the library (FIFO from node 0, neighbours ascending, restarts at the
    smallest unvisited id), cut into M blocks; the graph keeps its ids, so the blocks are scattered id sets.  part[] and
    every derived structure against the oracle's own traversal."""
    from sat_synth import rmat_graph
    if case == "five":
        rowptr, col = csr_from_edges(5, five_node["edges"])
        M = 2
    elif case == "random-disconnected":
        rowptr, col = random_graph(np.random.default_rng(11), 400, 0.004)
        M = 5
    elif case == "edgeless":
        rowptr, col = random_graph(np.random.default_rng(12), 50, 0.0)
        M = 3
    else:
        rowptr, col = rmat_graph(4, 15, 21_000, n_samples=150_000)       # seeded id permutation, no relabelling
        M = 8
    part = orc.bfs_blocks(rowptr, col, M)
    ctx = B.sat_create(0, 0)
    try:
        B.sat_graph_load(ctx, rowptr, col)
        B.sat_partition(ctx, M, B.SAT_PART_BFS_BLOCKS)
        _compare_partition(B, ctx, rowptr, col, part, M)
        if case == "five":
            assert part.tolist() == five_node["part"]
    finally:
        B.sat_destroy(ctx)


def test_device_resident_inputs(B):
    import torch
    wl = make_workload("tiny", with_dense=False)
    ctx = B.sat_create(0, 0)
    try:
        B.sat_graph_load(ctx, torch.from_numpy(wl.rowptr).cuda(), torch.from_numpy(wl.col).cuda())
        B.sat_partition(ctx, wl.M, B.SAT_PART_GIVEN, torch.from_numpy(wl.part_given).cuda())
        _compare_partition(B, ctx, wl.rowptr, wl.col, wl.part_given, wl.M)
    finally:
        B.sat_destroy(ctx)


def test_malformed_inputs_are_rejected(B):
    """Host-side failure handling: every malformed input returns an error status and the context stays usable."""
    rowptr, col = csr_from_edges(5, [[0, 1], [1, 2], [2, 3], [3, 4], [1, 3]])
    ctx = B.sat_create(0, 0)
    try:
        def expect(status, fn):
            with pytest.raises(B.SatError) as ei:
                fn()
            assert ei.value.status == status, ei.value

        expect(B.SAT_ESTATE, lambda: B.sat_partition(ctx, 2, B.SAT_PART_CONTIG_BLOCKS))
        bad = rowptr.copy()
        bad[2] = bad[3] + 1
        expect(B.SAT_EDATA, lambda: B.sat_graph_load(ctx, bad, col))
        c2 = col.copy()
        c2[0] = 7
        expect(B.SAT_EDATA, lambda: B.sat_graph_load(ctx, rowptr, c2))          # column out of range
        c3 = col.copy()
        c3[0] = 0
        expect(B.SAT_EDATA, lambda: B.sat_graph_load(ctx, rowptr, c3))          # self-loop (and asymmetric)
        c4 = col.copy()
        c4[1], c4[2] = col[2], col[1]
        expect(B.SAT_EDATA, lambda: B.sat_graph_load(ctx, rowptr, c4))          # unsorted row
        rp5, c5 = csr_from_edges(5, [[0, 1], [1, 2]])
        c5 = c5.copy()
        c5[0] = 3                                                                # (0,3) without (3,0)
        expect(B.SAT_EDATA, lambda: B.sat_graph_load(ctx, rp5, c5))
        B.sat_graph_load(ctx, rowptr, col)                                       # still usable
        expect(B.SAT_EINVAL, lambda: B.sat_partition(ctx, 0, B.SAT_PART_CONTIG_BLOCKS))
        expect(B.SAT_EINVAL, lambda: B.sat_partition(ctx, 9, B.SAT_PART_CONTIG_BLOCKS))
        expect(B.SAT_EINVAL, lambda: B.sat_partition(ctx, 2, B.SAT_PART_GIVEN, np.array([0, 1, 2, 0, 1], dtype=np.int32)))
        expect(B.SAT_ESTATE, lambda: B.sat_cache_init(ctx, [4], 2))
        B.sat_partition(ctx, 2, B.SAT_PART_CONTIG_BLOCKS)
        expect(B.SAT_EINVAL, lambda: B.sat_cache_init(ctx, [4], 0))              # tau = 0
        expect(B.SAT_ESTATE, lambda: B.sat_cache_commit(ctx))
        expect(B.SAT_EINVAL, lambda: B.sat_part_sizes(ctx, 5))
        B.sat_cache_init(ctx, [4], 2)
        import torch
        g = torch.zeros((3, 4), device="cuda")
        W = torch.zeros((4, 4), device="cuda")
        expect(B.SAT_ESTATE, lambda: B.sat_layer_bwd(ctx, 0, 1, g, W, W.clone(), None, 0))   # backward before forward
        odd = torch.zeros((3, 5), device="cuda")[:, :4]
        expect(B.SAT_EINVAL, lambda: B.sat_layer_fwd(ctx, 0, 1, odd, odd, W, None, 0, g))    # ld not a multiple of 4
        # a rejected graph leaves the loaded graph, its partition and the cache as they were
        before = B.sat_part_lists(ctx, 1)
        expect(B.SAT_EDATA, lambda: B.sat_graph_load(ctx, rowptr, c2))
        expect(B.SAT_EDATA, lambda: B.sat_graph_load(ctx, bad, col))
        after = B.sat_part_lists(ctx, 1)
        assert all(np.array_equal(before[k], after[k]) for k in before)
        assert B.sat_cache_state(ctx) == (0, 0)
        B.sat_sync_status(ctx)
    finally:
        B.sat_destroy(ctx)
