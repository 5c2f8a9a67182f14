"""GPU parity: ep_partition_quality and ep_reorder against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2604_01000_b200 as ep
    c = ep.Context(0)
    yield c
    c.check()
    c.close()


def _quality_matches(ctx, rowptr, colidx, assign, K):
    got = ctx.partition_quality(rowptr, colidx, assign, K)
    torch.cuda.synchronize()
    ctx.check()
    ref = oracle.partition_quality(rowptr.cpu().numpy(), colidx.cpu().numpy(), assign.cpu().numpy(), K)
    assert int(got.edge_cut.item()) == ref.edge_cut
    np.testing.assert_array_equal(got.part_vertices.cpu().numpy(), ref.part_vertices)
    np.testing.assert_array_equal(got.part_edges.cpu().numpy(), ref.part_edges)
    return ref


def _random_labels(N, K, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randint(0, K, (N,), generator=g, dtype=torch.int32).cuda()


@pytest.mark.parametrize("name", ["cfg1", "cfg2"])
def test_full_small_configs(ctx, name):
    w = synth.WORKLOADS[name]
    rowptr, colidx = synth.graph(w, device="cuda")
    z = synth.component_labels(w, torch.arange(w.N, device="cuda"))
    assign = (z % w.K).to(torch.int32)
    ref = _quality_matches(ctx, rowptr, colidx, assign, w.K)
    assert ref.edge_cut % 2 == 0 and ref.part_edges.sum() == colidx.numel()
    _quality_matches(ctx, rowptr.to(torch.int64), colidx, assign, w.K)
    _quality_matches(ctx, rowptr, colidx, _random_labels(w.N, w.K, 1), w.K)


@pytest.mark.parametrize("name,N", [("cfg3", 6_007), ("cfg4", 50_021), ("cfg5", 100_003)])
def test_scaled_configs(ctx, name, N):
    w = synth.scaled(synth.WORKLOADS[name], N)
    rowptr, colidx = synth.graph(w, device="cuda")
    _quality_matches(ctx, rowptr, colidx, _random_labels(N, w.K, 2), w.K)


@pytest.mark.parametrize("name,N,K,slice_kb", [("cfg5", 100_003, 64, 16), ("cfg4", 50_021, 32, 7), ("cfg4", 50_021, 300, 30),
                                               ("cfg5", 100_003, 64, 1)])
def test_vertex_range_slices_give_the_same_counts(ctx, name, N, K, slice_kb):
    """Labels too large for the L2 are gathered slice by slice of the vertex range, one pass over the column ids
    per slice.  A small slice limit forces that path on a small graph (2 to 8 slices, uneven last slice, int64 and
    int32 row pointers, a bad column id reported once): same counts as the oracle, bit for bit."""
    w = synth.scaled(synth.WORKLOADS[name], N)
    rowptr, colidx = synth.graph(w, device="cuda")
    assign = _random_labels(N, K, 5)
    ctx.set_quality_slice_kb(slice_kb)
    try:
        _quality_matches(ctx, rowptr, colidx, assign, K)
        _quality_matches(ctx, rowptr.to(torch.int64), colidx, assign, K)
        bad = colidx.clone()
        bad[7] = N + 5                                            # out of range: reported, never followed
        got = ctx.partition_quality(rowptr, bad, assign, K)
        torch.cuda.synchronize()
        assert ctx.poll_status() == 4                             # EP_ERR_BAD_INDEX, whatever the slice it falls in
        keep = torch.ones_like(bad, dtype=torch.bool)
        keep[7] = False
        ref = oracle.partition_quality(rowptr.cpu().numpy(), colidx.cpu().numpy(), assign.cpu().numpy(), K)
        src = torch.searchsorted(rowptr[1:].contiguous(), torch.tensor([7], device="cuda"), right=True)
        was_cut = int(assign[src] != assign[colidx[7]])
        assert int(got.edge_cut.item()) == ref.edge_cut - was_cut
    finally:
        ctx.set_quality_slice_kb(56 * 1024)


@pytest.mark.parametrize("N,K", [(6_007, 2), (6_007, 16), (6_007, 17), (6_007, 200), (9_001, 256), (5_003, 300),
                                 (100_003, 16), (60_013, 200), (180_001, 9)])
def test_dense_graph_label_tables_in_shared_memory(ctx, N, K):
    """Dense graphs with few vertices: the kernel variants that keep all labels in shared memory, as nibbles
    (K <= 16) or bytes (K <= 256), and the global-memory gather beyond.  The larger N are tables of which only one
    copy fits on an SM: the 1024-thread form whose four thread groups share it."""
    w = synth.scaled(synth.WORKLOADS["cfg3"], N)
    rowptr, colidx = synth.graph(w, device="cuda")
    _quality_matches(ctx, rowptr, colidx, _random_labels(N, K, N + K), K)
    _quality_matches(ctx, rowptr.to(torch.int64), colidx, _random_labels(N, K, N + K + 1), K)


@pytest.mark.parametrize("K", [1, 2, 255, 256, 257, 5000, 70_000])
def test_label_widths(ctx, K):
    N = 80_000
    w = synth.scaled(synth.WORKLOADS["cfg2"], N)
    rowptr, colidx = synth.graph(w, device="cuda")
    _quality_matches(ctx, rowptr, colidx, _random_labels(N, K, K), K)


def test_odd_csr_shapes(ctx):
    rng = np.random.default_rng(9)
    N = 30_000
    deg = rng.integers(0, 4, size=N)
    deg[rng.integers(0, N, size=50)] = rng.integers(5_000, 30_000, size=50)       # rows far longer than a tile
    deg[1000:9000] = 0                                                            # a long run of empty rows
    deg[-5:] = 0                                                                  # empty rows at the end
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    nnz = int(rowptr[-1])
    colidx = rng.integers(0, N, size=nnz).astype(np.int32)                        # unsorted, duplicates, self-loops
    colidx[:100] = np.repeat(np.arange(10, dtype=np.int32), 10)
    for dtype in (torch.int32, torch.int64):
        rp = torch.from_numpy(rowptr).to(dtype).cuda()
        for K in (3, 300):
            _quality_matches(ctx, rp, torch.from_numpy(colidx).cuda(), _random_labels(N, K, 4), K)


def test_odd_csr_shapes_one_table_per_sm(ctx):
    """Long rows, empty runs and unsorted entries through the 1024-thread form (table too large for two blocks)."""
    rng = np.random.default_rng(19)
    N = 110_000
    deg = rng.integers(0, 200, size=N)
    deg[rng.integers(0, N, size=40)] = rng.integers(5_000, 40_000, size=40)
    deg[2000:30_000] = 0
    deg[-3:] = 0
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    nnz = int(rowptr[-1])
    assert nnz * 2 >= N * 148
    colidx = rng.integers(0, N, size=nnz).astype(np.int32)
    for dtype in (torch.int32, torch.int64):
        rp = torch.from_numpy(rowptr).to(dtype).cuda()
        for K in (5, 130):
            _quality_matches(ctx, rp, torch.from_numpy(colidx).cuda(), _random_labels(N, K, 4), K)


@pytest.mark.parametrize("nnz", [0, 1, 3, 4, 5, 1023, 1024, 1025, 2047, 2049, 8191, 8192, 8193, 16_387])
def test_tile_boundaries(ctx, nnz):
    rng = np.random.default_rng(nnz)
    N = 97
    cuts = np.sort(rng.integers(0, nnz + 1, size=N - 1))
    rowptr = np.concatenate([[0], cuts, [nnz]]).astype(np.int32)
    colidx = rng.integers(0, N, size=nnz).astype(np.int32)
    ci = torch.from_numpy(colidx).cuda() if nnz else torch.empty(0, dtype=torch.int32, device="cuda")
    _quality_matches(ctx, torch.from_numpy(rowptr).cuda(), ci, _random_labels(N, 5, 7), 5)


@pytest.mark.parametrize("K", [3, 16, 200, 70_000])
@pytest.mark.parametrize("shape", ["short_rows", "dense_small", "starts_on_chunk_boundaries"])
def test_row_starts_everywhere_in_a_chunk(ctx, shape, K):
    """A warp works through 1024-entry chunks of the CSR arrays and rebuilds every entry's row from the row starts inside
    its chunk: hundreds of one- and two-entry rows per chunk (more than the 32 whose look-ups run ahead), rows that
    start inside a four-entry vector, on a chunk's first entry or on its last, with the labels gathered from global
    memory, from a byte table and from a nibble table in shared memory."""
    rng = np.random.default_rng(K + len(shape))
    if shape == "short_rows":
        N = 60_000
        deg = rng.integers(0, 4, size=N)
    elif shape == "dense_small":
        N = 3_000                                       # 148 N <= 2 nnz: the labels go to shared memory when K <= 256
        deg = rng.integers(150, 260, size=N)
    else:
        N = 4_000
        deg = rng.integers(100, 400, size=N)
        pos = 0
        for i in range(N):                              # every seventh row ends on a multiple of 1024, one before or one after
            if i % 7 == 0:
                end = (pos + int(deg[i]) + 1023) // 1024 * 1024 + (i // 7) % 3 - 1
                deg[i] = end - pos
            pos += int(deg[i])
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    nnz = int(rowptr[-1])
    colidx = rng.integers(0, N, size=nnz).astype(np.int32)
    labels = _random_labels(N, K, 11)
    for dtype in (torch.int32, torch.int64):
        _quality_matches(ctx, torch.from_numpy(rowptr).to(dtype).cuda(), torch.from_numpy(colidx).cuda(), labels, K)


def test_bad_indices_raise_a_status_without_faulting(ctx):
    rowptr = torch.tensor([0, 2, 4, 6], dtype=torch.int32).cuda()
    colidx = torch.tensor([1, 2, 0, 99, 0, 1], dtype=torch.int32).cuda()          # 99 is outside [0, N)
    assign = torch.tensor([0, 1, 0], dtype=torch.int32).cuda()
    ctx.partition_quality(rowptr, colidx, assign, 2)
    assert ctx.poll_status() == 4
    ctx.partition_quality(rowptr, colidx.clamp(max=2), torch.tensor([0, 7, 0], dtype=torch.int32).cuda(), 2)
    assert ctx.poll_status() == 4                                                 # label outside [0, K)
    ctx.partition_quality(torch.tensor([0, 4, 2, 6], dtype=torch.int32).cuda(), colidx.clamp(max=2), assign, 2)
    assert ctx.poll_status() == 4                                                 # row pointer goes backwards
    ctx.reorder(torch.tensor([0, 5, 1], dtype=torch.int32).cuda(), 2)
    assert ctx.poll_status() == 4
    assert ctx.poll_status() == 0


# ---------------------------------------------------------------------------------------------- reorder
@pytest.mark.parametrize("N,K", [(1, 1), (31, 2), (4096, 4), (4097, 4), (10_000, 4), (100_003, 32), (250_007, 256),
                                 (250_007, 257), (300_001, 4096), (150_000, 70_000), (1_000_003, 64)])
def test_reorder_is_the_stable_sort(ctx, N, K):
    assign = _random_labels(N, K, N + K)
    if K > 3:
        assign[assign == 2] = 3                                                   # an empty partition
    got = ctx.reorder(assign, K)
    torch.cuda.synchronize()
    ctx.check()
    perm, inv = oracle.reorder(assign.cpu().numpy(), K)
    np.testing.assert_array_equal(got.perm.cpu().numpy(), perm)
    np.testing.assert_array_equal(got.inv_perm.cpu().numpy(), inv)
    only = ctx.reorder(assign, K, inverse=False)
    assert only.inv_perm is None and torch.equal(only.perm, got.perm)


def test_reorder_of_kmeans_labels_groups_the_planted_graph(ctx):
    """End to end on the tiny config: cluster, score, reorder; the K-Means partition must cut far
    fewer entries than a random one (statistical sanity, not parity)."""
    w = synth.WORKLOADS["cfg1"]
    emb = synth.embeddings(w, device="cuda")
    init = emb[synth.init_centroid_rows(w, device="cuda")].contiguous()
    rowptr, colidx = synth.graph(w, device="cuda")
    km = ctx.kmeans(emb, w.K, w.iters, init)
    q = _quality_matches(ctx, rowptr, colidx, km.assign, w.K)
    rnd = _quality_matches(ctx, rowptr, colidx, _random_labels(w.N, w.K, 5), w.K)
    assert q.edge_cut < 0.6 * rnd.edge_cut
    assert abs(rnd.edge_cut / colidx.numel() - (1 - 1 / w.K)) < 0.02
    r = ctx.reorder(km.assign, w.K)
    lab = km.assign[r.perm.long()]
    assert torch.all(lab[1:] >= lab[:-1])


def test_host_buffer_entry_points_match_the_device_ones(ctx):
    w = synth.scaled(synth.WORKLOADS["cfg2"], 30_011)
    emb = synth.embeddings(w, device="cuda")
    init = emb[synth.init_centroid_rows(w, device="cuda")].contiguous()
    rowptr, colidx = synth.graph(w, device="cuda")
    km = ctx.kmeans(emb, w.K, 4, init, objective=True)
    q = ctx.partition_quality(rowptr, colidx, km.assign, w.K)
    r = ctx.reorder(km.assign, w.K)
    torch.cuda.synchronize()
    hk = ctx.kmeans_host(emb.cpu().pin_memory(), w.K, 4, init.cpu(), objective=True)
    torch.cuda.synchronize()
    assert torch.equal(hk.assign, km.assign.cpu()) and torch.equal(hk.centroids, km.centroids.cpu())
    assert torch.equal(hk.objective, km.objective.cpu())
    hq = ctx.partition_quality_host(rowptr.cpu(), colidx.cpu().pin_memory(), hk.assign, w.K)
    hr = ctx.reorder_host(hk.assign, w.K)
    torch.cuda.synchronize()
    ctx.check()
    assert torch.equal(hq.edge_cut, q.edge_cut.cpu()) and torch.equal(hq.part_vertices, q.part_vertices.cpu())
    assert torch.equal(hq.part_edges, q.part_edges.cpu())
    assert torch.equal(hr.perm, r.perm.cpu()) and torch.equal(hr.inv_perm, r.inv_perm.cpu())


@pytest.mark.parametrize("cluster_size", [-1, 0, 2, 8, 16])
def test_gather_yardsticks_sum_what_they_gather(ctx, cluster_size):
    """ep_probe_gather is the edge-cut pass reduced to its label lookups (a measuring stick for the bench): whatever
    memory serves the lookups, the sum must be that of the gathered bytes; entries outside [0, N) are skipped."""
    import paper_2604_01000_b200 as ep
    w = synth.scaled(synth.WORKLOADS["cfg3"], 40_009)
    rowptr, colidx = synth.graph(w, device="cuda")
    table = (synth.component_labels(w, torch.arange(w.N, device="cuda")) % 251).to(torch.uint8)
    colidx = colidx.clone()
    colidx[::1013] = -1                                   # a few entries that point nowhere
    colidx[5::4099] = w.N
    try:
        got = ctx.probe_gather(colidx, table, cluster_size)
    except ep.EmbedPartError as exc:
        if cluster_size == 16 and exc.status == 2:
            pytest.skip("no cluster of 16 blocks on this device")
        raise
    torch.cuda.synchronize()
    ctx.check()
    ok = (colidx >= 0) & (colidx < w.N)
    want = int(table[colidx[ok].long()].long().sum().item())
    assert int(got.item()) == want


@pytest.mark.parametrize("reorder_K", [0, 300])
def test_whole_path_on_host_buffers_equals_the_separate_calls(ctx, reorder_K):
    """ep_partition_and_reorder_host uploads every input once and runs the same kernels as the separate calls: its
    outputs are theirs, bit for bit, and the graph passes equal the oracle's."""
    w = synth.scaled(synth.WORKLOADS["cfg4"], 30_011)
    emb = synth.embeddings(w, device="cuda")
    rows = synth.init_centroid_rows(w, max(w.K, reorder_K), device="cuda")
    init, init2 = emb[rows[: w.K]].contiguous(), (emb[rows[:reorder_K]].contiguous() if reorder_K else None)
    rowptr, colidx = synth.graph(w, device="cuda")
    km = ctx.kmeans(emb, w.K, 5, init)
    fine = ctx.kmeans(emb, reorder_K, 2, init2) if reorder_K else km
    q = ctx.partition_quality(rowptr, colidx, km.assign, w.K)
    r = ctx.reorder(fine.assign, reorder_K or w.K)
    torch.cuda.synchronize()
    hk, hq, hr, hfine = ctx.partition_and_reorder_host(
        emb.cpu().pin_memory(), w.K, 5, init.cpu(), rowptr.cpu(), colidx.cpu().pin_memory(), reorder_K=reorder_K,
        reorder_iters=2, reorder_init=init2.cpu() if reorder_K else None)
    torch.cuda.synchronize()
    ctx.check()
    assert torch.equal(hk.assign, km.assign.cpu()) and torch.equal(hk.centroids, km.centroids.cpu())
    assert int(hq.edge_cut.item()) == int(q.edge_cut.item())
    assert torch.equal(hq.part_vertices, q.part_vertices.cpu()) and torch.equal(hq.part_edges, q.part_edges.cpu())
    assert torch.equal(hr.perm, r.perm.cpu()) and torch.equal(hr.inv_perm, r.inv_perm.cpu())
    if reorder_K:
        assert torch.equal(hfine, fine.assign.cpu())
    ref = oracle.partition_quality(rowptr.cpu().numpy(), colidx.cpu().numpy(), hk.assign.numpy(), w.K)
    assert int(hq.edge_cut.item()) == ref.edge_cut
    perm, inv = oracle.reorder(fine.assign.cpu().numpy(), reorder_K or w.K)
    np.testing.assert_array_equal(hr.perm.numpy(), perm)
    np.testing.assert_array_equal(hr.inv_perm.numpy(), inv)
