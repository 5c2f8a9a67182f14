"""Shape fuzz: hypothesis draws the shapes (rows not a multiple of any tile, every dimension class, cluster counts on
both sides of every path switch, empty rows, self-loops, duplicate entries, both row-pointer widths) and every draw is
compared with the oracle under the usual criteria.  Derandomised, so a failure reproduces."""
import numpy as np
import pytest
import torch
from hypothesis import given, settings, strategies as st, HealthCheck

import oracle
from parity import check_run_against_oracle

pytestmark = pytest.mark.gpu

FUZZ = settings(max_examples=40, deadline=None, derandomize=True, suppress_health_check=list(HealthCheck))


@pytest.fixture(scope="module")
def ctx():
    import paper_2604_01000_b200 as ep
    c = ep.Context(0)
    yield c
    c.set_kmeans_path("auto")
    c.check()
    c.close()


@FUZZ
@given(N=st.integers(1, 6000), d4=st.integers(1, 80), K=st.sampled_from([1, 2, 3, 4, 8, 16, 17, 32, 33, 64, 65, 100, 256, 257, 1024]),
       iters=st.integers(0, 3), path=st.sampled_from(["auto", "simt", "tensor"]), offset=st.sampled_from([0.0, 0.0, 5.0]),
       seed=st.integers(0, 2 ** 31 - 1))
def test_kmeans_shapes(ctx, N, d4, K, iters, path, offset, seed):
    d = 4 * d4
    K = min(K, N)
    rng = np.random.default_rng(seed)
    centres = rng.normal(size=(max(K, 2), d)) * 2
    emb_h = (centres[rng.integers(0, max(K, 2), size=N)] + rng.normal(size=(N, d)) + offset).astype(np.float32)
    init_h = emb_h[rng.permutation(N)[:K]].copy()
    ctx.set_kmeans_path(path)
    try:
        check_run_against_oracle(ctx, torch.from_numpy(emb_h).cuda(), torch.from_numpy(init_h).cuda(), K, iters,
                                 pinned_iterations=(1,) if iters > 0 else ())
    finally:
        ctx.set_kmeans_path("auto")


@FUZZ
@given(N=st.integers(1, 20000), mean_deg=st.sampled_from([0.0, 0.5, 3.0, 40.0, 300.0]), K=st.sampled_from([1, 2, 5, 16, 17, 64, 256, 300, 5000]),
       wide=st.booleans(), slice_kb=st.sampled_from([0, 1, 4]), seed=st.integers(0, 2 ** 31 - 1))
def test_graph_pass_shapes(ctx, N, mean_deg, K, wide, slice_kb, seed):
    rng = np.random.default_rng(seed)
    K = min(K, max(N, 1))
    deg = rng.poisson(mean_deg, size=N).astype(np.int64)
    if N > 3:
        deg[rng.integers(0, N, size=2)] = 0                                    # empty rows
        deg[rng.integers(0, N)] += int(20 * mean_deg)                          # one heavy row
    rowptr = np.concatenate([[0], np.cumsum(deg)])
    nnz = int(rowptr[-1])
    colidx = rng.integers(0, N, size=nnz).astype(np.int32)                     # duplicates and self-loops included
    assign = rng.integers(0, K, size=N).astype(np.int32)
    rp = torch.from_numpy(rowptr.astype(np.int64 if wide else np.int32)).cuda()
    ci = torch.from_numpy(colidx).cuda() if nnz else torch.zeros(0, dtype=torch.int32, device="cuda")
    a = torch.from_numpy(assign).cuda()
    if slice_kb:
        ctx.set_quality_slice_kb(slice_kb)
    try:
        q = ctx.partition_quality(rp, ci, a, K)
    finally:
        ctx.set_quality_slice_kb(56 * 1024)
    r = ctx.reorder(a, K)
    bw = ctx.graph_bandwidth(rp, ci, r.inv_perm)
    torch.cuda.synchronize()
    ctx.check()
    ref = oracle.partition_quality(rowptr, colidx, assign, K)
    assert int(q.edge_cut.item()) == ref.edge_cut
    np.testing.assert_array_equal(q.part_vertices.cpu().numpy(), ref.part_vertices)
    np.testing.assert_array_equal(q.part_edges.cpu().numpy(), ref.part_edges)
    perm, inv = oracle.reorder(assign, K)
    np.testing.assert_array_equal(r.perm.cpu().numpy(), perm)
    np.testing.assert_array_equal(r.inv_perm.cpu().numpy(), inv)
    ref_bw = oracle.graph_bandwidth(rowptr, colidx, inv)
    assert int(bw.bandwidth_sum.item()) == ref_bw.bandwidth_sum
    np.testing.assert_array_equal(bw.vertex_bandwidth.cpu().numpy(), ref_bw.vertex_bandwidth)
