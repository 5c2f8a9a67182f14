"""GPU parity at the configs' full sizes, in the launch configuration bench.py times.

cfg2 (N = 169,343, d = 128, K = 8, 30 iterations) and cfg3 (N = 232,965, d = 256, K = 16, 30 iterations, 114.6 M CSR
entries) are small enough for the oracle to run whole: every output is compared with it element by element.

cfg4 (N = 2,449,029, d = 128, nnz ~ 123.5 M): the oracle cannot run whole Lloyd iterations at this size in seconds, so:
labels are compared on a seeded row sample against the oracle's assignment step from the GPU's own
C_{T-1}; centroids against an independent fp64 mean of the rows carrying each label; the rest through
properties that hold at any size.  The graph passes are integer and are compared in full."""
import numpy as np
import pytest
import torch

import oracle
import synth
from parity import assert_labels_match, check_run_against_oracle, CENTROID_RTOL, rms_row_norm

pytestmark = pytest.mark.gpu

SAMPLE = 20_000


@pytest.fixture(scope="module")
def ctx():
    import paper_2604_01000_b200 as ep
    c = ep.Context(0)
    yield c
    c.check()
    c.close()


@pytest.fixture(scope="module")
def cfg4():
    w = synth.WORKLOADS["cfg4"]
    emb = synth.embeddings(w, device="cuda")
    rows = synth.init_centroid_rows(w, max(w.K, w.reorder_K), device="cuda")
    return w, emb, rows


class _Step:
    def __init__(self, assign, best1, best2):
        self.assign, self.best1, self.best2 = assign, best1, best2


def _check_run(ctx, emb, init, K, T, w):
    prev = ctx.kmeans(emb, K, T - 1, init, objective=True)
    last = ctx.kmeans(emb, K, T, init, objective=True)
    torch.cuda.synchronize()
    ctx.check()
    N = emb.shape[0]
    a = last.assign
    assert int(a.min()) >= 0 and int(a.max()) < K
    # the first T-1 iterations of the longer run are the shorter run, bit for bit
    assert torch.equal(last.objective[: T - 1], prev.objective)
    assert bool(torch.all(last.objective[1:] <= last.objective[:-1] * (1 + 1e-7)))
    # resuming from C_{T-1} gives the same last iteration
    step = ctx.kmeans(emb, K, 1, prev.centroids)
    assert torch.equal(step.assign, a) and torch.equal(step.centroids, last.centroids)
    # labels on a row sample: the oracle's assignment step against the GPU's C_{T-1}
    s = synth.subsample_rows(w, SAMPLE, device="cuda")
    xs = emb[s].cpu().numpy()
    c_prev = prev.centroids.cpu().numpy().astype(np.float64)
    ra, b1, b2 = oracle.assign_step(xs, c_prev)
    flips = assert_labels_match(a[s].cpu().numpy(), _Step(ra, b1, b2), xs, c_prev)
    assert flips <= SAMPLE // 1000
    # every non-empty centroid is the mean of its rows (independent fp64 sums on the device)
    sums = torch.zeros((K, emb.shape[1]), dtype=torch.float64, device="cuda")
    chunk = 1 << 19
    for r0 in range(0, N, chunk):
        sums.index_add_(0, a[r0:r0 + chunk].long(), emb[r0:r0 + chunk].double())
    cnt = torch.bincount(a.long(), minlength=K)
    assert int(cnt.sum()) == N
    mean = sums / cnt.clamp(min=1).double()[:, None]
    got = last.centroids.double()
    keep = cnt == 0
    assert torch.equal(got[keep].float(), prev.centroids[keep])          # empty clusters keep their centroid
    err = (got - mean).norm(dim=1)[~keep]
    scale = torch.clamp(mean.norm(dim=1)[~keep], min=1e-3 * rms_row_norm(xs))
    assert bool(torch.all(err <= CENTROID_RTOL * scale)), float((err / scale).max())
    # the objective of the last iteration, recomputed in fp64 on the sample's share: J >= sum over the sample
    d_s = ((torch.from_numpy(xs).double() - torch.from_numpy(c_prev)[torch.from_numpy(ra).long()]) ** 2).sum()
    assert float(last.objective[-1]) >= float(d_s) * (1 - 1e-6)


def test_cfg4_partition_run_full_size(ctx, cfg4):
    w, emb, rows = cfg4
    _check_run(ctx, emb, emb[rows[: w.K]].contiguous(), w.K, 4, w)


def test_cfg4_reordering_run_full_size(ctx, cfg4):
    w, emb, rows = cfg4
    _check_run(ctx, emb, emb[rows[: w.reorder_K]].contiguous(), w.reorder_K, 2, w)


def test_cfg4_graph_passes_full_size(ctx, cfg4):
    w, emb, rows = cfg4
    rowptr, colidx = synth.graph(w, device="cuda")
    km = ctx.kmeans(emb, w.K, 3, emb[rows[: w.K]].contiguous())
    q = ctx.partition_quality(rowptr, colidx, km.assign, w.K)
    fine = ctx.kmeans(emb, w.reorder_K, 1, emb[rows[: w.reorder_K]].contiguous())
    r = ctx.reorder(fine.assign, w.reorder_K)
    torch.cuda.synchronize()
    ctx.check()
    a = km.assign.cpu().numpy()
    ref = oracle.partition_quality(rowptr.cpu().numpy(), colidx.cpu().numpy(), a, w.K)
    assert int(q.edge_cut.item()) == ref.edge_cut and ref.edge_cut % 2 == 0
    np.testing.assert_array_equal(q.part_vertices.cpu().numpy(), ref.part_vertices)
    np.testing.assert_array_equal(q.part_edges.cpu().numpy(), ref.part_edges)
    assert int(ref.part_edges.sum()) == colidx.numel() and int(ref.part_vertices.sum()) == w.N
    perm, inv = oracle.reorder(fine.assign.cpu().numpy(), w.reorder_K)
    np.testing.assert_array_equal(r.perm.cpu().numpy(), perm)
    np.testing.assert_array_equal(r.inv_perm.cpu().numpy(), inv)
    # the numbering that the reordering run produced, scored the way Section 4.5.1 scores it (Eq. 3-5)
    bw = ctx.graph_bandwidth(rowptr, colidx, r.inv_perm)
    torch.cuda.synchronize()
    ctx.check()
    ref_bw = oracle.graph_bandwidth(rowptr.cpu().numpy(), colidx.cpu().numpy(), inv)
    assert int(bw.bandwidth_sum.item()) == ref_bw.bandwidth_sum
    np.testing.assert_array_equal(bw.vertex_bandwidth.cpu().numpy(), ref_bw.vertex_bandwidth)
    # ... and the graph stored under that numbering
    rp2, ci2 = ctx.relabel_graph(rowptr, colidx, r.perm, r.inv_perm)
    torch.cuda.synchronize()
    ctx.check()
    ref_rp, ref_ci = oracle.relabel_graph(rowptr.cpu().numpy(), colidx.cpu().numpy(), perm, inv)
    np.testing.assert_array_equal(rp2.cpu().numpy().astype(np.int64), ref_rp)
    np.testing.assert_array_equal(ci2.cpu().numpy(), ref_ci)
    # one application of the migration policy (Algorithm 4) to the K=32 partition at full size
    deg = np.diff(rowptr.cpu().numpy().astype(np.int64))
    cap = int(1.05 * w.N / w.K)
    words = torch.randint(-2 ** 31, 2 ** 31, (w.N,), generator=torch.Generator().manual_seed(5), dtype=torch.int64).to(torch.int32)
    moved_labels = km.assign.clone()
    state = ctx.migrate(rowptr, moved_labels, w.K, cap, int(deg.max()), words.cuda())
    torch.cuda.synchronize()
    ctx.check()
    ref_labels, ref_moved = oracle.migrate(rowptr.cpu().numpy(), a, w.K, cap, words.numpy().view(np.uint32))
    np.testing.assert_array_equal(moved_labels.cpu().numpy(), ref_labels)
    assert int(state[2].item()) == ref_moved


@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_cfg2_cfg3_whole_config_against_the_oracle(ctx, name):
    """The config as stated (full N, K, iteration count): K-Means end to end and iteration by iteration, then every
    graph pass on the full graph, bit for bit."""
    w = synth.WORKLOADS[name]
    emb = synth.embeddings(w, device="cuda")
    init = emb[synth.init_centroid_rows(w, device="cuda")].contiguous()
    check_run_against_oracle(ctx, emb, init, w.K, w.iters, pinned_iterations=(1, 2, w.iters // 2, w.iters))
    km = ctx.kmeans(emb, w.K, w.iters, init)
    del emb
    rowptr, colidx = synth.graph(w, device="cuda")
    q = ctx.partition_quality(rowptr, colidx, km.assign, w.K)
    r = ctx.reorder(km.assign, w.K)
    bw = ctx.graph_bandwidth(rowptr, colidx, r.inv_perm)
    rp2, ci2 = ctx.relabel_graph(rowptr, colidx, r.perm, r.inv_perm)
    torch.cuda.synchronize()
    ctx.check()
    a = km.assign.cpu().numpy()
    rp_h, ci_h = rowptr.cpu().numpy(), colidx.cpu().numpy()
    ref = oracle.partition_quality(rp_h, ci_h, a, w.K)
    assert int(q.edge_cut.item()) == ref.edge_cut and ref.edge_cut % 2 == 0
    np.testing.assert_array_equal(q.part_vertices.cpu().numpy(), ref.part_vertices)
    np.testing.assert_array_equal(q.part_edges.cpu().numpy(), ref.part_edges)
    perm, inv = oracle.reorder(a, w.K)
    np.testing.assert_array_equal(r.perm.cpu().numpy(), perm)
    np.testing.assert_array_equal(r.inv_perm.cpu().numpy(), inv)
    ref_bw = oracle.graph_bandwidth(rp_h, ci_h, inv)
    assert int(bw.bandwidth_sum.item()) == ref_bw.bandwidth_sum
    np.testing.assert_array_equal(bw.vertex_bandwidth.cpu().numpy(), ref_bw.vertex_bandwidth)
    ref_rp, ref_ci = oracle.relabel_graph(rp_h, ci_h, perm, inv)
    np.testing.assert_array_equal(rp2.cpu().numpy().astype(np.int64), ref_rp)
    np.testing.assert_array_equal(ci2.cpu().numpy(), ref_ci)
