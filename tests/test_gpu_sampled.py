"""GPU parity: ep_kmeans_sampled / ep_gather_rows (sampling-based clustering, Section 5 "Implementation")
against the oracle."""
from types import SimpleNamespace

import numpy as np
import pytest
import torch

import oracle
import synth
from parity import assert_centroids_close, assert_labels_match, check_run_against_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2604_01000_b200 as ep
    c = ep.Context(0)
    yield c
    c.check()
    c.close()


def _run(ctx, w, per_cluster, iters, path="auto"):
    emb = synth.embeddings(w, device="cuda")
    M = min(w.N, per_cluster * w.K)
    rows = synth.subsample_rows(w, M, device="cuda").to(torch.int64).contiguous()
    init = emb[rows[: w.K]].contiguous()
    ctx.set_kmeans_path(path)
    try:
        got = ctx.kmeans_sampled(emb, w.K, iters, rows, init)
        torch.cuda.synchronize()
        ctx.check()
    finally:
        ctx.set_kmeans_path("auto")
    emb_h, rows_h, init_h = emb.cpu().numpy(), rows.cpu().numpy(), init.cpu().numpy()
    a = got.assign.cpu().numpy()
    c = got.centroids.cpu().numpy()
    assert a.min() >= 0 and a.max() < w.K
    # the training step is ep_kmeans on the gathered rows, bit for bit ...
    sample = emb[rows].contiguous()
    ctx.set_kmeans_path(path)
    try:
        trained = ctx.kmeans(sample, w.K, iters, init)
        assert torch.equal(trained.centroids, got.centroids)
        # ... and that run against the oracle's: whole, and its last iteration on its own (with a few dozen rows per
        # cluster one near-tied row that changes sides moves a centroid by percents, so the whole-run comparison
        # may end at the first such row: see check_run_against_oracle)
        check_run_against_oracle(ctx, sample, init, w.K, iters, pinned_iterations=(1, iters))
    finally:
        ctx.set_kmeans_path("auto")
    # the last step pinned on its own: the labels of all rows against the centroids the library returned
    a2, b1, b2 = oracle.assign_step(emb_h, c.astype(np.float64))
    assert_labels_match(a, SimpleNamespace(assign=a2, best1=b1, best2=b2), emb_h, c.astype(np.float64))
    # end to end against the oracle's own centroids, when no near tie parted the two training runs
    ref = oracle.sampled_kmeans(emb_h, rows_h, w.K, iters, init_h)
    if np.array_equal(trained.assign.cpu().numpy(), oracle.kmeans(emb_h[rows_h], w.K, iters, init_h).assign):
        assert_centroids_close(c, ref.centroids, emb_h[rows_h])
        assert_labels_match(a, ref, emb_h, ref.centroids)


@pytest.mark.parametrize("name,N,per_cluster,iters", [("cfg1", 10_000, 512, 5), ("cfg2", 30_011, 512, 10),
                                                      ("cfg4", 40_009, 64, 6), ("cfg5", 50_021, 128, 8),
                                                      ("cfg3", 9_973, 512, 4)])
def test_sampled_clustering_matches_the_oracle(ctx, name, N, per_cluster, iters):
    w = synth.scaled(synth.WORKLOADS[name], N) if N != synth.WORKLOADS[name].N else synth.WORKLOADS[name]
    _run(ctx, w, per_cluster, iters)


def test_sampled_clustering_with_many_clusters_and_on_the_cuda_cores(ctx):
    w = synth.scaled(synth.WORKLOADS["cfg4"], 30_011, K=300)
    _run(ctx, w, 32, 3)
    _run(ctx, synth.scaled(synth.WORKLOADS["cfg2"], 20_011), 256, 5, path="simt")


def test_gather_rows_is_a_row_copy(ctx):
    w = synth.scaled(synth.WORKLOADS["cfg3"], 5_003)
    emb = synth.embeddings(w, device="cuda")
    rows = torch.randint(0, w.N, (1_237,), generator=torch.Generator().manual_seed(1)).cuda()
    out = ctx.gather_rows(emb, rows)
    torch.cuda.synchronize()
    ctx.check()
    np.testing.assert_array_equal(out.cpu().numpy(), emb.cpu().numpy()[rows.cpu().numpy()])
    ctx.gather_rows(emb, torch.tensor([0, w.N], dtype=torch.int64).cuda())       # a row number outside [0, N)
    assert ctx.poll_status() == 4 and ctx.poll_status() == 0


def test_argument_errors(ctx):
    import paper_2604_01000_b200 as ep
    emb = torch.zeros(100, 32, device="cuda")
    rows = torch.arange(10, dtype=torch.int64, device="cuda")
    with pytest.raises(ep.EmbedPartError):
        ctx.kmeans_sampled(emb, 16, 2, rows, emb[:16].contiguous())              # fewer sampled rows than clusters
    with pytest.raises(ep.EmbedPartError):
        ctx.kmeans_sampled(emb, 4, 0, rows, emb[:4].contiguous())                # no iteration on the sample
