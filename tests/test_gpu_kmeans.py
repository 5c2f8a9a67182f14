"""GPU parity: ep_kmeans (through the C ABI) against the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
import synth
from parity import (assert_centroids_are_means, assert_centroids_close, assert_labels_match,
                    assert_objective_close)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2604_01000_b200 as ep
    c = ep.Context(0)
    yield c
    c.check()
    c.close()


def _inputs(w, device="cuda"):
    emb = synth.embeddings(w, device=device)
    init = emb[synth.init_centroid_rows(w, device=device)].contiguous()
    return emb, init


def _run_and_compare(ctx, emb, init, K, iters, path="auto", single_steps=True):
    ctx.set_kmeans_path(path)
    emb_h = emb.cpu().numpy()
    init_h = init.cpu().numpy()
    ref = oracle.kmeans(emb_h, K, iters, init_h)
    got = ctx.kmeans(emb, K, iters, init, objective=True)
    torch.cuda.synchronize()
    ctx.check()
    a = got.assign.cpu().numpy()
    assert a.min() >= 0 and a.max() < K
    prev = oracle.kmeans(emb_h, K, max(iters - 1, 0), init_h).centroids if iters > 0 else init_h.astype(np.float64)
    flips = assert_labels_match(a, ref, emb_h, prev)
    assert_centroids_close(got.centroids.cpu().numpy(), ref.centroids, emb_h)
    assert_objective_close(got.objective.cpu().numpy(), ref.objective, emb_h)
    if single_steps and iters > 1:
        # pin each step on its own: one GPU iteration from the oracle's C_{t-1} (rounded to fp32)
        for t in sorted({1, iters // 2, iters - 1}):
            c_prev = oracle.kmeans(emb_h, K, t, init_h).centroids.astype(np.float32)
            step_ref = oracle.kmeans(emb_h, K, 1, c_prev)
            step = ctx.kmeans(emb, K, 1, torch.from_numpy(c_prev).cuda())
            assert_labels_match(step.assign.cpu().numpy(), step_ref, emb_h, c_prev.astype(np.float64))
            assert_centroids_close(step.centroids.cpu().numpy(), step_ref.centroids, emb_h)
    ctx.set_kmeans_path("auto")
    return flips


def test_cfg1_full(ctx):
    w = synth.WORKLOADS["cfg1"]
    emb, init = _inputs(w)
    _run_and_compare(ctx, emb, init, w.K, w.iters)


@pytest.mark.parametrize("name,N,iters", [("cfg2", 20_011, 30), ("cfg3", 9_973, 30), ("cfg4", 30_011, 12),
                                          ("cfg5", 25_013, 8)])
def test_scaled_configs(ctx, name, N, iters):
    """The paper-shaped configs at a row count the oracle finishes in seconds: several blocks, ragged tail."""
    w = synth.scaled(synth.WORKLOADS[name], N)
    emb, init = _inputs(w)
    _run_and_compare(ctx, emb, init, w.K, iters)


@pytest.mark.parametrize("K,N,d,iters", [(300, 12_007, 128, 3), (1024, 9_001, 64, 2), (4096, 20_003, 128, 2),
                                         (65, 5_003, 256, 3), (200, 3_001, 512, 2)])
def test_large_k_label_only_path(ctx, K, N, d, iters):
    w = synth.scaled(synth.WORKLOADS["cfg4"], N, d=d, K=K)
    emb, init = _inputs(w)
    _run_and_compare(ctx, emb, init, K, iters, single_steps=False)


@pytest.mark.parametrize("K,N,d,iters", [(2, 1_000, 32, 3), (5, 129, 64, 2), (32, 30_011, 128, 4), (64, 25_013, 128, 3),
                                         (100, 7_001, 100, 2), (256, 9_973, 256, 2), (257, 6_007, 36, 2),
                                         (300, 12_007, 128, 3), (1024, 9_001, 64, 2), (4096, 20_003, 128, 2),
                                         (700, 3_001, 224, 2), (16, 9_973, 256, 3), (32, 5_003, 200, 2), (5, 700, 132, 2),
                                         (1, 300, 256, 2)])
def test_tensor_core_path(ctx, K, N, d, iters):
    """The tcgen05 screening + fp32 resolve path, forced for every shape it accepts: labels must be the
    exact fp32 argmin, so the same tolerances apply as on the CUDA-core path."""
    w = synth.scaled(synth.WORKLOADS["cfg4"], N, d=d, K=K)
    emb, init = _inputs(w)
    _run_and_compare(ctx, emb, init, K, iters, path="tensor", single_steps=False)


def test_tensor_core_path_in_row_chunks(ctx):
    """A candidate buffer of 1 MiB forces several row chunks per iteration; the result must not change."""
    w = synth.scaled(synth.WORKLOADS["cfg4"], 60_013, K=2048)
    emb, init = _inputs(w)
    ctx.set_kmeans_path("tensor")
    whole = ctx.kmeans(emb, w.K, 2, init, objective=True)
    ctx.set_kmeans_cand_mb(1)
    try:
        parts = ctx.kmeans(emb, w.K, 2, init, objective=True)
    finally:
        ctx.set_kmeans_cand_mb(1024)
        ctx.set_kmeans_path("auto")
    assert torch.equal(whole.assign, parts.assign) and torch.equal(whole.centroids, parts.centroids)
    ref = oracle.kmeans(emb.cpu().numpy(), w.K, 2, init.cpu().numpy())
    prev = oracle.kmeans(emb.cpu().numpy(), w.K, 1, init.cpu().numpy()).centroids
    assert_labels_match(parts.assign.cpu().numpy(), ref, emb.cpu().numpy(), prev)
    assert_centroids_close(parts.centroids.cpu().numpy(), ref.centroids, emb.cpu().numpy())


def test_tensor_core_path_ties_and_duplicates(ctx):
    """Integer-valued rows and duplicated centroids: TF32 is exact here, ties must go to the lowest index."""
    rng = np.random.default_rng(5)
    base = rng.integers(-4, 5, size=(300, 32)).astype(np.float32)
    emb_h = np.concatenate([base, base[:77]])
    init_h = np.concatenate([base[:150], base[:150], np.full((1, 32), 1e3, np.float32)])   # every centroid twice; last stays empty
    emb, init = torch.from_numpy(emb_h).cuda(), torch.from_numpy(init_h).cuda()
    ctx.set_kmeans_path("tensor")
    try:
        got = ctx.kmeans(emb, 301, 2, init, objective=True)
    finally:
        ctx.set_kmeans_path("auto")
    ref = oracle.kmeans(emb_h, 301, 2, init_h)
    np.testing.assert_array_equal(got.assign.cpu().numpy(), ref.assign)
    assert_centroids_close(got.centroids.cpu().numpy(), ref.centroids, emb_h)


def test_fused_tensor_core_pass_ties_duplicates_and_repeatability(ctx):
    """K <= 64: the single-kernel tensor-core pass.  Duplicated centroids tie exactly, so those rows must
    go through its fp32 queue and come out on the lowest index; two runs must agree bit for bit."""
    rng = np.random.default_rng(6)
    base = rng.integers(-4, 5, size=(50, 64)).astype(np.float32)
    emb_h = np.concatenate([base, base, base[:29]] * 3)
    init_h = np.concatenate([base[:40], base[:40], np.full((1, 64), 1e3, np.float32)])
    emb, init = torch.from_numpy(emb_h).cuda(), torch.from_numpy(init_h).cuda()
    ctx.set_kmeans_path("tensor")
    try:
        got = ctx.kmeans(emb, 81, 2, init, objective=True)
        w = synth.scaled(synth.WORKLOADS["cfg4"], 70_001)
        e2, i2 = _inputs(w)
        a = ctx.kmeans(e2, w.K, 5, i2, objective=True)
        b = ctx.kmeans(e2, w.K, 5, i2, objective=True)
    finally:
        ctx.set_kmeans_path("auto")
    ref = oracle.kmeans(emb_h, 81, 2, init_h)
    np.testing.assert_array_equal(got.assign.cpu().numpy(), ref.assign)
    assert_centroids_close(got.centroids.cpu().numpy(), ref.centroids, emb_h)
    assert torch.equal(a.assign, b.assign) and torch.equal(a.centroids, b.centroids) and torch.equal(a.objective, b.objective)


@pytest.mark.parametrize("K,d", [(64, 128), (37, 96), (11, 256)])
def test_fused_tensor_core_pass_with_very_uneven_clusters(ctx, K, d):
    """The fused pass shares its clusters out among the accumulate warps by the counts of the previous iteration.
    Here one mixture component holds 70 % of the rows and every centroid starts inside a component of its own, so one
    cluster takes more than half of every tile while the others get a handful of rows each; the sums must not depend on who
    owns what: parity with the oracle over several iterations, and the resume identity across the change of owners."""
    rng = np.random.default_rng(100 + K)
    N = 20_011
    centres = rng.normal(size=(K, d)).astype(np.float32)
    share = rng.random(N)
    comp = np.where(share < 0.7, 0, rng.integers(1, K, size=N))
    comp[:K] = np.arange(K)                                    # every component has a row, and a centroid starts on it
    emb_h = (centres[comp] + 0.5 * rng.normal(size=(N, d))).astype(np.float32)
    init_h = emb_h[:K].copy()
    emb, init = torch.from_numpy(emb_h).cuda(), torch.from_numpy(init_h).cuda()
    _run_and_compare(ctx, emb, init, K, 4)
    three = ctx.kmeans(emb, K, 3, init)
    four = ctx.kmeans(emb, K, 4, init)
    step = ctx.kmeans(emb, K, 1, three.centroids)       # first iteration of a call: the default owners
    assert torch.equal(step.assign, four.assign) and torch.equal(step.centroids, four.centroids)


def _pin_every_iteration(ctx, emb, init, K, T, path):
    """Rows far from the origin next to tiny clusters make whole runs fragile: one near-tied row that changes sides
    (which the match criterion allows) moves a five-row centroid by a fifth of a distance, and the trajectories part
    for good.  So every iteration of the library's run is pinned on its own: iteration t against ONE oracle step from
    the library's own C_{t-1} (labels: no row with a clear nearest centroid may differ; centroids: the oracle's where
    the memberships agree, the mean of the rows that carry each label everywhere).  The whole run is compared with the
    oracle's whole run as well, up to the first iteration in which a near-tied row legitimately changed sides."""
    ctx.set_kmeans_path(path)
    try:
        emb_h, init_h = emb.cpu().numpy(), init.cpu().numpy()
        c_prev = init_h
        diverged_at = None
        for t in range(1, T + 1):
            got = ctx.kmeans(emb, K, t, init)                 # a t-iteration run is the prefix of the longer ones
            torch.cuda.synchronize()
            ctx.check()
            a = got.assign.cpu().numpy()
            c = got.centroids.cpu().numpy()
            step_ref = oracle.kmeans(emb_h, K, 1, c_prev)
            flips = assert_labels_match(a, step_ref, emb_h, c_prev.astype(np.float64))
            assert_centroids_are_means(c, emb_h, a, c_prev)
            if flips == 0:
                assert_centroids_close(c, step_ref.centroids, emb_h)
            if diverged_at is None:
                whole = oracle.kmeans(emb_h, K, t, init_h)
                if assert_labels_match(a, whole) > 0:          # raises on a clear mismatch; > 0: near ties changed sides
                    diverged_at = t
                else:
                    assert_centroids_close(c, whole.centroids, emb_h)
            c_prev = c
        return diverged_at
    finally:
        ctx.set_kmeans_path("auto")


def _clump_far_from_origin(K, d, N=20_011):
    """70 % of the rows in one tight clump far from the origin: |x|^2 about 9 d, squared distances between the rows
    of the clump about 0.18 d, so |x|^2 is fifty times the distances the labels are decided on; the initial centroids
    are random rows, most of them inside the clump, which the clustering therefore cuts into many near-tied pieces."""
    rng = np.random.default_rng(100 + K)
    centres = rng.normal(size=(K, d)).astype(np.float32) * 3
    comp = np.where(rng.random(N) < 0.7, 0, rng.integers(1, K, size=N))
    emb_h = (centres[comp] + 0.3 * rng.normal(size=(N, d))).astype(np.float32)
    init_h = emb_h[rng.permutation(N)[:K]].copy()
    return torch.from_numpy(emb_h).cuda(), torch.from_numpy(init_h).cuda()


@pytest.mark.parametrize("K,d,path", [(11, 256, "tensor"), (37, 96, "tensor"), (64, 128, "tensor"),
                                      (11, 256, "simt"), (37, 96, "simt"), (64, 128, "simt"),
                                      (130, 128, "tensor"), (300, 64, "tensor"), (300, 64, "simt")])
def test_rows_far_from_the_origin_keep_the_match_criterion(ctx, K, d, path):
    """|x|^2 far above the distances: the score |c|^2 - 2 x.c carries a rounding error relative to the NORMS, the
    criterion (labels agree unless the two nearest distances differ by less than 1e-5 relative) is stated on the
    DISTANCES.  Every kernel family therefore settles its close calls by sum_j (x_j - c_j)^2: the fused tensor-core
    pass (K <= 64), the CUDA-core kernels (fused for K <= 256, chunked beyond), the large-K tensor-core path."""
    emb, init = _clump_far_from_origin(K, d)
    _pin_every_iteration(ctx, emb, init, K, 4, path)


@pytest.mark.parametrize("path", ["auto", "simt"])
@pytest.mark.parametrize("name,N,K", [("cfg4", 30_011, 32), ("cfg3", 9_973, 16), ("cfg4", 20_011, 200)])
def test_uncentred_mixture_keeps_the_match_criterion(ctx, name, N, K, path):
    """The benchmark mixtures moved away from the origin by 8 in every coordinate (|x|^2 about 64 d, forty times the
    squared distances between components): a translation changes no distance, so the labels must still be the
    oracle's."""
    w = synth.scaled(synth.WORKLOADS[name], N, K=K)
    emb, init = _inputs(w)
    emb += 8.0
    init += 8.0
    _pin_every_iteration(ctx, emb, init, K, 3, path)


@pytest.mark.parametrize("N,d,K", [(1, 4, 1), (2, 8, 2), (33, 4, 3), (257, 1024, 5), (1000, 12, 1), (515, 100, 9),
                                   (64, 36, 64), (4097, 260, 17), (100, 516, 7)])
def test_shapes_and_edges(ctx, N, d, K):
    rng = np.random.default_rng(N * 131 + d)
    centres = rng.normal(size=(max(K, 2), d)) * 3
    emb_h = (centres[rng.integers(0, max(K, 2), size=N)] + rng.normal(size=(N, d))).astype(np.float32)
    init_h = emb_h[rng.permutation(N)[:K]].copy()
    emb, init = torch.from_numpy(emb_h).cuda(), torch.from_numpy(init_h).cuda()
    _run_and_compare(ctx, emb, init, K, 4, single_steps=False)


def test_empty_cluster_duplicates_and_ties(ctx):
    rng = np.random.default_rng(3)
    base = rng.integers(-4, 5, size=(40, 16)).astype(np.float32)
    emb_h = np.concatenate([base, base, base[:7]])                 # duplicate rows
    init_h = np.concatenate([base[:3], base[:1], np.full((1, 16), 1e3, np.float32)])   # centroid 3 duplicates 0; 4 stays empty
    emb, init = torch.from_numpy(emb_h).cuda(), torch.from_numpy(init_h).cuda()
    got = ctx.kmeans(emb, 5, 3, init, objective=True)
    ref = oracle.kmeans(emb_h, 5, 3, init_h)
    a = got.assign.cpu().numpy()
    assert not (a == 4).any()
    np.testing.assert_array_equal(got.centroids[4].cpu().numpy(), init_h[4])           # kept as it was
    np.testing.assert_array_equal(a, ref.assign)                   # integer data: ties resolved to the lowest index
    assert_centroids_close(got.centroids.cpu().numpy(), ref.centroids, emb_h)
    assert_objective_close(got.objective.cpu().numpy(), ref.objective, emb_h)


def test_iters_zero_assigns_only(ctx):
    w = synth.scaled(synth.WORKLOADS["cfg2"], 7_777)
    emb, init = _inputs(w)
    got = ctx.kmeans(emb, w.K, 0, init, objective=True)
    ref = oracle.kmeans(emb.cpu().numpy(), w.K, 0, init.cpu().numpy())
    assert torch.equal(got.centroids, init)
    assert_labels_match(got.assign.cpu().numpy(), ref)
    assert_objective_close(got.objective.cpu().numpy(), ref.objective, emb.cpu().numpy())


def test_runs_are_bit_identical_and_resumable(ctx):
    w = synth.scaled(synth.WORKLOADS["cfg3"], 40_009)
    emb, init = _inputs(w)
    a = ctx.kmeans(emb, w.K, 6, init, objective=True)
    b = ctx.kmeans(emb, w.K, 6, init, objective=True)
    assert torch.equal(a.assign, b.assign) and torch.equal(a.centroids, b.centroids)
    assert torch.equal(a.objective, b.objective)
    first = ctx.kmeans(emb, w.K, 2, init, objective=True)
    rest = ctx.kmeans(emb, w.K, 4, first.centroids, objective=True)
    assert torch.equal(rest.assign, a.assign) and torch.equal(rest.centroids, a.centroids)
    assert torch.equal(torch.cat([first.objective, rest.objective]), a.objective)
    assert torch.all(a.objective[1:] <= a.objective[:-1] * (1 + 1e-7))               # never increases


def test_argument_errors_are_reported_not_faulted(ctx):
    import paper_2604_01000_b200 as ep
    emb = torch.zeros((10, 8), device="cuda")
    with pytest.raises(ep.EmbedPartError):
        ctx.kmeans(emb, 11, 1, torch.zeros((11, 8), device="cuda"))                    # K > N
    with pytest.raises(ep.EmbedPartError):
        ctx.kmeans(torch.zeros((10, 6), device="cuda"), 2, 1, torch.zeros((2, 6), device="cuda"))   # d % 4
    with pytest.raises(ep.EmbedPartError):
        ctx.kmeans(emb, 2, -1, torch.zeros((2, 8), device="cuda"))
    with pytest.raises(ValueError):
        ctx.kmeans(emb.cpu(), 2, 1, torch.zeros((2, 8), device="cuda"))
    lib = ep.load_library()
    import ctypes
    rc = lib.ep_kmeans(ctx._h, ctypes.c_void_p(emb.data_ptr()), 10, 8, 2, 1, ctypes.c_void_p(emb.data_ptr()),
                       ctypes.c_void_p(emb.data_ptr()), ctypes.c_void_p(emb.data_ptr()), None, None, 0, None)
    assert rc == 3                                                                      # EP_ERR_WORKSPACE
    assert b"workspace" in lib.ep_last_error(ctx._h)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0


def test_two_contexts_on_two_streams_do_not_disturb_each_other(ctx):
    """Two independent clustering runs issued side by side (own context and workspace each, own stream each) give
    what they give one after the other."""
    import paper_2604_01000_b200 as ep
    w = synth.scaled(synth.WORKLOADS["cfg4"], 60_013)
    emb, init = _inputs(w)
    init2 = emb[synth.init_centroid_rows(w, 300, device="cuda")].contiguous()
    alone_a = ctx.kmeans(emb, w.K, 6, init)
    alone_b = ctx.kmeans(emb, 300, 3, init2)
    torch.cuda.synchronize()
    other = ep.Context(0)
    try:
        sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
        sa.wait_stream(torch.cuda.current_stream())
        sb.wait_stream(torch.cuda.current_stream())
        for _ in range(3):
            with torch.cuda.stream(sa):
                got_a = ctx.kmeans(emb, w.K, 6, init)
            with torch.cuda.stream(sb):
                got_b = other.kmeans(emb, 300, 3, init2)
        torch.cuda.synchronize()
        ctx.check()
        other.check()
    finally:
        other.close()
    assert torch.equal(got_a.assign, alone_a.assign) and torch.equal(got_a.centroids, alone_a.centroids)
    assert torch.equal(got_b.assign, alone_b.assign) and torch.equal(got_b.centroids, alone_b.centroids)


@pytest.mark.parametrize("name,N,iters", [("cfg1", 10_000, 6), ("cfg3", 30_011, 4), ("cfg5", 40_009, 3)])
def test_one_launch_for_all_iterations_equals_one_launch_per_iteration(ctx, name, N, iters):
    """The fused small-K pass either runs every iteration of a call inside one launch (the blocks update the centroids
    themselves between grid-wide barriers) or takes one launch per iteration plus the update kernel.  Same labels; the
    centroids agree to the last bits (the two fold the blocks' partial sums in fp64 in different fixed orders); both
    repeat bit for bit; both match the oracle."""
    w = synth.scaled(synth.WORKLOADS[name], N)
    emb, init = _inputs(w)
    got = {}
    try:
        for mode in (1, 2):
            ctx.set_kmeans_iterations_per_launch(mode)
            a = ctx.kmeans(emb, w.K, iters, init, objective=True)
            b = ctx.kmeans(emb, w.K, iters, init, objective=True)
            assert torch.equal(a.assign, b.assign) and torch.equal(a.centroids, b.centroids) and torch.equal(a.objective, b.objective)
            got[mode] = a
            _run_and_compare(ctx, emb, init, w.K, iters, single_steps=False)
            ctx.set_kmeans_iterations_per_launch(mode)           # _run_and_compare leaves the path on "auto", not this option
            first = ctx.kmeans(emb, w.K, 1, init)
            rest = ctx.kmeans(emb, w.K, iters - 1, first.centroids)
            assert torch.equal(rest.assign, a.assign) and torch.equal(rest.centroids, a.centroids)      # resumable
    finally:
        ctx.set_kmeans_iterations_per_launch(0)
    assert torch.equal(got[1].assign, got[2].assign)
    torch.testing.assert_close(got[1].centroids, got[2].centroids, rtol=1e-6, atol=1e-7)
    torch.testing.assert_close(got[1].objective, got[2].objective, rtol=1e-9, atol=0)
