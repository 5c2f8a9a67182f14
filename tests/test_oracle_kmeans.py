"""Pins for the oracle's K-Means (CPU only): hand traces, brute force, closed forms, invariants,
and a library special case.  None of these re-type the oracle's own formula."""
import itertools
import json
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _cases():
    with open(os.path.join(GOLDEN, "lloyd_hand_cases.json")) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c["name"][:40])
def test_hand_traces(case):
    emb = np.array(case["emb"], np.float32)
    init = np.array(case["init"], np.float32)
    for step in case["trace"]:
        r = oracle.kmeans(emb, init.shape[0], step["iters"], init)
        assert r.assign.tolist() == step["assign"]
        np.testing.assert_allclose(r.centroids, np.array(step["centroids"], np.float64), rtol=1e-14, atol=0)
        np.testing.assert_allclose(r.objective, np.array(step["objective"], np.float64), rtol=1e-13, atol=0)


def _cost_py(emb, cent, labels):
    """Objective of a labelling, with exact rational-free but independent arithmetic (math.fsum)."""
    terms = []
    for i, k in enumerate(labels):
        for j in range(emb.shape[1]):
            terms.append((float(emb[i, j]) - float(cent[k, j])) ** 2)
    return math.fsum(terms)


@pytest.mark.parametrize("seed,N,K,d", [(0, 7, 3, 2), (1, 8, 2, 3), (2, 6, 4, 1), (3, 5, 3, 5)])
def test_assignment_is_the_exhaustive_optimum(seed, N, K, d):
    """For fixed centroids the assignment step must minimise the objective over ALL K^N labellings."""
    rng = np.random.default_rng(seed)
    emb = rng.integers(-6, 7, size=(N, d)).astype(np.float32)
    cent = rng.integers(-6, 7, size=(K, d)).astype(np.float32)
    a, b1, b2 = oracle.assign_step(emb, cent.astype(np.float64))
    best = min(_cost_py(emb, cent, lab) for lab in itertools.product(range(K), repeat=N))
    assert _cost_py(emb, cent, a.tolist()) == pytest.approx(best, rel=1e-14, abs=0)
    assert math.fsum(b1.tolist()) == pytest.approx(best, rel=1e-14, abs=0)
    # among equal-cost choices the lowest index must have been taken, and best2 is the runner-up
    for i in range(N):
        dists = [math.fsum((float(emb[i, j]) - float(cent[k, j])) ** 2 for j in range(d)) for k in range(K)]
        assert a[i] == dists.index(min(dists))
        assert b1[i] == pytest.approx(sorted(dists)[0], rel=1e-14, abs=0)
        assert b2[i] == pytest.approx(sorted(dists)[1], rel=1e-14, abs=0)


def test_duplicate_centroids_lowest_index_and_runner_up():
    emb = np.array([[1.0, 2.0], [3.0, -1.0]], np.float32)
    cent = np.array([[9, 9], [1, 2], [1, 2], [3, -1]], np.float64)
    a, b1, b2 = oracle.assign_step(emb, cent)
    assert a.tolist() == [1, 3]
    assert b1.tolist() == [0.0, 0.0]
    assert b2.tolist() == [0.0, 13.0]          # the duplicate is the runner-up for row 0


def test_k1_is_the_global_mean():
    rng = np.random.default_rng(5)
    emb = rng.normal(size=(257, 12)).astype(np.float32)
    r = oracle.kmeans(emb, 1, 3, emb[:1])
    assert not r.assign.any()
    mean = np.array([math.fsum(emb[:, j].astype(np.float64).tolist()) / 257 for j in range(12)])
    np.testing.assert_allclose(r.centroids[0], mean, rtol=1e-13, atol=1e-15)
    assert np.isinf(r.best2).all()
    # J_1 is measured against the initial centroid (row 0), J_2 against the mean: the variance identity
    tot = math.fsum(((emb.astype(np.float64) - mean) ** 2).ravel().tolist())
    assert r.objective[1] == pytest.approx(tot, rel=1e-12)
    assert r.objective[2] == pytest.approx(tot, rel=1e-12)
    shift = 257 * math.fsum(((emb[0].astype(np.float64) - mean) ** 2).tolist())
    assert r.objective[0] == pytest.approx(tot + shift, rel=1e-12)   # parallel-axis theorem


def test_k_equals_n_is_a_fixed_point():
    rng = np.random.default_rng(6)
    emb = rng.normal(size=(23, 4)).astype(np.float32)
    r = oracle.kmeans(emb, 23, 2, emb)
    assert r.assign.tolist() == list(range(23))
    np.testing.assert_array_equal(r.centroids, emb.astype(np.float64))
    assert r.objective.tolist() == [0.0, 0.0]


def _mixture(seed, N, d, comps, spread=12.0, std=0.5):
    rng = np.random.default_rng(seed)
    centres = rng.normal(size=(comps, d)) * spread
    z = rng.integers(0, comps, size=N)
    return (centres[z] + std * rng.normal(size=(N, d))).astype(np.float32), z


def test_invariants_mean_counts_monotone_objective():
    emb, _ = _mixture(7, 3000, 16, 9, spread=1.0, std=1.0)     # overlapping blobs: many iterations matter
    K, T = 6, 12
    init = emb[:K]
    r = oracle.kmeans(emb, K, T, init)
    # (1) every non-empty centroid is the mean of the rows that carry its label (independent fp64 sum)
    x64 = emb.astype(np.float64)
    for k in range(K):
        rows = x64[r.assign == k]
        assert len(rows) > 0
        mean = np.array([math.fsum(rows[:, j].tolist()) for j in range(16)]) / len(rows)
        np.testing.assert_allclose(r.centroids[k], mean, rtol=1e-12, atol=1e-14)
    assert np.bincount(r.assign, minlength=K).sum() == 3000
    # (2) the objective never increases
    assert np.all(np.diff(r.objective) <= 1e-9 * r.objective[:-1])
    assert r.objective[0] > r.objective[-1]
    # (3) J_t is the cost of the assignment of step t against C_{t-1}: recompute the last one
    prev = oracle.kmeans(emb, K, T - 1, init).centroids
    a = r.assign
    J = math.fsum(((x64 - prev[a]) ** 2).ravel().tolist())
    assert r.objective[-1] == pytest.approx(J, rel=1e-12)
    # (4) best1 / best2 agree with a dense numpy distance matrix
    D = ((x64[:, None, :] - prev[None, :, :]) ** 2).sum(-1)
    np.testing.assert_array_equal(a, D.argmin(1))
    Ds = np.sort(D, axis=1)
    np.testing.assert_allclose(r.best1, Ds[:, 0], rtol=1e-12)
    np.testing.assert_allclose(r.best2, Ds[:, 1], rtol=1e-12)


def test_resume_equals_one_long_run_when_centroids_are_fp32_representable():
    # integer coordinates and power-of-two cluster sizes keep every centroid exactly representable in
    # fp32, so handing C_T back through the fp32 init argument loses nothing
    emb = np.array([[0, 0], [0, 8], [8, 0], [8, 8], [100, 100], [100, 108], [108, 100], [108, 108]], np.float32)
    init = np.array([[0, 0], [100, 100]], np.float32)
    full = oracle.kmeans(emb, 2, 4, init)
    first = oracle.kmeans(emb, 2, 1, init)
    rest = oracle.kmeans(emb, 2, 3, first.centroids.astype(np.float32))
    np.testing.assert_array_equal(full.centroids, rest.centroids)
    np.testing.assert_array_equal(full.assign, rest.assign)
    np.testing.assert_array_equal(full.objective[1:], rest.objective)


def test_separated_mixture_converges_to_component_means_and_stays():
    emb, z = _mixture(8, 4000, 8, 5, spread=30.0, std=0.5)
    first = [int(np.flatnonzero(z == c)[0]) for c in range(5)]
    r = oracle.kmeans(emb, 5, 2, emb[first])
    np.testing.assert_array_equal(r.assign, z)
    for c in range(5):
        np.testing.assert_allclose(r.centroids[c], emb[z == c].astype(np.float64).mean(0), rtol=1e-10, atol=1e-12)
    again = oracle.kmeans(emb, 5, 3, emb[first])
    np.testing.assert_allclose(again.centroids, r.centroids, rtol=1e-13)
    assert again.objective[2] == pytest.approx(again.objective[1], rel=1e-13)


def test_empty_cluster_keeps_its_centroid_and_objective_stays_monotone():
    emb, _ = _mixture(9, 500, 4, 3, spread=5.0)
    far = np.full((1, 4), 1e3, np.float32)
    init = np.concatenate([emb[:3], far])
    r = oracle.kmeans(emb, 4, 5, init)
    assert (r.assign != 3).all()
    np.testing.assert_array_equal(r.centroids[3], far[0].astype(np.float64))
    assert np.all(np.diff(r.objective) <= 0)


def test_iters_zero_is_assign_only():
    emb, _ = _mixture(10, 300, 6, 4)
    init = emb[10:14]
    r0 = oracle.kmeans(emb, 4, 0, init)
    r1 = oracle.kmeans(emb, 4, 1, init)
    np.testing.assert_array_equal(r0.assign, r1.assign)
    np.testing.assert_array_equal(r0.centroids, init.astype(np.float64))
    assert r0.objective.shape == (1,) and r0.objective[0] == r1.objective[0]


def test_thread_count_does_not_change_the_result():
    emb, _ = _mixture(11, 5000, 32, 7, spread=1.5, std=1.0)
    n = oracle.num_threads()
    try:
        oracle.set_num_threads(1)
        a = oracle.kmeans(emb, 7, 6, emb[:7])
        oracle.set_num_threads(max(2, n))
        b = oracle.kmeans(emb, 7, 6, emb[:7])
    finally:
        oracle.set_num_threads(n)
    np.testing.assert_array_equal(a.assign, b.assign)
    np.testing.assert_array_equal(a.centroids, b.centroids)
    np.testing.assert_array_equal(a.objective, b.objective)


def test_library_special_case_sklearn_lloyd():
    """scikit-learn's Lloyd with explicit init, one restart, zero tolerance and max_iter = T ends on
    the same centroids C_T (its labels follow another convention, so only centroids are compared)."""
    sk = pytest.importorskip("sklearn.cluster")
    emb, _ = _mixture(12, 2000, 10, 6, spread=1.2, std=1.0)
    K, T = 5, 7
    init = emb[100:100 + K]
    r = oracle.kmeans(emb, K, T, init)
    assert np.bincount(r.assign, minlength=K).min() > 0
    import warnings
    with warnings.catch_warnings():
        warnings.simplefilter("ignore")
        km = sk.KMeans(n_clusters=K, init=init.astype(np.float64), n_init=1, max_iter=T, tol=0.0,
                       algorithm="lloyd").fit(emb.astype(np.float64))
    np.testing.assert_allclose(km.cluster_centers_, r.centroids, rtol=1e-9, atol=1e-10)


# ------------------------------------------------------------------------- sampling-based clustering
def test_sampled_kmeans_with_every_row_in_the_sample_is_one_more_full_batch_assignment():
    """Sample = all rows: the centroids are full-batch Lloyd's C_T, and the labels are the assignment that
    full-batch Lloyd makes in iteration T + 1 (which is made against C_T)."""
    rng = np.random.default_rng(21)
    emb = rng.normal(size=(400, 6)).astype(np.float32)
    init = emb[:5].copy()
    T = 3
    s = oracle.sampled_kmeans(emb, np.arange(400), 5, T, init)
    full_T = oracle.kmeans(emb, 5, T, init)
    full_T1 = oracle.kmeans(emb, 5, T + 1, init)
    np.testing.assert_allclose(s.centroids, full_T.centroids, rtol=0, atol=0)
    np.testing.assert_array_equal(s.assign, full_T1.assign)
    np.testing.assert_allclose(s.objective, full_T.objective, rtol=0, atol=0)


def test_sampled_kmeans_labels_are_nearest_centroids_by_enumeration():
    rng = np.random.default_rng(22)
    emb = rng.integers(-5, 6, size=(40, 3)).astype(np.float32)
    rows = rng.permutation(40)[:12]
    s = oracle.sampled_kmeans(emb, rows, 3, 2, emb[rows[:3]])
    # the centroids depend on the sampled rows only
    again = oracle.kmeans(emb[rows], 3, 2, emb[rows[:3]])
    np.testing.assert_array_equal(s.centroids, again.centroids)
    for i in range(40):
        d = [float(((emb[i].astype(np.float64) - s.centroids[k]) ** 2).sum()) for k in range(3)]
        assert s.assign[i] == int(np.argmin(d)) and s.best1[i] == min(d)    # argmin returns the lowest index on ties
    # rows outside the sample do not move the centroids
    emb2 = emb.copy()
    outside = np.setdiff1d(np.arange(40), rows)
    emb2[outside] += 100.0
    np.testing.assert_array_equal(oracle.sampled_kmeans(emb2, rows, 3, 2, emb[rows[:3]]).centroids, s.centroids)


def test_sampled_kmeans_recovers_a_well_separated_mixture_from_a_small_sample():
    rng = np.random.default_rng(23)
    K, per, d = 4, 300, 8
    centres = rng.normal(size=(K, d)) * 50
    z = np.repeat(np.arange(K), per)
    emb = (centres[z] + rng.normal(size=(K * per, d))).astype(np.float32)
    rows = np.concatenate([np.flatnonzero(z == k)[:8] for k in range(K)])          # 8 rows of each component
    init = emb[[np.flatnonzero(z == k)[0] for k in range(K)]]
    s = oracle.sampled_kmeans(emb, rows, K, 2, init)
    np.testing.assert_array_equal(s.assign, z)
    for k in range(K):
        np.testing.assert_allclose(s.centroids[k], emb[rows[z[rows] == k]].astype(np.float64).mean(0), rtol=1e-12)


def test_sampled_kmeans_rejects_bad_samples():
    emb = np.zeros((10, 4), np.float32)
    with pytest.raises(ValueError):
        oracle.sampled_kmeans(emb, [0, 1, 1], 2, 1, emb[:2])          # a row twice
    with pytest.raises(ValueError):
        oracle.sampled_kmeans(emb, [0, 10], 2, 1, emb[:2])            # outside [0, N)
    with pytest.raises(ValueError):
        oracle.sampled_kmeans(emb, [0], 2, 1, emb[:2])                # fewer rows than clusters
    with pytest.raises(ValueError):
        oracle.sampled_kmeans(emb, [0, 1], 2, 0, emb[:2])             # no iteration
