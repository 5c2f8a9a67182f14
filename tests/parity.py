"""Shared comparison rules for the GPU-vs-oracle parity tests.

Tolerances (fp32 kernels against the fp64 oracle):
  * centroid k passes when |c_gpu - c_ref|_2 <= 1e-4 * max(|c_ref|_2, 1e-3 * rms row norm);
  * a row's label must equal the oracle's unless the oracle's two smallest distances d1 <= d2
    satisfy d2 - d1 <= 1e-5 * d2 (too close to call in fp32); such a row must still carry the
    label of one of its near-tied centroids, checked through its distance;
  * objective J_t: |J_gpu - J_ref| <= 1e-5 * J_ref + 1e-6 * sum_i |x_i|^2;
  * integer outputs (edge cut, partition loads, permutation) are bit-exact.
"""
import numpy as np

CENTROID_RTOL = 1e-4
GAP_RTOL = 1e-5
OBJECTIVE_RTOL = 1e-5


def rms_row_norm(emb: np.ndarray) -> float:
    return float(np.sqrt((emb.astype(np.float64) ** 2).sum(1).mean()))


def assert_centroids_close(c_gpu: np.ndarray, c_ref: np.ndarray, emb: np.ndarray, rtol=CENTROID_RTOL):
    c_gpu = np.asarray(c_gpu, np.float64)
    err = np.linalg.norm(c_gpu - c_ref, axis=1)
    scale = np.maximum(np.linalg.norm(c_ref, axis=1), 1e-3 * rms_row_norm(emb))
    bad = np.flatnonzero(err > rtol * scale)
    assert bad.size == 0, f"centroids {bad[:8]} off by {err[bad[:8]] / scale[bad[:8]]} (relative)"


def assert_labels_match(a_gpu: np.ndarray, ref, emb: np.ndarray = None, prev_centroids: np.ndarray = None,
                        gap_rtol=GAP_RTOL):
    """ref: oracle result with .assign, .best1, .best2 for the same assignment step."""
    a_gpu = np.asarray(a_gpu)
    diff = np.flatnonzero(a_gpu != ref.assign)
    if diff.size == 0:
        return 0
    gap = ref.best2[diff] - ref.best1[diff]
    clear = diff[gap > gap_rtol * ref.best2[diff]]
    assert clear.size == 0, (f"{clear.size} rows with a clear nearest centroid got another label, e.g. row "
                             f"{clear[0]}: gpu {a_gpu[clear[0]]} oracle {ref.assign[clear[0]]}")
    if emb is not None and prev_centroids is not None:
        # a near-tied row must still sit on one of the tied centroids
        x = emb[diff].astype(np.float64)
        dist = ((x - prev_centroids[a_gpu[diff]]) ** 2).sum(1)
        assert np.all(dist - ref.best1[diff] <= 2 * gap_rtol * np.maximum(ref.best2[diff], 1e-30))
    return int(diff.size)


def assert_objective_close(j_gpu, j_ref, emb, rtol=OBJECTIVE_RTOL):
    """The library forms J = sum|x|^2 - 2 sum_k c_k.S_k + sum_k n_k |c_k|^2 from its fp32 cluster sums,
    so its absolute error scales with sum|x|^2 (1e-6 of it is allowed) on top of rtol * J."""
    j_gpu = np.asarray(j_gpu, np.float64)
    x2 = float((emb.astype(np.float64) ** 2).sum())
    np.testing.assert_allclose(j_gpu, j_ref, rtol=rtol, atol=1e-6 * x2)


def assert_centroids_are_means(c_gpu: np.ndarray, emb: np.ndarray, a_gpu: np.ndarray, c_prev: np.ndarray,
                               rtol=CENTROID_RTOL):
    """The update step on its own, whatever the labels are: every centroid is the fp64 mean of the rows that carry
    its label, and a centroid without rows keeps its previous value (fp32 bits)."""
    K = c_gpu.shape[0]
    x = emb.astype(np.float64)
    sums = np.zeros((K, emb.shape[1]))
    np.add.at(sums, a_gpu, x)
    cnt = np.bincount(a_gpu, minlength=K)
    empty = cnt == 0
    np.testing.assert_array_equal(np.asarray(c_gpu)[empty], np.asarray(c_prev, np.float32)[empty])
    mean = sums[~empty] / cnt[~empty, None]
    err = np.linalg.norm(np.asarray(c_gpu, np.float64)[~empty] - mean, axis=1)
    scale = np.maximum(np.linalg.norm(mean, axis=1), 1e-3 * rms_row_norm(emb))
    assert np.all(err <= rtol * scale), f"a centroid is off its rows' mean by {float((err / scale).max())} (relative)"


def check_run_against_oracle(ctx, emb, init, K, T, pinned_iterations=()):
    """A T-iteration run of the library (device tensors emb, init) against the oracle's T-iteration run under the
    match criteria, and the iterations in `pinned_iterations` each on their own.

    Whole run: labels, centroids and objective trace under the criteria above.  A near-tied row is allowed to change
    sides, and when one does the two trajectories may part from the next iteration on (its centroid moves by
    distance / cluster size, which can exceed the 1e-5 gap of other rows).  If the whole-run comparison finds rows
    with a clear nearest centroid on another label, the first iteration at which the runs differ is located by
    bisection, and the test only passes when every row that differs THERE is a near tie; the iteration and the
    number of such rows are reported in a warning.

    Pinned iteration t: the library's labels after t iterations against one oracle step from the library's own
    C_{t-1}; its centroids against the oracle's where the memberships agree, and against the mean of the rows that
    carry each label in any case.  This holds whatever happened before t."""
    import warnings
    import oracle
    import torch
    emb_h, init_h = emb.cpu().numpy(), init.cpu().numpy()

    def run(t, objective=False):
        r = ctx.kmeans(emb, K, t, init, objective=objective)
        torch.cuda.synchronize()
        ctx.check()
        return r

    got = run(T, objective=True)
    a = got.assign.cpu().numpy()
    assert a.min() >= 0 and a.max() < K
    ref = oracle.kmeans(emb_h, K, T, init_h)
    try:
        flips = assert_labels_match(a, ref)
        assert_centroids_close(got.centroids.cpu().numpy(), ref.centroids, emb_h)
        assert_objective_close(got.objective.cpu().numpy(), ref.objective, emb_h)
    except AssertionError:
        lo, hi = 1, T                                   # smallest t whose labels differ from the oracle's at all
        while lo < hi:
            mid = (lo + hi) // 2
            same = np.array_equal(run(mid).assign.cpu().numpy(), oracle.kmeans(emb_h, K, mid, init_h).assign)
            lo, hi = (mid + 1, hi) if same else (lo, mid)
        first = oracle.kmeans(emb_h, K, lo, init_h)
        flips = assert_labels_match(run(lo).assign.cpu().numpy(), first)      # raises unless all of them are near ties
        assert flips > 0, "the runs differ although no near-tied row changed sides"
        warnings.warn(f"trajectories part at iteration {lo} of {T}: {flips} near-tied rows changed sides there")
        pinned_iterations = sorted(set(pinned_iterations) | {lo, min(lo + 1, T), T})
    for t in pinned_iterations:
        c_prev = run(t - 1).centroids.cpu().numpy() if t > 1 else init_h
        g = run(t)
        at, ct = g.assign.cpu().numpy(), g.centroids.cpu().numpy()
        step_ref = oracle.kmeans(emb_h, K, 1, c_prev)
        step_flips = assert_labels_match(at, step_ref, emb_h, c_prev.astype(np.float64))
        assert_centroids_are_means(ct, emb_h, at, c_prev)
        if step_flips == 0:
            assert_centroids_close(ct, step_ref.centroids, emb_h)
    return flips
