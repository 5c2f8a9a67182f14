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
