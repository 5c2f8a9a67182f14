"""Pins for the oracle's edge cut / partition loads and reordering (CPU only)."""
import json
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _cases():
    with open(os.path.join(GOLDEN, "edge_cut_hand_cases.json")) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c["name"][:40])
def test_hand_counted_graphs(case):
    q = oracle.partition_quality(case["rowptr"], case["colidx"], case["assign"], case["K"])
    assert q.edge_cut == case["edge_cut"]
    assert q.part_vertices.tolist() == case["part_vertices"]
    assert q.part_edges.tolist() == case["part_edges"]


def _random_csr(rng, N, p, symmetric=True, loops=False):
    A = rng.random((N, N)) < p
    if symmetric:
        A = A | A.T
    if not loops:
        np.fill_diagonal(A, False)
    rowptr = np.concatenate([[0], np.cumsum(A.sum(1))]).astype(np.int64)
    colidx = np.nonzero(A)[1].astype(np.int32)
    return A, rowptr, colidx


@pytest.mark.parametrize("seed", range(6))
def test_brute_force_dense_adjacency(seed):
    rng = np.random.default_rng(seed)
    N, K = int(rng.integers(2, 11)), int(rng.integers(1, 5))
    A, rowptr, colidx = _random_csr(rng, N, 0.4, symmetric=bool(seed % 2), loops=True)
    assign = rng.integers(0, K, size=N).astype(np.int32)
    cut = sum(1 for u in range(N) for v in range(N) if A[u, v] and assign[u] != assign[v])
    q = oracle.partition_quality(rowptr, colidx, assign, K)
    assert q.edge_cut == cut
    assert q.part_vertices.tolist() == [int((assign == p).sum()) for p in range(K)]
    assert q.part_edges.tolist() == [int(A[assign == p].sum()) for p in range(K)]


def test_closed_forms_and_ranges():
    rng = np.random.default_rng(42)
    N = 300
    A, rowptr, colidx = _random_csr(rng, N, 0.05, symmetric=True, loops=True)
    nnz = len(colidx)
    loops = int(np.trace(A))
    assert loops > 0
    same = oracle.partition_quality(rowptr, colidx, np.zeros(N, np.int32), 3)
    assert same.edge_cut == 0 and same.part_vertices.tolist() == [N, 0, 0] and same.part_edges.tolist() == [nnz, 0, 0]
    # balance = max/mean = K when one partition holds everything (Eq. 2)
    assert same.part_vertices.max() / (N / 3) == 3
    alone = oracle.partition_quality(rowptr, colidx, np.arange(N, dtype=np.int32), N)
    assert alone.edge_cut == nnz - loops                   # every entry but the self-loops is cut
    mod = oracle.partition_quality(rowptr, colidx, (np.arange(N) % 4).astype(np.int32), 4)
    assert mod.part_vertices.tolist() == [75] * 4          # balance exactly 1 when K divides N
    assert mod.part_vertices.max() / (N / 4) == 1
    assert 0 <= mod.edge_cut <= nnz and mod.edge_cut % 2 == 0     # symmetric graph: cut entries pair up
    assert mod.part_vertices.sum() == N and mod.part_edges.sum() == nnz


def test_library_special_case_scipy():
    sp = pytest.importorskip("scipy.sparse")
    rng = np.random.default_rng(3)
    N, K = 500, 7
    _, rowptr, colidx = _random_csr(rng, N, 0.03)
    assign = rng.integers(0, K, size=N).astype(np.int32)
    M = sp.csr_matrix((np.ones(len(colidx)), colidx, rowptr), shape=(N, N))
    onehot = sp.csr_matrix((np.ones(N), (np.arange(N), assign)), shape=(N, K))
    block = (onehot.T @ M @ onehot).toarray()              # block[p, q] = entries from p to q
    q = oracle.partition_quality(rowptr, colidx, assign, K)
    assert q.edge_cut == int(block.sum() - np.trace(block))
    assert q.part_edges.tolist() == block.sum(1).astype(int).tolist()


def test_random_assignment_cuts_about_one_minus_one_over_k():
    """Statistical sanity: a uniform random partition cuts a fraction 1 - sum (n_p/N)^2 of the entries."""
    rng = np.random.default_rng(4)
    N, K = 2000, 8
    _, rowptr, colidx = _random_csr(rng, N, 0.02)
    assign = rng.integers(0, K, size=N).astype(np.int32)
    q = oracle.partition_quality(rowptr, colidx, assign, K)
    expect = 1 - ((q.part_vertices / N) ** 2).sum()
    assert abs(q.edge_cut / len(colidx) - expect) < 0.01


def test_rejects_bad_inputs():
    with pytest.raises(ValueError):
        oracle.partition_quality([0, 1], [0], [2], 2)
    with pytest.raises(ValueError):
        oracle.partition_quality([0, 1], [5], [0], 2)
    with pytest.raises(ValueError):
        oracle.reorder([0, 3], 3)


# ---------------------------------------------------------------------------------------------- reorder
@pytest.mark.parametrize("seed", range(8))
def test_reorder_equals_sorting_by_label_then_id(seed):
    rng = np.random.default_rng(seed)
    N, K = int(rng.integers(1, 200)), int(rng.integers(1, 12))
    assign = rng.integers(0, K, size=N).astype(np.int32)
    perm, inv = oracle.reorder(assign, K)
    assert perm.tolist() == sorted(range(N), key=lambda v: (int(assign[v]), v))
    np.testing.assert_array_equal(perm, np.argsort(assign, kind="stable"))
    assert sorted(perm.tolist()) == list(range(N))                       # bijection
    np.testing.assert_array_equal(inv[perm], np.arange(N))
    np.testing.assert_array_equal(perm[inv], np.arange(N))


def test_reorder_brute_force_definition():
    # "vertices of the same partition get consecutive ids": walk partitions in order, vertices in order
    assign = np.array([2, 0, 2, 1, 0, 2, 1, 1, 0, 3], np.int32)
    want = [v for p in range(5) for v in range(len(assign)) if assign[v] == p]
    perm, inv = oracle.reorder(assign, 5)
    assert perm.tolist() == want == [1, 4, 8, 3, 6, 7, 0, 2, 5, 9]
    assert inv.tolist() == [6, 0, 7, 3, 1, 8, 4, 5, 2, 9]


def test_reorder_structure_on_a_larger_case():
    rng = np.random.default_rng(77)
    N, K = 50_000, 300
    assign = rng.integers(0, K, size=N).astype(np.int32)
    assign[assign == 17] = 18                                            # an empty partition
    perm, inv = oracle.reorder(assign, K)
    lab = assign[perm]
    assert np.all(np.diff(lab) >= 0)                                     # grouped, ascending partitions
    same = np.diff(lab) == 0
    assert np.all(np.diff(perm)[same] > 0)                               # original order inside a partition
    counts = np.bincount(assign, minlength=K)
    starts = np.concatenate([[0], np.cumsum(counts)[:-1]])
    for p in (0, 16, 18, K - 1):
        seg = perm[starts[p]: starts[p] + counts[p]]
        assert np.all(assign[seg] == p)
    assert counts[17] == 0


# ---------------------------------------------------------------------------------- graph bandwidth
def _bandwidth_cases():
    with open(os.path.join(GOLDEN, "graph_bandwidth_hand_cases.json")) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _bandwidth_cases(), ids=lambda c: c["name"][:40])
def test_bandwidth_hand_cases(case):
    b = oracle.graph_bandwidth(case["rowptr"], case["colidx"], case["pi"])
    assert b.vertex_bandwidth.tolist() == case["vertex_bandwidth"]
    assert b.bandwidth_sum == case["bandwidth_sum"] == sum(case["vertex_bandwidth"])
    assert b.average == case["bandwidth_sum"] / len(case["pi"])


@pytest.mark.parametrize("seed", range(6))
def test_bandwidth_brute_force_dense_adjacency(seed):
    """Eq. 3-5 written as a double loop over a dense adjacency matrix, any numbering."""
    rng = np.random.default_rng(100 + seed)
    N = int(rng.integers(2, 11))
    A, rowptr, colidx = _random_csr(rng, N, 0.35, symmetric=bool(seed % 2), loops=True)
    pi = rng.permutation(N).astype(np.int32)
    beta = [max([abs(int(pi[v]) - int(pi[u])) for u in range(N) if A[v, u]], default=0) for v in range(N)]
    b = oracle.graph_bandwidth(rowptr, colidx, pi)
    assert b.vertex_bandwidth.tolist() == beta and b.bandwidth_sum == sum(beta)


def test_bandwidth_closed_forms_and_invariances():
    rng = np.random.default_rng(7)
    # complete graph, identity numbering: the farthest neighbour of v is vertex 0 or vertex n-1
    n = 9
    A = ~np.eye(n, dtype=bool)
    rowptr = np.arange(n + 1, dtype=np.int64) * (n - 1)
    colidx = np.nonzero(A)[1].astype(np.int32)
    b = oracle.graph_bandwidth(rowptr, colidx, np.arange(n))
    assert b.vertex_bandwidth.tolist() == [max(v, n - 1 - v) for v in range(n)]
    # any graph, any numbering
    N = 200
    A, rowptr, colidx = _random_csr(rng, N, 0.03, symmetric=True)
    pi = rng.permutation(N).astype(np.int32)
    b = oracle.graph_bandwidth(rowptr, colidx, pi)
    deg = np.diff(rowptr)
    assert ((b.vertex_bandwidth >= 0) & (b.vertex_bandwidth <= N - 1)).all()
    assert (b.vertex_bandwidth[deg == 0] == 0).all() and (b.vertex_bandwidth[deg > 0] >= 1).all()
    # mirror image of the numbering: every gap is unchanged
    assert np.array_equal(oracle.graph_bandwidth(rowptr, colidx, N - 1 - pi).vertex_bandwidth, b.vertex_bandwidth)
    # renaming the vertices by pi and numbering the renamed graph by the identity is the same layout
    A2 = np.zeros_like(A)
    A2[np.ix_(pi, pi)] = A
    rowptr2 = np.concatenate([[0], np.cumsum(A2.sum(1))]).astype(np.int64)
    colidx2 = np.nonzero(A2)[1].astype(np.int32)
    b2 = oracle.graph_bandwidth(rowptr2, colidx2, np.arange(N))
    assert np.array_equal(b2.vertex_bandwidth[pi], b.vertex_bandwidth) and b2.bandwidth_sum == b.bandwidth_sum
    # a symmetric graph: the largest vertex bandwidth is attained at both ends of the widest edge
    assert (b.vertex_bandwidth == b.vertex_bandwidth.max()).sum() >= 2


def test_bandwidth_of_partition_ordered_numbering_beats_a_random_one():
    """Statistical sanity (Section 4.5.1): numbering a planted-partition graph by its blocks keeps
    neighbours closer than a random numbering does."""
    rng = np.random.default_rng(3)
    N, K = 400, 8
    block = rng.integers(0, K, size=N)
    P = np.where(block[:, None] == block[None, :], 0.10, 0.002)
    A = rng.random((N, N)) < P
    A = A | A.T
    np.fill_diagonal(A, False)
    rowptr = np.concatenate([[0], np.cumsum(A.sum(1))]).astype(np.int64)
    colidx = np.nonzero(A)[1].astype(np.int32)
    _, inv = oracle.reorder(block.astype(np.int32), K)
    grouped = oracle.graph_bandwidth(rowptr, colidx, inv).average
    shuffled = oracle.graph_bandwidth(rowptr, colidx, rng.permutation(N)).average
    assert grouped < shuffled


def test_bandwidth_rejects_bad_input():
    with pytest.raises(ValueError):
        oracle.graph_bandwidth([0, 1, 2], [1, 0], [0, 0])            # not a bijection
    with pytest.raises(ValueError):
        oracle.graph_bandwidth([0, 1, 2], [1, 5], [0, 1])            # neighbour outside [0, N)


# ------------------------------------------------------------------- the graph under a new numbering
def test_relabel_hand_case():
    """Path 0-1-2-3 numbered 2,0,3,1 (perm = [1,3,0,2]): worked by hand.
    new vertex 0 = old 1 (neighbours 0,2 -> 2,3); 1 = old 3 (2 -> 3); 2 = old 0 (1 -> 0); 3 = old 2 (1,3 -> 0,1)."""
    rowptr, colidx = [0, 1, 3, 5, 6], [1, 0, 2, 1, 3, 2]
    perm, inv = [1, 3, 0, 2], [2, 0, 3, 1]
    rp, ci = oracle.relabel_graph(rowptr, colidx, perm, inv)
    assert rp.tolist() == [0, 2, 3, 4, 6] and ci.tolist() == [2, 3, 3, 0, 0, 1]


@pytest.mark.parametrize("seed", range(4))
def test_relabel_is_the_same_graph_under_other_names(seed):
    rng = np.random.default_rng(200 + seed)
    N, K = int(rng.integers(5, 40)), 4
    A, rowptr, colidx = _random_csr(rng, N, 0.2, symmetric=bool(seed % 2), loops=True)
    assign = rng.integers(0, K, size=N).astype(np.int32)
    perm, inv = oracle.reorder(assign, K)
    rp, ci = oracle.relabel_graph(rowptr, colidx, perm, inv)
    # adjacency matrix renamed on both axes
    A2 = np.zeros_like(A)
    for i in range(N):
        A2[i, ci[rp[i]:rp[i + 1]]] = True
    assert np.array_equal(A2, A[np.ix_(perm, perm)])
    assert np.array_equal(np.diff(rp), np.diff(rowptr)[perm])
    # the metrics do not care about names: cut with renamed labels, bandwidth with the identity numbering
    q, q2 = oracle.partition_quality(rowptr, colidx, assign, K), oracle.partition_quality(rp, ci, assign[perm], K)
    assert q.edge_cut == q2.edge_cut and q.part_vertices.tolist() == q2.part_vertices.tolist()
    b, b2 = oracle.graph_bandwidth(rowptr, colidx, inv), oracle.graph_bandwidth(rp, ci, np.arange(N))
    assert b.bandwidth_sum == b2.bandwidth_sum and np.array_equal(b2.vertex_bandwidth, b.vertex_bandwidth[perm])
    # identity numbering changes nothing; relabelling back restores every row, entry order included
    ident = np.arange(N, dtype=np.int32)
    rp0, ci0 = oracle.relabel_graph(rowptr, colidx, ident, ident)
    assert np.array_equal(rp0, rowptr) and np.array_equal(ci0, colidx)
    rp3, ci3 = oracle.relabel_graph(rp, ci, inv, perm)
    assert np.array_equal(rp3, rowptr) and np.array_equal(ci3, colidx)


def test_permute_rows_and_bad_permutations():
    rng = np.random.default_rng(9)
    emb = rng.normal(size=(17, 8)).astype(np.float32)
    perm = rng.permutation(17).astype(np.int32)
    out = oracle.permute_rows(emb, perm)
    assert np.array_equal(out, emb[perm])
    with pytest.raises(ValueError):
        oracle.permute_rows(emb, np.zeros(17, np.int32))
    with pytest.raises(ValueError):
        oracle.relabel_graph([0, 1, 2], [1, 0], [0, 1], [1, 0])        # inv_perm is not the inverse
