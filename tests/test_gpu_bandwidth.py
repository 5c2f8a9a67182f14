"""GPU parity: ep_graph_bandwidth (Section 4.5.1, Eq. 3-5) against the oracle, bit for bit."""
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


def _matches(ctx, rowptr, colidx, pi):
    got = ctx.graph_bandwidth(rowptr, colidx, pi)
    only_sum = ctx.graph_bandwidth(rowptr, colidx, pi, per_vertex=False)
    torch.cuda.synchronize()
    ctx.check()
    ref = oracle.graph_bandwidth(rowptr.cpu().numpy(), colidx.cpu().numpy(), pi.cpu().numpy())
    np.testing.assert_array_equal(got.vertex_bandwidth.cpu().numpy(), ref.vertex_bandwidth)
    assert int(got.bandwidth_sum.item()) == ref.bandwidth_sum
    assert only_sum.vertex_bandwidth is None and int(only_sum.bandwidth_sum.item()) == ref.bandwidth_sum
    return ref


def _random_numbering(N, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randperm(N, generator=g).to(torch.int32).cuda()


@pytest.mark.parametrize("name", ["cfg1", "cfg2"])
def test_full_small_configs(ctx, name):
    w = synth.WORKLOADS[name]
    rowptr, colidx = synth.graph(w, device="cuda")
    ident = torch.arange(w.N, dtype=torch.int32, device="cuda")
    _matches(ctx, rowptr, colidx, ident)
    _matches(ctx, rowptr.to(torch.int64), colidx, _random_numbering(w.N, 1))


@pytest.mark.parametrize("name,N", [("cfg3", 6_007), ("cfg4", 50_021), ("cfg5", 100_003)])
def test_scaled_configs(ctx, name, N):
    w = synth.scaled(synth.WORKLOADS[name], N)
    rowptr, colidx = synth.graph(w, device="cuda")
    _matches(ctx, rowptr, colidx, _random_numbering(N, 2))


def test_numbering_by_kmeans_clusters_narrows_the_planted_graph(ctx):
    """The path the metric is for: cluster, reorder, score the new numbering (statistical sanity)."""
    w = synth.WORKLOADS["cfg1"]
    emb = synth.embeddings(w, device="cuda")
    init = emb[synth.init_centroid_rows(w, 8, device="cuda")].contiguous()
    rowptr, colidx = synth.graph(w, device="cuda")
    km = ctx.kmeans(emb, 8, 10, init)
    order = ctx.reorder(km.assign, 8)
    grouped = _matches(ctx, rowptr, colidx, order.inv_perm)
    shuffled = _matches(ctx, rowptr, colidx, _random_numbering(w.N, 3))
    assert grouped.bandwidth_sum < shuffled.bandwidth_sum


def test_odd_csr_shapes(ctx):
    rng = np.random.default_rng(11)
    N = 30_000
    deg = rng.integers(0, 4, size=N)
    deg[rng.integers(0, N, size=50)] = rng.integers(5_000, 30_000, size=50)       # rows far longer than a tile
    deg[1000:9000] = 0                                                            # a long run of empty rows
    deg[-5:] = 0                                                                  # empty rows at the end
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    nnz = int(rowptr[-1])
    colidx = rng.integers(0, N, size=nnz).astype(np.int32)                        # unsorted, duplicates, self-loops
    for dtype in (torch.int32, torch.int64):
        rp = torch.from_numpy(rowptr).to(dtype).cuda()
        _matches(ctx, rp, torch.from_numpy(colidx).cuda(), _random_numbering(N, 4))


@pytest.mark.parametrize("nnz", [0, 1, 3, 4, 5, 4095, 4096, 4097, 8191, 8192, 8193, 16_387])
def test_tile_boundaries(ctx, nnz):
    rng = np.random.default_rng(nnz + 1)
    N = 97
    cuts = np.sort(rng.integers(0, nnz + 1, size=N - 1))
    rowptr = np.concatenate([[0], cuts, [nnz]]).astype(np.int32)
    colidx = rng.integers(0, N, size=nnz).astype(np.int32)
    ci = torch.from_numpy(colidx).cuda() if nnz else torch.empty(0, dtype=torch.int32, device="cuda")
    _matches(ctx, torch.from_numpy(rowptr).cuda(), ci, _random_numbering(N, 5))


def test_single_vertex_and_self_loops(ctx):
    rowptr = torch.tensor([0, 2], dtype=torch.int32).cuda()
    colidx = torch.tensor([0, 0], dtype=torch.int32).cuda()
    ref = _matches(ctx, rowptr, colidx, torch.zeros(1, dtype=torch.int32).cuda())
    assert ref.bandwidth_sum == 0


def test_bad_indices_raise_a_status_without_faulting(ctx):
    rowptr = torch.tensor([0, 2, 4, 6], dtype=torch.int32).cuda()
    colidx = torch.tensor([1, 2, 0, 99, 0, 1], dtype=torch.int32).cuda()          # 99 is outside [0, N)
    pi = torch.tensor([0, 1, 2], dtype=torch.int32).cuda()
    got = ctx.graph_bandwidth(rowptr, colidx, pi)
    assert ctx.poll_status() == 4
    assert got.vertex_bandwidth.tolist() == [2, 1, 2]                             # the bad entry is skipped
    ctx.graph_bandwidth(torch.tensor([0, 4, 2, 6], dtype=torch.int32).cuda(), colidx.clamp(max=2), pi)
    assert ctx.poll_status() == 4                                                 # row pointer goes backwards
    assert ctx.poll_status() == 0


def test_host_buffer_variant(ctx):
    w = synth.scaled(synth.WORKLOADS["cfg4"], 20_011)
    rowptr, colidx = synth.graph(w, device="cpu")
    pi = torch.randperm(w.N, generator=torch.Generator().manual_seed(6)).to(torch.int32)
    out = ctx.graph_bandwidth_host(rowptr.pin_memory(), colidx.pin_memory(), pi.pin_memory())
    torch.cuda.synchronize()
    ctx.check()
    ref = oracle.graph_bandwidth(rowptr.numpy(), colidx.numpy(), pi.numpy())
    assert int(out.bandwidth_sum.item()) == ref.bandwidth_sum
    np.testing.assert_array_equal(out.vertex_bandwidth.numpy(), ref.vertex_bandwidth)
