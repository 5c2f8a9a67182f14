"""GPU parity: ep_relabel_graph / ep_permute_rows (the graph and the rows under the new numbering,
Section 4.5.1) against the oracle, bit for bit."""
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


def _labels(N, K, seed):
    return torch.randint(0, K, (N,), generator=torch.Generator().manual_seed(seed), dtype=torch.int32).cuda()


def _matches(ctx, rowptr, colidx, K, seed):
    N = rowptr.numel() - 1
    order = ctx.reorder(_labels(N, K, seed), K)
    new_rowptr, new_colidx = ctx.relabel_graph(rowptr, colidx, order.perm, order.inv_perm)
    torch.cuda.synchronize()
    ctx.check()
    rp, ci = oracle.relabel_graph(rowptr.cpu().numpy(), colidx.cpu().numpy(), order.perm.cpu().numpy(),
                                  order.inv_perm.cpu().numpy())
    assert new_rowptr.dtype == rowptr.dtype
    np.testing.assert_array_equal(new_rowptr.cpu().numpy().astype(np.int64), rp)
    np.testing.assert_array_equal(new_colidx.cpu().numpy(), ci)
    return order, new_rowptr, new_colidx


@pytest.mark.parametrize("name", ["cfg1", "cfg2"])
def test_full_small_configs(ctx, name):
    w = synth.WORKLOADS[name]
    rowptr, colidx = synth.graph(w, device="cuda")
    _matches(ctx, rowptr, colidx, w.K, 1)
    _matches(ctx, rowptr.to(torch.int64), colidx, 300, 2)


@pytest.mark.parametrize("name,N", [("cfg3", 6_007), ("cfg4", 50_021), ("cfg5", 100_003)])
def test_scaled_configs_and_metrics_survive_the_renaming(ctx, name, N):
    w = synth.scaled(synth.WORKLOADS[name], N)
    rowptr, colidx = synth.graph(w, device="cuda")
    order, rp2, ci2 = _matches(ctx, rowptr, colidx, 64, 3)
    # the bandwidth of the numbering on the old graph = the bandwidth of the identity numbering on the new one
    a = ctx.graph_bandwidth(rowptr, colidx, order.inv_perm)
    b = ctx.graph_bandwidth(rp2, ci2, torch.arange(N, dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert int(a.bandwidth_sum.item()) == int(b.bandwidth_sum.item())
    assert torch.equal(b.vertex_bandwidth, a.vertex_bandwidth[order.perm.long()])


def test_odd_csr_shapes(ctx):
    rng = np.random.default_rng(13)
    N = 30_000
    deg = rng.integers(0, 4, size=N)
    deg[rng.integers(0, N, size=50)] = rng.integers(3_000, 30_000, size=50)       # rows on both sides of the block-per-row limit
    deg[1000:9000] = 0
    deg[-5:] = 0
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    colidx = rng.integers(0, N, size=int(rowptr[-1])).astype(np.int32)            # unsorted, duplicates, self-loops
    for dtype in (torch.int32, torch.int64):
        _matches(ctx, torch.from_numpy(rowptr).to(dtype).cuda(), torch.from_numpy(colidx).cuda(), 7, 4)


@pytest.mark.parametrize("N", [1, 2, 2047, 2048, 2049, 70_001, 600_011])
def test_prefix_sum_sizes(ctx, N):
    """Row counts around the scan tile (2048 lengths) and beyond one block of tile totals."""
    rng = np.random.default_rng(N)
    deg = rng.integers(0, 3, size=N)
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int32)
    nnz = int(rowptr[-1])
    colidx = rng.integers(0, N, size=nnz).astype(np.int32)
    ci = torch.from_numpy(colidx).cuda() if nnz else torch.empty(0, dtype=torch.int32, device="cuda")
    _matches(ctx, torch.from_numpy(rowptr).cuda(), ci, min(N, 5), 5)


def test_permute_rows(ctx):
    w = synth.scaled(synth.WORKLOADS["cfg3"], 9_973)
    emb = synth.embeddings(w, device="cuda")
    order = ctx.reorder(_labels(w.N, 16, 6), 16)
    out = ctx.permute_rows(emb, order.perm)
    torch.cuda.synchronize()
    ctx.check()
    np.testing.assert_array_equal(out.cpu().numpy(), oracle.permute_rows(emb.cpu().numpy(), order.perm.cpu().numpy()))


def test_bad_indices_raise_a_status_without_faulting(ctx):
    rowptr = torch.tensor([0, 2, 4, 6], dtype=torch.int32).cuda()
    colidx = torch.tensor([1, 2, 0, 99, 0, 1], dtype=torch.int32).cuda()          # 99 is outside [0, N)
    ident = torch.arange(3, dtype=torch.int32).cuda()
    ctx.relabel_graph(rowptr, colidx, ident, ident)
    assert ctx.poll_status() == 4
    ctx.relabel_graph(rowptr, colidx.clamp(max=2), torch.tensor([0, 7, 2], dtype=torch.int32).cuda(), ident)
    assert ctx.poll_status() == 4                                                 # perm value outside [0, N)
    ctx.permute_rows(torch.zeros(3, 8, device="cuda"), torch.tensor([0, 1, 3], dtype=torch.int32).cuda())
    assert ctx.poll_status() == 4 and ctx.poll_status() == 0
