"""GPU parity: ep_migrate / ep_balance (Algorithm 4 and the balancing loop of Algorithm 3) against the
oracle, bit for bit; the random words are inputs to both."""
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


def _words(shape, seed):
    """32 random bits per entry as an int32 tensor (the library reads them as unsigned)."""
    g = torch.Generator().manual_seed(seed)
    return torch.randint(-2 ** 31, 2 ** 31, shape, generator=g, dtype=torch.int64).to(torch.int32)


def _skewed_labels(N, K, seed):
    rng = np.random.default_rng(seed)
    return torch.from_numpy(rng.choice(K, size=N, p=rng.dirichlet(np.ones(K) * 0.6)).astype(np.int32))


def _one_round(ctx, rowptr, N, K, seed, member_frac=None, beta=1.05):
    assign = _skewed_labels(N, K, seed)
    member = None
    if member_frac is not None:
        member = (torch.rand(N, generator=torch.Generator().manual_seed(seed + 1)) < member_frac).to(torch.uint8)
    S = N if member is None else int(member.sum())
    C = int(np.floor(beta * S / K))
    rw = _words((N,), seed + 2)
    deg = np.diff(rowptr.cpu().numpy().astype(np.int64))
    a_dev = assign.clone().cuda()
    state = ctx.migrate(rowptr, a_dev, K, C, int(deg.max()), rw.cuda(), None if member is None else member.cuda())
    torch.cuda.synchronize()
    ctx.check()
    ref, moved = oracle.migrate(rowptr.cpu().numpy(), assign.numpy(), K, C, rw.numpy().view(np.uint32),
                                None if member is None else member.numpy())
    np.testing.assert_array_equal(a_dev.cpu().numpy(), ref)
    assert int(state[2].item()) == moved
    return moved


@pytest.mark.parametrize("name,N,K", [("cfg1", 10_000, 4), ("cfg2", 50_021, 8), ("cfg4", 120_011, 32), ("cfg5", 80_003, 64)])
def test_one_application_matches_the_oracle(ctx, name, N, K):
    w = synth.WORKLOADS[name] if synth.WORKLOADS[name].N == N else synth.scaled(synth.WORKLOADS[name], N)
    rowptr, _ = synth.graph(w, device="cuda")
    assert _one_round(ctx, rowptr, N, K, 1) > 0
    assert _one_round(ctx, rowptr.to(torch.int64), N, K, 2, member_frac=0.3) > 0


def test_equal_degrees_and_empty_rows(ctx):
    """Ties everywhere: the lower vertex id must go first."""
    N, K = 40_000, 5
    deg = np.zeros(N, np.int64)
    deg[::3] = 2
    deg[5::7] = 1
    rowptr = torch.from_numpy(np.concatenate([[0], np.cumsum(deg)]).astype(np.int32)).cuda()
    _one_round(ctx, rowptr, N, K, 3)
    _one_round(ctx, rowptr, N, K, 4, member_frac=0.5, beta=1.0)


def test_balanced_input_is_left_alone(ctx):
    N, K = 10_000, 4
    rowptr = torch.arange(N + 1, dtype=torch.int32).cuda()
    assign = (torch.arange(N) % K).to(torch.int32).cuda()
    before = assign.clone()
    state = ctx.migrate(rowptr, assign, K, N // K, 1, _words((N,), 5).cuda())
    torch.cuda.synchronize()
    assert state.tolist() == [0, 0, 0, 0] and torch.equal(assign, before)


@pytest.mark.parametrize("K,member_frac", [(8, None), (32, 0.65), (3, 0.1)])
def test_balancing_loop_matches_the_oracle_and_reaches_the_bound(ctx, K, member_frac):
    w = synth.scaled(synth.WORKLOADS["cfg4"], 60_013)
    N = w.N
    rowptr, _ = synth.graph(w, device="cuda")
    assign = _skewed_labels(N, K, 7)
    member = None if member_frac is None else (torch.rand(N, generator=torch.Generator().manual_seed(8)) < member_frac).to(torch.uint8)
    S = N if member is None else int(member.sum())
    beta = 1.05
    C = int(np.floor(beta * S / K))
    rounds = _words((12, N), 9)
    deg = np.diff(rowptr.cpu().numpy().astype(np.int64))
    a_dev = assign.clone().cuda()
    used = ctx.balance(rowptr, a_dev, K, C, int(deg.max()), rounds.cuda(), None if member is None else member.cuda())
    ctx.check()
    ref, ref_rounds = oracle.balance(rowptr.cpu().numpy(), assign.numpy(), K, C, rounds.numpy().view(np.uint32),
                                     None if member is None else member.numpy().astype(bool))
    np.testing.assert_array_equal(a_dev.cpu().numpy(), ref)
    assert used == ref_rounds >= 1
    sel = np.ones(N, bool) if member is None else member.numpy().astype(bool)
    load = np.bincount(ref[sel], minlength=K)
    assert load.max() <= C and load.max() / (S / K) <= beta                      # vertex balance (Eq. 2) within beta


def test_errors(ctx):
    import paper_2604_01000_b200 as ep
    N, K = 1000, 4
    rowptr = torch.arange(N + 1, dtype=torch.int32).cuda()
    assign = torch.zeros(N, dtype=torch.int32).cuda()
    with pytest.raises(ep.EmbedPartError):                                        # capacity x K cannot hold the set
        ctx.balance(rowptr, assign, K, 100, 1, _words((3, N), 1).cuda())
    with pytest.raises(ep.EmbedPartError):                                        # key range too large
        ctx.migrate(rowptr, assign, 1024, 10, 2 ** 21, _words((N,), 1).cuda())
    bad = assign.clone()
    bad[5] = 9                                                                    # label outside [0, K)
    ctx.migrate(rowptr, bad, K, 400, 1, _words((N,), 2).cuda())
    assert ctx.poll_status() == 4 and ctx.poll_status() == 0


def test_phase_two_as_a_whole(ctx):
    """ep_cluster_and_balance against the oracle's composition (K-Means labels up to near-ties, so the
    comparison is made stage by stage: the balancing stages on the library's own K-Means labels)."""
    w = synth.scaled(synth.WORKLOADS["cfg4"], 40_009)
    N, K = w.N, 8
    emb = synth.embeddings(w, device="cuda")
    init = emb[synth.init_centroid_rows(w, K, device="cuda")].contiguous()
    rowptr, _ = synth.graph(w, device="cuda")
    split = torch.from_numpy(np.random.default_rng(1).choice(3, size=N, p=[0.5, 0.2, 0.3]).astype(np.uint8))
    caps = [int(np.floor(1.05 * int((split == s).sum()) / K)) for s in range(3)]
    words = _words((3, 10, N), 11)
    deg = np.diff(rowptr.cpu().numpy().astype(np.int64))
    got, used = ctx.cluster_and_balance(emb, K, 6, init, rowptr, int(deg.max()), split.cuda(), caps, words.cuda())
    ctx.check()
    km = ctx.kmeans(emb, K, 6, init)                                   # the same first stage on its own
    torch.cuda.synchronize()
    assert torch.equal(got.centroids, km.centroids)
    ref = km.assign.cpu().numpy()
    ref_used = []
    for s in range(3):
        ref, r = oracle.balance(rowptr.cpu().numpy(), ref, K, caps[s], words[s].numpy().view(np.uint32), (split == s).numpy())
        ref_used.append(r)
    np.testing.assert_array_equal(got.assign.cpu().numpy(), ref)
    assert used == ref_used
    for s in range(3):
        assert np.bincount(ref[(split == s).numpy()], minlength=K).max() <= caps[s]


def test_loose_degree_bound_takes_the_four_pass_sort(ctx):
    """A degree bound far above the real degrees makes the sort key wider than 24 bits (four radix passes);
    the result does not depend on the bound."""
    w = synth.scaled(synth.WORKLOADS["cfg4"], 50_021)
    rowptr, _ = synth.graph(w, device="cuda")
    N, K = w.N, 32
    assign = _skewed_labels(N, K, 21)
    C = int(np.floor(1.05 * N / K))
    rw = _words((N,), 22)
    deg = np.diff(rowptr.cpu().numpy().astype(np.int64))
    tight, loose = assign.clone().cuda(), assign.clone().cuda()
    ctx.migrate(rowptr, tight, K, C, int(deg.max()), rw.cuda())
    ctx.migrate(rowptr, loose, K, C, (1 << 24) - 1, rw.cuda())                    # K (D + 1) = 2^29
    torch.cuda.synchronize()
    ctx.check()
    ref, _ = oracle.migrate(rowptr.cpu().numpy(), assign.numpy(), K, C, rw.numpy().view(np.uint32))
    np.testing.assert_array_equal(tight.cpu().numpy(), ref)
    np.testing.assert_array_equal(loose.cpu().numpy(), ref)
