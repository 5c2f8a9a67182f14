"""Pins for the oracle's migration policy (Algorithm 4) and balancing loop (Algorithm 3); CPU only."""
import numpy as np
import pytest

import oracle


def _rowptr(deg):
    return np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)


def test_hand_case():
    """8 vertices, k = 3, C = 3.  Partition 0 holds {0,1,2,3,4} (L = 5, m = 2), partition 1 {5,6} (f = 1),
    partition 2 {7} (f = 2), F = 3.  Degrees of partition 0: 4,1,3,1,2 -> the two smallest are vertices 1 and 3
    (equal degree: lower id first).  Free capacity laid end to end: t = 0 -> partition 1, t = 1, 2 -> partition 2.
    rand 0 gives t = 0; rand 2^31 gives floor(0.5 * 3) = 1."""
    deg = [4, 1, 3, 1, 2, 7, 7, 7]
    assign = [0, 0, 0, 0, 0, 1, 1, 2]
    rand = np.zeros(8, np.uint32)
    rand[3] = 1 << 31
    out, moved = oracle.migrate(_rowptr(deg), assign, 3, 3, rand)
    assert moved == 2 and out.tolist() == [0, 1, 0, 2, 0, 1, 1, 2]
    # the largest word lands in the last unit of free capacity
    rand[1] = 0xFFFFFFFF
    out, _ = oracle.migrate(_rowptr(deg), assign, 3, 3, rand)
    assert out.tolist() == [0, 2, 0, 2, 0, 1, 1, 2]


@pytest.mark.parametrize("seed", range(6))
def test_one_round_against_numpy(seed):
    rng = np.random.default_rng(300 + seed)
    N, K = int(rng.integers(30, 400)), int(rng.integers(2, 7))
    deg = rng.integers(0, 6, size=N)                                   # many equal degrees
    assign = rng.choice(K, size=N, p=rng.dirichlet(np.ones(K) * 0.7)).astype(np.int32)
    member = rng.random(N) < 0.8 if seed % 2 else None
    sel = np.ones(N, bool) if member is None else member
    S = int(sel.sum())
    C = int(np.floor(1.05 * S / K))
    rand = rng.integers(0, 2 ** 32, size=N, dtype=np.uint64).astype(np.uint32)
    load = np.bincount(assign[sel], minlength=K)
    if (load > C).any() and not (load < C).any():
        pytest.skip("nothing underloaded")
    out, moved = oracle.migrate(_rowptr(deg), assign, K, C, rand, member)
    # who moves: per overloaded partition the m smallest by (degree, id), members only
    expect = assign.copy()
    free = np.where(load < C, C - load, 0)
    cum = np.cumsum(free)
    F = int(cum[-1])
    for i in np.flatnonzero(load > C):
        ids = np.flatnonzero(sel & (assign == i))
        order = ids[np.lexsort((ids, deg[ids]))]
        for v in order[: load[i] - C]:
            t = (int(rand[v]) * F) >> 32
            expect[v] = int(np.searchsorted(cum, t, side="right"))
    assert np.array_equal(out, expect) and moved == int((out != assign).sum())
    new_load = np.bincount(out[sel], minlength=K)
    assert (new_load[load > C] == C).all()                             # every overloaded partition lands on C
    assert (out[~sel] == assign[~sel]).all()                           # vertices outside S never move
    assert set(out[out != assign].tolist()) <= set(np.flatnonzero(load < C).tolist())
    assert new_load.sum() == S


def test_destinations_follow_free_capacity():
    """Evenly spaced random words: the share of each underloaded partition is its share of the free capacity."""
    K, C = 4, 1000
    assign = np.concatenate([np.zeros(2200, np.int32), np.full(700, 1), np.full(900, 2), np.full(200, 3)]).astype(np.int32)
    N = assign.size                                                    # S = 4000, loads 2200/700/900/200, m_0 = 1200
    deg = np.arange(N)                                                 # vertex id order = degree order
    rand = np.array([-((-(i % 1200) << 32) // 1200) for i in range(N)], dtype=np.uint64).astype(np.uint32)   # ceil(i 2^32 / F): t = i
    out, moved = oracle.migrate(_rowptr(deg), assign, K, C, rand)
    assert moved == 1200 and (out[1200:2200] == 0).all()               # the 1200 lowest degrees left partition 0
    got = np.bincount(out[:1200], minlength=K)
    assert got.tolist() == [0, 300, 100, 800]                          # f = 300, 100, 800 of F = 1200


def test_nothing_to_do_and_nowhere_to_go():
    deg = np.ones(6, np.int64)
    out, moved = oracle.migrate(_rowptr(deg), [0, 0, 1, 1, 2, 2], 3, 2, np.zeros(6, np.uint32))
    assert moved == 0 and out.tolist() == [0, 0, 1, 1, 2, 2]
    with pytest.raises(ValueError):
        oracle.migrate(_rowptr(deg), [0, 0, 0, 0, 1, 1], 2, 2, np.zeros(6, np.uint32))   # C * K < |S|


@pytest.mark.parametrize("seed", range(3))
def test_balancing_loop_reaches_the_bound(seed):
    rng = np.random.default_rng(400 + seed)
    N, K, beta = 5000, 8, 1.05
    deg = rng.integers(1, 50, size=N)
    assign = rng.choice(K, size=N, p=rng.dirichlet(np.ones(K) * 0.5)).astype(np.int32)
    member = rng.random(N) < 0.6
    S = int(member.sum())
    C = int(np.floor(beta * S / K))
    rounds_words = rng.integers(0, 2 ** 32, size=(20, N), dtype=np.uint64).astype(np.uint32)
    out, rounds = oracle.balance(_rowptr(deg), assign, K, C, rounds_words, member)
    load = np.bincount(out[member], minlength=K)
    assert load.max() <= C and load.max() / (S / K) <= beta            # Eq. 2 at most beta
    assert 1 <= rounds <= 20 and (out[~member] == assign[~member]).all()
    # migration prefers low degrees: the moved vertices have a lower mean degree than those that stayed
    moved = member & (out != assign)
    assert deg[moved].mean() < deg[member & ~moved].mean()


def test_phase_two_as_a_whole():
    """Algorithm 3: clustering, then the three balancing loops in the order training, validation, rest."""
    rng = np.random.default_rng(77)
    N, K, d = 3000, 6, 8
    centres = rng.normal(size=(K, d)) * 4
    z = rng.choice(K, size=N, p=[0.4, 0.25, 0.15, 0.1, 0.06, 0.04])
    emb = (centres[z] + rng.normal(size=(N, d))).astype(np.float32)
    deg = rng.integers(1, 30, size=N)
    split = rng.choice(3, size=N, p=[0.5, 0.2, 0.3]).astype(np.uint8)
    caps = [int(np.floor(1.05 * (split == s).sum() / K)) for s in range(3)]
    words = rng.integers(0, 2 ** 32, size=(3, 10, N), dtype=np.uint64).astype(np.uint32)
    init = emb[:K].copy()
    assign, cent, used = oracle.cluster_and_balance(emb, K, 5, init, _rowptr(deg), split, caps, words)
    km = oracle.kmeans(emb, K, 5, init)
    np.testing.assert_array_equal(cent, km.centroids)                  # balancing moves labels, not centroids
    for s in range(3):
        load = np.bincount(assign[split == s], minlength=K)
        assert load.max() <= caps[s] and load.sum() == (split == s).sum()
    assert all(r >= 1 for r in used)                                   # the mixture is skewed: every set needed work
    # the sets do not interfere: balancing each set on its own from the K-Means labels gives the same labels
    for s in range(3):
        alone, _ = oracle.balance(_rowptr(deg), km.assign, K, caps[s], words[s], split == s)
        assert np.array_equal(alone[split == s], assign[split == s])
