"""The seeded input generators: reproducible, sliceable, and shaped as the recipe says (CPU only)."""
import numpy as np
import torch

import synth


def test_hash_matches_a_scalar_reimplementation():
    idx = torch.tensor([0, 1, 2, 12345678901, (1 << 40) + 7], dtype=torch.int64)
    got = synth.hash64(99, 3, idx).tolist()
    M = (1 << 64) - 1
    base = synth._mix_py(synth._mix_py(99) ^ ((3 + 1) * 0xD1342543DE82EF95 & M))
    for i, g in zip(idx.tolist(), got):
        x = (i * 0x9E3779B97F4A7C15 + base) & M
        x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & M
        x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & M
        x ^= x >> 31
        assert g & M == x


def test_embeddings_are_reproducible_and_sliceable():
    w = synth.scaled(synth.WORKLOADS["cfg2"], 5000)
    full = synth.embeddings(w, chunk_rows=1 << 20)
    again = synth.embeddings(w, chunk_rows=777)
    assert torch.equal(full, again)
    part = synth.embeddings(w, row_start=1234, row_end=2345)
    assert torch.equal(part, full[1234:2345])
    rows = torch.tensor([4999, 0, 17, 17, 2500])
    assert torch.allclose(synth.embedding_rows(w, rows), full[rows], rtol=0, atol=1e-6)
    assert full.dtype == torch.float32 and full.shape == (5000, 128)


def test_mixture_statistics():
    w = synth.scaled(synth.WORKLOADS["cfg1"], 40_000)
    emb = synth.embeddings(w)
    z = synth.component_labels(w, torch.arange(w.N))
    counts = torch.bincount(z, minlength=w.ncomp)
    assert counts.min() > 0.9 * w.N / w.ncomp and counts.max() < 1.1 * w.N / w.ncomp
    centres = synth.component_centres(w, "cpu")
    resid = emb - centres[z]
    assert abs(resid.std().item() - w.sigma) < 0.01
    assert abs(resid.mean().item()) < 0.01
    assert abs(centres.std().item() - 1.0) < 0.15


def test_initial_centroid_rows_are_distinct_and_seeded():
    w = synth.WORKLOADS["cfg1"]
    r = synth.init_centroid_rows(w, 64)
    assert len(set(r.tolist())) == 64 and r.min() >= 0 and r.max() < w.N
    assert torch.equal(r[:4], synth.init_centroid_rows(w))
    w2 = synth.scaled(w, w.N, seed=w.seed + 1)
    assert not torch.equal(synth.init_centroid_rows(w2, 64), r)


def _check_graph(w, buckets=None):
    kw = {} if buckets is None else {"max_bucket_entries": buckets}
    rowptr, colidx = synth.graph(w, **kw)
    rp = rowptr.numpy().astype(np.int64)
    ci = colidx.numpy()
    N = w.N
    assert rp[0] == 0 and rp[-1] == len(ci) and np.all(np.diff(rp) >= 0)
    assert ci.min() >= 0 and ci.max() < N
    src = np.repeat(np.arange(N), np.diff(rp))
    assert np.all(src != ci)                                             # no self-loops
    key = src.astype(np.int64) * N + ci
    assert np.all(np.diff(key) > 0)                                      # rows sorted, no duplicates
    rev = np.sort(ci.astype(np.int64) * N + src)
    assert np.array_equal(rev, key)                                      # symmetric
    return rp, ci, src


def test_planted_partition_graph():
    w = synth.WORKLOADS["cfg1"]
    rp, ci, src = _check_graph(w)
    assert abs(len(ci) / w.N - 10) < 0.5
    z = synth.component_labels(w, torch.arange(w.N)).numpy()
    intra = (z[src] == z[ci]).mean()
    assert 0.78 < intra < 0.88                                           # 0.8 + chance hits of the global draws
    assert rowptr_dtype(w) == torch.int32


def rowptr_dtype(w):
    return synth.graph(synth.scaled(w, 50, 200))[0].dtype


def test_power_law_graph_and_bucketed_generation_agree():
    w = synth.scaled(synth.WORKLOADS["cfg5"], 20_000)
    rp, ci, src = _check_graph(w)
    deg = np.diff(rp)
    assert 22 < deg.mean() <= 29.2                                       # de-duplication inside the small components trims it
    assert deg.max() > 8 * deg.mean()                                    # heavy tail
    rowptr_b, colidx_b = synth.graph(w, max_bucket_entries=150_000)      # several source-row buckets
    assert rowptr_b.dtype == torch.int64
    assert np.array_equal(rowptr_b.numpy(), rp) and np.array_equal(colidx_b.numpy(), ci)
