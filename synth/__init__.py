"""Seeded synthetic inputs shaped like the paper's workloads (Table 1 graphs).

This module serves both the CPU oracle's tests and the CUDA path's tests and
benchmark.  It holds NONE of the method's arithmetic (no distances, no
clustering, no cut counting): it only draws embeddings, initial-centroid row
ids and CSR graphs from a counter-based hash, with plain torch tensor ops, on
whichever device it is asked to use.  The public datasets themselves are not
reproduced; only their vertex / edge counts are used.

Everything is a pure function of (seed, stream, index), so any slice can be
regenerated on its own.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Optional, Tuple

import torch

# ----------------------------------------------------------------------------------------------
# counter-based hash -> uniforms / normals
# ----------------------------------------------------------------------------------------------
_M64 = (1 << 64) - 1
_GOLD = 0x9E3779B97F4A7C15
_MUL1 = 0xBF58476D1CE4E5B9
_MUL2 = 0x94D049BB133111EB

STREAM_CENTRES, STREAM_LABELS, STREAM_NOISE, STREAM_DEGREES, STREAM_EDGES, STREAM_INIT, STREAM_SUBSAMPLE = range(7)


def _s64(x: int) -> int:
    """Python int -> the same 64 bits as a signed value (what a torch int64 holds)."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix_py(x: int) -> int:
    x = (x + _GOLD) & _M64
    x = ((x ^ (x >> 30)) * _MUL1) & _M64
    x = ((x ^ (x >> 27)) * _MUL2) & _M64
    return x ^ (x >> 31)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def hash64(seed: int, stream: int, idx: torch.Tensor) -> torch.Tensor:
    """64 well-mixed bits per index (a splitmix64-style finaliser); int64 in, int64 out."""
    base = _mix_py(_mix_py(seed & _M64) ^ ((stream + 1) * 0xD1342543DE82EF95 & _M64))
    x = idx * _s64(_GOLD) + _s64(base)
    x = (x ^ _lsr(x, 30)) * _s64(_MUL1)
    x = (x ^ _lsr(x, 27)) * _s64(_MUL2)
    return x ^ _lsr(x, 31)


def uniform53(seed: int, stream: int, idx: torch.Tensor) -> torch.Tensor:
    """float64 uniforms in (0, 1)."""
    h = _lsr(hash64(seed, stream, idx), 11)
    return (h.to(torch.float64) + 0.5) * (1.0 / (1 << 53))


def normal_pairs(seed: int, stream: int, pair_idx: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
    """Two independent fp32 standard normals per index (Box-Muller on 24-bit uniforms)."""
    h = hash64(seed, stream, pair_idx)
    u1 = ((_lsr(h, 40) & 0xFFFFFF).to(torch.float32) + 1.0) * (1.0 / (1 << 24))   # (0, 1]
    u2 = (_lsr(h, 8) & 0xFFFFFF).to(torch.float32) * (1.0 / (1 << 24))            # [0, 1)
    r = torch.sqrt(-2.0 * torch.log(u1))
    ang = (2.0 * math.pi) * u2
    return r * torch.cos(ang), r * torch.sin(ang)


# ----------------------------------------------------------------------------------------------
# workload table
# ----------------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    N: int
    d: int
    ncomp: int          # Gaussian mixture components
    sigma: float        # per-coordinate noise std
    K: int              # partitions
    iters: int          # Lloyd iterations
    nnz_target: int     # directed CSR entries aimed for (before de-duplication)
    p_in: float         # probability an edge stays inside its source's component
    alpha: float        # Pareto exponent of the expected degrees; 0 = uniform degrees
    rowptr64: bool = False
    reorder_K: int = 0  # extra clustering run for reordering (0 = none)
    reorder_iters: int = 0


_SEED0 = 0xE3BED000

WORKLOADS = {
    # tiny planted-partition case
    "cfg1": Workload("cfg1", _SEED0 + 1, 10_000, 64, 8, 0.5, 4, 20, 100_000, 0.80, 0.0),
    # vertex / edge counts of the paper's Table 1: arxiv, reddit, products, papers100M
    "cfg2": Workload("cfg2", _SEED0 + 2, 169_343, 128, 40, 0.7, 8, 30, 2 * 1_166_243, 0.70, 2.1),
    "cfg3": Workload("cfg3", _SEED0 + 3, 232_965, 256, 41, 0.7, 16, 30, 114_615_892, 0.60, 2.1),
    "cfg4": Workload("cfg4", _SEED0 + 4, 2_449_029, 128, 47, 0.7, 32, 30, 123_718_280, 0.65, 2.1,
                     reorder_K=4096, reorder_iters=10),
    "cfg5": Workload("cfg5", _SEED0 + 5, 111_059_956, 128, 172, 0.7, 64, 20, 2 * 1_615_685_872, 0.60, 2.1,
                     rowptr64=True),
}


def scaled(w: Workload, N: int, nnz_target: Optional[int] = None, **kw) -> Workload:
    """The same recipe at another vertex count (mean degree kept unless nnz_target is given)."""
    if nnz_target is None:
        nnz_target = max(2, int(round(w.nnz_target * (N / w.N))))
    return replace(w, N=N, nnz_target=nnz_target, name=f"{w.name}@{N}", **kw)


# ----------------------------------------------------------------------------------------------
# embeddings
# ----------------------------------------------------------------------------------------------
def component_labels(w: Workload, rows: torch.Tensor) -> torch.Tensor:
    """Mixture component of each vertex id in `rows` (int64 tensor); iid uniform."""
    h = _lsr(hash64(w.seed, STREAM_LABELS, rows), 1)
    return h % w.ncomp


def component_centres(w: Workload, device) -> torch.Tensor:
    """ncomp x d fp32 centres ~ N(0, I)."""
    npairs = (w.ncomp * w.d + 1) // 2
    z0, z1 = normal_pairs(w.seed, STREAM_CENTRES, torch.arange(npairs, dtype=torch.int64, device=device))
    return torch.stack((z0, z1), dim=1).reshape(-1)[: w.ncomp * w.d].reshape(w.ncomp, w.d).contiguous()


def embeddings(w: Workload, device="cpu", row_start: int = 0, row_end: Optional[int] = None,
               out: Optional[torch.Tensor] = None, chunk_rows: int = 1 << 20) -> torch.Tensor:
    """Rows [row_start, row_end) of the N x d fp32 embedding matrix: centre of the row's component
    plus sigma * N(0, I) noise.  d must be even."""
    assert w.d % 2 == 0
    row_end = w.N if row_end is None else row_end
    n = row_end - row_start
    if out is None:
        out = torch.empty((n, w.d), dtype=torch.float32, device=device)
    assert out.shape == (n, w.d) and out.dtype == torch.float32
    device = out.device
    centres = component_centres(w, device)
    half = w.d // 2
    for r0 in range(row_start, row_end, chunk_rows):
        r1 = min(row_end, r0 + chunk_rows)
        rows = torch.arange(r0, r1, dtype=torch.int64, device=device)
        z = component_labels(w, rows)
        pair = torch.arange(r0 * half, r1 * half, dtype=torch.int64, device=device)
        n0, n1 = normal_pairs(w.seed, STREAM_NOISE, pair)
        noise = torch.stack((n0, n1), dim=1).reshape(r1 - r0, w.d)
        del n0, n1, pair
        dst = out[r0 - row_start: r1 - row_start]
        torch.index_select(centres, 0, z, out=dst)
        dst.add_(noise, alpha=w.sigma)
        del noise
    return out


def embedding_rows(w: Workload, rows: torch.Tensor) -> torch.Tensor:
    """The embedding rows of an arbitrary id list (same values as `embeddings` produces)."""
    device = rows.device
    rows = rows.to(torch.int64)
    centres = component_centres(w, device)
    half = w.d // 2
    pair = (rows[:, None] * half + torch.arange(half, dtype=torch.int64, device=device)[None, :]).reshape(-1)
    n0, n1 = normal_pairs(w.seed, STREAM_NOISE, pair)
    noise = torch.stack((n0, n1), dim=1).reshape(rows.numel(), w.d)
    return centres[component_labels(w, rows)] + w.sigma * noise


def first_of_permutation(w: Workload, stream: int, count: int, device="cpu") -> torch.Tensor:
    """The first `count` entries of a seeded permutation of [0, N): vertex ids ordered by a hash
    key (ties, which 63-bit keys all but exclude, broken by id)."""
    keys = _lsr(hash64(w.seed, stream, torch.arange(w.N, dtype=torch.int64, device=device)), 1)
    if count * 8 < w.N:
        kth = torch.topk(keys, count, largest=False, sorted=True)
        return kth.indices
    return torch.sort(keys, stable=True).indices[:count]


def init_centroid_rows(w: Workload, K: Optional[int] = None, device="cpu") -> torch.Tensor:
    """Row ids whose embeddings serve as initial centroids: first K of a seeded permutation."""
    return first_of_permutation(w, STREAM_INIT, w.K if K is None else K, device)


def subsample_rows(w: Workload, count: int, device="cpu") -> torch.Tensor:
    return first_of_permutation(w, STREAM_SUBSAMPLE, count, device)


# ----------------------------------------------------------------------------------------------
# graphs
# ----------------------------------------------------------------------------------------------
def _expected_degrees(w: Workload, device) -> torch.Tensor:
    """Chung-Lu weights in expected-degree units (float64, one per vertex)."""
    if w.alpha <= 0:
        return torch.full((w.N,), w.nnz_target / w.N, dtype=torch.float64, device=device)
    u = uniform53(w.seed, STREAM_DEGREES, torch.arange(w.N, dtype=torch.int64, device=device))
    wt = u.pow(-1.0 / w.alpha)                              # Pareto, x_m = 1
    cap = math.sqrt(float(w.nnz_target))
    for _ in range(8):                                      # rescale to the target mean, then cap
        wt = torch.clamp(wt * (w.nnz_target / float(wt.sum())), max=cap)
    return wt


def graph(w: Workload, device="cpu", edge_chunk: int = 1 << 25, max_bucket_entries: int = 600_000_000
          ) -> Tuple[torch.Tensor, torch.Tensor]:
    """Symmetric CSR (rowptr int32 or int64 per w.rowptr64, colidx int32): sorted rows, no
    self-loops, no duplicates, vertex ids carry no locality.

    nnz_target/2 undirected edges are drawn: the source u in proportion to its expected degree;
    the target v, with probability p_in, in proportion to expected degree among the vertices of u's
    mixture component, else among all vertices.  Both directions are stored.  The vertex count may
    make this a multi-gigabyte job, so directed entries are produced per source-row bucket, each
    bucket re-deriving the edge list from the hash."""
    N = w.N
    n_und = w.nnz_target // 2
    ids = torch.arange(N, dtype=torch.int64, device=device)
    comp = component_labels(w, ids)
    order = torch.sort(comp, stable=True).indices            # vertices grouped by component
    deg = _expected_degrees(w, device)
    cum = torch.cumsum(deg[order], 0)
    total = float(cum[-1])
    counts = torch.bincount(comp, minlength=w.ncomp)
    ends = torch.cumsum(counts, 0)
    starts = ends - counts
    zero = torch.zeros(1, dtype=torch.float64, device=device)
    cum0 = torch.cat((zero, cum))                            # cum0[i] = weight before sorted slot i
    comp_lo = cum0[starts]
    comp_hi = cum0[ends]
    del ids, deg

    n_buckets = max(1, -(-2 * n_und // max_bucket_entries))
    rows_per_bucket = -(-N // n_buckets)
    rowptr_dtype = torch.int64 if w.rowptr64 else torch.int32
    deg_out = torch.zeros(N, dtype=torch.int64, device=device)
    col_parts = []
    for b in range(n_buckets):
        lo_row, hi_row = b * rows_per_bucket, min(N, (b + 1) * rows_per_bucket)
        keys = []
        for e0 in range(0, n_und, edge_chunk):
            e1 = min(n_und, e0 + edge_chunk)
            e = torch.arange(e0, e1, dtype=torch.int64, device=device)
            t_u = uniform53(w.seed, STREAM_EDGES, 3 * e) * total
            su = torch.searchsorted(cum, t_u, right=True).clamp_(max=N - 1)
            u = order[su]
            inside = uniform53(w.seed, STREAM_EDGES, 3 * e + 1) < w.p_in
            cu = comp[u]
            lo = torch.where(inside, comp_lo[cu], zero)
            hi = torch.where(inside, comp_hi[cu], cum0[-1:])
            t_v = lo + uniform53(w.seed, STREAM_EDGES, 3 * e + 2) * (hi - lo)
            sv = torch.searchsorted(cum, t_v, right=True).clamp_(max=N - 1)
            v = order[sv]
            del e, t_u, su, inside, cu, lo, hi, t_v, sv
            for a, c in ((u, v), (v, u)):
                m = (a != c) & (a >= lo_row) & (a < hi_row)
                keys.append(a[m] * N + c[m])
            del u, v
        k = torch.cat(keys) if len(keys) > 1 else keys[0]
        del keys
        k = torch.unique(k, sorted=True)
        src = torch.div(k, N, rounding_mode="floor")
        col_parts.append((k - src * N).to(torch.int32))
        deg_out += torch.bincount(src, minlength=N)
        del k, src
    colidx = torch.cat(col_parts) if len(col_parts) > 1 else col_parts[0]
    rowptr = torch.zeros(N + 1, dtype=torch.int64, device=device)
    torch.cumsum(deg_out, 0, out=rowptr[1:])
    return rowptr.to(rowptr_dtype), colidx.contiguous()
