"""ctypes wrapper around ``ep_oracle.c`` (numpy in, numpy out).

TEST INFRASTRUCTURE.  The C file holds all of the arithmetic; this module only
compiles it with gcc and marshals arrays.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess
from typing import NamedTuple, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ep_oracle.c")
_lib = None

# -O3 -march=native as the CPU-baseline plan asks; -ffp-contract=off keeps every operation the separately rounded
# IEEE double operation the C file states (no fused multiply-add), so the optimisation level changes no result.
_CFLAGS = ["-O3", "-march=native", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-std=c11"]


def _host_tag() -> str:
    """-march=native code only runs on the kind of CPU it was built on: the library's name carries a tag of the
    host's instruction-set flags, so a tree carried to another machine rebuilds there."""
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    return hashlib.sha1((flags + " ".join(_CFLAGS)).encode()).hexdigest()[:10]


def _lib_path() -> str:
    return os.path.join(_HERE, "libep_oracle.%s.so" % _host_tag())


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP on) and return the library path."""
    lib = _lib_path()
    if force or not os.path.exists(lib) or os.path.getmtime(lib) < os.path.getmtime(_SRC):
        tmp = lib + ".tmp.%d" % os.getpid()
        cmd = ["gcc", *_CFLAGS, "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True, capture_output=True, text=True)
        os.replace(tmp, lib)
    return lib


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        p = ctypes.c_void_p
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
        lib.oracle_assign.argtypes = [p, ctypes.c_int64, ctypes.c_int32, p, ctypes.c_int32, p, p, p]
        lib.oracle_assign.restype = None
        lib.oracle_kmeans.argtypes = [p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                      p, p, p, p, p, p]
        lib.oracle_kmeans.restype = ctypes.c_int
        lib.oracle_partition_quality.argtypes = [p, p, p, ctypes.c_int64, ctypes.c_int32, p, p, p]
        lib.oracle_partition_quality.restype = None
        lib.oracle_reorder.argtypes = [p, ctypes.c_int64, ctypes.c_int32, p, p]
        lib.oracle_reorder.restype = ctypes.c_int
        lib.oracle_graph_bandwidth.argtypes = [p, p, p, ctypes.c_int64, p, p]
        lib.oracle_graph_bandwidth.restype = None
        lib.oracle_migrate.argtypes = [p, ctypes.c_int64, ctypes.c_int32, p, ctypes.c_int64, p, p]
        lib.oracle_migrate.restype = ctypes.c_int64
        lib.oracle_relabel_graph.argtypes = [p, p, p, p, ctypes.c_int64, p, p]
        lib.oracle_relabel_graph.restype = None
        lib.oracle_permute_rows.argtypes = [p, ctypes.c_int64, ctypes.c_int32, p, p]
        lib.oracle_permute_rows.restype = None
        _lib = lib
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def _f32_matrix(a, name: str) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    if a.ndim != 2:
        raise ValueError(f"{name} must be 2-D")
    return a


def _labels(a, n: int, K: int) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.int32)
    if a.shape != (n,):
        raise ValueError("assign must have one entry per vertex")
    if n and (a.min() < 0 or a.max() >= K):
        raise ValueError("assign value outside [0, K)")
    return a


class KMeansResult(NamedTuple):
    assign: np.ndarray      # int32 [N]
    centroids: np.ndarray   # float64 [K, d]
    objective: np.ndarray   # float64 [max(iters, 1)]
    best1: np.ndarray       # float64 [N]  smallest distance of the returned assignment
    best2: np.ndarray       # float64 [N]  second smallest (inf when K == 1)


def kmeans(emb, K: int, iters: int, init_centroids) -> KMeansResult:
    emb = _f32_matrix(emb, "emb")
    init = _f32_matrix(init_centroids, "init_centroids")
    N, d = emb.shape
    if init.shape != (K, d):
        raise ValueError("init_centroids must be K x d")
    if iters < 0 or K < 1 or N < 1:
        raise ValueError("bad K / iters / N")
    assign = np.empty(N, np.int32)
    cent = np.empty((K, d), np.float64)
    obj = np.empty(max(iters, 1), np.float64)
    b1 = np.empty(N, np.float64)
    b2 = np.empty(N, np.float64)
    rc = _load().oracle_kmeans(_ptr(emb), N, d, K, iters, _ptr(init), _ptr(assign), _ptr(cent),
                               _ptr(obj), _ptr(b1), _ptr(b2))
    if rc != 0:
        raise MemoryError("oracle_kmeans")
    return KMeansResult(assign, cent, obj, b1, b2)


def assign_step(emb, centroids):
    """One assignment step against fp64 centroids: (assign, best1, best2)."""
    emb = _f32_matrix(emb, "emb")
    C = np.ascontiguousarray(centroids, dtype=np.float64)
    N, d = emb.shape
    K = C.shape[0]
    if C.shape != (K, d):
        raise ValueError("centroids must be K x d")
    assign = np.empty(N, np.int32)
    b1 = np.empty(N, np.float64)
    b2 = np.empty(N, np.float64)
    _load().oracle_assign(_ptr(emb), N, d, _ptr(C), K, _ptr(assign), _ptr(b1), _ptr(b2))
    return assign, b1, b2


def sampled_kmeans(emb, sample_rows, K: int, iters: int, init_centroids) -> KMeansResult:
    """Sampling-based clustering (Section 5, "Implementation": the centroids are computed from a sample of
    the embeddings, 2^9 per cluster in the paper; every embedding is then given to its nearest centroid).

    Steps, in that order: X_S = the rows `sample_rows` of emb (distinct row numbers); C_T = the centroids of
    `iters` Lloyd iterations over X_S from `init_centroids`; a_i = argmin_k |x_i - C_T[k]|^2 for every row i
    of emb (lowest index on ties).  Returned: that assignment, C_T, the objective trace of the iterations on
    the sample, and the two smallest distances of every row to C_T."""
    emb = _f32_matrix(emb, "emb")
    rows = np.ascontiguousarray(sample_rows, dtype=np.int64)
    N = emb.shape[0]
    if rows.ndim != 1 or rows.size < K or rows.min() < 0 or rows.max() >= N or np.unique(rows).size != rows.size:
        raise ValueError("sample_rows must be at least K distinct row numbers in [0, N)")
    if iters < 1:
        raise ValueError("the centroids need at least one iteration on the sample")
    trained = kmeans(emb[rows], K, iters, init_centroids)
    assign, b1, b2 = assign_step(emb, trained.centroids)
    return KMeansResult(assign, trained.centroids, trained.objective, b1, b2)


class QualityResult(NamedTuple):
    edge_cut: int
    part_vertices: np.ndarray  # int64 [K]
    part_edges: np.ndarray     # int64 [K]


def partition_quality(rowptr, colidx, assign, K: int) -> QualityResult:
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    colidx = np.ascontiguousarray(colidx, dtype=np.int32)
    N = rowptr.shape[0] - 1
    assign = _labels(assign, N, K)
    if rowptr[0] != 0 or rowptr[-1] != colidx.shape[0] or np.any(np.diff(rowptr) < 0):
        raise ValueError("rowptr is not a CSR row pointer for colidx")
    if colidx.size and (colidx.min() < 0 or colidx.max() >= N):
        raise ValueError("colidx value outside [0, N)")
    cut = ctypes.c_uint64(0)
    pv = np.empty(K, np.int64)
    pe = np.empty(K, np.int64)
    _load().oracle_partition_quality(_ptr(rowptr), _ptr(colidx), _ptr(assign), N, K,
                                     ctypes.addressof(cut), _ptr(pv), _ptr(pe))
    return QualityResult(int(cut.value), pv, pe)


def reorder(assign, K: int):
    """(perm, inv_perm): perm[new_id] = old id, inv_perm[old id] = new id."""
    assign = np.ascontiguousarray(assign, dtype=np.int32)
    N = assign.shape[0]
    assign = _labels(assign, N, K)
    perm = np.empty(N, np.int32)
    inv = np.empty(N, np.int32)
    rc = _load().oracle_reorder(_ptr(assign), N, K, _ptr(perm), _ptr(inv))
    if rc != 0:
        raise MemoryError("oracle_reorder")
    return perm, inv


class BandwidthResult(NamedTuple):
    bandwidth_sum: int              # sum over v of beta_v; the average graph bandwidth is bandwidth_sum / N
    vertex_bandwidth: np.ndarray    # int32 [N]

    @property
    def average(self) -> float:
        return self.bandwidth_sum / max(1, self.vertex_bandwidth.shape[0])


def graph_bandwidth(rowptr, colidx, pi) -> BandwidthResult:
    """Vertex bandwidths and their sum for the numbering pi (pi[v] = new id of v)."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    colidx = np.ascontiguousarray(colidx, dtype=np.int32)
    pi = np.ascontiguousarray(pi, dtype=np.int32)
    N = rowptr.shape[0] - 1
    if pi.shape != (N,):
        raise ValueError("pi must have one entry per vertex")
    if rowptr[0] != 0 or rowptr[-1] != colidx.shape[0] or np.any(np.diff(rowptr) < 0):
        raise ValueError("rowptr is not a CSR row pointer for colidx")
    if colidx.size and (colidx.min() < 0 or colidx.max() >= N):
        raise ValueError("colidx value outside [0, N)")
    if N and not np.array_equal(np.sort(pi), np.arange(N, dtype=np.int32)):
        raise ValueError("pi is not a bijection of [0, N)")
    total = ctypes.c_uint64(0)
    vb = np.empty(N, np.int32)
    _load().oracle_graph_bandwidth(_ptr(rowptr), _ptr(colidx), _ptr(pi), N, ctypes.addressof(total), _ptr(vb))
    return BandwidthResult(int(total.value), vb)


def _permutation_pair(perm, inv_perm, N: int):
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    inv = np.ascontiguousarray(inv_perm, dtype=np.int32)
    if perm.shape != (N,) or inv.shape != (N,) or not np.array_equal(np.sort(perm), np.arange(N, dtype=np.int32)):
        raise ValueError("perm must be a permutation of [0, N)")
    if not np.array_equal(inv[perm], np.arange(N, dtype=np.int32)):
        raise ValueError("inv_perm is not the inverse of perm")
    return perm, inv


def relabel_graph(rowptr, colidx, perm, inv_perm):
    """(new_rowptr int64, new_colidx int32): row i = old row perm[i] with ids mapped through inv_perm."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    colidx = np.ascontiguousarray(colidx, dtype=np.int32)
    N = rowptr.shape[0] - 1
    perm, inv = _permutation_pair(perm, inv_perm, N)
    if rowptr[0] != 0 or rowptr[-1] != colidx.shape[0] or np.any(np.diff(rowptr) < 0):
        raise ValueError("rowptr is not a CSR row pointer for colidx")
    if colidx.size and (colidx.min() < 0 or colidx.max() >= N):
        raise ValueError("colidx value outside [0, N)")
    new_rowptr = np.empty(N + 1, np.int64)
    new_colidx = np.empty(colidx.shape[0], np.int32)
    _load().oracle_relabel_graph(_ptr(rowptr), _ptr(colidx), _ptr(perm), _ptr(inv), N, _ptr(new_rowptr), _ptr(new_colidx))
    return new_rowptr, new_colidx


def permute_rows(emb, perm):
    """out[i] = emb[perm[i]]."""
    emb = _f32_matrix(emb, "emb")
    N, d = emb.shape
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    if perm.shape != (N,) or not np.array_equal(np.sort(perm), np.arange(N, dtype=np.int32)):
        raise ValueError("perm must be a permutation of [0, N)")
    out = np.empty_like(emb)
    _load().oracle_permute_rows(_ptr(emb), N, d, _ptr(perm), _ptr(out))
    return out


def migrate(rowptr, assign, K: int, capacity: int, rand_words, member=None):
    """One application of the migration policy (Algorithm 4): (new assign, vertices moved).
    rand_words: one uint32 per vertex; member: boolean mask of the candidate set (None = all)."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    N = rowptr.shape[0] - 1
    out = _labels(assign, N, K).copy()
    rw = np.ascontiguousarray(rand_words, dtype=np.uint32)
    if rw.shape != (N,):
        raise ValueError("rand_words must have one entry per vertex")
    mem = None if member is None else np.ascontiguousarray(member, dtype=np.uint8)
    if mem is not None and mem.shape != (N,):
        raise ValueError("member must have one entry per vertex")
    if capacity < 0 or np.any(np.diff(rowptr) < 0):
        raise ValueError("bad capacity or row pointer")
    moved = int(_load().oracle_migrate(_ptr(rowptr), N, K, _ptr(mem), int(capacity), _ptr(rw), _ptr(out)))
    if moved == -1:
        raise ValueError("overloaded partitions but no free capacity: capacity * K < |S|")
    if moved < 0:
        raise MemoryError("oracle_migrate")
    return out, moved


def balance(rowptr, assign, K: int, capacity: int, rand_rounds, member=None):
    """The loop of Algorithm 3 for one vertex set: apply the migration policy, each round with the next row
    of rand_rounds, while any partition holds more than `capacity` vertices of the set.
    Returns (assign, rounds used)."""
    rand_rounds = np.ascontiguousarray(rand_rounds, dtype=np.uint32)
    out = np.ascontiguousarray(assign, dtype=np.int32)
    sel = slice(None) if member is None else np.asarray(member, dtype=bool)
    rounds = 0
    while np.bincount(out[sel], minlength=K).max(initial=0) > capacity:
        if rounds == rand_rounds.shape[0]:
            raise RuntimeError("not balanced within the given rounds")
        out, _ = migrate(rowptr, out, K, capacity, rand_rounds[rounds], member)
        rounds += 1
    return out, rounds


def cluster_and_balance(emb, K: int, iters: int, init_centroids, rowptr, split, capacities, rand_rounds):
    """Phase 2 as a whole (Algorithm 3): P <- KMeans(E, k), then the balancing loop for the training vertices,
    then for the validation vertices, then for the remaining ones, each with its own capacity.

    split[v] is 0 (training), 1 (validation) or 2 (rest); capacities = (C_train, C_val, C_rest);
    rand_rounds[s] is the [max_rounds, N] array of random words of set s.
    Returns (assign, centroids, rounds used per set)."""
    split = np.ascontiguousarray(split, dtype=np.uint8)
    km = kmeans(emb, K, iters, init_centroids)
    if split.shape != (km.assign.shape[0],) or split.max(initial=0) > 2:
        raise ValueError("split must hold 0, 1 or 2 for every vertex")
    assign = km.assign
    used = []
    for s in range(3):
        assign, r = balance(rowptr, assign, K, int(capacities[s]), rand_rounds[s], split == s)
        used.append(r)
    return assign, km.centroids, used
