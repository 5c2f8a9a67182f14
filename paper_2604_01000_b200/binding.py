"""ctypes binding of the C ABI in include/embedpart.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes
import os
import threading
from typing import NamedTuple, Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_NAME = "libembedpart.so"

EXPORTED_SYMBOLS = (
    "ep_create", "ep_destroy", "ep_status_string", "ep_last_error", "ep_poll_status", "ep_set_option",
    "ep_get_option", "ep_kmeans_workspace_bytes", "ep_kmeans", "ep_quality_workspace_bytes",
    "ep_partition_quality", "ep_reorder_workspace_bytes", "ep_reorder", "ep_profile_read", "ep_launch_count",
    "ep_kmeans_host_arena_bytes", "ep_kmeans_host", "ep_quality_host_arena_bytes", "ep_partition_quality_host",
    "ep_reorder_host_arena_bytes", "ep_reorder_host", "ep_reorder_static", "ep_debug_counters",
    "ep_graph_bandwidth_workspace_bytes", "ep_graph_bandwidth", "ep_graph_bandwidth_host_arena_bytes",
    "ep_graph_bandwidth_host", "ep_kmeans_sampled_workspace_bytes", "ep_kmeans_sampled", "ep_gather_rows",
    "ep_relabel_graph_workspace_bytes", "ep_relabel_graph", "ep_permute_rows",
    "ep_balance_workspace_bytes", "ep_migrate", "ep_balance",
    "ep_cluster_and_balance_workspace_bytes", "ep_cluster_and_balance", "ep_selftest_wait_timeout", "ep_probe_gather",
    "ep_partition_and_reorder_host_arena_bytes", "ep_partition_and_reorder_host",
)

EP_OK = 0
EP_OPT_KMEANS_PATH = 1
EP_OPT_PROFILE = 2
EP_OPT_TIMER_GROUP = 3
EP_OPT_KMEANS_CAND_MB = 4
EP_OPT_QUALITY_SLICE_KB = 5
EP_OPT_KMEANS_ITERATIONS_PER_LAUNCH = 6
TIMER_COUNT = 9
TIMERS = {"kmeans_assign": 0, "kmeans_update": 1, "edge_cut": 2, "quality_prep": 3, "reorder": 4,
          "kmeans_resolve": 5, "graph_bandwidth": 6, "relabel": 7, "balance": 8}
KMEANS_PATHS = {"auto": 0, "simt": 1, "tensor": 2}


class EmbedPartError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"embedpart status {status}: {what}")
        self.status = status


def library_path() -> str:
    """The built library; the bounds-checked build when EP_USE_DEBUG_LIBRARY=1 is set before the first use."""
    if os.environ.get("EP_USE_DEBUG_LIBRARY", "") == "1":
        return os.path.join(_PKG, "libembedpart_debug.so")
    return os.path.join(_PKG, _LIB_NAME)


_lib = None
_lib_lock = threading.Lock()


def load_library() -> ctypes.CDLL:
    """Loads the built library; raises if it is missing (there is no fallback)."""
    global _lib
    with _lib_lock:
        if _lib is None:
            path = library_path()
            if not os.path.exists(path):
                raise FileNotFoundError(
                    f"{path} is missing: build it with `python -m paper_2604_01000_b200.build` "
                    "(needs nvcc); this package has no CPU fallback")
            lib = ctypes.CDLL(path)
            vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
            lib.ep_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int]
            lib.ep_create.restype = ctypes.c_int
            lib.ep_destroy.argtypes = [vp]
            lib.ep_destroy.restype = ctypes.c_int
            lib.ep_status_string.argtypes = [ctypes.c_int]
            lib.ep_status_string.restype = ctypes.c_char_p
            lib.ep_last_error.argtypes = [vp]
            lib.ep_last_error.restype = ctypes.c_char_p
            lib.ep_poll_status.argtypes = [vp]
            lib.ep_poll_status.restype = ctypes.c_int
            lib.ep_set_option.argtypes = [vp, ctypes.c_int, ctypes.c_int]
            lib.ep_set_option.restype = ctypes.c_int
            lib.ep_get_option.argtypes = [vp, ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
            lib.ep_get_option.restype = ctypes.c_int
            lib.ep_kmeans_workspace_bytes.argtypes = [vp, i64, i32, i32]
            lib.ep_kmeans_workspace_bytes.restype = sz
            lib.ep_kmeans.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp]
            lib.ep_kmeans.restype = ctypes.c_int
            lib.ep_quality_workspace_bytes.argtypes = [vp, i64, i64, i32]
            lib.ep_quality_workspace_bytes.restype = sz
            lib.ep_partition_quality.argtypes = [vp, vp, i32, vp, i64, vp, i64, i32, vp, vp, vp, vp, sz, vp]
            lib.ep_partition_quality.restype = ctypes.c_int
            lib.ep_reorder_workspace_bytes.argtypes = [vp, i64, i32]
            lib.ep_reorder_workspace_bytes.restype = sz
            lib.ep_reorder.argtypes = [vp, vp, i64, i32, vp, vp, vp, sz, vp]
            lib.ep_reorder.restype = ctypes.c_int
            lib.ep_profile_read.argtypes = [vp, ctypes.c_int, ctypes.POINTER(ctypes.c_double),
                                            ctypes.POINTER(ctypes.c_int64)]
            lib.ep_profile_read.restype = ctypes.c_int
            lib.ep_debug_counters.argtypes = [vp, ctypes.POINTER(ctypes.c_int64)]
            lib.ep_debug_counters.restype = ctypes.c_int
            lib.ep_selftest_wait_timeout.argtypes = [vp, i64, vp, vp]
            lib.ep_selftest_wait_timeout.restype = ctypes.c_int
            lib.ep_probe_gather.argtypes = [vp, vp, i64, vp, i64, i32, vp, vp]
            lib.ep_probe_gather.restype = ctypes.c_int
            lib.ep_partition_and_reorder_host_arena_bytes.argtypes = [vp, i64, i32, i32, i32, i64, i32]
            lib.ep_partition_and_reorder_host_arena_bytes.restype = sz
            lib.ep_partition_and_reorder_host.argtypes = [vp, vp, i64, i32, i32, i32, vp, i32, i32, vp, vp, i32, vp, i64,
                                                          vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
            lib.ep_partition_and_reorder_host.restype = ctypes.c_int
            lib.ep_launch_count.argtypes = [vp]
            lib.ep_launch_count.restype = ctypes.c_int64
            lib.ep_kmeans_host_arena_bytes.argtypes = [vp, i64, i32, i32, i32]
            lib.ep_kmeans_host_arena_bytes.restype = sz
            lib.ep_kmeans_host.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp]
            lib.ep_kmeans_host.restype = ctypes.c_int
            lib.ep_quality_host_arena_bytes.argtypes = [vp, i64, i64, i32, i32]
            lib.ep_quality_host_arena_bytes.restype = sz
            lib.ep_partition_quality_host.argtypes = [vp, vp, i32, vp, i64, vp, i64, i32, vp, vp, vp, vp, sz, vp]
            lib.ep_partition_quality_host.restype = ctypes.c_int
            lib.ep_reorder_host_arena_bytes.argtypes = [vp, i64, i32]
            lib.ep_reorder_host_arena_bytes.restype = sz
            lib.ep_reorder_host.argtypes = [vp, vp, i64, i32, vp, vp, vp, sz, vp]
            lib.ep_reorder_host.restype = ctypes.c_int
            lib.ep_reorder_static.argtypes = [vp, i64, i32, vp, vp, vp, vp]
            lib.ep_reorder_static.restype = ctypes.c_int
            lib.ep_kmeans_sampled_workspace_bytes.argtypes = [vp, i64, i32, i32, i64]
            lib.ep_kmeans_sampled_workspace_bytes.restype = sz
            lib.ep_kmeans_sampled.argtypes = [vp, vp, i64, i32, i32, i32, vp, i64, vp, vp, vp, vp, sz, vp]
            lib.ep_kmeans_sampled.restype = ctypes.c_int
            lib.ep_gather_rows.argtypes = [vp, vp, i64, i32, vp, i64, vp, vp]
            lib.ep_gather_rows.restype = ctypes.c_int
            lib.ep_cluster_and_balance_workspace_bytes.argtypes = [vp, i64, i32, i32, i64]
            lib.ep_cluster_and_balance_workspace_bytes.restype = sz
            lib.ep_cluster_and_balance.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp, i32, i64, vp, vp, vp, i32, vp, vp, vp,
                                                   vp, sz, vp]
            lib.ep_cluster_and_balance.restype = ctypes.c_int
            lib.ep_balance_workspace_bytes.argtypes = [vp, i64, i32, i64]
            lib.ep_balance_workspace_bytes.restype = sz
            lib.ep_migrate.argtypes = [vp, vp, i32, i64, i32, vp, i64, i64, vp, vp, vp, vp, sz, vp]
            lib.ep_migrate.restype = ctypes.c_int
            lib.ep_balance.argtypes = [vp, vp, i32, i64, i32, vp, i64, i64, vp, i32, vp, vp, vp, sz, vp]
            lib.ep_balance.restype = ctypes.c_int
            lib.ep_relabel_graph_workspace_bytes.argtypes = [vp, i64, i64]
            lib.ep_relabel_graph_workspace_bytes.restype = sz
            lib.ep_relabel_graph.argtypes = [vp, vp, i32, vp, i64, vp, vp, i64, vp, vp, vp, sz, vp]
            lib.ep_relabel_graph.restype = ctypes.c_int
            lib.ep_permute_rows.argtypes = [vp, vp, i64, i32, vp, vp, vp]
            lib.ep_permute_rows.restype = ctypes.c_int
            lib.ep_graph_bandwidth_workspace_bytes.argtypes = [vp, i64, i64]
            lib.ep_graph_bandwidth_workspace_bytes.restype = sz
            lib.ep_graph_bandwidth.argtypes = [vp, vp, i32, vp, i64, vp, i64, vp, vp, vp, sz, vp]
            lib.ep_graph_bandwidth.restype = ctypes.c_int
            lib.ep_graph_bandwidth_host_arena_bytes.argtypes = [vp, i64, i64, i32]
            lib.ep_graph_bandwidth_host_arena_bytes.restype = sz
            lib.ep_graph_bandwidth_host.argtypes = [vp, vp, i32, vp, i64, vp, i64, vp, vp, vp, sz, vp]
            lib.ep_graph_bandwidth_host.restype = ctypes.c_int
            _lib = lib
    return _lib


def _dev_ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _check_cuda(t: torch.Tensor, dtype, name: str, device: torch.device) -> torch.Tensor:
    if not isinstance(t, torch.Tensor) or not t.is_cuda or t.device != device:
        raise ValueError(f"{name} must be a CUDA tensor on {device}")
    if t.dtype != dtype:
        raise ValueError(f"{name} must have dtype {dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t


class Context:
    """Owns an ep_ctx for one device and a grow-only workspace tensor."""

    def __init__(self, device: int | torch.device | None = None):
        if device is None:
            device = torch.cuda.current_device()
        self.device = torch.device("cuda", device if isinstance(device, int) else (device.index or 0))
        self._lib = load_library()
        h = ctypes.c_void_p()
        rc = self._lib.ep_create(ctypes.byref(h), self.device.index)
        if rc != EP_OK:
            raise EmbedPartError(rc, self._lib.ep_status_string(rc).decode())
        self._h = h
        self._ws: Optional[torch.Tensor] = None

    def close(self):
        if getattr(self, "_h", None):
            self._lib.ep_destroy(self._h)
            self._h = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    # -- helpers ------------------------------------------------------------------------------
    def _raise(self, rc: int):
        msg = self._lib.ep_status_string(rc).decode()
        detail = self._lib.ep_last_error(self._h).decode()
        raise EmbedPartError(rc, f"{msg}: {detail}" if detail else msg)

    def workspace(self, nbytes: int) -> torch.Tensor:
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = None
            self._ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=self.device)
        return self._ws

    def poll_status(self) -> int:
        return int(self._lib.ep_poll_status(self._h))

    def check(self):
        """Synchronises and raises if a kernel flagged bad input since the last check."""
        rc = self.poll_status()
        if rc != EP_OK:
            self._raise(rc)

    def set_kmeans_path(self, path: str):
        rc = self._lib.ep_set_option(self._h, EP_OPT_KMEANS_PATH, KMEANS_PATHS[path])
        if rc != EP_OK:
            self._raise(rc)

    def set_profile(self, on: bool):
        rc = self._lib.ep_set_option(self._h, EP_OPT_PROFILE, 1 if on else 0)
        if rc != EP_OK:
            self._raise(rc)

    def set_timer_group(self, group: int):
        rc = self._lib.ep_set_option(self._h, EP_OPT_TIMER_GROUP, group)
        if rc != EP_OK:
            self._raise(rc)

    def set_kmeans_cand_mb(self, mib: int):
        """Upper bound (MiB) of the tensor-core path's candidate buffer; set before calling kmeans."""
        rc = self._lib.ep_set_option(self._h, EP_OPT_KMEANS_CAND_MB, mib)
        if rc != EP_OK:
            self._raise(rc)

    def set_kmeans_iterations_per_launch(self, mode: int):
        """0 or 2 = all iterations in one launch (default), 1 = one launch per Lloyd iteration (fused small-K pass)."""
        rc = self._lib.ep_set_option(self._h, EP_OPT_KMEANS_ITERATIONS_PER_LAUNCH, int(mode))
        if rc != EP_OK:
            self._raise(rc)

    def set_quality_slice_kb(self, kib: int):
        """Largest label slice (KiB) ep_partition_quality gathers from in one pass over the column ids."""
        rc = self._lib.ep_set_option(self._h, EP_OPT_QUALITY_SLICE_KB, kib)
        if rc != EP_OK:
            self._raise(rc)

    def profile_read(self, timer: str, group: int = 0):
        """(total milliseconds, timed intervals) of one library timer since its last read."""
        ms, n = ctypes.c_double(0), ctypes.c_int64(0)
        rc = self._lib.ep_profile_read(self._h, group * TIMER_COUNT + TIMERS[timer], ctypes.byref(ms),
                                       ctypes.byref(n))
        if rc != EP_OK:
            self._raise(rc)
        return ms.value, n.value

    def debug_counters(self):
        """The library's 8 diagnostic counters (kept while profiling is on); reading clears them."""
        out = (ctypes.c_int64 * 8)()
        rc = self._lib.ep_debug_counters(self._h, out)
        if rc != EP_OK:
            self._raise(rc)
        return list(out)

    def selftest_wait_timeout(self, limit_clocks: int) -> torch.Tensor:
        """Makes a bounded device wait run out (see ep_selftest_wait_timeout); returns the 3 diagnostic words."""
        out = torch.zeros(3, dtype=torch.int64, device=self.device)
        rc = self._lib.ep_selftest_wait_timeout(self._h, int(limit_clocks), ctypes.c_void_p(out.data_ptr()), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return out

    def probe_gather(self, colidx: torch.Tensor, table: torch.Tensor, cluster_size: int = 0) -> torch.Tensor:
        """Yardstick: sum of table[colidx[e]] over all entries (see ep_probe_gather); returns the 1-element sum."""
        if colidx.dtype != torch.int32 or table.dtype != torch.uint8 or not colidx.is_cuda or not table.is_cuda:
            raise ValueError("colidx must be a CUDA int32 tensor, table a CUDA uint8 tensor")
        out = torch.zeros(1, dtype=torch.int64, device=self.device)
        rc = self._lib.ep_probe_gather(self._h, ctypes.c_void_p(colidx.data_ptr()), colidx.numel(),
                                       ctypes.c_void_p(table.data_ptr()), table.numel(), int(cluster_size),
                                       ctypes.c_void_p(out.data_ptr()), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return out

    def launch_count(self) -> int:
        return int(self._lib.ep_launch_count(self._h))

    def _stream(self):
        return ctypes.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)

    # -- calls --------------------------------------------------------------------------------
    def kmeans(self, emb, K: int, iters: int, init_centroids, objective: bool = False):
        emb = _check_cuda(emb, torch.float32, "emb", self.device)
        init = _check_cuda(init_centroids, torch.float32, "init_centroids", self.device)
        if emb.dim() != 2 or init.dim() != 2 or init.shape != (K, emb.shape[1]):
            raise ValueError("emb must be N x d and init_centroids K x d")
        N, d = emb.shape
        need = self._lib.ep_kmeans_workspace_bytes(self._h, N, d, K)
        if need == 0:
            raise EmbedPartError(1, f"shape out of range: N={N} d={d} K={K}")
        ws = self.workspace(need)
        assign = torch.empty(N, dtype=torch.int32, device=self.device)
        cent = torch.empty((K, d), dtype=torch.float32, device=self.device)
        obj = torch.empty(max(iters, 1), dtype=torch.float64, device=self.device) if objective else None
        with torch.cuda.device(self.device):
            rc = self._lib.ep_kmeans(self._h, _dev_ptr(emb), N, d, K, iters, _dev_ptr(init), _dev_ptr(assign),
                                     _dev_ptr(cent), _dev_ptr(obj), _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return KMeansResult(assign, cent, obj)

    def gather_rows(self, emb, rows):
        """out[i] = emb[rows[i]] (rows: int64 CUDA tensor)."""
        emb = _check_cuda(emb, torch.float32, "emb", self.device)
        rows = _check_cuda(rows, torch.int64, "rows", self.device)
        N, d = emb.shape
        out = torch.empty(rows.numel(), d, dtype=torch.float32, device=self.device)
        with torch.cuda.device(self.device):
            rc = self._lib.ep_gather_rows(self._h, _dev_ptr(emb), N, d, _dev_ptr(rows), rows.numel(), _dev_ptr(out),
                                          self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return out

    def kmeans_sampled(self, emb, K: int, iters: int, sample_rows, init_centroids):
        """Centroids from `iters` Lloyd iterations over the rows `sample_rows`, then every row of emb assigned
        to its nearest centroid: (assign, centroids, None)."""
        emb = _check_cuda(emb, torch.float32, "emb", self.device)
        rows = _check_cuda(sample_rows, torch.int64, "sample_rows", self.device)
        init = _check_cuda(init_centroids, torch.float32, "init_centroids", self.device)
        N, d = emb.shape
        if init.shape != (K, d):
            raise ValueError("init_centroids must be K x d")
        M = rows.numel()
        need = self._lib.ep_kmeans_sampled_workspace_bytes(self._h, N, d, K, M)
        if need == 0:
            raise EmbedPartError(1, f"shape out of range: N={N} d={d} K={K} M={M}")
        ws = self.workspace(need)
        assign = torch.empty(N, dtype=torch.int32, device=self.device)
        cent = torch.empty(K, d, dtype=torch.float32, device=self.device)
        with torch.cuda.device(self.device):
            rc = self._lib.ep_kmeans_sampled(self._h, _dev_ptr(emb), N, d, K, iters, _dev_ptr(rows), M, _dev_ptr(init),
                                             _dev_ptr(assign), _dev_ptr(cent), _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return KMeansResult(assign, cent, None)

    def partition_quality(self, rowptr, colidx, assign, K: int):
        if rowptr.dtype not in (torch.int32, torch.int64):
            raise ValueError("rowptr must be int32 or int64")
        rowptr = _check_cuda(rowptr, rowptr.dtype, "rowptr", self.device)
        colidx = _check_cuda(colidx, torch.int32, "colidx", self.device)
        assign = _check_cuda(assign, torch.int32, "assign", self.device)
        N, nnz = assign.numel(), colidx.numel()
        if rowptr.numel() != N + 1:
            raise ValueError("rowptr must have N + 1 entries")
        need = self._lib.ep_quality_workspace_bytes(self._h, N, nnz, K)
        if need == 0:
            raise EmbedPartError(1, f"shape out of range: N={N} nnz={nnz} K={K}")
        ws = self.workspace(need)
        cut = torch.empty(1, dtype=torch.int64, device=self.device)
        pv = torch.empty(K, dtype=torch.int64, device=self.device)
        pe = torch.empty(K, dtype=torch.int64, device=self.device)
        with torch.cuda.device(self.device):
            rc = self._lib.ep_partition_quality(self._h, _dev_ptr(rowptr), int(rowptr.dtype == torch.int64),
                                                _dev_ptr(colidx), nnz, _dev_ptr(assign), N, K, _dev_ptr(cut),
                                                _dev_ptr(pv), _dev_ptr(pe), _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return QualityResult(cut, pv, pe)

    def reorder(self, assign, K: int, inverse: bool = True):
        assign = _check_cuda(assign, torch.int32, "assign", self.device)
        N = assign.numel()
        need = self._lib.ep_reorder_workspace_bytes(self._h, N, K)
        if need == 0:
            raise EmbedPartError(1, f"shape out of range: N={N} K={K}")
        ws = self.workspace(need)
        perm = torch.empty(N, dtype=torch.int32, device=self.device)
        inv = torch.empty(N, dtype=torch.int32, device=self.device) if inverse else None
        with torch.cuda.device(self.device):
            rc = self._lib.ep_reorder(self._h, _dev_ptr(assign), N, K, _dev_ptr(perm), _dev_ptr(inv), _dev_ptr(ws),
                                      ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return ReorderResult(perm, inv)

    def _balance_args(self, rowptr, assign, K, max_degree, member):
        if rowptr.dtype not in (torch.int32, torch.int64):
            raise ValueError("rowptr must be int32 or int64")
        rowptr = _check_cuda(rowptr, rowptr.dtype, "rowptr", self.device)
        assign = _check_cuda(assign, torch.int32, "assign", self.device)
        if member is not None:
            member = _check_cuda(member, torch.uint8, "member", self.device)
        N = assign.numel()
        if rowptr.numel() != N + 1 or (member is not None and member.numel() != N):
            raise ValueError("rowptr must have N + 1 entries, member N")
        need = self._lib.ep_balance_workspace_bytes(self._h, N, K, max_degree)
        if need == 0:
            raise EmbedPartError(5, f"unsupported shape: N={N} K={K} max_degree={max_degree}")
        return rowptr, assign, member, N, self.workspace(need)

    def migrate(self, rowptr, assign, K: int, capacity: int, max_degree: int, rand_words, member=None):
        """One application of the migration policy (Algorithm 4), in place on `assign`; returns the int64 state
        tensor [vertices above capacity before, free capacity, vertices moved or -1, 0]."""
        rowptr, assign, member, N, ws = self._balance_args(rowptr, assign, K, max_degree, member)
        rand_words = _check_cuda(rand_words, torch.int32, "rand_words", self.device)   # 32 random bits per vertex
        if rand_words.numel() != N:
            raise ValueError("rand_words must have N entries")
        state = torch.zeros(4, dtype=torch.int64, device=self.device)
        with torch.cuda.device(self.device):
            rc = self._lib.ep_migrate(self._h, _dev_ptr(rowptr), int(rowptr.dtype == torch.int64), N, K, _dev_ptr(member),
                                      capacity, max_degree, _dev_ptr(rand_words), _dev_ptr(assign), _dev_ptr(state),
                                      _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return state

    def balance(self, rowptr, assign, K: int, capacity: int, max_degree: int, rand_rounds, member=None):
        """The loop of Algorithm 3 for one vertex set, in place on `assign`; rand_rounds is [max_rounds, N] int32
        (32 random bits each).  Returns the number of applications of the policy.  Synchronises the stream."""
        rowptr, assign, member, N, ws = self._balance_args(rowptr, assign, K, max_degree, member)
        rand_rounds = _check_cuda(rand_rounds, torch.int32, "rand_rounds", self.device)
        if rand_rounds.dim() != 2 or rand_rounds.shape[1] != N:
            raise ValueError("rand_rounds must be [max_rounds, N]")
        used = ctypes.c_int32(0)
        with torch.cuda.device(self.device):
            rc = self._lib.ep_balance(self._h, _dev_ptr(rowptr), int(rowptr.dtype == torch.int64), N, K, _dev_ptr(member),
                                      capacity, max_degree, _dev_ptr(rand_rounds), rand_rounds.shape[0], _dev_ptr(assign),
                                      ctypes.byref(used), _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return used.value

    def cluster_and_balance(self, emb, K: int, iters: int, init_centroids, rowptr, max_degree: int, split, capacities,
                            rand_rounds):
        """Phase 2 as a whole (Algorithm 3): K-Means, then the balancing loops of the training (split 0), validation
        (1) and remaining (2) vertices.  rand_rounds: [3, max_rounds, N] int32.  Returns (KMeansResult, rounds used
        per set).  Synchronises the stream."""
        emb = _check_cuda(emb, torch.float32, "emb", self.device)
        init = _check_cuda(init_centroids, torch.float32, "init_centroids", self.device)
        rowptr = _check_cuda(rowptr, rowptr.dtype, "rowptr", self.device)
        split = _check_cuda(split, torch.uint8, "split", self.device)
        rand_rounds = _check_cuda(rand_rounds, torch.int32, "rand_rounds", self.device)
        N, d = emb.shape
        if init.shape != (K, d) or rowptr.numel() != N + 1 or split.numel() != N:
            raise ValueError("init_centroids must be K x d, rowptr N + 1 entries, split N bytes")
        if rand_rounds.dim() != 3 or rand_rounds.shape[0] != 3 or rand_rounds.shape[2] != N:
            raise ValueError("rand_rounds must be [3, max_rounds, N]")
        need = self._lib.ep_cluster_and_balance_workspace_bytes(self._h, N, d, K, max_degree)
        if need == 0:
            raise EmbedPartError(1, f"shape out of range or unsupported: N={N} d={d} K={K} max_degree={max_degree}")
        ws = self.workspace(need)
        assign = torch.empty(N, dtype=torch.int32, device=self.device)
        cent = torch.empty(K, d, dtype=torch.float32, device=self.device)
        caps = (ctypes.c_int64 * 3)(*[int(c) for c in capacities])
        used = (ctypes.c_int32 * 3)()
        with torch.cuda.device(self.device):
            rc = self._lib.ep_cluster_and_balance(self._h, _dev_ptr(emb), N, d, K, iters, _dev_ptr(init), _dev_ptr(rowptr),
                                                  int(rowptr.dtype == torch.int64), max_degree, _dev_ptr(split), caps,
                                                  _dev_ptr(rand_rounds), rand_rounds.shape[1], _dev_ptr(assign),
                                                  _dev_ptr(cent), used, _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return KMeansResult(assign, cent, None), list(used)

    def relabel_graph(self, rowptr, colidx, perm, inv_perm):
        """(new_rowptr, new_colidx): the CSR graph with vertex perm[i] renamed i."""
        if rowptr.dtype not in (torch.int32, torch.int64):
            raise ValueError("rowptr must be int32 or int64")
        rowptr = _check_cuda(rowptr, rowptr.dtype, "rowptr", self.device)
        colidx = _check_cuda(colidx, torch.int32, "colidx", self.device)
        perm = _check_cuda(perm, torch.int32, "perm", self.device)
        inv_perm = _check_cuda(inv_perm, torch.int32, "inv_perm", self.device)
        N, nnz = perm.numel(), colidx.numel()
        if rowptr.numel() != N + 1 or inv_perm.numel() != N:
            raise ValueError("rowptr must have N + 1 entries, inv_perm N")
        need = self._lib.ep_relabel_graph_workspace_bytes(self._h, N, nnz)
        if need == 0:
            raise EmbedPartError(1, f"shape out of range: N={N} nnz={nnz}")
        ws = self.workspace(need)
        new_rowptr = torch.empty_like(rowptr)
        new_colidx = torch.empty_like(colidx)
        with torch.cuda.device(self.device):
            rc = self._lib.ep_relabel_graph(self._h, _dev_ptr(rowptr), int(rowptr.dtype == torch.int64), _dev_ptr(colidx),
                                            nnz, _dev_ptr(perm), _dev_ptr(inv_perm), N, _dev_ptr(new_rowptr),
                                            _dev_ptr(new_colidx), _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return new_rowptr, new_colidx

    def permute_rows(self, emb, perm):
        """out[i] = emb[perm[i]] (perm: int32 CUDA tensor of N entries)."""
        emb = _check_cuda(emb, torch.float32, "emb", self.device)
        perm = _check_cuda(perm, torch.int32, "perm", self.device)
        N, d = emb.shape
        if perm.numel() != N:
            raise ValueError("perm must have N entries")
        out = torch.empty_like(emb)
        with torch.cuda.device(self.device):
            rc = self._lib.ep_permute_rows(self._h, _dev_ptr(emb), N, d, _dev_ptr(perm), _dev_ptr(out), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return out

    def graph_bandwidth(self, rowptr, colidx, pi, per_vertex: bool = True):
        """Sum of the vertex bandwidths of the numbering pi (pi[v] = new id of v) and, if asked, each of them."""
        if rowptr.dtype not in (torch.int32, torch.int64):
            raise ValueError("rowptr must be int32 or int64")
        rowptr = _check_cuda(rowptr, rowptr.dtype, "rowptr", self.device)
        colidx = _check_cuda(colidx, torch.int32, "colidx", self.device)
        pi = _check_cuda(pi, torch.int32, "pi", self.device)
        N, nnz = pi.numel(), colidx.numel()
        if rowptr.numel() != N + 1:
            raise ValueError("rowptr must have N + 1 entries")
        need = self._lib.ep_graph_bandwidth_workspace_bytes(self._h, N, nnz)
        if need == 0:
            raise EmbedPartError(1, f"shape out of range: N={N} nnz={nnz}")
        ws = self.workspace(need)
        total = torch.empty(1, dtype=torch.int64, device=self.device)
        vb = torch.empty(N, dtype=torch.int32, device=self.device) if per_vertex else None
        with torch.cuda.device(self.device):
            rc = self._lib.ep_graph_bandwidth(self._h, _dev_ptr(rowptr), int(rowptr.dtype == torch.int64),
                                              _dev_ptr(colidx), nnz, _dev_ptr(pi), N, _dev_ptr(total), _dev_ptr(vb),
                                              _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return BandwidthResult(total, vb)

    # -- host-buffer calls (inputs and outputs are CPU tensors; copies are part of the call) -----
    def _host(self, t, dtype, name):
        if not isinstance(t, torch.Tensor) or t.is_cuda or t.dtype != dtype or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous CPU tensor of dtype {dtype}")
        return t

    def kmeans_host(self, emb, K: int, iters: int, init_centroids, objective: bool = False, out=None):
        emb = self._host(emb, torch.float32, "emb")
        init = self._host(init_centroids, torch.float32, "init_centroids")
        N, d = emb.shape
        need = self._lib.ep_kmeans_host_arena_bytes(self._h, N, d, K, iters)
        if need == 0:
            raise EmbedPartError(1, f"shape out of range: N={N} d={d} K={K}")
        ws = self.workspace(need)
        if out is None:
            out = KMeansResult(torch.empty(N, dtype=torch.int32).pin_memory(),
                               torch.empty((K, d), dtype=torch.float32).pin_memory(),
                               torch.empty(max(iters, 1), dtype=torch.float64).pin_memory() if objective else None)
        with torch.cuda.device(self.device):
            rc = self._lib.ep_kmeans_host(self._h, _dev_ptr(emb), N, d, K, iters, _dev_ptr(init),
                                          _dev_ptr(out.assign), _dev_ptr(out.centroids), _dev_ptr(out.objective),
                                          _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return out

    def partition_quality_host(self, rowptr, colidx, assign, K: int, out=None):
        rowptr = self._host(rowptr, rowptr.dtype, "rowptr")
        colidx = self._host(colidx, torch.int32, "colidx")
        assign = self._host(assign, torch.int32, "assign")
        N, nnz = assign.numel(), colidx.numel()
        is64 = int(rowptr.dtype == torch.int64)
        need = self._lib.ep_quality_host_arena_bytes(self._h, N, nnz, K, is64)
        if need == 0:
            raise EmbedPartError(1, f"shape out of range: N={N} nnz={nnz} K={K}")
        ws = self.workspace(need)
        if out is None:
            out = QualityResult(torch.empty(1, dtype=torch.int64).pin_memory(),
                                torch.empty(K, dtype=torch.int64).pin_memory(),
                                torch.empty(K, dtype=torch.int64).pin_memory())
        with torch.cuda.device(self.device):
            rc = self._lib.ep_partition_quality_host(self._h, _dev_ptr(rowptr), is64, _dev_ptr(colidx), nnz,
                                                     _dev_ptr(assign), N, K, _dev_ptr(out.edge_cut),
                                                     _dev_ptr(out.part_vertices), _dev_ptr(out.part_edges),
                                                     _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return out

    def graph_bandwidth_host(self, rowptr, colidx, pi, per_vertex: bool = True, out=None):
        rowptr = self._host(rowptr, rowptr.dtype, "rowptr")
        colidx = self._host(colidx, torch.int32, "colidx")
        pi = self._host(pi, torch.int32, "pi")
        N, nnz = pi.numel(), colidx.numel()
        is64 = int(rowptr.dtype == torch.int64)
        need = self._lib.ep_graph_bandwidth_host_arena_bytes(self._h, N, nnz, is64)
        if need == 0:
            raise EmbedPartError(1, f"shape out of range: N={N} nnz={nnz}")
        ws = self.workspace(need)
        if out is None:
            out = BandwidthResult(torch.empty(1, dtype=torch.int64).pin_memory(),
                                  torch.empty(N, dtype=torch.int32).pin_memory() if per_vertex else None)
        with torch.cuda.device(self.device):
            rc = self._lib.ep_graph_bandwidth_host(self._h, _dev_ptr(rowptr), is64, _dev_ptr(colidx), nnz, _dev_ptr(pi),
                                                   N, _dev_ptr(out.bandwidth_sum), _dev_ptr(out.vertex_bandwidth),
                                                   _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return out

    def reorder_host(self, assign, K: int, inverse: bool = True, out=None):
        assign = self._host(assign, torch.int32, "assign")
        N = assign.numel()
        need = self._lib.ep_reorder_host_arena_bytes(self._h, N, K)
        if need == 0:
            raise EmbedPartError(1, f"shape out of range: N={N} K={K}")
        ws = self.workspace(need)
        if out is None:
            out = ReorderResult(torch.empty(N, dtype=torch.int32).pin_memory(),
                                torch.empty(N, dtype=torch.int32).pin_memory() if inverse else None)
        with torch.cuda.device(self.device):
            rc = self._lib.ep_reorder_host(self._h, _dev_ptr(assign), N, K, _dev_ptr(out.perm), _dev_ptr(out.inv_perm),
                                           _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return out

    def partition_and_reorder_host_arena_bytes(self, N, d, K, reorder_K, nnz, rowptr64) -> int:
        return int(self._lib.ep_partition_and_reorder_host_arena_bytes(self._h, N, d, K, reorder_K, nnz, int(bool(rowptr64))))

    def partition_and_reorder_host(self, emb, K: int, iters: int, init_centroids, rowptr, colidx, reorder_K: int = 0,
                                   reorder_iters: int = 0, reorder_init=None, out=None):
        """The whole path on host buffers with every input uploaded once (ep_partition_and_reorder_host).
        Returns (KMeansResult, QualityResult, ReorderResult, labels of the second run or None); `out` may carry
        such a tuple of page-locked tensors to write into."""
        emb = self._host(emb, torch.float32, "emb")
        init = self._host(init_centroids, torch.float32, "init_centroids")
        colidx = self._host(colidx, torch.int32, "colidx")
        rowptr = self._host(rowptr, rowptr.dtype, "rowptr")
        init2 = self._host(reorder_init, torch.float32, "reorder_init") if reorder_K > 0 else None
        N, d = emb.shape
        nnz, is64 = colidx.numel(), int(rowptr.dtype == torch.int64)
        need = self._lib.ep_partition_and_reorder_host_arena_bytes(self._h, N, d, K, reorder_K, nnz, is64)
        if need == 0:
            raise EmbedPartError(1, f"shape out of range: N={N} d={d} K={K} reorder_K={reorder_K} nnz={nnz}")
        ws = self.workspace(need)
        if out is None:
            pin = lambda *shape, dtype: torch.empty(shape, dtype=dtype).pin_memory()   # noqa: E731
            out = (KMeansResult(pin(N, dtype=torch.int32), pin(K, d, dtype=torch.float32), None),
                   QualityResult(pin(1, dtype=torch.int64), pin(K, dtype=torch.int64), pin(K, dtype=torch.int64)),
                   ReorderResult(pin(N, dtype=torch.int32), pin(N, dtype=torch.int32)),
                   pin(N, dtype=torch.int32) if reorder_K > 0 else None)
        km, q, r, fine = out
        with torch.cuda.device(self.device):
            rc = self._lib.ep_partition_and_reorder_host(
                self._h, _dev_ptr(emb), N, d, K, iters, _dev_ptr(init), reorder_K, reorder_iters, _dev_ptr(init2),
                _dev_ptr(rowptr), is64, _dev_ptr(colidx), nnz, _dev_ptr(km.assign), _dev_ptr(km.centroids),
                _dev_ptr(q.edge_cut), _dev_ptr(q.part_vertices), _dev_ptr(q.part_edges), _dev_ptr(fine),
                _dev_ptr(r.perm), _dev_ptr(r.inv_perm), _dev_ptr(ws), ws.numel(), self._stream())
        if rc != EP_OK:
            self._raise(rc)
        return out


class KMeansResult(NamedTuple):
    assign: torch.Tensor                 # int32 [N]
    centroids: torch.Tensor              # float32 [K, d]
    objective: Optional[torch.Tensor]    # float64 [max(iters, 1)] or None


class QualityResult(NamedTuple):
    edge_cut: torch.Tensor               # int64 [1]: cut CSR entries
    part_vertices: torch.Tensor          # int64 [K]
    part_edges: torch.Tensor             # int64 [K]


class ReorderResult(NamedTuple):
    perm: torch.Tensor                   # int32 [N]: perm[new_id] = old id
    inv_perm: Optional[torch.Tensor]     # int32 [N]: inv_perm[old id] = new id


class BandwidthResult(NamedTuple):
    bandwidth_sum: torch.Tensor               # int64 [1]: sum of the vertex bandwidths (divide by N for the average)
    vertex_bandwidth: Optional[torch.Tensor]  # int32 [N]


_default: dict[int, Context] = {}


def default_context(device: Optional[int] = None) -> Context:
    idx = torch.cuda.current_device() if device is None else device
    if idx not in _default:
        _default[idx] = Context(idx)
    return _default[idx]


def ep_kmeans(emb, K, iters, init_centroids, objective=False) -> KMeansResult:
    """Lloyd K-Means: (assign, centroids, objective).  Asynchronous on the current stream."""
    return default_context(emb.device.index).kmeans(emb, K, iters, init_centroids, objective)


def ep_partition_quality(rowptr, colidx, assign, K) -> QualityResult:
    """Edge cut and partition loads of `assign` over the CSR graph."""
    return default_context(assign.device.index).partition_quality(rowptr, colidx, assign, K)


def ep_reorder(assign, K, inverse=True) -> ReorderResult:
    """Partition-ordered permutation (and its inverse)."""
    return default_context(assign.device.index).reorder(assign, K, inverse)


def ep_kmeans_sampled(emb, K, iters, sample_rows, init_centroids) -> KMeansResult:
    """Sampling-based clustering: centroids from the sampled rows, labels for every row."""
    return default_context(emb.device.index).kmeans_sampled(emb, K, iters, sample_rows, init_centroids)


def ep_graph_bandwidth(rowptr, colidx, pi, per_vertex=True) -> BandwidthResult:
    """Vertex bandwidths of the numbering pi over the CSR graph and their sum."""
    return default_context(pi.device.index).graph_bandwidth(rowptr, colidx, pi, per_vertex)


REORDER_STATIC_MAX_N = 1 << 22
REORDER_STATIC_MAX_K = 256


def ep_reorder_static(assign, K, inverse=True, status=None) -> ReorderResult:
    """ep_reorder through the entry point that needs neither a context nor a workspace (its scratch is
    built into the library); N <= REORDER_STATIC_MAX_N, K <= REORDER_STATIC_MAX_K.  `status`, if given,
    is a one-element int32 CUDA tensor that receives the device status.  The output tensors are still
    allocated here by torch: it is the library call that allocates nothing."""
    lib = load_library()
    if not assign.is_cuda or assign.dtype != torch.int32 or not assign.is_contiguous():
        raise ValueError("assign must be a contiguous int32 CUDA tensor")
    N = assign.numel()
    perm = torch.empty(N, dtype=torch.int32, device=assign.device)
    inv = torch.empty(N, dtype=torch.int32, device=assign.device) if inverse else None
    with torch.cuda.device(assign.device):
        rc = lib.ep_reorder_static(_dev_ptr(assign), N, K, _dev_ptr(perm), _dev_ptr(inv), _dev_ptr(status),
                                   ctypes.c_void_p(torch.cuda.current_stream(assign.device).cuda_stream))
    if rc != EP_OK:
        raise EmbedPartError(rc, lib.ep_status_string(rc).decode())
    return ReorderResult(perm, inv)
