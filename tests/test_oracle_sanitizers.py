"""The oracle's C code under AddressSanitizer and UndefinedBehaviorSanitizer.

The oracle is what every parity claim rests on, so its own memory accesses and integer arithmetic are checked once
with the compiler's sanitizers: the C file is built with -fsanitize=address,undefined into a library of its own and a
child process (the sanitizer runtime has to be loaded before Python) drives every entry point through small and
awkward inputs: empty rows, K = 1, K = N, a single vertex, duplicate entries, an empty candidate set.  Any report
from a sanitizer ends the child with a non-zero status."""
import os
import subprocess
import sys

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)

CHILD = r'''
import ctypes, sys
import numpy as np
sys.path.insert(0, %(root)r)
import oracle.ep_oracle as eo
eo._lib_path = lambda: %(lib)r          # the sanitized build
rng = np.random.default_rng(7)
for N, d, K, T in ((1, 4, 1, 2), (7, 8, 7, 3), (64, 12, 5, 4), (300, 32, 9, 0), (33, 4, 33, 1)):
    emb = rng.normal(size=(N, d)).astype(np.float32)
    init = emb[rng.permutation(N)[:K]].copy()
    r = eo.kmeans(emb, K, T, init)
    assert r.assign.min() >= 0 and r.assign.max() < K
    eo.assign_step(emb, r.centroids)
    if N >= 2 * K:
        eo.sampled_kmeans(emb, np.arange(0, N, 2), K, max(T, 1), emb[:K].copy())
for N, K in ((1, 1), (6, 2), (50, 7), (200, 200)):
    deg = rng.integers(0, 6, size=N)
    deg[rng.integers(0, N)] = 0
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    colidx = rng.integers(0, N, size=int(rowptr[-1])).astype(np.int32)        # duplicates and self-loops allowed
    assign = rng.integers(0, K, size=N).astype(np.int32)
    eo.partition_quality(rowptr, colidx, assign, K)
    perm, inv = eo.reorder(assign, K)
    eo.graph_bandwidth(rowptr, colidx, inv)
    eo.relabel_graph(rowptr, colidx, perm, inv)
    eo.permute_rows(rng.normal(size=(N, 4)).astype(np.float32), perm)
    words = rng.integers(0, 2 ** 32, size=N, dtype=np.uint64).astype(np.uint32)
    cap = -(-N // K) + 1
    eo.migrate(rowptr, assign, K, cap, words)
    eo.migrate(rowptr, assign, K, cap, words, member=np.zeros(N, np.uint8))   # an empty candidate set
    eo.balance(rowptr, assign, K, cap, rng.integers(0, 2 ** 32, size=(64, N), dtype=np.uint64).astype(np.uint32))
print("sanitized oracle ok")
'''


def test_oracle_runs_clean_under_address_and_undefined_behaviour_sanitizers(tmp_path):
    asan = subprocess.run(["gcc", "-print-file-name=libasan.so"], capture_output=True, text=True).stdout.strip()
    ubsan = subprocess.run(["gcc", "-print-file-name=libubsan.so"], capture_output=True, text=True).stdout.strip()
    if not (os.path.isabs(asan) and os.path.exists(asan) and os.path.isabs(ubsan) and os.path.exists(ubsan)):
        pytest.skip("gcc's sanitizer runtimes are not installed")
    lib = str(tmp_path / "libep_oracle_sanitized.so")
    src = os.path.join(ROOT, "oracle", "ep_oracle.c")
    subprocess.run(["gcc", "-O1", "-g", "-fno-omit-frame-pointer", "-fsanitize=address,undefined",
                    "-fno-sanitize-recover=undefined", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", lib, src, "-lm"],
                   check=True, capture_output=True, text=True)
    env = dict(os.environ, LD_PRELOAD=f"{asan}:{ubsan}", ASAN_OPTIONS="detect_leaks=0:abort_on_error=0:exitcode=97",
               UBSAN_OPTIONS="halt_on_error=1:exitcode=98", OMP_NUM_THREADS="2")
    r = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT, "lib": lib}], capture_output=True, text=True, env=env,
                       timeout=600)
    assert r.returncode == 0 and "sanitized oracle ok" in r.stdout, (r.returncode, r.stdout[-2000:], r.stderr[-4000:])
