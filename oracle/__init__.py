"""ctypes front end of the CPU oracle (oracle/bmu_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  The CUDA library never imports or calls it,
and this package imports nothing from the CUDA library.  All arithmetic lives
in the C file; this module only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bmu_oracle.c")
_LIB = os.path.join(_HERE, "libbmu_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE: no -ffast-math)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                           "-Wall", "-Wextra", _SRC, "-o", tmp, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        lib.oracle_norms.argtypes = [vp, i64, i64, vp]
        lib.oracle_norms.restype = None
        lib.oracle_eval.argtypes = [vp, i64, i64, vp, vp, vp, i64, i64]
        lib.oracle_eval.restype = ctypes.c_double
        lib.oracle_bmu.argtypes = [vp, i64, i64, vp, vp, vp, i64, vp, vp, vp, ci]
        lib.oracle_bmu.restype = ci
        lib.oracle_bmu2.argtypes = [vp, i64, i64, vp, vp, vp, i64, vp, vp, vp, vp, ci]
        lib.oracle_bmu2.restype = ci
        lib.oracle_scatter.argtypes = [vp, vp, i64, vp, i64, vp, vp]
        lib.oracle_scatter.restype = None
        lib.oracle_blur_plane.argtypes = [vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_double, vp]
        lib.oracle_blur_plane.restype = None
        lib.oracle_writeback.argtypes = [vp, vp, i64, i64, vp]
        lib.oracle_writeback.restype = None
        lib.oracle_map_errors.argtypes = [vp, vp, vp, i64, ctypes.c_int32, ctypes.c_int32,
                                          ctypes.c_int32, vp]
        lib.oracle_map_errors.restype = None
        lib.oracle_max_threads.argtypes = []
        lib.oracle_max_threads.restype = ci
        _lib = lib
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def norms(W) -> np.ndarray:
    """||w_j||^2 per neuron in float64.  W: [D, M] float32, feature-major."""
    W = _f32(W)
    D, M = W.shape
    out = np.empty(M, dtype=np.float64)
    _load().oracle_norms(_p(W), D, M, _p(out))
    return out


def bmu(W, rowptr, colidx, norms_=None, threads: int = 0):
    """(bmu int32 [N], d1 float64 [N], d2 float64 [N]) for a CSR corpus."""
    W = _f32(W)
    rowptr, colidx = _i32(rowptr), _i32(colidx)
    D, M = W.shape
    N = rowptr.shape[0] - 1
    n = norms(W) if norms_ is None else np.ascontiguousarray(norms_, dtype=np.float64)
    out_b = np.empty(N, dtype=np.int32)
    d1 = np.empty(N, dtype=np.float64)
    d2 = np.empty(N, dtype=np.float64)
    rc = _load().oracle_bmu(_p(W), D, M, _p(n), _p(rowptr), _p(colidx), N,
                            _p(out_b), _p(d1), _p(d2), int(threads))
    if rc != 0:
        raise MemoryError("oracle_bmu could not allocate its accumulators")
    return out_b, d1, d2


def bmu2(W, rowptr, colidx, norms_=None, threads: int = 0):
    """(bmu, d1, bmu2, d2): best and second-best unit of every document."""
    W = _f32(W)
    rowptr, colidx = _i32(rowptr), _i32(colidx)
    D, M = W.shape
    N = rowptr.shape[0] - 1
    n = norms(W) if norms_ is None else np.ascontiguousarray(norms_, dtype=np.float64)
    b1 = np.empty(N, dtype=np.int32)
    b2 = np.empty(N, dtype=np.int32)
    d1 = np.empty(N, dtype=np.float64)
    d2 = np.empty(N, dtype=np.float64)
    rc = _load().oracle_bmu2(_p(W), D, M, _p(n), _p(rowptr), _p(colidx), N,
                             _p(b1), _p(d1), _p(d2), _p(b2), int(threads))
    if rc != 0:
        raise MemoryError("oracle_bmu2 could not allocate its accumulators")
    return b1, d1, b2, d2


def eval_pair(W, rowptr, colidx, norms_, i: int, j: int) -> float:
    """Distance of document i to neuron j."""
    W = _f32(W)
    rowptr, colidx = _i32(rowptr), _i32(colidx)
    D, M = W.shape
    n = np.ascontiguousarray(norms_, dtype=np.float64)
    return float(_load().oracle_eval(_p(W), D, M, _p(n), _p(rowptr), _p(colidx),
                                     int(i), int(j)))


# ---- the rest of a batch epoch: scatter, blur, write-back (Table 4) ----------
def scatter(rowptr, colidx, bmu_, D: int, M: int):
    """(num uint64 [D, M], cnt uint64 [M]): how many documents of each unit have each feature."""
    rowptr, colidx, b = _i32(rowptr), _i32(colidx), _i32(bmu_)
    N = rowptr.shape[0] - 1
    num = np.zeros((D, M), dtype=np.uint64)
    cnt = np.zeros(M, dtype=np.uint64)
    _load().oracle_scatter(_p(rowptr), _p(colidx), N, _p(b), M, _p(num), _p(cnt))
    return num, cnt


def blur(planes, edge_x: int, edge_y: int, sigma: float) -> np.ndarray:
    """Truncated Gaussian neighbourhood sum of every plane ([..., edge_y * edge_x]) in float64."""
    a = np.ascontiguousarray(planes, dtype=np.float64)
    flat = a.reshape(-1, edge_x * edge_y)
    out = np.empty_like(flat)
    for r in range(flat.shape[0]):
        _load().oracle_blur_plane(_p(flat[r]), edge_x, edge_y, float(sigma), _p(out[r]))
    return out.reshape(a.shape)


def writeback(B, c, W) -> np.ndarray:
    """New codebook (float32 copy of W with W[f][j] = B[f][j] / c[j] where c[j] > 0)."""
    B = np.ascontiguousarray(B, dtype=np.float64)
    c = np.ascontiguousarray(c, dtype=np.float64)
    out = _f32(W).copy()
    D, M = out.shape
    _load().oracle_writeback(_p(B), _p(c), D, M, _p(out))
    return out


def map_errors(bmu, bmu2, dist, edge_x: int, edge_y: int, adjacency: int = 4) -> np.ndarray:
    """(mean squared quantisation error, mean quantisation error, topographic error) of a
    search with second-best units on an edge_y x edge_x map."""
    b1 = np.ascontiguousarray(bmu, dtype=np.int32)
    b2 = np.ascontiguousarray(bmu2, dtype=np.int32)
    d = _f32(dist)
    if adjacency not in (4, 8):
        raise ValueError("adjacency must be 4 or 8")
    out = np.zeros(3, dtype=np.float64)
    _load().oracle_map_errors(_p(b1), _p(b2), _p(d), b1.size, edge_x, edge_y, adjacency, _p(out))
    return out
