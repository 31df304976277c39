"""CPU oracle for the DEFT gradient-selection path: TEST INFRASTRUCTURE ONLY.

Thin ctypes/numpy marshalling around ``deft_oracle.cpp`` (plain single-threaded
C++, fp64 norms, sort-based selection, literal Algorithm 3 / Algorithm 4).  Only
the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library never does, and this package never imports the CUDA
library.  No arithmetic of the method lives in this file: every function below
only converts arguments and calls the C++ routine of the same name.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "deft_oracle.cpp")
_LIB = os.path.join(_HERE, "libdeft_oracle.so")

MODE_PAPER = 0
MODE_EXACT = 1


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared", "-pthread", _SRC, "-o", tmp]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_split_layers.restype = ctypes.c_int64
        _lib.oracle_allocate_k.restype = ctypes.c_int64
        _lib.oracle_rank_bin.restype = ctypes.c_int64
        _lib.oracle_partition_optimum.restype = ctypes.c_double
        _lib.oracle_select_rank.restype = ctypes.c_int64
        _lib.oracle_index_union.restype = ctypes.c_int64
        _lib.oracle_vector_norm.restype = ctypes.c_double
        _lib.oracle_error_eq2.restype = ctypes.c_double
        _lib.oracle_hardware_threads.restype = ctypes.c_int64
        _lib.oracle_select_rank_threads.restype = ctypes.c_int64
    return _lib


def _p(a):
    return ctypes.c_void_p(a.ctypes.data)


def _i64(x):
    return ctypes.c_int64(int(x))


def split_layers(tensor_sizes, n_workers):
    """Algorithm 2. Returns (layer_start[L+1] int64, layer_tensor[L] int32)."""
    sizes = np.ascontiguousarray(tensor_sizes, dtype=np.int64)
    cap = int(sizes.size) * int(n_workers)
    start = np.zeros(cap + 1, dtype=np.int64)
    tensor = np.zeros(cap, dtype=np.int32)
    L = _load().oracle_split_layers(_p(sizes), _i64(sizes.size), _i64(n_workers), _p(start), _p(tensor), _i64(cap))
    if L < 0:
        raise ValueError("oracle_split_layers: invalid input")
    return start[: L + 1].copy(), tensor[:L].copy()


def accumulate(e, g):
    """Algorithm 1 line 5, in place over ``e`` (fp32)."""
    assert e.dtype == np.float32 and g.dtype == np.float32 and e.flags.c_contiguous and g.flags.c_contiguous
    assert e.size == g.size
    _load().oracle_accumulate(_p(e), _p(g), _i64(e.size))
    return e


def layer_norms(acc, layer_start):
    """Per-layer L2 norms in fp64 (Section 4.2)."""
    assert acc.dtype == np.float32 and acc.flags.c_contiguous
    ls = np.ascontiguousarray(layer_start, dtype=np.int64)
    norms = np.zeros(ls.size - 1, dtype=np.float64)
    _load().oracle_layer_norms(_p(acc), _p(ls), _i64(ls.size - 1), _p(norms))
    return norms


def allocate_k(norms, layer_size, k, mode=MODE_EXACT):
    """Algorithm 3. Returns (k_l int64[L], sum_k)."""
    nr = np.ascontiguousarray(norms, dtype=np.float64)
    sz = np.ascontiguousarray(layer_size, dtype=np.int64)
    k_l = np.zeros(sz.size, dtype=np.int64)
    s = ctypes.c_int64(0)
    rc = _load().oracle_allocate_k(_p(nr), _p(sz), _i64(sz.size), _i64(k), _i64(mode), _p(k_l), ctypes.byref(s))
    if rc != 0:
        raise ValueError("oracle_allocate_k failed with %d" % rc)
    return k_l, int(s.value)


def partition(layer_size, k_l, n_workers):
    """Algorithm 4 packing. Returns (bin_of_layer int32[L], bin_load float64[N])."""
    sz = np.ascontiguousarray(layer_size, dtype=np.int64)
    kl = np.ascontiguousarray(k_l, dtype=np.int64)
    bins = np.zeros(sz.size, dtype=np.int32)
    load = np.zeros(int(n_workers), dtype=np.float64)
    _load().oracle_partition(_p(sz), _p(kl), _i64(sz.size), _i64(n_workers), _p(bins), _p(load))
    return bins, load


def partition_by_size(layer_size, n_workers):
    """Algorithm 4's packing with cost = layer size (load-model ablation). Returns (bins, loads)."""
    sz = np.ascontiguousarray(layer_size, dtype=np.int64)
    bins = np.zeros(sz.size, dtype=np.int32)
    load = np.zeros(int(n_workers), dtype=np.float64)
    _load().oracle_partition_by_size(_p(sz), _i64(sz.size), _i64(n_workers), _p(bins), _p(load))
    return bins, load


def rank_bin(iteration, rank, n_workers):
    """Algorithm 4 lines 1-2."""
    return int(_load().oracle_rank_bin(_i64(iteration), _i64(rank), _i64(n_workers)))


def partition_optimum(cost, n_workers):
    """Exhaustive minimum of the maximum bin load (tiny inputs only)."""
    c = np.ascontiguousarray(cost, dtype=np.float64)
    return float(_load().oracle_partition_optimum(_p(c), _i64(c.size), _i64(n_workers)))


def select_layer(acc, st, end, k):
    """Algorithm 5 on one layer: (values fp32[k], indices int64[k]), ascending index."""
    assert acc.dtype == np.float32 and acc.flags.c_contiguous
    val = np.zeros(int(k), dtype=np.float32)
    idx = np.zeros(int(k), dtype=np.int64)
    _load().oracle_select_layer(_p(acc), _i64(st), _i64(end), _i64(k), _p(val), _p(idx))
    return val, idx


def select_rank(acc, layer_start, k_l, my_layers):
    """Algorithm 5 over a rank's layers (ascending ids)."""
    assert acc.dtype == np.float32 and acc.flags.c_contiguous
    ls = np.ascontiguousarray(layer_start, dtype=np.int64)
    kl = np.ascontiguousarray(k_l, dtype=np.int64)
    my = np.ascontiguousarray(my_layers, dtype=np.int32)
    total = int(kl[my].sum()) if my.size else 0
    val = np.zeros(total, dtype=np.float32)
    idx = np.zeros(total, dtype=np.int64)
    got = _load().oracle_select_rank(_p(acc), _p(ls), _p(kl), _p(my), _i64(my.size), _p(val), _p(idx))
    assert got == total
    return val, idx


def topk(acc, k):
    """Conventional full-vector Top-k (Section 3.1): Algorithm 5 with one layer."""
    return select_layer(acc, 0, acc.size, k)


def residual_update(acc, idx):
    """Algorithm 1 lines 11-12, in place."""
    assert acc.dtype == np.float32 and acc.flags.c_contiguous
    ix = np.ascontiguousarray(idx, dtype=np.int64)
    _load().oracle_residual_update(_p(acc), _p(ix), _i64(ix.size))
    return acc


def threshold_select(acc, threshold):
    """Hard-threshold sparsifier (Section 3.2): entries with magnitude > threshold, ascending index."""
    assert acc.dtype == np.float32 and acc.flags.c_contiguous
    lib = _load()
    lib.oracle_threshold_select.restype = ctypes.c_int64
    n = lib.oracle_threshold_select(_p(acc), _i64(acc.size), ctypes.c_float(threshold), None, None, _i64(0))
    val = np.empty(n, dtype=np.float32)
    idx = np.empty(n, dtype=np.int64)
    lib.oracle_threshold_select(_p(acc), _i64(acc.size), ctypes.c_float(threshold), _p(val), _p(idx), _i64(n))
    return val, idx


def clt_leader(iteration, n_workers):
    """CLT-k (Section 3.1): the worker that selects in this iteration."""
    lib = _load()
    lib.oracle_clt_leader.restype = ctypes.c_int64
    return int(lib.oracle_clt_leader(_i64(iteration), _i64(n_workers)))


def gather_update(acc, idx):
    """CLT-k follower: own values at the leader's indices, then cleared (in place).  Returns the values."""
    assert acc.dtype == np.float32 and acc.flags.c_contiguous
    ix = np.ascontiguousarray(idx, dtype=np.int64)
    val = np.empty(ix.size, dtype=np.float32)
    _load().oracle_gather_update(_p(acc), _p(ix), _i64(ix.size), _p(val))
    return val


def my_layers(bin_of_layer, iteration, rank, n_workers):
    """Layer ids (ascending) whose bin is the one ``rank`` reads this iteration."""
    b = rank_bin(iteration, rank, n_workers)
    return np.nonzero(np.asarray(bin_of_layer) == b)[0].astype(np.int32)


def index_union(idx):
    """Algorithm 1 line 7: the set of the gathered indices, ascending."""
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    out = np.empty(idx.size, dtype=np.int64)
    n = _load().oracle_index_union(_p(idx), _i64(idx.size), _p(out))
    return out[:n].copy()


def sum_into(dst, src):
    """Algorithm 1 line 9 (the sum), fp32, in place over ``dst``."""
    assert dst.dtype == np.float32 and src.dtype == np.float32 and dst.size == src.size
    _load().oracle_sum_into(_p(dst), _p(src), _i64(dst.size))
    return dst


def average(total, n_workers):
    """Algorithm 1 line 9 (the 1/n), fp32, in place."""
    assert total.dtype == np.float32
    _load().oracle_average(_p(total), _i64(total.size), _i64(n_workers))
    return total


def vector_norm(x):
    """Eq. 2: L2 norm of a worker's residual, fp64."""
    assert x.dtype == np.float32 and x.flags.c_contiguous
    return float(_load().oracle_vector_norm(_p(x), _i64(x.size)))


def error_eq2(worker_errors):
    """Eq. 2: mean of the workers' errors."""
    w = np.ascontiguousarray(worker_errors, dtype=np.float64)
    return float(_load().oracle_error_eq2(_p(w), _i64(w.size)))


def hardware_threads():
    return int(_load().oracle_hardware_threads())


def select_rank_threads(acc, layer_start, k_l, my_layers, threads=0):
    """oracle select_rank with the rank's layers farmed out over host threads (timing leg).
    Returns (values, indices, threads used)."""
    layer_start = np.ascontiguousarray(layer_start, dtype=np.int64)
    k_l = np.ascontiguousarray(k_l, dtype=np.int64)
    my = np.ascontiguousarray(my_layers, dtype=np.int32)
    total = int(k_l[my].sum()) if my.size else 0
    val = np.empty(total, dtype=np.float32)
    idx = np.empty(total, dtype=np.int64)
    used = _load().oracle_select_rank_threads(_p(acc), _p(layer_start), _p(k_l), _p(my), _i64(my.size), _p(val), _p(idx),
                                              _i64(threads))
    return val, idx, int(used)
