"""Thin binding over libdeft.so (ctypes): the same names as the C ABI, argument marshalling only.

Host tables are numpy arrays, device buffers are torch CUDA tensors (used for memory and
streams only).  Nothing here computes anything of the method, and there is no fallback:
if the CUDA library is missing or fails to load, importing a device call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdeft.so")

OK = 0
WARN_K_INEXACT = 1
ERR_INVALID_ARG = -1
ERR_INFEASIBLE_K = -2
ERR_NONFINITE_NORM = -3
ERR_CAPACITY = -4
ERR_CUDA = -5
ERR_TOO_LARGE = -6
MODE_PAPER = 0
MODE_EXACT = 1


class DeftError(RuntimeError):
    def __init__(self, call: str, status: int, detail: str = ""):
        self.status = status
        super().__init__("%s failed: %s%s" % (call, status_string(status), detail))


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libdeft.so from the package directory.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                "libdeft.so is missing at %s: build it with `python -m paper_2307_03500_b200.build` "
                "(there is no CPU fallback)" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        c = ctypes
        vp, i32, i64, sz = c.c_void_p, c.c_int32, c.c_int64, c.c_size_t
        L.deft_status_string.restype = c.c_char_p
        L.deft_status_string.argtypes = [i32]
        L.deft_last_cuda_error.restype = i32
        L.deft_last_cuda_error.argtypes = []
        L.deft_debug_select_timing.restype = None
        L.deft_debug_select_timing.argtypes = [vp]
        L.deft_debug_select_kernel.restype = None
        L.deft_debug_select_kernel.argtypes = [i32]
        L.deft_debug_select_ring.restype = None
        L.deft_debug_select_ring.argtypes = [i32]
        L.deft_debug_step_staging.restype = None
        L.deft_debug_step_staging.argtypes = [i32]
        L.deft_select_stats.restype = i32
        L.deft_select_stats.argtypes = [vp, sz, i32, vp, vp]
        L.deft_select_launch_max_elems.restype = i64
        L.deft_select_launch_max_elems.argtypes = []
        L.deft_split_layers.restype = i32
        L.deft_split_layers.argtypes = [vp, i32, i32, vp, vp, i32, vp]
        L.deft_allocate_k.restype = i32
        L.deft_allocate_k.argtypes = [vp, vp, i32, i64, i32, vp, vp]
        L.deft_partition.restype = i32
        L.deft_partition.argtypes = [vp, vp, i32, i32, vp, vp]
        L.deft_rank_bin.restype = i32
        L.deft_rank_bin.argtypes = [i64, i32, i32]
        L.deft_bin_layers.restype = i32
        L.deft_bin_layers.argtypes = [vp, i32, i32, vp, i32, vp]
        L.deft_workspace_bytes.restype = sz
        L.deft_workspace_bytes.argtypes = [i64, i32]
        L.deft_layer_norms.restype = i32
        L.deft_layer_norms.argtypes = [vp, vp, i64, vp, i32, vp, vp, sz, vp]
        L.deft_layer_norms_static_max_slots.restype = i64
        L.deft_layer_norms_static_max_slots.argtypes = []
        L.deft_layer_norms_static.restype = i32
        L.deft_layer_norms_static.argtypes = [vp, vp, i64, vp, i32, vp, vp]
        L.deft_select.restype = i32
        L.deft_select.argtypes = [vp, vp, vp, vp, i32, vp, vp, i64, vp, sz, vp]
        L.deft_plan_bytes.restype = sz
        L.deft_plan_bytes.argtypes = [i32, i32]
        L.deft_plan_build.restype = i32
        L.deft_plan_build.argtypes = [vp, vp, vp, i32, i32, i64, vp, sz]
        L.deft_plan_rank_info.restype = i32
        L.deft_plan_rank_info.argtypes = [vp, i32, vp, vp, vp, vp]
        L.deft_plan_rank_table.restype = i32
        L.deft_plan_rank_table.argtypes = [vp, i32, vp, vp, vp, vp]
        L.deft_step.restype = i32
        L.deft_step.argtypes = [vp, vp, i64, vp, vp, i32, i32, i64, i32, i32, i64, i32, vp, vp, vp, vp, vp, vp, vp, sz,
                                vp, vp, vp, i64, vp, sz, vp, vp]
        L.deft_workspace_init.restype = i32
        L.deft_workspace_init.argtypes = [vp, sz, i32, vp]
        L.deft_threshold_select.restype = i32
        L.deft_threshold_select.argtypes = [vp, i64, ctypes.c_float, i32, vp, vp, i64, vp, vp, sz, vp]
        L.deft_clt_leader.restype = i32
        L.deft_clt_leader.argtypes = [i64, i32]
        L.deft_gather_update.restype = i32
        L.deft_gather_update.argtypes = [vp, i64, vp, i64, vp, vp]
        L.deft_plan_step.restype = i32
        L.deft_plan_step.argtypes = [vp, vp, i32, i32, i64, i32, i32, i64, vp, vp, vp, vp, vp, sz, vp, vp, sz, vp]
        L.deft_partition_model.restype = i32
        L.deft_partition_model.argtypes = [vp, vp, i32, i32, i32, vp, vp]
        L.deft_plan_upload.restype = i32
        L.deft_plan_upload.argtypes = [vp, vp, vp, sz, vp]
        L.deft_select_planned.restype = i32
        L.deft_select_planned.argtypes = [vp, vp, vp, i32, vp, vp, i64, vp, sz, vp]
        L.deft_select_update_all.restype = i32
        L.deft_select_update_all.argtypes = [vp, i64, vp, vp, vp, vp, i64, vp, sz, vp]
        L.deft_select_update_ranks.restype = i32
        L.deft_select_update_ranks.argtypes = [vp, i64, vp, vp, i32, i32, vp, vp, i64, vp, sz, vp, vp]
        L.deft_error_eq2.restype = i32
        L.deft_error_eq2.argtypes = [vp, i32, vp]
        L.deft_union_workspace_bytes.restype = sz
        L.deft_union_workspace_bytes.argtypes = [i64]
        L.deft_index_union.restype = i32
        L.deft_index_union.argtypes = [vp, i64, i64, vp, i64, vp, vp, sz, vp]
        L.deft_sum_into.restype = i32
        L.deft_sum_into.argtypes = [vp, vp, i64, vp]
        L.deft_average.restype = i32
        L.deft_average.argtypes = [vp, i64, i32, vp]
        L.deft_vector_norm_workspace_bytes.restype = sz
        L.deft_vector_norm_workspace_bytes.argtypes = [i64]
        L.deft_vector_norm.restype = i32
        L.deft_vector_norm.argtypes = [vp, i64, vp, vp, sz, vp]
        L.deft_residual_update.restype = i32
        L.deft_residual_update.argtypes = [vp, i64, vp, i64, vp]
        L.deft_topk_baseline.restype = i32
        L.deft_topk_baseline.argtypes = [vp, i64, i64, vp, vp, vp, sz, vp]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().deft_status_string(int(status)).decode()


def _check(call: str, status: int, allow_warn: bool = False) -> int:
    if status < 0 or (status > 0 and not allow_warn):
        detail = ""
        if status == ERR_CUDA:
            detail = " (cudaError %d)" % lib().deft_last_cuda_error()
        raise DeftError(call, status, detail)
    return status


def _np(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def _hp(a: Optional[np.ndarray]):
    return None if a is None else ctypes.c_void_p(a.ctypes.data)


def _dp(t, dtype=None):
    """Device pointer of a contiguous CUDA tensor."""
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError("expected dtype %s, got %s" % (dtype, t.dtype))
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


# ------------------------------------------------------------------------------------------
# host planners
# ------------------------------------------------------------------------------------------
def deft_split_layers(tensor_sizes, n_workers: int) -> Tuple[np.ndarray, np.ndarray]:
    """Algorithm 2 -> (layer_start int64[L+1], layer_tensor int32[L])."""
    sizes = _np(tensor_sizes, np.int64)
    L = ctypes.c_int32(0)
    st = lib().deft_split_layers(_hp(sizes), sizes.size, int(n_workers), _hp(np.zeros(1, np.int64)), None, 0,
                                 ctypes.byref(L))
    if st != ERR_CAPACITY:
        _check("deft_split_layers", st)
    cap = int(L.value)
    start = np.zeros(cap + 1, dtype=np.int64)
    tensor = np.zeros(cap, dtype=np.int32)
    _check("deft_split_layers",
           lib().deft_split_layers(_hp(sizes), sizes.size, int(n_workers), _hp(start), _hp(tensor), cap,
                                   ctypes.byref(L)))
    return start, tensor


def deft_allocate_k(norms, layer_size, k: int, mode: int = MODE_EXACT) -> Tuple[np.ndarray, int, int]:
    """Algorithm 3 -> (k_l int64[L], sum_k, status) ; status may be WARN_K_INEXACT in PAPER mode."""
    nr = _np(norms, np.float64)
    sz = _np(layer_size, np.int64)
    if nr.size != sz.size:
        raise ValueError("norms and layer_size differ in length")
    k_l = np.zeros(sz.size, dtype=np.int64)
    s = ctypes.c_int64(0)
    st = _check("deft_allocate_k",
                lib().deft_allocate_k(_hp(nr), _hp(sz), sz.size, int(k), int(mode), _hp(k_l), ctypes.byref(s)),
                allow_warn=True)
    return k_l, int(s.value), st


COST_EQ3 = 0
COST_SIZE = 1


def deft_partition_model(layer_size, k_l, n_workers: int, cost_model: int) -> Tuple[np.ndarray, np.ndarray]:
    """Algorithm 4's packing under a load model (COST_EQ3 / COST_SIZE) -> (bins int32[L], loads float64[N])."""
    sz = _np(layer_size, np.int64)
    kl = None if k_l is None else _np(k_l, np.int64)
    if kl is not None and kl.size != sz.size:
        raise ValueError("k_l and layer_size differ in length")
    bins = np.zeros(sz.size, dtype=np.int32)
    load = np.zeros(int(n_workers), dtype=np.float64)
    _check("deft_partition_model", lib().deft_partition_model(_hp(sz), _hp(kl), sz.size, int(n_workers),
                                                              int(cost_model), _hp(bins), _hp(load)))
    return bins, load


def deft_partition(layer_size, k_l, n_workers: int) -> Tuple[np.ndarray, np.ndarray]:
    """Algorithm 4 packing -> (bin_of_layer int32[L], bin_load float64[N])."""
    sz = _np(layer_size, np.int64)
    kl = _np(k_l, np.int64)
    if kl.size != sz.size:
        raise ValueError("k_l and layer_size differ in length")
    bins = np.zeros(sz.size, dtype=np.int32)
    load = np.zeros(int(n_workers), dtype=np.float64)
    _check("deft_partition", lib().deft_partition(_hp(sz), _hp(kl), sz.size, int(n_workers), _hp(bins), _hp(load)))
    return bins, load


def deft_rank_bin(iteration: int, rank: int, n_workers: int) -> int:
    b = lib().deft_rank_bin(int(iteration), int(rank), int(n_workers))
    if b < 0:
        raise DeftError("deft_rank_bin", ERR_INVALID_ARG)
    return int(b)


def deft_bin_layers(bin_of_layer, bin_id: int) -> np.ndarray:
    bins = _np(bin_of_layer, np.int32)
    out = np.zeros(bins.size, dtype=np.int32)
    n = ctypes.c_int32(0)
    _check("deft_bin_layers", lib().deft_bin_layers(_hp(bins), bins.size, int(bin_id), _hp(out), out.size,
                                                    ctypes.byref(n)))
    return out[: n.value].copy()


# ------------------------------------------------------------------------------------------
# device calls
# ------------------------------------------------------------------------------------------
def deft_workspace_bytes(max_elems: int, max_layers: int) -> int:
    return int(lib().deft_workspace_bytes(int(max_elems), int(max_layers)))


def alloc_workspace(max_elems: int, max_layers: int, device="cuda"):
    """A torch uint8 tensor of deft_workspace_bytes() bytes (torch allocations are 512-byte aligned)."""
    import torch
    ws = torch.empty(deft_workspace_bytes(max_elems, max_layers), dtype=torch.uint8, device=device)
    with torch.cuda.device(ws.device):
        _check("deft_workspace_init", lib().deft_workspace_init(_dp(ws), ws.numel(), int(max_layers), _stream(None)))
    return ws


def deft_layer_norms(resid_acc, grad, layer_start_d, norms_d, ws, stream=None) -> None:
    import torch
    n_g = resid_acc.numel()
    L = layer_start_d.numel() - 1
    if grad is not None and grad.numel() != n_g:
        raise ValueError("grad and resid_acc differ in length")
    if norms_d.numel() < L:
        raise ValueError("norms_d too small")
    _check("deft_layer_norms",
           lib().deft_layer_norms(_dp(resid_acc, torch.float32), _dp(grad, torch.float32), n_g,
                                  _dp(layer_start_d, torch.int64), L, _dp(norms_d, torch.float64),
                                  _dp(ws), ws.numel() * ws.element_size(), _stream(stream)))


def deft_layer_norms_static(resid_acc, grad, layer_start_d, norms_d, stream=None) -> None:
    """deft_layer_norms without a workspace, for callers that may not allocate device memory: the scratch is a
    fixed array inside the library (limit: ceil(n_g/8192) + L + 1 <= deft_layer_norms_static_max_slots())."""
    import torch
    n_g = resid_acc.numel()
    L = layer_start_d.numel() - 1
    if grad is not None and grad.numel() != n_g:
        raise ValueError("grad and resid_acc differ in length")
    if norms_d.numel() < L:
        raise ValueError("norms_d too small")
    _check("deft_layer_norms_static",
           lib().deft_layer_norms_static(_dp(resid_acc, torch.float32), _dp(grad, torch.float32), n_g,
                                         _dp(layer_start_d, torch.int64), L, _dp(norms_d, torch.float64),
                                         _stream(stream)))


def deft_select(acc, layer_start_h, k_l_h, my_layers_h, val_d, idx_d, ws, stream=None) -> int:
    """Algorithm 5 for one rank.  Returns the number of entries written (sum of k_l over my layers)."""
    import torch
    ls = _np(layer_start_h, np.int64)
    kl = _np(k_l_h, np.int64)
    my = _np(my_layers_h, np.int32)
    if kl.size != ls.size - 1:
        raise ValueError("k_l_h and layer_start_h disagree")
    if my.size and (my.min() < 0 or my.max() >= kl.size):
        raise ValueError("layer id out of range")
    cap = min(val_d.numel(), idx_d.numel())
    _check("deft_select",
           lib().deft_select(_dp(acc, torch.float32), _hp(ls), _hp(kl), _hp(my), my.size,
                             _dp(val_d, torch.float32), _dp(idx_d, torch.int64), cap, _dp(ws),
                             ws.numel() * ws.element_size(), _stream(stream)))
    return int(kl[my].sum()) if my.size else 0


def deft_debug_select_timing(timing_d) -> None:
    """Diagnostic phase stamps of the selection kernel: a zeroed CUDA uint64/int64 tensor of 1024, or None."""
    lib().deft_debug_select_timing(None if timing_d is None else _dp(timing_d))


def deft_debug_select_kernel(single_pass) -> None:
    """True / False: force the single-pass / the five-step selection kernel; None: by call size (default)."""
    lib().deft_debug_select_kernel(-1 if single_pass is None else (1 if single_pass else 0))


def deft_debug_select_ring(on: bool) -> None:
    """The single-pass kernel reads through a ring of bulk copies (True, the default) or with plain loads (False)."""
    lib().deft_debug_select_ring(1 if on else 0)


def deft_debug_step_staging(on: bool) -> None:
    """deft_step for all workers stages during the accumulate pass (True, the default) or leaves the read to the
    selection launch (False)."""
    lib().deft_debug_step_staging(1 if on else 0)


def deft_select_stats(ws, n_layers: int, stream=None) -> dict:
    out = np.zeros(8, dtype=np.uint64)
    _check("deft_select_stats", lib().deft_select_stats(_dp(ws), ws.numel() * ws.element_size(), n_layers,
                                                        _hp(out), _stream(stream)))
    return {"one_read": int(out[0]), "cut_failed": int(out[1]), "no_cut": int(out[2]), "ring_gave_up": int(out[3]), "staged_entries": int(out[4])}


def deft_select_launch_max_elems() -> int:
    return int(lib().deft_select_launch_max_elems())


def deft_plan_bytes(n_layers: int, n_workers: int) -> int:
    return int(lib().deft_plan_bytes(int(n_layers), int(n_workers)))


def deft_plan_build(layer_start_h, k_l_h, bin_of_layer_h, n_workers: int, iteration: int,
                    out: Optional[np.ndarray] = None) -> np.ndarray:
    """Builds the step's plan blob on the host.  ``out`` may be a uint8 numpy view of pinned memory."""
    ls = _np(layer_start_h, np.int64)
    kl = _np(k_l_h, np.int64)
    bins = _np(bin_of_layer_h, np.int32)
    L = kl.size
    if ls.size != L + 1 or bins.size != L:
        raise ValueError("layer_start_h, k_l_h and bin_of_layer_h disagree")
    need = deft_plan_bytes(L, n_workers)
    if need == 0:
        raise DeftError("deft_plan_bytes", ERR_INVALID_ARG)
    if out is None:
        out = np.empty(need, dtype=np.uint8)
    if out.dtype != np.uint8 or not out.flags.c_contiguous or out.size < need:
        raise ValueError("plan buffer must be contiguous uint8 of at least %d bytes" % need)
    _check("deft_plan_build", lib().deft_plan_build(_hp(ls), _hp(kl), _hp(bins), L, int(n_workers), int(iteration),
                                                    _hp(out), out.size))
    return out


def deft_plan_rank_info(plan_h: np.ndarray, rank: int) -> Tuple[int, int, int, int]:
    """(layers, elements scanned, entries selected, sum of k over lower ranks) of one rank."""
    n = ctypes.c_int32(0)
    e, k, o = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_int64(0)
    _check("deft_plan_rank_info", lib().deft_plan_rank_info(_hp(plan_h), int(rank), ctypes.byref(n), ctypes.byref(e),
                                                            ctypes.byref(k), ctypes.byref(o)))
    return int(n.value), int(e.value), int(k.value), int(o.value)


def deft_plan_rank_table(plan_h: np.ndarray, n_workers: int):
    """(layers int32[N], elements int64[N], entries int64[N], output offsets int64[N]) of all ranks."""
    n = np.zeros(n_workers, dtype=np.int32)
    e = np.zeros(n_workers, dtype=np.int64)
    k = np.zeros(n_workers, dtype=np.int64)
    o = np.zeros(n_workers, dtype=np.int64)
    _check("deft_plan_rank_table", lib().deft_plan_rank_table(_hp(plan_h), int(n_workers), _hp(n), _hp(e), _hp(k),
                                                              _hp(o)))
    return n, e, k, o


def deft_plan_upload(plan_h: np.ndarray, plan_d, ws, stream=None) -> None:
    if plan_d.numel() * plan_d.element_size() < plan_h.size:
        raise ValueError("plan_d smaller than the plan")
    _check("deft_plan_upload", lib().deft_plan_upload(_hp(plan_h), _dp(plan_d), _dp(ws),
                                                      ws.numel() * ws.element_size(), _stream(stream)))


def deft_plan_step(norms, layer_start_h, n_workers: int, k: int, mode: int, iteration: int, plan_h: np.ndarray,
                   plan_d, ws, stream=None, cost_model: int = 0):
    """Algorithm 3 + Algorithm 4 + plan build + plan upload in one call.
    Returns (k_l int64[L], sum_k, bin_of_layer int32[L], bin_load float64[N], status)."""
    nr = _np(norms, np.float64)
    ls = _np(layer_start_h, np.int64)
    L = nr.size
    if ls.size != L + 1:
        raise ValueError("norms and layer_start_h disagree")
    if plan_d.numel() * plan_d.element_size() < deft_plan_bytes(L, n_workers) or plan_h.dtype != np.uint8 or \
            not plan_h.flags.c_contiguous:
        raise ValueError("plan buffers too small or not contiguous uint8")
    k_l = np.empty(L, dtype=np.int64)
    bins = np.empty(L, dtype=np.int32)
    load = np.empty(int(n_workers), dtype=np.float64)
    s = ctypes.c_int64(0)
    st = _check("deft_plan_step",
                lib().deft_plan_step(_hp(nr), _hp(ls), L, int(n_workers), int(k), int(mode), int(cost_model),
                                     int(iteration), _hp(k_l),
                                     ctypes.byref(s), _hp(bins), _hp(load), _hp(plan_h), plan_h.size, _dp(plan_d),
                                     _dp(ws), ws.numel() * ws.element_size(), _stream(stream)),
                allow_warn=True)
    return k_l, int(s.value), bins, load, st


def deft_step(resid_acc, grad, layer_start_h, layer_start_d, n_workers: int, k: int, mode: int, cost_model: int,
              iteration: int, rank: int, norms_d, norms_h_pinned, k_l_out: np.ndarray, bins_out: np.ndarray,
              load_out: np.ndarray, plan_h: np.ndarray, plan_d, val_d, idx_d, ws, events=None, stream=None):
    """One whole step in one C call (rank = -1: all workers in one launch).  The output arrays
    (k_l_out int64[L], bins_out int32[L], load_out float64[N]) are filled in place.
    norms_h_pinned: a (pinned) torch float64 CPU tensor of L.  events: optional 4 torch CUDA events.
    Returns (sum_k, status)."""
    import torch
    ls = _np(layer_start_h, np.int64)
    L = ls.size - 1
    ev = None
    if events is not None:
        flat = []
        for e in events:
            if e.cuda_event == 0:   # torch creates the handle lazily, on first record
                e.record()
            flat.append(e.cuda_event)
        ev = (ctypes.c_void_p * 4)(*flat)
    s = ctypes.c_int64(0)
    st = _check("deft_step",
                lib().deft_step(_dp(resid_acc, torch.float32), None if grad is None else _dp(grad, torch.float32),
                                resid_acc.numel(), _hp(ls), _dp(layer_start_d, torch.int64), L, int(n_workers), int(k),
                                int(mode), int(cost_model), int(iteration), int(rank), _dp(norms_d, torch.float64),
                                ctypes.c_void_p(norms_h_pinned.data_ptr()), _hp(k_l_out), ctypes.byref(s),
                                _hp(bins_out), _hp(load_out), _hp(plan_h), plan_h.size, _dp(plan_d),
                                _dp(val_d, torch.float32), _dp(idx_d, torch.int64), min(val_d.numel(), idx_d.numel()),
                                _dp(ws), ws.numel() * ws.element_size(), ev, _stream(stream)),
                allow_warn=True)
    return int(s.value), st


def deft_select_planned(acc, plan_h: np.ndarray, plan_d, rank: int, val_d, idx_d, ws, stream=None) -> None:
    """Algorithm 5 for one rank of an uploaded plan (one kernel launch)."""
    import torch
    cap = min(val_d.numel(), idx_d.numel())
    _check("deft_select_planned",
           lib().deft_select_planned(_dp(acc, torch.float32), _hp(plan_h), _dp(plan_d), int(rank),
                                     _dp(val_d, torch.float32) if cap else None,
                                     _dp(idx_d, torch.int64) if cap else None, cap, _dp(ws),
                                     ws.numel() * ws.element_size(), _stream(stream)))


def deft_select_update_ranks(acc, plan_h: np.ndarray, plan_d, rank_begin: int, rank_end: int, val_d, idx_d, ws,
                             events=None, stream=None) -> None:
    """Selection + residual update for a range of simulated ranks (one C call).
    events: optional list of (before, between, after) torch.cuda.Event triples, one per rank."""
    import torch
    ev = None
    if events is not None:
        if len(events) != rank_end - rank_begin:
            raise ValueError("one event triple per rank expected")
        flat = []
        for tri in events:
            for e in tri:
                if e.cuda_event == 0:   # torch creates the handle lazily, on first record
                    e.record()
                flat.append(e.cuda_event)
        ev = (ctypes.c_void_p * len(flat))(*flat)
    _check("deft_select_update_ranks",
           lib().deft_select_update_ranks(_dp(acc, torch.float32), acc.numel(), _hp(plan_h), _dp(plan_d),
                                          int(rank_begin), int(rank_end), _dp(val_d, torch.float32),
                                          _dp(idx_d, torch.int64), min(val_d.numel(), idx_d.numel()), _dp(ws),
                                          ws.numel() * ws.element_size(), ev, _stream(stream)))


def deft_select_update_all(acc, plan_h: np.ndarray, plan_d, val_d, idx_d, ws, stream=None) -> None:
    """Selection + residual update for ALL simulated ranks of the plan in one launch."""
    import torch
    _check("deft_select_update_all",
           lib().deft_select_update_all(_dp(acc, torch.float32), acc.numel(), _hp(plan_h), _dp(plan_d),
                                        _dp(val_d, torch.float32), _dp(idx_d, torch.int64),
                                        min(val_d.numel(), idx_d.numel()), _dp(ws), ws.numel() * ws.element_size(),
                                        _stream(stream)))


def deft_threshold_select(acc, threshold: float, val_d, idx_d, count_d, ws, zero_selected: bool = False,
                          stream=None) -> None:
    """Hard-threshold sparsifier (Section 3.2): entries with magnitude > threshold, ascending index.
    count_d: CUDA int64 tensor of one element that receives the total count."""
    import torch
    cap = 0 if val_d is None or idx_d is None else min(val_d.numel(), idx_d.numel())
    _check("deft_threshold_select",
           lib().deft_threshold_select(_dp(acc, torch.float32), acc.numel(), float(threshold), int(bool(zero_selected)),
                                       _dp(val_d, torch.float32) if cap else None,
                                       _dp(idx_d, torch.int64) if cap else None, cap, _dp(count_d, torch.int64),
                                       _dp(ws), ws.numel() * ws.element_size(), _stream(stream)))


def deft_clt_leader(iteration: int, n_workers: int) -> int:
    r = int(lib().deft_clt_leader(int(iteration), int(n_workers)))
    if r < 0:
        raise DeftError("deft_clt_leader", ERR_INVALID_ARG)
    return r


def deft_gather_update(acc, idx_d, count: int, val_d, stream=None) -> None:
    """CLT-k follower: val_d[i] = acc[idx_d[i]], then that entry is cleared."""
    import torch
    if count > idx_d.numel() or count > val_d.numel():
        raise ValueError("count exceeds idx_d / val_d")
    _check("deft_gather_update",
           lib().deft_gather_update(_dp(acc, torch.float32), acc.numel(), _dp(idx_d, torch.int64), int(count),
                                    _dp(val_d, torch.float32), _stream(stream)))


def deft_error_eq2(worker_errors) -> float:
    w = _np(worker_errors, np.float64)
    out = np.zeros(1, dtype=np.float64)
    _check("deft_error_eq2", lib().deft_error_eq2(_hp(w), int(w.size), _hp(out)))
    return float(out[0])


def deft_union_workspace_bytes(n_g: int) -> int:
    return int(lib().deft_union_workspace_bytes(int(n_g)))


def deft_index_union(idx_d, count: int, n_g: int, union_d, count_d, ws, stream=None) -> None:
    """Sorted set of idx_d[:count] into union_d (as many as fit), its size into count_d (device int64)."""
    _check("deft_index_union", lib().deft_index_union(_dp(idx_d), int(count), int(n_g), _dp(union_d),
                                                      union_d.numel() if union_d is not None else 0, _dp(count_d),
                                                      _dp(ws), ws.numel() * ws.element_size(), _stream(stream)))


def deft_sum_into(dst, src, count: int, stream=None) -> None:
    _check("deft_sum_into", lib().deft_sum_into(_dp(dst), _dp(src), int(count), _stream(stream)))


def deft_average(sum_d, count: int, n_workers: int, stream=None) -> None:
    _check("deft_average", lib().deft_average(_dp(sum_d), int(count), int(n_workers), _stream(stream)))


def deft_vector_norm_workspace_bytes(n: int) -> int:
    return int(lib().deft_vector_norm_workspace_bytes(int(n)))


def deft_vector_norm(x, norm_d, ws, stream=None) -> None:
    _check("deft_vector_norm", lib().deft_vector_norm(_dp(x), x.numel(), _dp(norm_d), _dp(ws),
                                                      ws.numel() * ws.element_size(), _stream(stream)))


def deft_residual_update(acc, idx_d, count: int, stream=None) -> None:
    import torch
    if count > idx_d.numel():
        raise ValueError("count exceeds idx_d")
    _check("deft_residual_update",
           lib().deft_residual_update(_dp(acc, torch.float32), acc.numel(), _dp(idx_d, torch.int64), int(count),
                                      _stream(stream)))


def deft_topk_baseline(acc, k: int, val_d, idx_d, ws, stream=None) -> None:
    import torch
    if min(val_d.numel(), idx_d.numel()) < k:
        raise DeftError("deft_topk_baseline", ERR_CAPACITY)
    _check("deft_topk_baseline",
           lib().deft_topk_baseline(_dp(acc, torch.float32), acc.numel(), int(k), _dp(val_d, torch.float32),
                                    _dp(idx_d, torch.int64), _dp(ws), ws.numel() * ws.element_size(),
                                    _stream(stream)))
