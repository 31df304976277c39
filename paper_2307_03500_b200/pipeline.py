"""One DEFT sparsification step driven through the C ABI (orchestration only).

``DeftStep`` owns the device buffers a step needs (layer table, norms, workspace, output
slabs) and issues the calls in the order of the paper's Section 4: norms of the accumulated
vector -> local k (Algorithm 3) -> bins (Algorithm 4) -> per-rank selection (Algorithm 5) ->
residual update (Algorithm 1, lines 11-12).  Workers are simulated: the same GPU runs the
per-rank part once for every rank.  Every numeric step runs inside libdeft.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

from . import deft


@dataclass
class StepPlan:
    k_l: np.ndarray            # int64[L]
    sum_k: int
    bin_of_layer: np.ndarray   # int32[L]
    bin_load: np.ndarray       # float64[N]  (Eq. 4 per bin)
    rank_layers_n: np.ndarray  # int32[N]  layers of each rank
    rank_k: np.ndarray         # int64[N]  entries each rank selects
    rank_elems: np.ndarray     # int64[N]  elements each rank scans
    rank_out_off: np.ndarray   # int64[N+1] offsets into the output slabs
    plan_h: np.ndarray         # the uploaded plan blob (host copy)


class DeftStep:
    def __init__(self, tensor_sizes, n_workers: int, density: float, device="cuda:0",
                 mode: int = deft.MODE_EXACT, k: Optional[int] = None, cost_model: int = deft.COST_EQ3):
        self.device = torch.device(device)
        self.N = int(n_workers)
        self.mode = mode
        self.cost_model = cost_model
        self.layer_start, self.layer_tensor = deft.deft_split_layers(tensor_sizes, n_workers)
        self.layer_size = np.diff(self.layer_start)
        self.L = int(self.layer_size.size)
        self.n_g = int(self.layer_start[-1])
        self.k = int(k) if k is not None else max(1, int(math.floor(float(self.n_g) * density)))
        if mode == deft.MODE_EXACT:
            self.k = max(self.k, self.L)   # every layer keeps at least one entry (Algorithm 3)
        self.layer_start_d = torch.from_numpy(self.layer_start).to(self.device)
        self.norms_d = torch.empty(self.L, dtype=torch.float64, device=self.device)
        self.norms_h = torch.empty(self.L, dtype=torch.float64).pin_memory() if self.device.type == "cuda" \
            else torch.empty(self.L, dtype=torch.float64)
        self.ws = deft.alloc_workspace(self.n_g, self.L, self.device)
        cap = self.k + self.L + 64   # PAPER mode may overshoot by at most one per layer
        self.val_d = torch.empty(cap, dtype=torch.float32, device=self.device)
        self.idx_d = torch.empty(cap, dtype=torch.int64, device=self.device)
        nbytes = deft.deft_plan_bytes(self.L, self.N)
        self._plan_pin = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
        self.plan_h = self._plan_pin.numpy()
        self.plan_d = torch.empty(nbytes, dtype=torch.uint8, device=self.device)

    # -- step 1: accumulate + norms (device) ------------------------------------------------
    def layer_norms(self, resid: torch.Tensor, grad: Optional[torch.Tensor]) -> np.ndarray:
        deft.deft_layer_norms(resid, grad, self.layer_start_d, self.norms_d, self.ws)
        self.norms_h.copy_(self.norms_d, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        return self.norms_h.numpy()

    # -- steps 2 and 3: local k and bins (host) ---------------------------------------------
    def plan(self, norms: np.ndarray, iteration: int = 0) -> StepPlan:
        """Algorithm 3, Algorithm 4, then the plan of all N ranks built on the host and uploaded."""
        k_l, sum_k, bins, load, _ = deft.deft_plan_step(norms, self.layer_start, self.N, self.k, self.mode, iteration,
                                                        self.plan_h, self.plan_d, self.ws, cost_model=self.cost_model)
        n_layers, elems, rank_k, out_off = deft.deft_plan_rank_table(self.plan_h, self.N)
        off = np.zeros(self.N + 1, dtype=np.int64)
        off[:-1] = out_off
        off[-1] = out_off[-1] + rank_k[-1]
        return StepPlan(k_l, sum_k, bins, load, n_layers, rank_k, elems, off, self.plan_h)

    def rank_layers(self, plan: StepPlan, iteration: int, rank: int) -> np.ndarray:
        return deft.deft_bin_layers(plan.bin_of_layer, deft.deft_rank_bin(iteration, rank, self.N))

    # -- step 4: selection + residual update for one rank (device) --------------------------
    def select_rank(self, acc: torch.Tensor, plan: StepPlan, rank: int):
        a, b = int(plan.rank_out_off[rank]), int(plan.rank_out_off[rank + 1])
        val, idx = self.val_d[a:b], self.idx_d[a:b]
        if b > a:
            deft.deft_select_planned(acc, plan.plan_h, self.plan_d, rank, val, idx, self.ws)
        return val, idx

    def select_and_update_all(self, acc: torch.Tensor, plan: StepPlan, events=None, per_rank: bool = False) -> None:
        """Selection followed by the residual update for every simulated rank (one C call): all ranks in
        one launch, or — with `per_rank` or `events` — one launch per rank, rank after rank.
        `events`: optional list of (before, between, after) CUDA events per rank, recorded on the stream."""
        if events is None and not per_rank:
            deft.deft_select_update_all(acc, plan.plan_h, self.plan_d, self.val_d, self.idx_d, self.ws)
        else:
            deft.deft_select_update_ranks(acc, plan.plan_h, self.plan_d, 0, self.N, self.val_d, self.idx_d, self.ws,
                                          events)

    def residual_update(self, acc: torch.Tensor, idx: torch.Tensor) -> None:
        deft.deft_residual_update(acc, idx, idx.numel())

    # -- the whole step in ONE library call ---------------------------------------------------
    def step_fused(self, resid: torch.Tensor, grad: Optional[torch.Tensor], iteration: int = 0, rank: int = -1,
                   events=None, stream=None) -> StepPlan:
        """accumulate + norms -> host planning -> selection + residual update, one C call
        (`deft_step`): all simulated workers in one launch (rank = -1) or one worker.
        The pointers of the buffers this object owns are marshalled once and reused: the call is made
        every step and the device waits for the host between its two kernels."""
        import ctypes
        if not hasattr(self, "_k_l"):
            self._k_l = np.empty(self.L, dtype=np.int64)
            self._bins = np.empty(self.L, dtype=np.int32)
            self._load = np.empty(self.N, dtype=np.float64)
            self._ls_h = np.ascontiguousarray(self.layer_start, dtype=np.int64)
            self._sum_k = ctypes.c_int64(0)
            vp = ctypes.c_void_p
            self._fixed = dict(
                ls_h=vp(self._ls_h.ctypes.data), ls_d=vp(self.layer_start_d.data_ptr()), norms_d=vp(self.norms_d.data_ptr()),
                norms_h=vp(self.norms_h.data_ptr()), k_l=vp(self._k_l.ctypes.data), sum_k=ctypes.byref(self._sum_k),
                bins=vp(self._bins.ctypes.data), load=vp(self._load.ctypes.data), plan_h=vp(self.plan_h.ctypes.data),
                plan_d=vp(self.plan_d.data_ptr()), val_d=vp(self.val_d.data_ptr()), idx_d=vp(self.idx_d.data_ptr()),
                ws=vp(self.ws.data_ptr()), ws_bytes=self.ws.numel() * self.ws.element_size(),
                out_cap=min(self.val_d.numel(), self.idx_d.numel()), plan_cap=self.plan_h.size,
                norms_h_ptr=self.norms_h.data_ptr())
        f = self._fixed
        if f["norms_h_ptr"] != self.norms_h.data_ptr():      # the caller swapped the host buffer for the norms
            f["norms_h"] = ctypes.c_void_p(self.norms_h.data_ptr())
            f["norms_h_ptr"] = self.norms_h.data_ptr()
        if resid.dtype != torch.float32 or not resid.is_cuda or not resid.is_contiguous() or resid.numel() != self.n_g:
            raise ValueError("resid: a contiguous float32 CUDA tensor of n_g elements")
        if grad is not None and (grad.dtype != torch.float32 or not grad.is_cuda or not grad.is_contiguous()
                                 or grad.numel() != self.n_g):
            raise ValueError("grad: a contiguous float32 CUDA tensor of n_g elements")
        ev = None
        if events is not None:
            flat = []
            for e in events:
                if e.cuda_event == 0:   # torch creates the handle lazily, on first record
                    e.record()
                flat.append(e.cuda_event)
            ev = (ctypes.c_void_p * 4)(*flat)
        st = torch.cuda.current_stream(self.device) if stream is None else stream
        status = deft.lib().deft_step(
            ctypes.c_void_p(resid.data_ptr()), None if grad is None else ctypes.c_void_p(grad.data_ptr()), self.n_g,
            f["ls_h"], f["ls_d"], self.L, self.N, int(self.k), int(self.mode), int(self.cost_model), int(iteration),
            int(rank), f["norms_d"], f["norms_h"], f["k_l"], f["sum_k"], f["bins"], f["load"], f["plan_h"],
            f["plan_cap"], f["plan_d"], f["val_d"], f["idx_d"], f["out_cap"], f["ws"], f["ws_bytes"], ev,
            ctypes.c_void_p(st.cuda_stream))
        deft._check("deft_step", status, allow_warn=True)
        n_layers, elems, rank_k, out_off = deft.deft_plan_rank_table(self.plan_h, self.N)
        off = np.empty(self.N + 1, dtype=np.int64)
        off[:-1] = out_off
        off[-1] = out_off[-1] + rank_k[-1]
        return StepPlan(self._k_l.copy(), int(self._sum_k.value), self._bins.copy(), self._load.copy(), n_layers, rank_k,
                        elems, off, self.plan_h)

    # -- the whole step for all simulated ranks ---------------------------------------------
    def step(self, resid: torch.Tensor, grad: Optional[torch.Tensor], iteration: int = 0, events=None,
             per_rank: bool = False):
        """accumulate + norms -> plan -> (selection, residual update) for every rank.  Returns the plan and,
        per rank, views of its selected (values, indices)."""
        norms = self.layer_norms(resid, grad)
        plan = self.plan(norms, iteration)
        self.select_and_update_all(resid, plan, events, per_rank)
        off = plan.rank_out_off
        outs = [(self.val_d[int(off[r]):int(off[r + 1])], self.idx_d[int(off[r]):int(off[r + 1])])
                for r in range(self.N)]
        return plan, outs
