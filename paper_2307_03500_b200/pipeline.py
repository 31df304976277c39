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
    rank_layers: List[np.ndarray]   # per rank: ascending layer ids
    rank_k: np.ndarray         # int64[N]  entries each rank selects
    rank_elems: np.ndarray     # int64[N]  elements each rank scans
    rank_out_off: np.ndarray   # int64[N+1] offsets into the output slabs


class DeftStep:
    def __init__(self, tensor_sizes, n_workers: int, density: float, device="cuda:0",
                 mode: int = deft.MODE_EXACT, k: Optional[int] = None):
        self.device = torch.device(device)
        self.N = int(n_workers)
        self.mode = mode
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

    # -- step 1: accumulate + norms (device) ------------------------------------------------
    def layer_norms(self, resid: torch.Tensor, grad: Optional[torch.Tensor]) -> np.ndarray:
        deft.deft_layer_norms(resid, grad, self.layer_start_d, self.norms_d, self.ws)
        self.norms_h.copy_(self.norms_d, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        return self.norms_h.numpy()

    # -- steps 2 and 3: local k and bins (host) ---------------------------------------------
    def plan(self, norms: np.ndarray, iteration: int = 0) -> StepPlan:
        k_l, sum_k, _ = deft.deft_allocate_k(norms, self.layer_size, self.k, self.mode)
        bins, load = deft.deft_partition(self.layer_size, k_l, self.N)
        rank_layers = [deft.deft_bin_layers(bins, deft.deft_rank_bin(iteration, r, self.N)) for r in range(self.N)]
        rank_k = np.array([int(k_l[m].sum()) for m in rank_layers], dtype=np.int64)
        rank_elems = np.array([int(self.layer_size[m].sum()) for m in rank_layers], dtype=np.int64)
        off = np.zeros(self.N + 1, dtype=np.int64)
        np.cumsum(rank_k, out=off[1:])
        return StepPlan(k_l, sum_k, bins, load, rank_layers, rank_k, rank_elems, off)

    # -- step 4: selection + residual update for one rank (device) --------------------------
    def select_rank(self, acc: torch.Tensor, plan: StepPlan, rank: int):
        a, b = int(plan.rank_out_off[rank]), int(plan.rank_out_off[rank + 1])
        val, idx = self.val_d[a:b], self.idx_d[a:b]
        if b > a:
            deft.deft_select(acc, self.layer_start, plan.k_l, plan.rank_layers[rank], val, idx, self.ws)
        return val, idx

    def residual_update(self, acc: torch.Tensor, idx: torch.Tensor) -> None:
        deft.deft_residual_update(acc, idx, idx.numel())

    # -- the whole step for all simulated ranks ---------------------------------------------
    def step(self, resid: torch.Tensor, grad: Optional[torch.Tensor], iteration: int = 0):
        norms = self.layer_norms(resid, grad)
        plan = self.plan(norms, iteration)
        outs = []
        for r in range(self.N):
            val, idx = self.select_rank(resid, plan, r)
            outs.append((val, idx))
        # all ranks read the same accumulated vector, so zeroing starts after the last selection
        for val, idx in outs:
            self.residual_update(resid, idx)
        return plan, outs
