"""Algorithm 1 (distributed SGD with error feedback) with ONE worker per process and real collectives.

``simulate.MultiWorkerSim`` replays N workers on one device; this module is the same loop as it runs
on N GPUs: every process owns one worker's residual, computes on its own device through libdeft, and
talks to the others through ``torch.distributed`` (NCCL between GPUs; gloo on CPU for the tests).
The collectives are the ones Algorithm 1 and Algorithm 4 name:

  * broadcast from the iteration's delegate (worker ``iteration % N``, Algorithm 4 lines 1-2 and 19) of
    what it computed from ITS norms: the local k of every layer (Algorithm 3) and the bin of every layer
    (Algorithm 4) — 12 bytes per layer;
  * all-gather of the selected indices (Algorithm 1 line 7), padded to the largest list: the list
    sizes follow from k_l and the bins, which every worker holds, so no sizes are exchanged for DEFT;
  * all-reduce (sum) of the workers' values at the selected indices (line 9), then the 1/n;
  * all-gather of one double per worker for the error of Eq. 2.

Orchestration only.  Every numeric step is a call on an ``ops`` object: ``LibdeftOps`` (the default)
issues libdeft calls on the process's GPU and fails loudly without one; the CPU-side test of this
module plugs in stand-ins for the device calls so that the exchange pattern (padding, delegate
rotation, rank order of the gathered lists, the communication-volume figure) is exercised with gloo.

Reported per step: the actual density (Section 5.2: globally selected entries / n_g), the error of
Eq. 2, and max_i sum k_x, the per-worker index count that the all-gather's volume term of Section 5.4
(2(n - 1) max_i sum k_x beta) is made of.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch
import torch.distributed as dist

from . import deft


@dataclass
class StepReport:
    density: float          # |union of the selected indices| / n_g
    error: float            # Eq. 2
    max_rank_k: int         # max over workers of the indices a worker contributes (communication volume term)
    union: torch.Tensor     # int64 indices that took part in the update (rank order for DEFT, ascending otherwise)
    mean: torch.Tensor      # fp32 averaged values at those indices


class LibdeftOps:
    """The device side of one worker: libdeft calls on this process's GPU."""

    def __init__(self, tensor_sizes, n_workers: int, density: float, device):
        from .pipeline import DeftStep
        if not torch.cuda.is_available():
            raise RuntimeError("LibdeftOps needs a CUDA device: libdeft has no CPU path")
        self.ds = DeftStep(tensor_sizes, n_workers, density, device=device)
        self.device = self.ds.device
        self.n_g, self.L, self.k = self.ds.n_g, self.ds.L, self.ds.k
        self.layer_start = self.ds.layer_start
        cap = self.n_g
        self._val = torch.empty(self.k + self.L + 64, dtype=torch.float32, device=self.device)
        self._idx = torch.empty(self.k + self.L + 64, dtype=torch.int64, device=self.device)
        self._count = torch.zeros(1, dtype=torch.int64, device=self.device)
        self._norm = torch.zeros(1, dtype=torch.float64, device=self.device)
        self._ws_union = torch.empty(deft.deft_union_workspace_bytes(self.n_g), dtype=torch.uint8, device=self.device)
        self._ws_norm = torch.empty(deft.deft_vector_norm_workspace_bytes(self.n_g), dtype=torch.uint8, device=self.device)
        self._union = torch.empty(min(cap, (self.k + self.L + 64) * n_workers), dtype=torch.int64, device=self.device)

    def new_residual(self) -> torch.Tensor:
        return torch.zeros(self.n_g, dtype=torch.float32, device=self.device)

    def layer_norms(self, e, g) -> np.ndarray:
        return self.ds.layer_norms(e, g).copy()

    def select(self, e, k_l: np.ndarray, my_layers: np.ndarray):
        n = int(k_l[my_layers].sum()) if my_layers.size else 0
        if n:
            deft.deft_select(e, self.layer_start, k_l, my_layers, self._val[:n], self._idx[:n], self.ds.ws)
        return self._val[:n], self._idx[:n]

    def topk(self, e, k: int):
        deft.deft_topk_baseline(e, k, self._val[:k], self._idx[:k], self.ds.ws)
        return self._val[:k], self._idx[:k]

    def threshold_select(self, e, threshold: float):
        val = torch.empty(self.n_g, dtype=torch.float32, device=self.device)
        idx = torch.empty(self.n_g, dtype=torch.int64, device=self.device)
        deft.deft_threshold_select(e, threshold, val, idx, self._count, self.ds.ws)
        n = int(self._count.item())
        return val[:n], idx[:n]

    def index_union(self, idx: torch.Tensor) -> torch.Tensor:
        if idx.numel() > self._union.numel():
            self._union = torch.empty(min(self.n_g, idx.numel()), dtype=torch.int64, device=self.device)
        deft.deft_index_union(idx, idx.numel(), self.n_g, self._union, self._count, self._ws_union)
        return self._union[:int(self._count.item())]

    def gather_update(self, e, union: torch.Tensor) -> torch.Tensor:
        out = torch.empty(union.numel(), dtype=torch.float32, device=self.device)
        deft.deft_gather_update(e, union, union.numel(), out)
        return out

    def average(self, total: torch.Tensor, n_workers: int) -> None:
        deft.deft_average(total, total.numel(), n_workers)

    def vector_norm(self, e) -> float:
        deft.deft_vector_norm(e, self._norm, self._ws_norm)
        return float(self._norm.item())


class DistributedWorker:
    """Worker ``dist.get_rank()`` of ``dist.get_world_size()``: one Algorithm 1 iteration per ``step``."""

    def __init__(self, tensor_sizes, density: float, sparsifier: str = "deft", threshold: Optional[float] = None,
                 ops=None, device=None, group=None, mode: int = deft.MODE_EXACT):
        if sparsifier not in ("deft", "topk", "cltk", "hard_threshold"):
            raise ValueError(sparsifier)
        if sparsifier == "hard_threshold" and threshold is None:
            raise ValueError("hard_threshold needs a threshold")
        self.kind, self.threshold, self.group, self.mode = sparsifier, threshold, group, mode
        self.rank, self.N = dist.get_rank(group), dist.get_world_size(group)
        self.ops = ops if ops is not None else LibdeftOps(tensor_sizes, self.N, density, device)
        self.n_g, self.L, self.k = self.ops.n_g, self.ops.L, self.ops.k
        self.layer_start = np.asarray(self.ops.layer_start, dtype=np.int64)
        self.layer_size = np.diff(self.layer_start)
        self.e = self.ops.new_residual()
        self.iteration = 0

    # Algorithm 4 lines 1-2 and 19: the delegate's k_l and bins reach every worker
    def _shared_plan(self, norms: np.ndarray):
        delegate = self.iteration % self.N
        buf = torch.zeros(2 * self.L, dtype=torch.int64)
        if self.rank == delegate:
            k_l, _, _ = deft.deft_allocate_k(norms, self.layer_size, self.k, self.mode)
            bins, _ = deft.deft_partition(self.layer_size, k_l, self.N)
            buf[:self.L] = torch.from_numpy(np.asarray(k_l, dtype=np.int64))
            buf[self.L:] = torch.from_numpy(np.asarray(bins, dtype=np.int64))
        buf = buf.to(self.e.device)
        dist.broadcast(buf, src=delegate, group=self.group)
        host = buf.cpu().numpy()
        return host[:self.L].copy(), host[self.L:].astype(np.int32)

    def _all_gather_padded(self, idx: torch.Tensor, counts: List[int]) -> List[torch.Tensor]:
        """Every worker's list (``counts[r]`` entries from worker r), via one equal-sized all-gather."""
        width = max(max(counts), 1)
        mine = torch.zeros(width, dtype=torch.int64, device=idx.device)
        mine[:idx.numel()] = idx
        out = [torch.empty(width, dtype=torch.int64, device=idx.device) for _ in range(self.N)]
        dist.all_gather(out, mine, group=self.group)
        return [out[r][:counts[r]] for r in range(self.N)]

    def _counts(self, n_mine: int) -> List[int]:
        t = torch.zeros(self.N, dtype=torch.int64, device=self.e.device)
        t[self.rank] = n_mine
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=self.group)
        return [int(x) for x in t.cpu().tolist()]

    def step(self, grad) -> StepReport:
        """grad: this worker's gradient (already scaled by the learning rate), on the worker's device."""
        ops, N, t = self.ops, self.N, self.iteration
        norms = ops.layer_norms(self.e, grad)                                  # line 5 (+ the norms of Section 4.2)
        if self.kind == "deft":
            k_l, bins = self._shared_plan(norms)
            my = deft.deft_bin_layers(bins, deft.deft_rank_bin(t, self.rank, N))
            _, idx = ops.select(self.e, k_l, my)                               # line 6
            counts = [int(k_l[deft.deft_bin_layers(bins, deft.deft_rank_bin(t, r, N))].sum()) for r in range(N)]
            union = torch.cat(self._all_gather_padded(idx, counts))            # line 7: disjoint lists ARE the set
        elif self.kind == "topk":
            _, idx = ops.topk(self.e, self.k)
            counts = [self.k] * N
            union = ops.index_union(torch.cat(self._all_gather_padded(idx, counts)))
        elif self.kind == "cltk":
            leader = deft.deft_clt_leader(t, N)
            idx = torch.zeros(self.k, dtype=torch.int64, device=self.e.device)
            if self.rank == leader:
                idx.copy_(ops.topk(self.e, self.k)[1])
            dist.broadcast(idx, src=leader, group=self.group)
            counts = [self.k if r == leader else 0 for r in range(N)]
            union = idx
        else:
            _, idx = ops.threshold_select(self.e, self.threshold)
            counts = self._counts(int(idx.numel()))
            union = ops.index_union(torch.cat(self._all_gather_padded(idx, counts)))
        total = ops.gather_update(self.e, union)                               # lines 8, 11-12: own values, then cleared
        if union.numel():
            dist.all_reduce(total, op=dist.ReduceOp.SUM, group=self.group)     # line 9
        ops.average(total, N)
        errs = torch.zeros(N, dtype=torch.float64, device=self.e.device)      # Eq. 2
        errs[self.rank] = ops.vector_norm(self.e)
        dist.all_reduce(errs, op=dist.ReduceOp.SUM, group=self.group)
        self.iteration += 1
        return StepReport(union.numel() / self.n_g, deft.deft_error_eq2(errs.cpu().numpy()), max(counts), union, total)
