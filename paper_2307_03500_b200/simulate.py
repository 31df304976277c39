"""Algorithm 1 (distributed SGD with error feedback) for N workers simulated on ONE device.

Every worker keeps its own residual ``e_r`` and receives its own gradient; the collectives of
Algorithm 1 (all-gather of indices, all-reduce of values) become plain buffer sharing because all
workers live in one address space (``distributed.py`` is the same loop with one process per worker and
real collectives).  Orchestration only: every numeric step — the union of the index lists, the sum and
the average of the contributions, the error of Eq. 2 — is a libdeft call.

Sparsifiers (Section 3 and Section 4 of the paper):
  ``deft``            a delegate worker runs Algorithms 3 and 4 on its own norms and shares k_l and
                      the bins; worker r selects its layers from ITS accumulated vector (Algorithm 5);
                      the union has exactly sum(k_l) entries (no build-up)
  ``topk``            every worker selects its own top k; the union grows with N (gradient build-up)
  ``cltk``            the iteration's leader selects its top k; everybody uses the leader's indices
  ``hard_threshold``  every worker selects the entries above a fixed threshold

One step returns the actual density (Section 5.2: globally selected entries / n_g) and the error of
Eq. 2 (mean over workers of the L2 norm of the residual after the update).
"""
from __future__ import annotations

from typing import List, Optional

import numpy as np
import torch

from . import deft
from .pipeline import DeftStep


class MultiWorkerSim:
    def __init__(self, tensor_sizes, n_workers: int, density: float, sparsifier: str = "deft",
                 threshold: Optional[float] = None, device="cuda:0", delegate: int = 0):
        if sparsifier not in ("deft", "topk", "cltk", "hard_threshold"):
            raise ValueError(sparsifier)
        if sparsifier == "hard_threshold" and threshold is None:
            raise ValueError("hard_threshold needs a threshold")
        self.kind = sparsifier
        self.N = int(n_workers)
        self.threshold = threshold
        self.delegate = int(delegate)
        self.ds = DeftStep(tensor_sizes, n_workers, density, device=device)
        self.n_g, self.k = self.ds.n_g, self.ds.k
        dev = self.ds.device
        self.e: List[torch.Tensor] = [torch.zeros(self.n_g, dtype=torch.float32, device=dev) for _ in range(self.N)]
        per_worker = self.n_g if sparsifier == "hard_threshold" else self.k + self.ds.L + 64
        self.val = torch.empty(per_worker, dtype=torch.float32, device=dev)
        self.idx = torch.empty(per_worker, dtype=torch.int64, device=dev)
        # what the all-gather would deliver: every worker's list, side by side
        gathered = per_worker if sparsifier in ("deft", "cltk") else min(per_worker * self.N, self.n_g * self.N)
        self.gathered = torch.empty(gathered, dtype=torch.int64, device=dev)
        self.union = torch.empty(min(self.n_g, gathered), dtype=torch.int64, device=dev)
        self.contrib = torch.empty(self.union.numel(), dtype=torch.float32, device=dev)
        self.total = torch.empty(self.union.numel(), dtype=torch.float32, device=dev)
        self.count_d = torch.zeros(1, dtype=torch.int64, device=dev)
        self.norm_d = torch.zeros(1, dtype=torch.float64, device=dev)
        self.ws_union = torch.empty(deft.deft_union_workspace_bytes(self.n_g), dtype=torch.uint8, device=dev)
        self.ws_norm = torch.empty(deft.deft_vector_norm_workspace_bytes(self.n_g), dtype=torch.uint8, device=dev)
        self.iteration = 0
        self.last_union: Optional[torch.Tensor] = None
        self.last_mean: Optional[torch.Tensor] = None
        self.max_rank_k = 0

    # -- Eq. 2 -------------------------------------------------------------------------------
    def error(self) -> float:
        errs = np.empty(self.N, dtype=np.float64)
        for r in range(self.N):
            deft.deft_vector_norm(self.e[r], self.norm_d, self.ws_norm)
            errs[r] = float(self.norm_d.item())
        return deft.deft_error_eq2(errs)

    def _union_of(self, count: int) -> torch.Tensor:
        """Line 7: the set of the gathered indices (``self.gathered[:count]``)."""
        deft.deft_index_union(self.gathered, count, self.n_g, self.union, self.count_d, self.ws_union)
        return self.union[:int(self.count_d.item())]

    # -- Algorithm 1, lines 5-12, for all workers ---------------------------------------------
    def step(self, grads: List[torch.Tensor]):
        """grads[r]: worker r's gradient (already scaled by the learning rate).  Returns
        (actual density, error after the update)."""
        ds, N, t = self.ds, self.N, self.iteration
        norms_all = []
        for r in range(N):                                         # line 5: acc_r = e_r + g_r (in place)
            norms_all.append(ds.layer_norms(self.e[r], grads[r]).copy())
        if self.kind == "deft":
            plan = ds.plan(norms_all[self.delegate], t)            # Algorithms 3 + 4 on the delegate, shared
            for r in range(N):                                     # line 6: worker r, its layers, its vector
                ds.select_rank(self.e[r], plan, r)
            union = ds.idx_d[:plan.sum_k]                          # line 7: all-gather (ranks wrote side by side);
            self.max_rank_k = int(plan.rank_k.max())               # disjoint layers: the lists ARE the set
        elif self.kind == "topk":
            for r in range(N):
                deft.deft_topk_baseline(self.e[r], self.k, self.val[:self.k], self.gathered[r * self.k:(r + 1) * self.k], ds.ws)
            union = self._union_of(N * self.k)                     # line 7
            self.max_rank_k = self.k
        elif self.kind == "cltk":
            leader = deft.deft_clt_leader(t, N)
            deft.deft_topk_baseline(self.e[leader], self.k, self.val[:self.k], self.idx[:self.k], ds.ws)
            union = self.idx[:self.k]
            self.max_rank_k = self.k
        else:
            at = 0
            self.max_rank_k = 0
            for r in range(N):
                deft.deft_threshold_select(self.e[r], self.threshold, self.val, self.idx, self.count_d, ds.ws)
                n = int(self.count_d.item())
                if at + n > self.gathered.numel():
                    grown = torch.empty(max(at + n, 2 * self.gathered.numel()), dtype=torch.int64, device=ds.device)
                    grown[:at].copy_(self.gathered[:at])
                    self.gathered = grown
                self.gathered[at:at + n].copy_(self.idx[:n])
                at += n
                self.max_rank_k = max(self.max_rank_k, n)
            union = self._union_of(at)
        m = int(union.numel())
        if m > self.contrib.numel():
            self.contrib = torch.empty(m, dtype=torch.float32, device=ds.device)
            self.total = torch.empty(m, dtype=torch.float32, device=ds.device)
        total = self.total[:m]
        total.zero_()
        for r in range(N):                                         # lines 8-12: values at the union, cleared
            if m:
                deft.deft_gather_update(self.e[r], union, m, self.contrib)
                deft.deft_sum_into(total, self.contrib, m)         # line 9: the all-reduce's sum, in rank order
        deft.deft_average(total, m, N)                             # ... and its 1/n
        self.last_union, self.last_mean = union, total
        self.iteration += 1
        return m / self.n_g, self.error()
