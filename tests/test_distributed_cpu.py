"""Algorithm 1 with one worker per process and real collectives (``distributed.DistributedWorker``),
run as two gloo ranks on CPU.

libdeft has no CPU path, so the device side of a worker is replaced here by stand-ins built from the
oracle (test infrastructure); the host planners are the library's own.  What is under test is the
exchange: the delegate's broadcast and its rotation, the padded all-gather and the rank order of the
gathered lists, the all-reduce and the 1/n, the all-gather for Eq. 2, and the reported communication
figure.  Every rank's results are compared with the same iterations run in one process from oracle
pieces (two workers: the sum of two floats does not depend on the order, so the bar is bit equality).
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2307_03500_b200 import deft
from paper_2307_03500_b200 import workloads as W

STEPS = 3
THRESHOLD = 0.05


class OracleOps:
    """CPU stand-in for ``distributed.LibdeftOps``: the same calls, answered by the oracle."""

    def __init__(self, tensor_sizes, n_workers, density):
        self.layer_start, _ = oracle.split_layers(tensor_sizes, n_workers)
        self.n_g = int(self.layer_start[-1])
        self.L = self.layer_start.size - 1
        self.k = max(max(1, int(np.floor(float(self.n_g) * density))), self.L)

    def new_residual(self):
        return torch.zeros(self.n_g, dtype=torch.float32)

    def layer_norms(self, e, g):
        oracle.accumulate(e.numpy(), g.numpy())
        return oracle.layer_norms(e.numpy(), self.layer_start)

    def select(self, e, k_l, my_layers):
        val, idx = oracle.select_rank(e.numpy(), self.layer_start, k_l, my_layers)
        return torch.from_numpy(val), torch.from_numpy(idx)

    def topk(self, e, k):
        val, idx = oracle.topk(e.numpy(), k)
        return torch.from_numpy(val), torch.from_numpy(idx)

    def threshold_select(self, e, threshold):
        val, idx = oracle.threshold_select(e.numpy(), threshold)
        return torch.from_numpy(val), torch.from_numpy(idx)

    def index_union(self, idx):
        return torch.from_numpy(oracle.index_union(idx.numpy()))

    def gather_update(self, e, union):
        return torch.from_numpy(oracle.gather_update(e.numpy(), union.numpy()))

    def average(self, total, n_workers):
        oracle.average(total.numpy(), n_workers)

    def vector_norm(self, e):
        return oracle.vector_norm(e.numpy())


def _worker_grad(w, t, r):
    base = w.gradient(t)
    rng = np.random.default_rng(np.random.SeedSequence([w.seed, 0x51, t, r]))
    noise = rng.standard_normal(w.n_g, dtype=np.float32) * np.float32(0.5) * np.abs(base)
    return (base + noise).astype(np.float32)


def _single_process_reference(kind, w, N):
    """The same iterations from oracle pieces in one process.  The delegate of iteration t is worker t % N."""
    start, _ = oracle.split_layers(w.sizes, N)
    size = np.diff(start)
    k = max(max(1, int(np.floor(float(w.n_g) * w.density))), size.size)
    e = [np.zeros(w.n_g, dtype=np.float32) for _ in range(N)]
    out = []
    for t in range(STEPS):
        norms = []
        for r in range(N):
            oracle.accumulate(e[r], _worker_grad(w, t, r))
            norms.append(oracle.layer_norms(e[r], start))
        if kind == "deft":
            k_l, _ = oracle.allocate_k(norms[t % N], size, k, oracle.MODE_EXACT)
            bins, _ = oracle.partition(size, k_l, N)
            parts = [oracle.select_rank(e[r], start, k_l, oracle.my_layers(bins, t, r, N))[1] for r in range(N)]
            union = np.concatenate(parts)
            max_k = max(p.size for p in parts)
        elif kind == "topk":
            union = oracle.index_union(np.concatenate([oracle.topk(e[r], k)[1] for r in range(N)]))
            max_k = k
        elif kind == "cltk":
            union = oracle.topk(e[oracle.clt_leader(t, N)], k)[1]
            max_k = k
        else:
            parts = [oracle.threshold_select(e[r], THRESHOLD)[1] for r in range(N)]
            union = oracle.index_union(np.concatenate(parts))
            max_k = max(p.size for p in parts)
        mean = np.zeros(union.size, dtype=np.float32)
        for r in range(N):
            oracle.sum_into(mean, oracle.gather_update(e[r], union))
        oracle.average(mean, N)
        err = oracle.error_eq2([oracle.vector_norm(e[r]) for r in range(N)])
        out.append((union.copy(), mean.copy(), union.size / w.n_g, err, max_k, [x.copy() for x in e]))
    return out


def _rank_main(rank, world, port, kind, result_dir):
    from paper_2307_03500_b200.distributed import DistributedWorker
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    try:
        w = W.tiny()
        ops = OracleOps(w.sizes, world, w.density)
        worker = DistributedWorker(w.sizes, w.density, kind, threshold=THRESHOLD, ops=ops)
        ref = _single_process_reference(kind, w, world)
        for t in range(STEPS):
            rep = worker.step(torch.from_numpy(_worker_grad(w, t, rank)))
            union, mean, dens, err, max_k, e_ref = ref[t]
            assert np.array_equal(rep.union.numpy(), union), "union, step %d" % t
            assert rep.mean.numpy().tobytes() == mean.tobytes(), "averaged values, step %d" % t
            assert rep.density == dens and rep.max_rank_k == max_k
            assert abs(rep.error - err) <= 1e-12 * err
            assert worker.e.numpy().tobytes() == e_ref[rank].tobytes(), "residual, step %d" % t
            if kind in ("deft", "cltk"):
                assert rep.density == ops.k / ops.n_g                    # no build-up
            if kind == "topk":
                assert ops.k / ops.n_g < rep.density <= world * ops.k / ops.n_g   # build-up, bounded by N * k
        open(os.path.join(result_dir, "ok.%d" % rank), "w").write("ok")
    finally:
        dist.destroy_process_group()


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


@pytest.mark.parametrize("kind", ["deft", "topk", "cltk", "hard_threshold"])
def test_two_gloo_ranks_match_the_single_process_loop(kind, tmp_path):
    deft.lib()   # the host planners are the library's own: it must load without a GPU
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), kind, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        assert os.path.exists(os.path.join(str(tmp_path), "ok.%d" % r))
