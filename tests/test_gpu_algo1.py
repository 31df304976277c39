"""The device calls around the sparsifier that a multi-worker Algorithm 1 needs (union of the gathered
indices, sum and average of the contributions, Eq. 2's norm) against the oracle, and the one-process-
per-worker loop on a single GPU (one NCCL rank) against the same iterations from oracle pieces."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2307_03500_b200 import build as deft_build
from paper_2307_03500_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def deft():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    deft_build.build()
    from paper_2307_03500_b200 import deft as d
    d.lib()
    return d


@pytest.mark.parametrize("n_g,count", [(1, 1), (31, 5), (32, 40), (33, 33), (100003, 5000), (40_000_000, 3_000_000)])
def test_index_union_matches_oracle(deft, n_g, count):
    rng = np.random.default_rng(n_g)
    idx = rng.integers(0, n_g, size=count).astype(np.int64)
    if count > 10:
        idx[:5] = [0, n_g - 1, n_g - 1, 0, n_g // 2]                 # edges and duplicates
    want = oracle.index_union(idx)
    idx_d = torch.from_numpy(idx).cuda()
    out = torch.full((want.size + 8,), -7, dtype=torch.int64, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int64, device="cuda")
    ws = torch.empty(deft.deft_union_workspace_bytes(n_g), dtype=torch.uint8, device="cuda")
    for _ in range(2):                                               # the workspace is reusable as it is
        deft.deft_index_union(idx_d, count, n_g, out, cnt, ws)
        torch.cuda.synchronize()
        assert int(cnt.item()) == want.size
        assert out[:want.size].cpu().numpy().tolist() == want.tolist()
        assert torch.all(out[want.size:] == -7)
    small = torch.full((3,), -7, dtype=torch.int64, device="cuda")   # too small an output: counted, not written
    deft.deft_index_union(idx_d, count, n_g, small, cnt, ws)
    torch.cuda.synchronize()
    assert int(cnt.item()) == want.size and small.cpu().numpy().tolist()[:min(3, want.size)] == want[:3].tolist()


def test_sum_average_and_vector_norm_match_oracle(deft):
    rng = np.random.default_rng(31)
    for n in (1, 1000, 1_000_003):
        a = rng.standard_normal(n).astype(np.float32)
        b = (rng.standard_normal(n) * 1e-3).astype(np.float32)
        a_d, b_d = torch.from_numpy(a.copy()).cuda(), torch.from_numpy(b).cuda()
        deft.deft_sum_into(a_d, b_d, n)
        deft.deft_average(a_d, n, 7)
        torch.cuda.synchronize()
        want = oracle.average(oracle.sum_into(a.copy(), b), 7)
        assert a_d.cpu().numpy().tobytes() == want.tobytes()
        x = rng.standard_normal(n).astype(np.float32)
        x_d = torch.from_numpy(x).cuda()
        norm = torch.zeros(1, dtype=torch.float64, device="cuda")
        ws = torch.empty(deft.deft_vector_norm_workspace_bytes(n), dtype=torch.uint8, device="cuda")
        deft.deft_vector_norm(x_d, norm, ws)
        torch.cuda.synchronize()
        ref = oracle.vector_norm(x)
        assert abs(float(norm.item()) - ref) <= 1e-5 * ref
        assert x_d.cpu().numpy().tobytes() == x.tobytes()            # nothing written
    assert deft.deft_error_eq2([1.0, 2.0, 6.0]) == oracle.error_eq2([1.0, 2.0, 6.0]) == 3.0


def test_one_process_per_worker_loop_on_one_gpu(deft):
    """``distributed.DistributedWorker`` with the library's own device calls, as the only rank of an NCCL
    group: the collectives degenerate, everything else is the path N GPUs would run."""
    import torch.distributed as dist
    from paper_2307_03500_b200.distributed import DistributedWorker
    from tests.test_distributed_cpu import _single_process_reference, _worker_grad, STEPS, THRESHOLD
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29533")
    dist.init_process_group("nccl", rank=0, world_size=1)
    try:
        w = W.tiny()
        for kind in ("deft", "topk", "hard_threshold"):
            worker = DistributedWorker(w.sizes, w.density, kind, threshold=THRESHOLD, device="cuda:0")
            ref = _single_process_reference(kind, w, 1)
            for t in range(STEPS):
                rep = worker.step(torch.from_numpy(_worker_grad(w, t, 0)).cuda())
                union, mean, dens, err, max_k, e_ref = ref[t]
                assert np.array_equal(rep.union.cpu().numpy(), union)
                assert rep.mean.cpu().numpy().tobytes() == mean.tobytes()
                assert rep.density == dens and rep.max_rank_k == max_k
                assert abs(rep.error - err) <= 1e-5 * err
                assert worker.e.cpu().numpy().tobytes() == e_ref[0].tobytes()
    finally:
        dist.destroy_process_group()
