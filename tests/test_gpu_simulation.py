"""Algorithm 1 for N simulated workers with DIFFERENT gradients: the library-driven simulation
against the same loop composed from oracle functions (density, Eq. 2 error, union, averages)."""
import math

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


def _worker_grads(w, N, t):
    base = w.gradient(t)
    out = []
    for r in range(N):
        rng = np.random.default_rng(np.random.SeedSequence([w.seed, 0x51, t, r]))
        noise = rng.standard_normal(w.n_g, dtype=np.float32) * np.float32(0.5) * np.abs(base)
        out.append((base + noise).astype(np.float32))
    return out


def _oracle_step(kind, e, grads, start, size, k, N, t, threshold):
    """Algorithm 1 lines 5-12 for all workers, from oracle pieces.  e: list of residuals (in place)."""
    norms = []
    for r in range(N):
        oracle.accumulate(e[r], grads[r])
        norms.append(oracle.layer_norms(e[r], start))
    if kind == "deft":
        k_l, s = oracle.allocate_k(norms[0], size, k, oracle.MODE_EXACT)
        bins, _ = oracle.partition(size, k_l, N)
        parts = [oracle.select_rank(e[r], start, k_l, oracle.my_layers(bins, t, r, N))[1] for r in range(N)]
        union = np.concatenate(parts)                      # rank order, as the ranks' slabs lie side by side
        assert np.unique(union).size == union.size == s
    elif kind == "topk":
        union = oracle.index_union(np.concatenate([oracle.topk(e[r], k)[1] for r in range(N)]))
    elif kind == "cltk":
        union = oracle.topk(e[oracle.clt_leader(t, N)], k)[1]
    else:
        union = oracle.index_union(np.concatenate([oracle.threshold_select(e[r], threshold)[1] for r in range(N)]))
    mean = np.zeros(union.size, dtype=np.float32)
    for r in range(N):
        oracle.sum_into(mean, oracle.gather_update(e[r], union))
    oracle.average(mean, N)
    err = oracle.error_eq2([oracle.vector_norm(e[r]) for r in range(N)])
    return union, mean, union.size / e[0].size, err


@pytest.mark.parametrize("kind", ["deft", "topk", "cltk", "hard_threshold"])
def test_multi_worker_simulation_matches_oracle_loop(deft, kind):
    from paper_2307_03500_b200.simulate import MultiWorkerSim
    w = W.tiny()
    N = w.n_workers
    thr = 0.05
    sim = MultiWorkerSim(w.sizes, N, w.density, kind, threshold=thr)
    start, _ = oracle.split_layers(w.sizes, N)
    size = np.diff(start)
    e_cpu = [np.zeros(w.n_g, dtype=np.float32) for _ in range(N)]
    dens = []
    for t in range(4):
        grads = _worker_grads(w, N, t)
        d_gpu, err_gpu = sim.step([torch.from_numpy(g).cuda() for g in grads])
        union, mean, d_cpu, err_cpu = _oracle_step(kind, e_cpu, grads, start, size, sim.k, N, t, thr)
        assert d_gpu == d_cpu
        assert np.array_equal(sim.last_union.cpu().numpy(), union)
        assert sim.last_mean.cpu().numpy().tobytes() == mean.tobytes()
        for r in range(N):
            assert sim.e[r].cpu().numpy().tobytes() == e_cpu[r].tobytes()
        assert abs(err_gpu - err_cpu) <= 1e-5 * err_cpu
        dens.append(d_gpu)
    if kind in ("deft", "cltk"):
        assert all(abs(d - sim.k / w.n_g) < 1e-12 for d in dens)          # no build-up: density as set
    if kind == "topk":
        assert all(d > sim.k / w.n_g for d in dens)                       # build-up: union larger than k
        assert all(d <= N * sim.k / w.n_g for d in dens)
