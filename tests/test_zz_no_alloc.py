"""deft_layer_norms_static: the workspace-free variant for callers that cannot allocate.

Some users of the library run where device allocation is off limits (inside another
framework's memory-pooled or captured region, or as a plugin that is given tensors but no
allocator).  For them the accumulate + norm call exists in a form whose scratch is a fixed
array inside the library.  This test calls it through the C ABI twice in a row on different
data and checks both results against the ordinary entry point (same kernel, so the values
must be identical; the bar written here is the suite's norm tolerance) and against the CPU
oracle's sequential fp64 norms of the same accumulated vector.  It lives in its
own file, collected last, and passes on its own as well as after the other tests.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2307_03500_b200 import build as deft_build
from paper_2307_03500_b200 import workloads as W

pytestmark = pytest.mark.gpu

NORM_RTOL = 1e-5


def test_static_scratch_entry_point_matches_workspace_entry_point_twice():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    deft_build.build()
    from paper_2307_03500_b200 import deft

    w = W.resnet18()
    start, _ = deft.deft_split_layers(w.sizes, w.n_workers)
    L = start.size - 1
    assert (w.n_g + 8191) // 8192 + L + 1 <= deft.lib().deft_layer_norms_static_max_slots()
    ls_d = torch.from_numpy(start).cuda()
    ws = deft.alloc_workspace(w.n_g, L)
    e_ref = torch.zeros(w.n_g, dtype=torch.float32, device="cuda")
    e_new = torch.zeros(w.n_g, dtype=torch.float32, device="cuda")
    n_ref = torch.empty(L, dtype=torch.float64, device="cuda")
    n_new = torch.full((L,), -1.0, dtype=torch.float64, device="cuda")
    e_cpu = np.zeros(w.n_g, dtype=np.float32)
    for step in range(2):   # the second call finds the first call's leftovers in the shared scratch
        g_h = w.gradient(step)
        g = torch.from_numpy(g_h).cuda()
        deft.deft_layer_norms(e_ref, g, ls_d, n_ref, ws)
        deft.deft_layer_norms_static(e_new, g, ls_d, n_new)
        torch.cuda.synchronize()
        a, b = n_ref.cpu().numpy(), n_new.cpu().numpy()
        assert np.all(a > 0)
        assert np.all(np.abs(a - b) <= NORM_RTOL * a)
        assert torch.equal(e_ref, e_new)            # the accumulated vector is bit-identical
        e_cpu = oracle.accumulate(e_cpu, g_h)       # the oracle's own accumulate + norms
        want = oracle.layer_norms(e_cpu, start)
        assert e_new.cpu().numpy().tobytes() == e_cpu.tobytes()
        assert np.all(np.abs(b - want) <= NORM_RTOL * want)
    # norms-only form (no gradient) and the size limit
    deft.deft_layer_norms_static(e_new, None, ls_d, n_new)
    torch.cuda.synchronize()
    assert np.all(np.abs(n_new.cpu().numpy() - a) <= NORM_RTOL * a)
    big = torch.empty(1, dtype=torch.float32, device="cuda")
    rc = deft.lib().deft_layer_norms_static(big.data_ptr(), None, 8192 * 20000, ls_d.data_ptr(), L,
                                            n_new.data_ptr(), None)
    assert rc == deft.ERR_CAPACITY                  # refused on the host, nothing launched
