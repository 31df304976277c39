"""Parity of the comparison sparsifiers (Section 3: hard threshold, CLT-k) with the oracle."""
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


def _threshold(deft, x, lam, cap=None, zero=False):
    acc_d = torch.from_numpy(x).cuda()
    ws = deft.alloc_workspace(x.size, 1)
    want_val, want_idx = oracle.threshold_select(x, lam)
    cap = want_idx.size if cap is None else cap
    val_d = torch.full((cap + 4,), 7.0, dtype=torch.float32, device="cuda")
    idx_d = torch.full((cap + 4,), -7, dtype=torch.int64, device="cuda")
    cnt_d = torch.full((1,), -1, dtype=torch.int64, device="cuda")
    deft.deft_threshold_select(acc_d, lam, val_d[:cap] if cap else None, idx_d[:cap] if cap else None, cnt_d, ws,
                               zero_selected=zero)
    torch.cuda.synchronize()
    assert int(cnt_d.item()) == want_idx.size                      # the total, whatever the capacity
    m = min(cap, want_idx.size)
    assert np.array_equal(idx_d[:m].cpu().numpy(), want_idx[:m])   # the first `cap` in index order
    assert val_d[:m].cpu().numpy().tobytes() == want_val[:m].tobytes()
    assert torch.all(val_d[max(m, cap):] == 7.0) and torch.all(idx_d[max(m, cap):] == -7)
    if m < cap:
        assert torch.all(val_d[m:cap] == 7.0)
    after = acc_d.cpu().numpy()
    if zero:
        want = x.copy()
        want[want_idx] = 0.0
        assert after.tobytes() == want.tobytes()
    else:
        assert after.tobytes() == x.tobytes()


@pytest.mark.parametrize("kind", ["gauss", "wide_exponent", "few_values", "mostly_zero", "signed_zero", "denormal",
                                  "all_equal", "all_zero", "outlier"])
def test_threshold_select_adversarial(deft, kind):
    x = W.adversarial_vector(kind, 300_007, seed=31)
    for lam in (0.0, 0.25, 1.0, 2.5, 1e30):
        _threshold(deft, x, lam)


@pytest.mark.parametrize("n", [1, 2047, 2049, 4097, 1_000_003])
def test_threshold_select_sizes_capacity_and_zeroing(deft, n):
    x = W.adversarial_vector("gauss", n, seed=n % 89)
    _threshold(deft, x, 1.0)
    _threshold(deft, x, 0.5, zero=True)
    _threshold(deft, x, 0.1, cap=0)                     # count only
    _threshold(deft, x, 0.1, cap=max(1, n // 50), zero=True)   # fewer slots than selected entries
    _threshold(deft, x, 10.0)                           # nothing selected


def test_threshold_select_large_vector_round_robin_split(deft):
    n = 21_000_003
    x = W.adversarial_vector("gauss", n, seed=33)
    x[2_000_000:2_400_000] *= np.float32(40.0)         # a hot region: many entries from few tiles
    _threshold(deft, x, 3.0, zero=True)                 # ~0.3 % + the hot region
    _threshold(deft, x, 0.01)                           # nearly everything (every CTA spills)


def test_threshold_rejects_bad_arguments(deft):
    x = torch.zeros(100, dtype=torch.float32, device="cuda")
    ws = deft.alloc_workspace(100, 1)
    cnt = torch.zeros(1, dtype=torch.int64, device="cuda")
    with pytest.raises(deft.DeftError):
        deft.deft_threshold_select(x, float("nan"), None, None, cnt, ws)
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(deft.DeftError):
        deft.deft_threshold_select(x, 1.0, None, None, cnt, small)


def test_clt_k_leader_and_followers(deft):
    """One CLT-k iteration on 4 simulated workers: the leader's top-k, every worker's gather."""
    N, n, k = 4, 500_009, 5_000
    rng = np.random.default_rng(41)
    shared = rng.standard_normal(n).astype(np.float32)
    vecs = [(shared + 0.3 * rng.standard_normal(n).astype(np.float32)) for _ in range(N)]
    for it in (0, 1, 6):
        leader = deft.deft_clt_leader(it, N)
        assert leader == oracle.clt_leader(it, N)
        acc = [torch.from_numpy(v.copy()).cuda() for v in vecs]
        ws = deft.alloc_workspace(n, 1)
        lval = torch.empty(k, dtype=torch.float32, device="cuda")
        lidx = torch.empty(k, dtype=torch.int64, device="cuda")
        deft.deft_topk_baseline(acc[leader], k, lval, lidx, ws)
        want_val, want_idx = oracle.topk(vecs[leader], k)
        assert np.array_equal(lidx.cpu().numpy(), want_idx)
        for r in range(N):
            val = torch.full((k,), 9.0, dtype=torch.float32, device="cuda")
            deft.deft_gather_update(acc[r], lidx, k, val)
            torch.cuda.synchronize()
            ref = vecs[r].copy()
            want = oracle.gather_update(ref, want_idx)
            assert val.cpu().numpy().tobytes() == want.tobytes()
            assert acc[r].cpu().numpy().tobytes() == ref.tobytes()
        assert lval.cpu().numpy().tobytes() == want_val.tobytes()
    with pytest.raises(deft.DeftError):
        deft.deft_clt_leader(0, 0)
