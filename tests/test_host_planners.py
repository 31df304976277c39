"""The library's host planners (Algorithms 2-4) against the oracle, bit for bit, plus the
C-ABI surface: every symbol the header declares is exported, and bad arguments come back
as status codes.  No GPU needed (the library loads without a driver)."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2307_03500_b200 import build as deft_build
from paper_2307_03500_b200 import workloads as W

deft_build.build()
from paper_2307_03500_b200 import deft  # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "deft.h")).read()
    names = re.findall(r"DEFT_API\s+[\w\s\*]+?\b(deft_\w+)\s*\(", header)
    assert len(names) >= 12 and len(set(names)) == len(names)
    lib = ctypes.CDLL(deft.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings():
    assert deft.status_string(0) == "DEFT_OK"
    assert deft.status_string(-4) == "DEFT_ERR_CAPACITY"
    assert deft.lib().deft_last_cuda_error() == 0


@pytest.mark.parametrize("name,N", [("tiny", 4), ("resnet18", 16), ("lstm_lm", 16), ("bert_large", 32),
                                    ("gpt2_medium", 1), ("gpt2_medium", 8), ("gpt2_medium", 64)])
def test_split_layers_matches_oracle(name, N):
    sizes = W.WORKLOADS[name]().sizes
    a, at = deft.deft_split_layers(sizes, N)
    b, bt = oracle.split_layers(sizes, N)
    assert a.tolist() == b.tolist() and at.tolist() == bt.tolist()


def test_split_layers_random_and_errors():
    rng = np.random.default_rng(1)
    for _ in range(200):
        T = int(rng.integers(1, 12))
        sizes = rng.integers(1, 200, size=T)
        N = int(rng.integers(1, 20))
        a, at = deft.deft_split_layers(sizes, N)
        b, bt = oracle.split_layers(sizes, N)
        assert a.tolist() == b.tolist() and at.tolist() == bt.tolist()
    with pytest.raises(deft.DeftError):
        deft.deft_split_layers([4, 0, 3], 2)
    with pytest.raises(deft.DeftError):
        deft.deft_split_layers([4, 3], 0)


def _random_case(rng):
    L = int(rng.integers(1, 80))
    norms = np.exp(rng.uniform(-12, 5, size=L))
    which = rng.integers(0, 6)
    if which == 0:
        norms[rng.integers(0, L, size=max(1, L // 3))] = 0.0
    elif which == 1:
        norms[:] = norms[0]
    elif which == 2:
        norms = np.round(norms, 1)  # many ties
    sizes = rng.integers(1, 200000, size=L)
    if rng.integers(0, 3) == 0:
        sizes[rng.integers(0, L, size=max(1, L // 4))] = rng.integers(1, 5)
    n_g = int(sizes.sum())
    k = int(rng.integers(1, n_g + 1))
    return norms, sizes, k, L, n_g


def test_allocate_k_matches_oracle_bit_for_bit():
    rng = np.random.default_rng(2)
    for _ in range(500):
        norms, sizes, k, L, n_g = _random_case(rng)
        for mode in (deft.MODE_PAPER, deft.MODE_EXACT):
            if mode == deft.MODE_EXACT and not (L <= k <= n_g):
                with pytest.raises(deft.DeftError) as ei:
                    deft.deft_allocate_k(norms, sizes, k, mode)
                assert ei.value.status == deft.ERR_INFEASIBLE_K
                continue
            a, sa, st = deft.deft_allocate_k(norms, sizes, k, mode)
            b, sb = oracle.allocate_k(norms, sizes, k, mode)
            assert a.tolist() == b.tolist() and sa == sb
            assert st == (deft.OK if sa == k else deft.WARN_K_INEXACT)


def test_allocate_k_errors():
    with pytest.raises(deft.DeftError) as ei:
        deft.deft_allocate_k([1.0, float("inf")], [5, 5], 4)
    assert ei.value.status == deft.ERR_NONFINITE_NORM
    with pytest.raises(deft.DeftError) as ei:
        deft.deft_allocate_k([1.0, -1.0], [5, 5], 4)
    assert ei.value.status == deft.ERR_NONFINITE_NORM
    with pytest.raises(deft.DeftError) as ei:
        deft.deft_allocate_k([1.0, 1.0], [5, 0], 4)
    assert ei.value.status == deft.ERR_INVALID_ARG
    with pytest.raises(deft.DeftError) as ei:
        deft.deft_allocate_k([1.0], [5], 0)
    assert ei.value.status == deft.ERR_INVALID_ARG


def test_partition_matches_oracle_bit_for_bit():
    rng = np.random.default_rng(3)
    for _ in range(300):
        norms, sizes, k, L, n_g = _random_case(rng)
        k_l, _ = oracle.allocate_k(norms, sizes, k, oracle.MODE_PAPER)
        N = int(rng.integers(1, 70))
        a, la = deft.deft_partition(sizes, k_l, N)
        b, lb = oracle.partition(sizes, k_l, N)
        assert a.tolist() == b.tolist()
        assert la.tobytes() == lb.tobytes()
        # bins of a rotation are disjoint and cover every layer
        it = int(rng.integers(0, 1000))
        seen = []
        for r in range(N):
            bin_id = deft.deft_rank_bin(it, r, N)
            assert bin_id == oracle.rank_bin(it, r, N)
            mine = deft.deft_bin_layers(a, bin_id)
            assert mine.tolist() == oracle.my_layers(b, it, r, N).tolist()
            seen += mine.tolist()
        assert sorted(seen) == list(range(L))


def test_partition_by_size_matches_oracle_bit_for_bit():
    rng = np.random.default_rng(4)
    for _ in range(200):
        norms, sizes, k, L, n_g = _random_case(rng)
        N = int(rng.integers(1, 70))
        a, la = deft.deft_partition_model(sizes, None, N, deft.COST_SIZE)
        b, lb = oracle.partition_by_size(sizes, N)
        assert a.tolist() == b.tolist()
        assert la.tobytes() == lb.tobytes()
        k_l, _ = oracle.allocate_k(norms, sizes, k, oracle.MODE_PAPER)
        c, lc = deft.deft_partition_model(sizes, k_l, N, deft.COST_EQ3)      # the Eq. 3 model through the same call
        d, ld = oracle.partition(sizes, k_l, N)
        assert c.tolist() == d.tolist() and lc.tobytes() == ld.tobytes()
    with pytest.raises(deft.DeftError):
        deft.deft_partition_model([5, 5], [1, 1], 2, 7)
    with pytest.raises(deft.DeftError):
        deft.deft_partition_model([5, 5], None, 2, deft.COST_EQ3)


def test_partition_errors():
    with pytest.raises(deft.DeftError):
        deft.deft_partition([5, 5], [1, 0], 2)
    with pytest.raises(deft.DeftError):
        deft.deft_partition([5, 5], [1, 1], 0)
    with pytest.raises(deft.DeftError):
        deft.deft_rank_bin(0, 4, 4)


def test_workspace_bytes_is_monotone_and_covers_staging():
    a = deft.deft_workspace_bytes(1 << 20, 16)
    b = deft.deft_workspace_bytes(1 << 21, 16)
    c = deft.deft_workspace_bytes(1 << 20, 64)
    assert 8 * (1 << 20) < a < b and a < c
    assert deft.deft_workspace_bytes(0, 4) == 0


def test_device_calls_reject_bad_arguments_without_touching_the_gpu():
    L = deft.lib()
    assert L.deft_layer_norms(None, None, 10, None, 1, None, None, 0, None) == deft.ERR_INVALID_ARG
    assert L.deft_select(None, None, None, None, 0, None, None, 0, None, 0, None) == deft.OK   # empty rank
    assert L.deft_select(None, None, None, None, 3, None, None, 0, None, 0, None) == deft.ERR_INVALID_ARG
    assert L.deft_topk_baseline(None, 10, 3, None, None, None, 0, None) == deft.ERR_INVALID_ARG
    assert L.deft_residual_update(None, 10, None, 0, None) == deft.OK
    assert L.deft_residual_update(None, 10, None, 11, None) == deft.ERR_INVALID_ARG
    # misaligned vector / ids not ascending / k_l out of range are caught on the host
    ls = np.array([0, 100, 200], dtype=np.int64)
    kl = np.array([5, 500], dtype=np.int64)
    my = np.array([1, 0], dtype=np.int32)
    fake = ctypes.c_void_p(0x1000)
    p = lambda a: ctypes.c_void_p(a.ctypes.data)
    assert L.deft_select(ctypes.c_void_p(0x1004), p(ls), p(kl), p(my), 2, fake, fake, 600, fake, 1 << 20, None) \
        == deft.ERR_INVALID_ARG
    assert L.deft_select(fake, p(ls), p(kl), p(my), 2, fake, fake, 600, fake, 1 << 20, None) == deft.ERR_INVALID_ARG
    my = np.array([0, 1], dtype=np.int32)
    assert L.deft_select(fake, p(ls), p(kl), p(my), 2, fake, fake, 600, fake, 1 << 20, None) == deft.ERR_INVALID_ARG
    kl[1] = 50
    assert L.deft_select(fake, p(ls), p(kl), p(my), 2, fake, fake, 10, fake, 1 << 20, None) == deft.ERR_CAPACITY
    assert L.deft_select(fake, p(ls), p(kl), p(my), 2, fake, fake, 600, fake, 64, None) == deft.ERR_CAPACITY


def test_size_limits_are_the_header_s():
    """The header's limits are the ones the host code enforces: a layer of DEFT_MAX_LAYER_ELEMS elements is
    planned, one element more is an invalid argument (before anything touches a GPU); the status that says
    "beyond one launch" has its own name."""
    header = open(os.path.join(ROOT, "include", "deft.h")).read()
    limit = int(re.search(r"#define\s+DEFT_MAX_LAYER_ELEMS\s+(\d+)LL", header).group(1))
    assert limit == 2 ** 31 - 1
    assert int(re.search(r"#define\s+DEFT_ERR_TOO_LARGE\s+(-\d+)", header).group(1)) == deft.ERR_TOO_LARGE
    assert deft.status_string(deft.ERR_TOO_LARGE) == "DEFT_ERR_TOO_LARGE"
    bins = np.array([0, 1], dtype=np.int32)
    k_l = np.array([7, 9], dtype=np.int64)
    ok = deft.deft_plan_build(np.array([0, limit, limit + 4096], dtype=np.int64), k_l, bins, 2, 0)
    n_layers, elems, k, off = deft.deft_plan_rank_table(ok, 2)
    assert n_layers.tolist() == [1, 1] and elems.tolist() == [limit, 4096] and k.tolist() == [7, 9] and off.tolist() == [0, 7]
    with pytest.raises(deft.DeftError) as ei:
        deft.deft_plan_build(np.array([0, limit + 1, limit + 4097], dtype=np.int64), k_l, bins, 2, 0)
    assert ei.value.status == deft.ERR_INVALID_ARG
    # Top-k and the hard threshold take the same limit for their n (checked before the pointers are used)
    L = deft.lib()
    fake = ctypes.c_void_p(0x1000)
    assert L.deft_topk_baseline(fake, limit + 1, 3, fake, fake, fake, 1 << 40, None) == deft.ERR_INVALID_ARG
    # the workspace for the largest layer is a finite, monotone number
    assert deft.deft_workspace_bytes(limit, 1) > 8 * limit
