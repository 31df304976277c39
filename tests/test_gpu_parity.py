"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element.

Bars: indices, values, k_l and partitions are bit-exact; norms agree to 1e-5 relative
(fp32 squares over runs of 8 elements, fp64 beyond, against the oracle's sequential fp64).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2307_03500_b200 import build as deft_build
from paper_2307_03500_b200 import workloads as W

pytestmark = pytest.mark.gpu

NORM_RTOL = 1e-5


@pytest.fixture(scope="module")
def deft():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    deft_build.build()
    from paper_2307_03500_b200 import deft as d
    d.lib()
    return d


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _gpu_norms(deft, e, g, layer_start):
    e_d = _dev(e)
    g_d = _dev(g) if g is not None else None
    ls_d = _dev(np.asarray(layer_start, dtype=np.int64))
    L = len(layer_start) - 1
    norms_d = torch.full((L,), -1.0, dtype=torch.float64, device="cuda")
    ws = deft.alloc_workspace(e.size, L)
    deft.deft_layer_norms(e_d, g_d, ls_d, norms_d, ws)
    torch.cuda.synchronize()
    return e_d.cpu().numpy(), norms_d.cpu().numpy()


def _gpu_select(deft, acc_d, layer_start, k_l, my, ws=None, n_elems=None):
    total = int(np.asarray(k_l)[my].sum()) if len(my) else 0
    val_d = torch.full((total + 8,), 7.0, dtype=torch.float32, device="cuda")
    idx_d = torch.full((total + 8,), -7, dtype=torch.int64, device="cuda")
    if ws is None:
        ws = deft.alloc_workspace(int(layer_start[-1]), len(layer_start) - 1)
    n = deft.deft_select(acc_d, layer_start, k_l, my, val_d, idx_d, ws)
    torch.cuda.synchronize()
    assert n == total
    # canaries behind the output are untouched
    assert torch.all(val_d[total:] == 7.0) and torch.all(idx_d[total:] == -7)
    return val_d[:total].cpu().numpy(), idx_d[:total].cpu().numpy()


# ------------------------------------------------------------------------------------------
# step 1: accumulate + norms
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("wl", ["tiny", "resnet18", "bert_div64", "gpt2_div64_N64"])
def test_accumulate_and_norms(deft, wl):
    w = {"tiny": W.tiny(), "resnet18": W.resnet18(), "bert_div64": W.scaled_down(W.bert_large(), 64),
         "gpt2_div64_N64": W.scaled_down(W.gpt2_medium(64, 0.01), 64)}[wl]
    rng = np.random.default_rng(7)
    e = (rng.standard_normal(w.n_g, dtype=np.float32) * np.float32(1e-3))
    g = w.gradient(0)
    start, _ = oracle.split_layers(w.sizes, w.n_workers)
    want_acc = oracle.accumulate(e.copy(), g)
    want = oracle.layer_norms(want_acc, start)
    got_acc, got = _gpu_norms(deft, e, g, start)
    assert got_acc.tobytes() == want_acc.tobytes()          # one fp32 add per element: bit-exact
    assert np.all(np.abs(got - want) <= NORM_RTOL * want)
    assert np.all((want > 0) | (got == 0))
    # run-to-run bit-identical
    _, again = _gpu_norms(deft, e, g, start)
    assert again.tobytes() == got.tobytes()
    # norms-only mode: nothing written, same norms
    kept, only = _gpu_norms(deft, want_acc, None, start)
    assert kept.tobytes() == want_acc.tobytes() and only.tobytes() == got.tobytes()


def test_norms_ragged_layers_and_closed_forms(deft):
    # layer boundaries that are not multiples of anything, tiny layers, a zero layer, a tail
    sizes = [1, 3, 8191, 8192, 8193, 10, 64, 37 * 37, 100, 5, 20001]
    start = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    rng = np.random.default_rng(8)
    e = rng.standard_normal(int(start[-1]), dtype=np.float32)
    e[start[7]:start[8]] = 1.0     # all ones, 37*37 elements -> norm 37
    e[start[8]:start[9]] = 0.0     # zero layer
    got_acc, got = _gpu_norms(deft, e, None, start)
    want = oracle.layer_norms(e, start)
    assert np.all(np.abs(got - want) <= NORM_RTOL * want)
    assert got[7] == 37.0 and got[8] == 0.0


# ------------------------------------------------------------------------------------------
# the whole path on the paper-shaped workloads (scaled so the oracle sorts in seconds)
# ------------------------------------------------------------------------------------------
def _whole_path(deft, w, steps=1, mode=None, iteration=0):
    from paper_2307_03500_b200.pipeline import DeftStep
    mode = deft.MODE_EXACT if mode is None else mode
    N = w.n_workers
    ds = DeftStep(w.sizes, N, w.density, mode=mode)
    start, _ = oracle.split_layers(w.sizes, N)
    assert ds.layer_start.tolist() == start.tolist()
    size = np.diff(start)
    e_cpu = np.zeros(w.n_g, dtype=np.float32)
    e_gpu = torch.zeros(w.n_g, dtype=torch.float32, device="cuda")
    for t in range(steps):
        g = w.gradient(t)
        g_d = _dev(g)
        # GPU
        norms_gpu = ds.layer_norms(e_gpu, g_d).copy()
        # oracle
        oracle.accumulate(e_cpu, g)
        norms_cpu = oracle.layer_norms(e_cpu, start)
        assert e_gpu.cpu().numpy().tobytes() == e_cpu.tobytes()
        assert np.all(np.abs(norms_gpu - norms_cpu) <= NORM_RTOL * norms_cpu)
        # both planners get identical norms (the GPU's): k_l and bins must then be bit-exact
        plan = ds.plan(norms_gpu, iteration + t)
        k_l, s = oracle.allocate_k(norms_gpu, size, ds.k, mode)
        bins, load = oracle.partition(size, k_l, N)
        assert plan.k_l.tolist() == k_l.tolist() and plan.sum_k == s
        assert plan.bin_of_layer.tolist() == bins.tolist() and plan.bin_load.tobytes() == load.tobytes()
        if mode == deft.MODE_EXACT:
            assert s == ds.k
        seen = np.zeros(w.n_g, dtype=np.int8)
        all_idx = []
        for r in range(N):
            my = oracle.my_layers(bins, iteration + t, r, N)
            assert ds.rank_layers(plan, iteration + t, r).tolist() == my.tolist()
            val_d, idx_d = ds.select_rank(e_gpu, plan, r)
            torch.cuda.synchronize()
            want_val, want_idx = oracle.select_rank(e_cpu, start, k_l, my)
            assert idx_d.cpu().numpy().tolist() == want_idx.tolist()
            assert val_d.cpu().numpy().tobytes() == want_val.tobytes()
            seen[want_idx] += 1
            all_idx.append(idx_d)
        assert seen.max() == 1 and int(seen.sum()) == s       # disjoint, density kept
        # all ranks in one launch (selection + zeroing): same bytes as the per-rank calls
        val_pr, idx_pr = ds.val_d[:s].clone(), ds.idx_d[:s].clone()
        e_all = e_gpu.clone()
        ds.val_d.fill_(7.0)
        ds.idx_d.fill_(-7)
        deft.deft_plan_upload(plan.plan_h, ds.plan_d, ds.ws)   # the per-layer scratch state is single-use
        ds.select_and_update_all(e_all, plan)
        torch.cuda.synchronize()
        assert torch.equal(ds.idx_d[:s], idx_pr) and ds.val_d[:s].cpu().numpy().tobytes() == val_pr.cpu().numpy().tobytes()
        assert torch.all(ds.idx_d[s:] == -7)
        for idx_d in all_idx:
            ds.residual_update(e_gpu, idx_d)
        torch.cuda.synchronize()
        oracle.residual_update(e_cpu, np.nonzero(seen)[0])
        assert e_gpu.cpu().numpy().tobytes() == e_cpu.tobytes()
        assert e_all.cpu().numpy().tobytes() == e_cpu.tobytes()


def test_whole_path_tiny(deft):
    _whole_path(deft, W.tiny())
    _whole_path(deft, W.tiny(), mode=0, iteration=5)


def test_whole_path_resnet18(deft):
    _whole_path(deft, W.resnet18())


def test_whole_path_lstm_three_steps_with_residual(deft):
    _whole_path(deft, W.scaled_down(W.lstm_lm(), 16), steps=3)


def test_whole_path_bert_shaped(deft):
    _whole_path(deft, W.scaled_down(W.bert_large(), 32))


@pytest.mark.parametrize("N,d", [(1, 0.1), (8, 0.01), (64, 0.001)])
def test_whole_path_gpt2_shaped(deft, N, d):
    _whole_path(deft, W.scaled_down(W.gpt2_medium(N, d), 32))


# ------------------------------------------------------------------------------------------
# selection edge cases
# ------------------------------------------------------------------------------------------
KINDS = ["gauss", "few_values", "all_equal", "all_zero", "signed_zero", "mostly_zero", "outlier",
         "bf16_like", "denormal", "wide_exponent"]


@pytest.mark.parametrize("kind", KINDS)
def test_select_adversarial_layers(deft, kind):
    # one vector holding layers of awkward sizes at awkward offsets; every layer is its own case
    sizes = [1, 10, 31, 32, 33, 4095, 4096, 4097, 5, 12289, 20000, 3]
    start = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    x = W.adversarial_vector(kind, int(start[-1]), seed=3)
    acc_d = _dev(x)
    ws = deft.alloc_workspace(x.size, len(sizes))
    for pick in ("one", "all", "mid", "most"):
        k_l = np.array([{"one": 1, "all": s, "mid": max(1, s // 3), "most": max(1, s - 1)}[pick] for s in sizes],
                       dtype=np.int64)
        for my in ([0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11], [5], [1, 4, 7, 10], [11]):
            my = np.array(my, dtype=np.int32)
            val, idx = _gpu_select(deft, acc_d, start, k_l, my, ws)
            want_val, want_idx = oracle.select_rank(x, start, k_l, my)
            assert idx.tolist() == want_idx.tolist(), (kind, pick, my.tolist())
            assert val.tobytes() == want_val.tobytes()


def test_select_threshold_value_repeated_across_tiles(deft):
    # the k-th magnitude occurs many times, spread over several tiles and both signs
    n = 50000
    rng = np.random.default_rng(5)
    x = rng.standard_normal(n, dtype=np.float32) * np.float32(0.1)
    x[np.abs(x) > 0.25] = 0.1
    rep = rng.choice(n, size=3000, replace=False)
    x[rep] = np.where(rng.random(3000) < 0.5, 0.25, -0.25).astype(np.float32)
    big = rng.choice(np.setdiff1d(np.arange(n), rep), size=100, replace=False)
    x[big] = 1.0 + rng.random(100).astype(np.float32)
    acc_d = _dev(x)
    start = np.array([0, n], dtype=np.int64)
    for k in (100, 101, 1500, 3099, 3100, 3101):
        val, idx = _gpu_select(deft, acc_d, start, np.array([k]), np.array([0], dtype=np.int32))
        want_val, want_idx = oracle.select_layer(x, 0, n, k)
        assert idx.tolist() == want_idx.tolist() and val.tobytes() == want_val.tobytes()


def test_empty_rank_and_single_layer_equals_topk(deft):
    x = W.adversarial_vector("gauss", 70001, seed=6)
    acc_d = _dev(x)
    ws = deft.alloc_workspace(x.size, 4)
    start = np.array([0, 70001], dtype=np.int64)
    val_d = torch.empty(16, dtype=torch.float32, device="cuda")
    idx_d = torch.empty(16, dtype=torch.int64, device="cuda")
    assert deft.deft_select(acc_d, start, np.array([5]), np.array([], dtype=np.int32), val_d, idx_d, ws) == 0
    k = 701
    v1, i1 = _gpu_select(deft, acc_d, start, np.array([k]), np.array([0], dtype=np.int32), ws)
    val_d = torch.empty(k, dtype=torch.float32, device="cuda")
    idx_d = torch.empty(k, dtype=torch.int64, device="cuda")
    deft.deft_topk_baseline(acc_d, k, val_d, idx_d, ws)
    torch.cuda.synchronize()
    want_val, want_idx = oracle.topk(x, k)
    assert idx_d.cpu().numpy().tolist() == want_idx.tolist() == i1.tolist()
    assert val_d.cpu().numpy().tobytes() == want_val.tobytes() == v1.tobytes()


@pytest.mark.parametrize("n,k", [(1, 1), (4097, 4097), (1 << 20, 1), (3_000_001, 30_000), (3_000_001, 2_999_999)])
def test_topk_baseline(deft, n, k):
    x = W.adversarial_vector("gauss", n, seed=n % 97)
    acc_d = _dev(x)
    ws = deft.alloc_workspace(n, 1)
    val_d = torch.empty(k, dtype=torch.float32, device="cuda")
    idx_d = torch.empty(k, dtype=torch.int64, device="cuda")
    deft.deft_topk_baseline(acc_d, k, val_d, idx_d, ws)
    torch.cuda.synchronize()
    want_val, want_idx = oracle.topk(x, k)
    assert np.array_equal(idx_d.cpu().numpy(), want_idx)
    assert val_d.cpu().numpy().tobytes() == want_val.tobytes()


@pytest.mark.parametrize("kind,k", [("clustered", 21_000), ("clustered", 2_100_000), ("few_values", 300_001)])
def test_topk_single_large_layer_round_robin_split(deft, kind, k):
    """One layer large enough that the kernel deals its tiles out to the CTAs round-robin
    (several thousand tiles per CTA-round, a ragged last super-tile, an unaligned start)."""
    n = 21_000_003
    if kind == "clustered":     # the large entries sit in a few narrow regions
        x = W.adversarial_vector("gauss", n + 3, seed=5)
        x[1_000_000:1_300_000] *= np.float32(50.0)
        x[-70_000:] *= np.float32(80.0)
    else:                       # eight distinct magnitudes: the threshold value repeats millions of times
        x = W.adversarial_vector("few_values", n + 3, seed=6)
    acc_d = _dev(x)
    start = np.array([3, n + 3], dtype=np.int64)      # layer starts 12 bytes into the buffer
    ws = deft.alloc_workspace(n, 1)
    val_d = torch.empty(k, dtype=torch.float32, device="cuda")
    idx_d = torch.empty(k, dtype=torch.int64, device="cuda")
    deft.deft_select(acc_d, start, np.array([k], dtype=np.int64), np.array([0], dtype=np.int32), val_d, idx_d, ws)
    torch.cuda.synchronize()
    want_val, want_idx = oracle.select_layer(x, 3, n + 3, k)
    assert np.array_equal(idx_d.cpu().numpy(), want_idx)
    assert val_d.cpu().numpy().tobytes() == want_val.tobytes()


def test_large_multi_layer_rank_cost_weighted_split(deft):
    """A rank large enough (> 64 tiles per CTA) that the kernel re-deals its tiles by estimated
    cost after the first read: layers whose density of selected entries differs by five orders
    of magnitude, small and tiny layers between large ones, layers skipped by the rank."""
    sizes = [5_000_000, 3_000_001, 20_000, 1_000, 8_000_005, 1_500_000, 6_000_000, 17, 2_500_000]
    start = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    x = W.adversarial_vector("gauss", int(start[-1]), seed=12)
    x[start[4]:start[4] + 2_000_000] *= np.float32(30.0)          # the large entries of layer 4 sit at its head
    x[start[6]:start[7]] = W.adversarial_vector("few_values", sizes[6], seed=13)
    k_l = np.array([5, 900_000, 100, 10, 8_000, 1, 600_000, 17, 2_499_999], dtype=np.int64)
    my = np.array([0, 1, 2, 3, 4, 6, 7, 8], dtype=np.int32)       # layer 5 belongs to another rank
    acc_d = _dev(x)
    ws = deft.alloc_workspace(int(start[-1]), len(sizes))
    want_val, want_idx = oracle.select_rank(x, start, k_l, my)
    for rep in range(2):        # the second call runs with the cuts remembered from the first
        val, idx = _gpu_select(deft, acc_d, start, k_l, my, ws=ws)
        assert np.array_equal(idx, want_idx)
        assert val.tobytes() == want_val.tobytes()
    x2 = (x * np.float32(0.97)).astype(np.float32)      # cuts slightly too high for every layer
    x2[start[0]:start[1]] = x[start[0]:start[1]] * np.float32(3.0)
    want_val, want_idx = oracle.select_rank(x2, start, k_l, my)
    val, idx = _gpu_select(deft, _dev(x2), start, k_l, my, ws=ws)
    assert np.array_equal(idx, want_idx) and val.tobytes() == want_val.tobytes()


@pytest.mark.parametrize("scale_first", [1.0, 16.0, 1.0 / 16.0, 1e-6, 1e6])
def test_speculative_cut_from_previous_call_never_changes_the_result(deft, scale_first):
    """The kernel stages entries above a cut remembered from the previous call on the same
    workspace.  Whatever that cut is — exact, far too high (second read needed), far too low
    (nearly everything staged) — the selection must equal the oracle's."""
    w = W.scaled_down(W.gpt2_medium(4, 0.01), 32)
    x = w.gradient(0)
    start, _ = oracle.split_layers(w.sizes, 4)
    size = np.diff(start)
    k_l = np.maximum(1, size // 97)
    k_l[::5] = np.maximum(1, size[::5] // 3)                    # some layers too dense for a speculative cut
    my = np.arange(size.size, dtype=np.int32)
    ws = deft.alloc_workspace(int(start[-1]), size.size)
    first = (x * np.float32(scale_first)).astype(np.float32)
    first[start[3]:start[4]] = x[start[3]:start[4]] * np.float32(1e3)      # one layer's cut moves the other way
    got0 = _gpu_select(deft, _dev(first), start, k_l, my, ws=ws)
    want0 = oracle.select_rank(first, start, k_l, my)
    assert np.array_equal(got0[1], want0[1]) and got0[0].tobytes() == want0[0].tobytes()
    want = oracle.select_rank(x, start, k_l, my)
    for _ in range(2):                                           # second call: cuts from `first`; third: from x itself
        got = _gpu_select(deft, _dev(x), start, k_l, my, ws=ws)
        assert np.array_equal(got[1], want[1]) and got[0].tobytes() == want[0].tobytes()
    # a subset of the layers, Top-k and a hard threshold share the workspace (and its remembered cuts)
    sub = my[1::2]
    got = _gpu_select(deft, _dev(x), start, k_l, sub, ws=ws)
    wsub = oracle.select_rank(x, start, k_l, sub)
    assert np.array_equal(got[1], wsub[1]) and got[0].tobytes() == wsub[0].tobytes()


@pytest.mark.parametrize("seed", list(range(24)))
def test_random_layer_structures(deft, seed):
    """Random layer tables (tiny, direct-sized, streamed and large layers in any order, unaligned
    boundaries), random k_l from 1 to the whole layer, a random subset of the layers as the rank,
    per-layer value distributions from the edge-case generators; every call repeated on the same
    workspace so that the second one runs with remembered cuts."""
    rng = np.random.default_rng(1000 + seed)
    L = int(rng.integers(1, 40))
    kinds = ["gauss", "wide_exponent", "few_values", "mostly_zero", "all_equal", "bf16_like", "outlier", "denormal"]
    sizes = []
    for _ in range(L):
        c = rng.integers(0, 4)
        sizes.append(int([rng.integers(1, 100), rng.integers(1000, 20_000), rng.integers(16_000, 17_000),
                          rng.integers(100_000, 400_000)][c]))
    if seed % 6 == 0:
        sizes[int(rng.integers(0, L))] = int(rng.integers(1_500_000, 2_500_000))
    start = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    x = np.empty(int(start[-1]), dtype=np.float32)
    for l in range(L):
        x[start[l]:start[l + 1]] = W.adversarial_vector(kinds[int(rng.integers(0, len(kinds)))], sizes[l],
                                                        seed=seed * 131 + l) * np.float32(10.0 ** rng.integers(-3, 4))
    k_l = np.empty(L, dtype=np.int64)
    for l in range(L):
        c = rng.integers(0, 4)
        k_l[l] = [1, sizes[l], max(1, sizes[l] // 100), int(rng.integers(1, sizes[l] + 1))][c]
    my = np.sort(rng.choice(L, size=int(rng.integers(1, L + 1)), replace=False)).astype(np.int32)
    acc_d = _dev(x)
    ws = deft.alloc_workspace(int(start[-1]), L)
    want = oracle.select_rank(x, start, k_l, my)
    for rep in range(2):
        got = _gpu_select(deft, acc_d, start, k_l, my, ws=ws)
        assert np.array_equal(got[1], want[1]), (seed, rep)
        assert got[0].tobytes() == want[0].tobytes(), (seed, rep)
    # the vector changes a little, the cuts remembered from before are reused
    x2 = x.copy()
    x2[::3] *= np.float32(1.07)
    want2 = oracle.select_rank(x2, start, k_l, my)
    got2 = _gpu_select(deft, _dev(x2), start, k_l, my, ws=ws)
    assert np.array_equal(got2[1], want2[1]) and got2[0].tobytes() == want2[0].tobytes()


def test_nan_and_infinities_sort_by_bit_pattern(deft):
    """Magnitude order is the IEEE bit pattern with the sign cleared: NaN above infinity above
    every finite value; the selected values come back bit for bit (payloads, signs)."""
    n = 70_001
    x = W.adversarial_vector("gauss", n, seed=77)
    bits = x.view(np.uint32)
    bits[5] = 0x7FC00001          # quiet NaN with a payload
    bits[60_000] = 0xFFC00000     # negative NaN
    bits[123] = 0x7F800000        # +inf
    bits[40_000] = 0xFF800000     # -inf
    bits[999] = 0x7F7FFFFF        # largest finite
    start = np.array([0, 30_000, n], dtype=np.int64)
    for k_l in ([1, 1], [2, 3], [30_000, 100]):
        k_l = np.array(k_l, dtype=np.int64)
        my = np.array([0, 1], dtype=np.int32)
        got = _gpu_select(deft, _dev(x), start, k_l, my)
        want = oracle.select_rank(x, start, k_l, my)
        assert np.array_equal(got[1], want[1]) and got[0].tobytes() == want[0].tobytes()
    got = _gpu_select(deft, _dev(x), start, np.array([3, 2], dtype=np.int64), np.array([0, 1], dtype=np.int32))
    assert sorted(got[1].tolist()) == [5, 123, 999, 40_000, 60_000]


def test_whole_step_in_one_call_matches_the_separate_calls(deft):
    from paper_2307_03500_b200.pipeline import DeftStep
    w = W.scaled_down(W.bert_large(), 64)
    N = w.n_workers
    ds_a = DeftStep(w.sizes, N, w.density)
    ds_b = DeftStep(w.sizes, N, w.density)
    e_a = torch.zeros(w.n_g, dtype=torch.float32, device="cuda")
    e_b = torch.zeros_like(e_a)
    for t in range(3):
        g_d = _dev(w.gradient(t))
        plan_a, _ = ds_a.step(e_a, g_d, iteration=t)                 # separate calls, all workers in one launch
        plan_b = ds_b.step_fused(e_b, g_d, iteration=t)              # the same through deft_step
        torch.cuda.synchronize()
        assert plan_a.sum_k == plan_b.sum_k and plan_a.k_l.tolist() == plan_b.k_l.tolist()
        assert torch.equal(ds_a.norms_d, ds_b.norms_d)                # the step's accumulate pass takes the roots itself: same bits
        assert plan_a.bin_of_layer.tolist() == plan_b.bin_of_layer.tolist()
        assert plan_a.bin_load.tobytes() == plan_b.bin_load.tobytes()
        s = plan_a.sum_k
        assert torch.equal(ds_a.idx_d[:s], ds_b.idx_d[:s]) and torch.equal(ds_a.val_d[:s], ds_b.val_d[:s])
        assert torch.equal(e_a, e_b)
    # one worker only: its entries at the head of the output, only its entries cleared
    ds_c = DeftStep(w.sizes, N, w.density)
    e_c = torch.zeros_like(e_a)
    g_d = _dev(w.gradient(0))
    r = 3
    plan_c = ds_c.step_fused(e_c, g_d, iteration=0, rank=r)
    torch.cuda.synchronize()
    acc = oracle.accumulate(np.zeros(w.n_g, dtype=np.float32), w.gradient(0))
    start, _ = oracle.split_layers(w.sizes, N)
    my = oracle.my_layers(plan_c.bin_of_layer, 0, r, N)
    want_val, want_idx = oracle.select_rank(acc, start, plan_c.k_l, my)
    kr = int(plan_c.rank_k[r])
    assert np.array_equal(ds_c.idx_d[:kr].cpu().numpy(), want_idx)
    assert ds_c.val_d[:kr].cpu().numpy().tobytes() == want_val.tobytes()
    acc[want_idx] = 0.0
    assert e_c.cpu().numpy().tobytes() == acc.tobytes()


def test_select_is_bit_deterministic_run_to_run(deft):
    w = W.scaled_down(W.gpt2_medium(4, 0.01), 16)
    x = w.gradient(0)
    acc_d = _dev(x)
    start, _ = oracle.split_layers(w.sizes, 4)
    size = np.diff(start)
    k_l = np.maximum(1, size // 100)
    my = np.arange(0, size.size, 2, dtype=np.int32)
    a = _gpu_select(deft, acc_d, start, k_l, my)
    b = _gpu_select(deft, acc_d, start, k_l, my)
    assert a[0].tobytes() == b[0].tobytes() and a[1].tobytes() == b[1].tobytes()


def test_residual_update(deft):
    x = W.adversarial_vector("gauss", 100003, seed=8)
    acc_d = _dev(x)
    _, idx = oracle.topk(x, 5000)
    idx_d = _dev(idx)
    deft.deft_residual_update(acc_d, idx_d, idx.size)
    deft.deft_residual_update(acc_d, idx_d, 0)
    torch.cuda.synchronize()
    want = oracle.residual_update(x.copy(), idx)
    assert acc_d.cpu().numpy().tobytes() == want.tobytes()


def test_capacity_errors_are_reported_not_faulted(deft):
    x = W.adversarial_vector("gauss", 10000, seed=1)
    acc_d = _dev(x)
    start = np.array([0, 10000], dtype=np.int64)
    val_d = torch.empty(10, dtype=torch.float32, device="cuda")
    idx_d = torch.empty(10, dtype=torch.int64, device="cuda")
    ws = deft.alloc_workspace(10000, 1)
    with pytest.raises(deft.DeftError) as ei:
        deft.deft_select(acc_d, start, np.array([11]), np.array([0], dtype=np.int32), val_d, idx_d, ws)
    assert ei.value.status == deft.ERR_CAPACITY
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(deft.DeftError) as ei:
        deft.deft_select(acc_d, start, np.array([5]), np.array([0], dtype=np.int32), val_d, idx_d, small)
    assert ei.value.status == deft.ERR_CAPACITY


# ------------------------------------------------------------------------------------------
# the forms of the selection kernel, the workspace's memory, limits
# ------------------------------------------------------------------------------------------
def test_every_form_of_the_selection_kernel_gives_the_same_bits(deft):
    """Five-step kernel, single-pass kernel with plain loads, single-pass kernel reading through its ring
    of bulk copies: three steps with the residual carried over (so that the later calls run on remembered
    cuts), every form on its own workspace, each compared with the oracle."""
    from paper_2307_03500_b200.pipeline import DeftStep
    w = W.scaled_down(W.bert_large(), 16)
    N = w.n_workers
    start, _ = oracle.split_layers(w.sizes, N)
    size = np.diff(start)
    forms = [(False, True), (True, False), (True, True)]     # (single pass, ring)
    try:
        runs = []
        for single, ring in forms:
            deft.deft_debug_select_kernel(single)
            deft.deft_debug_select_ring(ring)
            ds = DeftStep(w.sizes, N, w.density)
            e = torch.zeros(w.n_g, dtype=torch.float32, device="cuda")
            outs = []
            for t in range(3):
                plan = ds.step_fused(e, _dev(w.gradient(t)), iteration=t)
                torch.cuda.synchronize()
                outs.append((plan, ds.val_d[:plan.sum_k].cpu().numpy(), ds.idx_d[:plan.sum_k].cpu().numpy(), e.cpu().numpy()))
            st = deft.deft_select_stats(ds.ws, ds.L)
            assert st["ring_gave_up"] == 0
            if single:   # the second and third step found cuts for the layers of the first
                assert st["one_read"] > 0
            runs.append(outs)
    finally:
        deft.deft_debug_select_kernel(None)
        deft.deft_debug_select_ring(True)
    acc = np.zeros(w.n_g, dtype=np.float32)
    for t in range(3):
        oracle.accumulate(acc, w.gradient(t))
        plan = runs[0][t][0]
        want_val, want_idx = [], []
        for r in range(N):
            v, i = oracle.select_rank(acc, start, plan.k_l, oracle.my_layers(plan.bin_of_layer, t, r, N))
            want_val.append(v)
            want_idx.append(i)
        want_val, want_idx = np.concatenate(want_val), np.concatenate(want_idx)
        acc[want_idx] = 0.0
        for outs in runs:
            _, val, idx, e_now = outs[t]
            assert np.array_equal(idx, want_idx) and val.tobytes() == want_val.tobytes()
            assert e_now.tobytes() == acc.tobytes()
    assert size.sum() == w.n_g


@pytest.mark.parametrize("density", [0.03, 0.2])
def test_whole_step_with_layers_the_staging_pass_cannot_serve(deft, density):
    """Two layers that select more entries each than one CTA finishes behind the staging accumulate pass
    (density 0.03), or that are too dense for a cut at all (0.2): the step drops what was staged, or stages
    nothing, and selects the ordinary way.  Three steps against the oracle."""
    from paper_2307_03500_b200.pipeline import DeftStep
    sizes = [3_000_000, 2_500_001]
    ds = DeftStep(sizes, 1, density)
    n = int(sum(sizes))
    e = torch.zeros(n, dtype=torch.float32, device="cuda")
    acc = np.zeros(n, dtype=np.float32)
    start = np.asarray(ds.layer_start)
    for t in range(3):
        g = W.adversarial_vector("gauss", n, seed=70 + t)
        plan = ds.step_fused(e, _dev(g), iteration=t)
        torch.cuda.synchronize()
        oracle.accumulate(acc, g)
        k_l, _ = oracle.allocate_k(oracle.layer_norms(acc, start), np.diff(start), ds.k, oracle.MODE_EXACT)
        assert plan.k_l.tolist() == k_l.tolist()
        want_val, want_idx = oracle.select_rank(acc, start, k_l, np.arange(len(sizes), dtype=np.int32))
        assert np.array_equal(ds.idx_d[:plan.sum_k].cpu().numpy(), want_idx)
        assert ds.val_d[:plan.sum_k].cpu().numpy().tobytes() == want_val.tobytes()
        acc[want_idx] = 0.0
        assert e.cpu().numpy().tobytes() == acc.tobytes()


@pytest.mark.parametrize("L", [1, 2, 3, 4])
def test_few_large_layers_keep_their_remembered_cuts_across_the_norms_pass(deft, L):
    """The norms pass and the selection share one workspace.  With one to four layers of a few million
    elements the norm partials are many and the remembered cuts few: the second step must still find the
    cuts of the first (every streamed layer finished in one read), and both steps must match the oracle."""
    from paper_2307_03500_b200.pipeline import DeftStep
    sizes = [3_000_000 + 4099 * i for i in range(L)]
    ds = DeftStep(sizes, 1, 0.002)
    assert ds.L == L
    n = int(sum(sizes))
    e = torch.zeros(n, dtype=torch.float32, device="cuda")
    start = np.asarray(ds.layer_start)
    before = deft.deft_select_stats(ds.ws, ds.L)
    mid = None
    for t in range(2):
        acc = W.adversarial_vector("gauss", n, seed=40 + t)      # a fresh draw of the same distribution, no gradient added
        e.copy_(_dev(acc))
        plan = ds.step_fused(e, None, iteration=t)
        torch.cuda.synchronize()
        k_l, _ = oracle.allocate_k(oracle.layer_norms(acc, start), np.diff(start), ds.k, oracle.MODE_EXACT)
        assert plan.k_l.tolist() == k_l.tolist()
        want_val, want_idx = oracle.select_rank(acc, start, k_l, np.arange(L, dtype=np.int32))
        assert np.array_equal(ds.idx_d[:plan.sum_k].cpu().numpy(), want_idx)
        assert ds.val_d[:plan.sum_k].cpu().numpy().tobytes() == want_val.tobytes()
        acc[want_idx] = 0.0
        assert e.cpu().numpy().tobytes() == acc.tobytes()
        st = deft.deft_select_stats(ds.ws, ds.L)
        if t == 1:
            assert st["cut_failed"] == before["cut_failed"], "the cuts of the first step were lost or wrong"
            assert st["no_cut"] == mid["no_cut"], "the second step had no cut for a layer the first step finished"
            assert st["one_read"] == mid["one_read"] + L
        mid = st


def test_whole_step_with_pageable_host_norms(deft):
    """deft_step hands the norms to the host through norms_h: pinned memory is read in place while the
    device still works; ordinary pageable memory takes the copy-and-wait path.  Same result."""
    from paper_2307_03500_b200.pipeline import DeftStep
    w = W.scaled_down(W.bert_large(), 64)
    N = w.n_workers
    ds_a = DeftStep(w.sizes, N, w.density)
    ds_b = DeftStep(w.sizes, N, w.density)
    ds_b.norms_h = torch.empty(ds_b.L, dtype=torch.float64)        # pageable
    assert not ds_b.norms_h.is_pinned()
    e_a = torch.zeros(w.n_g, dtype=torch.float32, device="cuda")
    e_b = torch.zeros_like(e_a)
    for t in range(2):
        g_d = _dev(w.gradient(t))
        plan_a = ds_a.step_fused(e_a, g_d, iteration=t)
        plan_b = ds_b.step_fused(e_b, g_d, iteration=t)
        torch.cuda.synchronize()
        assert plan_a.k_l.tolist() == plan_b.k_l.tolist() and plan_a.bin_of_layer.tolist() == plan_b.bin_of_layer.tolist()
        s = plan_a.sum_k
        assert torch.equal(ds_a.idx_d[:s], ds_b.idx_d[:s]) and torch.equal(ds_a.val_d[:s], ds_b.val_d[:s])
        assert torch.equal(e_a, e_b)
        assert ds_a.norms_h.numpy().tobytes() == ds_b.norms_h.numpy().tobytes()


def test_beyond_one_launch_is_reported_not_attempted(deft):
    """A single layer larger than what one selection launch can scan (every CTA owns a bounded number of
    tiles) comes back as DEFT_ERR_TOO_LARGE before any kernel runs: the vector is never read, so it can be
    left uninitialised.  About 16 GB of device memory for the vector and the workspace."""
    n = deft.deft_select_launch_max_elems() + 4096
    assert n < 2 ** 31 - 1
    free, _ = torch.cuda.mem_get_info()
    need = 4 * n + deft.deft_workspace_bytes(n, 1) + (1 << 30)
    if free < need:
        pytest.skip("needs %.0f GB of free device memory" % (need / 1e9))
    acc_d = torch.empty(n, dtype=torch.float32, device="cuda")
    ws = deft.alloc_workspace(n, 1)
    val_d = torch.full((16,), 7.0, dtype=torch.float32, device="cuda")
    idx_d = torch.full((16,), -7, dtype=torch.int64, device="cuda")
    with pytest.raises(deft.DeftError) as ei:
        deft.deft_topk_baseline(acc_d, 8, val_d[:8], idx_d[:8], ws)
    assert ei.value.status == deft.ERR_TOO_LARGE
    torch.cuda.synchronize()
    assert torch.all(val_d == 7.0) and torch.all(idx_d == -7)
    del acc_d, ws
    torch.cuda.empty_cache()


def test_staging_in_the_accumulate_pass_never_changes_the_result(deft):
    """deft_step for all workers stages above the remembered cuts while it accumulates, before this step's
    norms and k_l exist.  Steps whose gradients jump up (far too many entries staged: the per-tile lists
    overflow) and down (too few staged) must come out like every other step: the layers concerned are
    searched in full.  Every step is compared with the oracle, and with the same step without staging."""
    from paper_2307_03500_b200.pipeline import DeftStep
    w = W.scaled_down(W.bert_large(), 16)
    N = w.n_workers
    start, _ = oracle.split_layers(w.sizes, N)
    scales = [1.0, 1.0, 1.0, 64.0, 1.0, 1.0 / 4096.0, 1.0, 1.0]
    try:
        deft.deft_debug_select_kernel(True)      # the vector is below the size at which the default takes this path
        ds = {True: DeftStep(w.sizes, N, w.density), False: DeftStep(w.sizes, N, w.density)}
        e = {True: torch.zeros(w.n_g, dtype=torch.float32, device="cuda"),
             False: torch.zeros(w.n_g, dtype=torch.float32, device="cuda")}
        acc = np.zeros(w.n_g, dtype=np.float32)
        for t, sc in enumerate(scales):
            g = (w.gradient(t) * np.float32(sc)).astype(np.float32)
            g_d = _dev(g)
            plans = {}
            for staged in (True, False):
                deft.deft_debug_step_staging(staged)
                plans[staged] = ds[staged].step_fused(e[staged], g_d, iteration=t)
                torch.cuda.synchronize()
            oracle.accumulate(acc, g)
            plan = plans[True]
            assert plan.k_l.tolist() == plans[False].k_l.tolist()
            want_val, want_idx = [], []
            for r in range(N):
                v, i = oracle.select_rank(acc, start, plan.k_l, oracle.my_layers(plan.bin_of_layer, t, r, N))
                want_val.append(v)
                want_idx.append(i)
            want_val, want_idx = np.concatenate(want_val), np.concatenate(want_idx)
            acc[want_idx] = 0.0
            for staged in (True, False):
                s = plan.sum_k
                assert np.array_equal(ds[staged].idx_d[:s].cpu().numpy(), want_idx), (t, staged)
                assert ds[staged].val_d[:s].cpu().numpy().tobytes() == want_val.tobytes(), (t, staged)
                assert e[staged].cpu().numpy().tobytes() == acc.tobytes(), (t, staged)
        st = deft.deft_select_stats(ds[True].ws, ds[True].L)
        assert st["one_read"] > 0 and st["staged_entries"] > 0      # layers were finished from what the pass staged
        assert st["cut_failed"] > 0                                   # and the jumps made cuts fail
    finally:
        deft.deft_debug_select_kernel(None)
        deft.deft_debug_step_staging(True)


def test_many_steps_staged_and_unstaged_agree(deft):
    """Sixty steps with the residual carried over, gradients repeated, rescaled and now and then jumping by
    a factor of 16 or 1/64: the step that stages in its accumulate pass and the step whose selection launch
    reads the vector itself (alternating between its two ways of reading) must leave the same bytes
    every time.  (The unstaged step is compared with the oracle elsewhere.)"""
    from paper_2307_03500_b200.pipeline import DeftStep
    w = W.scaled_down(W.bert_large(), 16)
    N = w.n_workers
    rng = np.random.default_rng(5)
    try:
        deft.deft_debug_select_kernel(True)
        ds_a, ds_b = DeftStep(w.sizes, N, w.density), DeftStep(w.sizes, N, w.density)
        e_a = torch.zeros(w.n_g, dtype=torch.float32, device="cuda")
        e_b = torch.zeros_like(e_a)
        for t in range(60):
            g = W.device_gradient(w, t % 5 if t % 11 < 4 else 100 + t, "cuda")
            g.mul_(float(np.exp(rng.normal(0, 0.15))) * (16.0 if t % 17 == 16 else 1.0) * (1 / 64.0 if t % 23 == 22 else 1.0))
            deft.deft_debug_step_staging(True)
            deft.deft_debug_select_ring(True)
            plan_a = ds_a.step_fused(e_a, g, t)
            deft.deft_debug_step_staging(False)
            deft.deft_debug_select_ring(t % 2 == 0)
            plan_b = ds_b.step_fused(e_b, g, t)
            torch.cuda.synchronize()
            s = plan_a.sum_k
            assert plan_a.k_l.tolist() == plan_b.k_l.tolist(), t
            assert torch.equal(ds_a.idx_d[:s], ds_b.idx_d[:s]) and torch.equal(ds_a.val_d[:s], ds_b.val_d[:s]), t
            assert torch.equal(e_a, e_b), t
        st = deft.deft_select_stats(ds_a.ws, ds_a.L)
        assert st["one_read"] > 0 and st["cut_failed"] > 0 and st["ring_gave_up"] == 0
    finally:
        deft.deft_debug_select_kernel(None)
        deft.deft_debug_step_staging(True)
        deft.deft_debug_select_ring(True)
