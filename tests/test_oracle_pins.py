"""Pins for the CPU oracle: it is checked against things other than itself.

Hand-evaluated cases (tests/golden), closed forms, invariants the paper states,
library routines (numpy.linalg.norm, torch.topk), exact rational arithmetic and
brute force on tiny inputs.  None of this needs a GPU.
"""
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2307_03500_b200 import workloads as W


@pytest.fixture(scope="module")
def golden(golden_dir):
    with open(os.path.join(golden_dir, "hand_worked.json")) as f:
        return json.load(f)


# --------------------------------------------------------------------------
# Algorithm 2
# --------------------------------------------------------------------------
def test_split_hand_worked(golden):
    for c in golden["split_layers"]:
        start, tensor = oracle.split_layers(c["sizes"], c["n_workers"])
        assert start.tolist() == c["layer_start"], c["cite"]
        assert tensor.tolist() == c["layer_tensor"], c["cite"]


@pytest.mark.parametrize("name,N,L_expected", [
    ("tiny", 4, 14), ("resnet18", 16, 122), ("lstm_lm", 16, 101), ("bert_large", 32, 416),
    ("gpt2_medium", 1, 292), ("gpt2_medium", 4, 292), ("gpt2_medium", 8, 299), ("gpt2_medium", 16, 307),
    ("gpt2_medium", 32, 323), ("gpt2_medium", 64, 355),
])
def test_split_invariants(name, N, L_expected):
    w = W.WORKLOADS[name]()
    sizes = np.asarray(w.sizes, dtype=np.int64)
    n_g = int(sizes.sum())
    start, tensor = oracle.split_layers(sizes, N)
    L = start.size - 1
    # count: T - (#split) + N * (#split), computed from the definition "size > n_g / N"
    n_split = int(sum(1 for s in w.sizes if s * N > n_g))
    assert L == len(w.sizes) - n_split + N * n_split == L_expected
    # contiguous cover of [0, n_g)
    assert start[0] == 0 and start[-1] == n_g and np.all(np.diff(start) > 0)
    # Section 4.1: no layer above ceil(n_g / N)
    assert int(np.diff(start).max()) <= -(-n_g // N)
    # fragments of one tensor: sizes differ by at most one, larger ones first, sum to the tensor
    for t, s in enumerate(w.sizes):
        frag = np.diff(start)[tensor == t]
        assert int(frag.sum()) == s
        if s * N > n_g:
            assert frag.size == N and frag.max() - frag.min() <= 1 and np.all(np.diff(frag) <= 0)
            assert int((frag == frag.max()).sum()) == (s % N if s % N else N)
        else:
            assert frag.size == 1


def test_split_drops_empty_fragments():
    # 3 elements over 4 workers: quotient 0, remainder 3 -> three 1-element layers
    start, tensor = oracle.split_layers([3, 1], 4)
    assert start.tolist() == [0, 1, 2, 3, 4] and tensor.tolist() == [0, 0, 0, 1]


# --------------------------------------------------------------------------
# accumulate + norms
# --------------------------------------------------------------------------
def test_accumulate_is_one_fp32_add():
    rng = np.random.default_rng(5)
    e = rng.standard_normal(10007, dtype=np.float32)
    g = (rng.standard_normal(10007) * 1e-3).astype(np.float32)
    want = (e.astype(np.float64) + g.astype(np.float64)).astype(np.float32)  # exact sum, one rounding
    got = oracle.accumulate(e.copy(), g)
    assert got.tobytes() == want.tobytes()


def test_norms_closed_forms():
    # all-ones layer of m*m elements -> m exactly; powers of two; zero layer -> 0
    m = 37
    acc = np.concatenate([
        np.ones(m * m, dtype=np.float32),
        np.zeros(100, dtype=np.float32),
        np.array([3.0, -4.0], dtype=np.float32),
        np.full(4, 2.0 ** -70, dtype=np.float32) * np.array([1, -1, 1, -1], dtype=np.float32),
        np.array([-0.0], dtype=np.float32),
    ])
    start = np.array([0, m * m, m * m + 100, m * m + 102, m * m + 106, m * m + 107])
    n = oracle.layer_norms(acc, start)
    assert n[0] == float(m) and n[1] == 0.0 and n[2] == 5.0 and n[3] == 2.0 ** -69 and n[4] == 0.0


def test_norms_match_numpy_library():
    w = W.tiny()
    acc = w.gradient(0)
    start, _ = oracle.split_layers(w.sizes, w.n_workers)
    n = oracle.layer_norms(acc, start)
    for l in range(start.size - 1):
        ref = np.linalg.norm(acc[start[l]:start[l + 1]].astype(np.float64))
        assert abs(n[l] - ref) <= 1e-13 * ref
        ref2 = math.sqrt(math.fsum(float(x) * float(x) for x in acc[start[l]:start[l + 1]][:2000])) if l == 1 else None
        if ref2 is not None:  # layer 1 has 64 elements: exactly-rounded sum
            assert abs(n[l] - ref2) <= 4e-16 * ref2


# --------------------------------------------------------------------------
# Algorithm 3
# --------------------------------------------------------------------------
def test_allocate_hand_worked(golden):
    for c in golden["allocate_k"]:
        kp, sp = oracle.allocate_k(c["norms"], c["sizes"], c["k"], oracle.MODE_PAPER)
        assert kp.tolist() == c["paper"] and sp == sum(c["paper"]), c["cite"]
        ke, se = oracle.allocate_k(c["norms"], c["sizes"], c["k"], oracle.MODE_EXACT)
        assert ke.tolist() == c["exact"] and se == c["k"], c["cite"]


def _alg3_exact_rational(norms, sizes, k):
    """Algorithm 3 in exact rational arithmetic (what the recursion means before rounding)."""
    L = len(norms)
    order = sorted(range(L), key=lambda l: (-norms[l], l))
    fr = [Fraction(x) for x in norms]
    k_remain = Fraction(k)
    norm_remain = sum(fr[l] for l in order)
    out = [0] * L
    near_integer = False
    for p, l in enumerate(order):
        k_temp = k_remain * fr[l] / norm_remain if norm_remain > 0 else Fraction(0)
        # the last layer's ratio is exactly 1 and a zero norm gives exactly 0 in fp64 too
        exact_in_fp64 = (p == L - 1) or fr[l] == 0
        if not exact_in_fp64 and abs(k_temp - round(k_temp)) < Fraction(1, 10 ** 9):
            near_integer = True
        fl = math.floor(k_temp)
        out[l] = sizes[l] if sizes[l] < k_temp else max(1, fl)
        k_remain -= out[l]
        norm_remain -= fr[l]
    return out, near_integer


def test_allocate_matches_exact_rational_arithmetic():
    rng = np.random.default_rng(11)
    checked = 0
    for trial in range(400):
        L = int(rng.integers(1, 13))
        norms = np.exp(rng.uniform(-6, 3, size=L))
        if trial % 7 == 0:
            norms[rng.integers(0, L)] = 0.0
        sizes = rng.integers(1, 5000, size=L)
        k = int(rng.integers(1, max(2, int(sizes.sum()))))
        want, near = _alg3_exact_rational(norms.tolist(), sizes.tolist(), k)
        if near:
            continue  # a product within 1e-9 of an integer: fp64 may legitimately floor differently
        got, s = oracle.allocate_k(norms, sizes, k, oracle.MODE_PAPER)
        assert got.tolist() == want
        assert s == sum(want)
        checked += 1
    assert checked > 300


def test_allocate_invariants_and_exact_sum():
    rng = np.random.default_rng(12)
    for trial in range(300):
        L = int(rng.integers(1, 60))
        norms = np.exp(rng.uniform(-9, 4, size=L))
        sizes = rng.integers(1, 100000, size=L)
        n_g = int(sizes.sum())
        k = int(rng.integers(L, n_g + 1))
        for mode in (oracle.MODE_PAPER, oracle.MODE_EXACT):
            k_l, s = oracle.allocate_k(norms, sizes, k, mode)
            assert np.all(k_l >= 1) and np.all(k_l <= sizes) and s == int(k_l.sum())
            if mode == oracle.MODE_EXACT:
                assert s == k


def _exact_repair(k_paper, norms, sizes, k):
    """The EXACT mode's integer repair restated: shortfall handed out in priority order up to
    each layer's size; surplus taken back one per layer per round, in priority order, never
    below 1 (priority = norm descending, equal norms by lower layer id)."""
    out = list(k_paper)
    order = sorted(range(len(out)), key=lambda l: (-norms[l], l))
    rem = k - sum(out)
    for l in order:
        add = min(sizes[l] - out[l], max(rem, 0))
        out[l] += add
        rem -= add
    while rem < 0:
        for l in order:
            if rem < 0 and out[l] > 1:
                out[l] -= 1
                rem += 1
    return out


def test_allocate_exact_repair_follows_priority_order():
    # PAPER mode is pinned by exact rational arithmetic above; EXACT = PAPER + the repair.  The cases
    # are built so that the repair fires (many near-zero norms: floor-1 surplus; small sizes under large
    # norms: size-clamp shortfall) and priority order is a random permutation of id order.
    rng = np.random.default_rng(17)
    fired_short = fired_surplus = differs_from_id_order = 0
    for trial in range(600):
        L = int(rng.integers(2, 24))
        norms = np.exp(rng.uniform(-2, 3, size=L))
        tiny = rng.random(L) < (0.5 if trial % 2 else 0.1)
        norms[tiny] = rng.choice([0.0, 1e-9, 1e-7], size=int(tiny.sum()))
        sizes = rng.integers(1, 40, size=L) if trial % 2 == 0 else rng.integers(50, 500, size=L)
        n_g = int(sizes.sum())
        k = int(rng.integers(L, n_g + 1))
        kp, sp = oracle.allocate_k(norms, sizes, k, oracle.MODE_PAPER)
        ke, se = oracle.allocate_k(norms, sizes, k, oracle.MODE_EXACT)
        want = _exact_repair(kp.tolist(), norms.tolist(), sizes.tolist(), k)
        assert ke.tolist() == want and se == k
        fired_short += sp < k
        fired_surplus += sp > k
        # the same repair walked in id order (what a wrong implementation would do)
        by_id = _exact_repair(kp.tolist(), [0.0] * L, sizes.tolist(), k)
        differs_from_id_order += by_id != want
    assert fired_short > 50 and fired_surplus > 50 and differs_from_id_order > 50


def test_allocate_special_cases():
    # one layer: min(size, k)
    assert oracle.allocate_k([2.5], [100], 7, oracle.MODE_PAPER)[0].tolist() == [7]
    assert oracle.allocate_k([2.5], [5], 7, oracle.MODE_PAPER)[0].tolist() == [5]
    # equal norms, ample sizes: k_l follows floor(k_remain / layers_left)
    L, k = 9, 1000
    k_l, s = oracle.allocate_k([1.0] * L, [10 ** 6] * L, k, oracle.MODE_PAPER)
    k_remain, want = k, []
    for p in range(L):
        want.append(k_remain // (L - p))
        k_remain -= want[-1]
    assert k_l.tolist() == want and s == k
    # doubling every norm changes nothing (only ratios enter)
    rng = np.random.default_rng(3)
    norms = np.exp(rng.uniform(-3, 3, size=20))
    sizes = rng.integers(100, 10000, size=20)
    a = oracle.allocate_k(norms, sizes, 5000, oracle.MODE_PAPER)[0]
    b = oracle.allocate_k(norms * 2.0, sizes, 5000, oracle.MODE_PAPER)[0]
    assert a.tolist() == b.tolist()


def test_allocate_proportionality_bound():
    # Without clamp events, layer at priority position p obeys
    #   k*norm/S_0 - 1 < k_l <= k*norm/S_0 + p*norm/S_p      (S_p = norm sum from position p on)
    rng = np.random.default_rng(13)
    for trial in range(100):
        L = int(rng.integers(2, 30))
        norms = np.exp(rng.uniform(-1, 1, size=L))
        sizes = np.full(L, 10 ** 9)
        k = int(rng.integers(200 * L, 10 ** 6))
        k_l, s = oracle.allocate_k(norms, sizes, k, oracle.MODE_PAPER)
        assert s == k and np.all(k_l > 1)
        order = np.argsort(-norms, kind="stable")
        S = np.cumsum(norms[order][::-1])[::-1]
        for p, l in enumerate(order):
            share = k * norms[l] / S[0]
            assert share - 1 - 1e-6 < k_l[l] <= share + p * norms[l] / S[p] + 1e-6


def test_allocate_rejects_bad_input():
    with pytest.raises(ValueError):
        oracle.allocate_k([1.0, float("nan")], [10, 10], 5, oracle.MODE_PAPER)
    with pytest.raises(ValueError):
        oracle.allocate_k([1.0, 1.0], [10, 10], 1, oracle.MODE_EXACT)   # k < L
    with pytest.raises(ValueError):
        oracle.allocate_k([1.0, 1.0], [10, 10], 21, oracle.MODE_EXACT)  # k > n_g


# --------------------------------------------------------------------------
# Algorithm 4
# --------------------------------------------------------------------------
def test_partition_hand_worked(golden):
    for c in golden["partition"]:
        bins, load = oracle.partition(c["sizes"], c["k_l"], c["n_workers"])
        assert bins.tolist() == c["bin_of_layer"], c["cite"]
        if c["load_in_units_of_ln_k"] is not None:
            unit = math.log(c["k_l"][0])
            assert np.allclose(load, np.array(c["load_in_units_of_ln_k"]) * unit, rtol=1e-14)
    for c in golden["rank_bin"]:
        assert oracle.rank_bin(c["iteration"], c["rank"], c["n_workers"]) == c["bin"], c["cite"]


def test_partition_is_lpt_within_graham_bound_of_exhaustive_optimum():
    rng = np.random.default_rng(21)
    for trial in range(60):
        L = int(rng.integers(1, 10))
        N = int(rng.integers(1, 5))
        sizes = rng.integers(1, 1000, size=L)
        k_l = np.minimum(sizes, rng.integers(1, 50, size=L))
        cost = sizes * np.log(k_l.astype(np.float64))
        bins, load = oracle.partition(sizes, k_l, N)
        # loads are what the assignment says
        for b in range(N):
            assert abs(load[b] - cost[bins == b].sum()) <= 1e-9 * max(1.0, cost.sum())
        assert bins.min() >= 0 and bins.max() < N
        opt = oracle.partition_optimum(cost, N)
        mk = load.max()
        assert mk >= opt - 1e-9
        assert mk <= (4.0 / 3.0 - 1.0 / (3.0 * N)) * opt + 1e-9          # Graham's LPT bound
        assert mk >= max(cost.max(), cost.sum() / N) - 1e-9
        assert mk <= cost.sum() / N + (1.0 - 1.0 / N) * cost.max() + 1e-9
        if N == 1 or L <= N:
            assert abs(mk - opt) <= 1e-9


def test_partition_optimum_brute_force_is_right_on_a_known_case():
    # {5,4} | {3,3,3}: optimum 9, while largest-first packing gives 10
    assert oracle.partition_optimum([5, 4, 3, 3, 3], 2) == 9.0
    assert oracle.partition_optimum([7.0], 3) == 7.0
    assert oracle.partition_optimum([1, 1, 1, 1, 1, 1], 3) == 2.0


def test_partition_equal_costs_divide_evenly():
    bins, load = oracle.partition([10] * 12, [4] * 12, 4)
    assert sorted(np.bincount(bins, minlength=4).tolist()) == [3, 3, 3, 3]
    assert np.allclose(load, 30 * math.log(4))


def test_partition_by_size_hand_case_and_bounds():
    # sizes 5,4,3,3,3 on two bins, largest first into the lighter bin (first bin on ties):
    # 5->b0, 4->b1, 3->b1 (4<5), 3->b0 (5<7), 3->b1 (7<8): loads 8 | 10
    bins, load = oracle.partition_by_size([5, 4, 3, 3, 3], 2)
    assert bins.tolist() == [0, 1, 1, 0, 1] and load.tolist() == [8.0, 10.0]
    rng = np.random.default_rng(23)
    for trial in range(40):
        L = int(rng.integers(1, 10))
        N = int(rng.integers(1, 5))
        sizes = rng.integers(1, 1000, size=L)
        bins, load = oracle.partition_by_size(sizes, N)
        for b in range(N):
            assert load[b] == float(sizes[bins == b].sum())             # integer-valued doubles: exact
        opt = oracle.partition_optimum(sizes.astype(np.float64), N)
        assert opt - 1e-9 <= load.max() <= (4.0 / 3.0 - 1.0 / (3.0 * N)) * opt + 1e-9
    # with equal k_l the two load models rank the layers alike and pack identically
    sizes = rng.integers(100, 10_000, size=25)
    b_eq3, _ = oracle.partition(sizes, np.full(25, 7), 4)
    b_size, _ = oracle.partition_by_size(sizes, 4)
    assert b_eq3.tolist() == b_size.tolist()


# --------------------------------------------------------------------------
# Algorithm 5 / Top-k
# --------------------------------------------------------------------------
def test_select_hand_worked(golden):
    for c in golden["select"]:
        x = np.array(c["x"], dtype=np.float32)
        val, idx = oracle.select_layer(x, c["st"], c["end"], c["k"])
        assert idx.tolist() == c["idx"] and val.tolist() == c["val"], c["cite"]


def _brute_force_select(x, st, end, k):
    keys = x.view(np.uint32) & np.uint32(0x7FFFFFFF)
    chosen = []
    taken = set()
    for _ in range(k):  # k times: scan for the largest remaining magnitude, first occurrence
        best = -1
        for i in range(st, end):
            if i in taken:
                continue
            if best < 0 or keys[i] > keys[best]:
                best = i
        taken.add(best)
        chosen.append(best)
    chosen.sort()
    return chosen


@pytest.mark.parametrize("kind", ["gauss", "few_values", "all_equal", "all_zero", "signed_zero",
                                  "mostly_zero", "outlier", "bf16_like", "denormal", "wide_exponent"])
def test_select_matches_brute_force(kind):
    for n, k in [(1, 1), (10, 1), (10, 10), (33, 7), (200, 31), (257, 200)]:
        x = W.adversarial_vector(kind, n, seed=n)
        val, idx = oracle.select_layer(x, 0, n, k)
        want = _brute_force_select(x, 0, n, k)
        assert idx.tolist() == want
        assert val.tobytes() == x[want].tobytes()


def test_select_matches_torch_topk_when_magnitudes_are_distinct():
    rng = np.random.default_rng(31)
    n = 200000
    x = rng.permutation(n).astype(np.float32) + 1.0   # distinct magnitudes
    x *= rng.choice([-1.0, 1.0], size=n).astype(np.float32)
    for st, end, k in [(0, n, 1000), (1234, 150001, 17), (n - 5000, n, 4999)]:
        val, idx = oracle.select_layer(x, st, end, k)
        ref = torch.topk(torch.from_numpy(x[st:end]).abs(), k).indices.numpy() + st
        assert idx.tolist() == sorted(ref.tolist())
        assert val.tobytes() == x[idx].tobytes()


def test_select_threshold_invariants_with_ties():
    x = W.adversarial_vector("few_values", 50000, seed=9)
    keys = (x.view(np.uint32) & np.uint32(0x7FFFFFFF)).astype(np.int64)
    for k in (1, 777, 25000, 49999, 50000):
        val, idx = oracle.select_layer(x, 0, x.size, k)
        assert idx.size == k and np.all(np.diff(idx) > 0)
        sel = np.zeros(x.size, dtype=bool)
        sel[idx] = True
        if k < x.size:
            thr = keys[sel].min()
            assert thr >= keys[~sel].max()
            # among entries equal to the threshold the selected ones are the lowest indices
            eq = np.nonzero(keys == thr)[0]
            n_eq_sel = int(sel[eq].sum())
            assert np.all(sel[eq[:n_eq_sel]]) and not np.any(sel[eq[n_eq_sel:]])


def test_single_layer_deft_is_conventional_topk():
    x = W.adversarial_vector("gauss", 30000, seed=2)
    v1, i1 = oracle.topk(x, 300)
    v2, i2 = oracle.select_rank(x, [0, x.size], [300], [0])
    assert i1.tolist() == i2.tolist() and v1.tobytes() == v2.tobytes()


# --------------------------------------------------------------------------
# residual update and the whole path
# --------------------------------------------------------------------------
def test_residual_update_properties():
    x = W.adversarial_vector("gauss", 40000, seed=4)
    val, idx = oracle.topk(x, 4000)
    before = x.copy()
    oracle.residual_update(x, idx)
    sel = np.zeros(x.size, dtype=bool)
    sel[idx] = True
    assert x[~sel].tobytes() == before[~sel].tobytes()
    assert np.all(x[sel].view(np.uint32) == 0)   # +0.0f
    e0 = float(np.sum(before.astype(np.float64) ** 2))
    e1 = float(np.sum(val.astype(np.float64) ** 2)) + float(np.sum(x.astype(np.float64) ** 2))
    assert abs(e0 - e1) <= 1e-12 * e0
    # selecting everything leaves an all-zero residual
    val, idx = oracle.topk(before, before.size)
    y = before.copy()
    oracle.residual_update(y, idx)
    assert not y.any()


@pytest.mark.parametrize("wl", ["tiny", "resnet_div16", "bert_div256", "gpt2_div256"])
def test_whole_path_partitions_are_disjoint_and_density_is_kept(wl):
    w = {"tiny": W.tiny(),
         "resnet_div16": W.scaled_down(W.resnet18(), 16),
         "bert_div256": W.scaled_down(W.bert_large(), 256),
         "gpt2_div256": W.scaled_down(W.gpt2_medium(8, 0.01), 256)}[wl]
    N = w.n_workers
    acc = oracle.accumulate(np.zeros(w.n_g, dtype=np.float32), w.gradient(0))
    start, _ = oracle.split_layers(w.sizes, N)
    size = np.diff(start)
    norms = oracle.layer_norms(acc, start)
    k = max(w.k, size.size)
    k_l, s = oracle.allocate_k(norms, size, k, oracle.MODE_EXACT)
    assert s == k
    bins, load = oracle.partition(size, k_l, N)
    seen = np.zeros(w.n_g, dtype=np.int32)
    layers_seen = []
    for it in (0, 3):
        seen[:] = 0
        layers_seen.clear()
        for r in range(N):
            my = oracle.my_layers(bins, it, r, N)
            layers_seen += my.tolist()
            val, idx = oracle.select_rank(acc, start, k_l, my)
            assert idx.size == int(k_l[my].sum())
            assert np.all(np.diff(idx) > 0)
            seen[idx] += 1
        assert sorted(layers_seen) == list(range(size.size))      # bins cover every layer once
        assert seen.max() == 1 and int(seen.sum()) == k           # no overlap, no build-up: density kept
    # per-layer counts
    for l in range(size.size):
        assert int(seen[start[l]:start[l + 1]].sum()) == k_l[l]


# ------------------------------------------------------------------------------------------
# comparison sparsifiers (Section 3): hard threshold, CLT-k
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("kind", ["gauss", "wide_exponent", "few_values", "mostly_zero", "signed_zero", "denormal"])
def test_threshold_select_equals_numpy_mask(kind):
    x = W.adversarial_vector(kind, 50_003, seed=21)
    for lam in (0.0, 1e-30, 0.25, 0.5, 1.0, 3.0, 1e30):
        val, idx = oracle.threshold_select(x, lam)
        want = np.nonzero(np.abs(x) > np.float32(lam))[0]       # library routine on finite data
        assert np.array_equal(idx, want)
        assert val.tobytes() == x[want].tobytes()


def test_threshold_select_hand_cases():
    x = np.array([0.5, -0.5, 0.25, -0.0, 0.0, np.inf, -np.inf, 1e-45, -3.0], dtype=np.float32)
    val, idx = oracle.threshold_select(x, 0.5)                    # strict: 0.5 itself is not selected
    assert idx.tolist() == [5, 6, 8] and val.tolist() == [np.inf, -np.inf, -3.0]
    val, idx = oracle.threshold_select(x, 0.0)                    # everything but the zeros (the denormal counts)
    assert idx.tolist() == [0, 1, 2, 5, 6, 7, 8]
    val, idx = oracle.threshold_select(x, np.inf)
    assert idx.size == 0
    y = np.array([1.0, np.nan, 2.0], dtype=np.float32)            # NaN sorts above everything, as in Algorithm 5
    assert oracle.threshold_select(y, 1e38)[1].tolist() == [1]
    assert oracle.threshold_select(x, -0.5)[1].tolist() == [5, 6, 8]   # the threshold's sign is ignored


def test_threshold_at_the_kth_magnitude_reproduces_topk_when_magnitudes_are_distinct():
    rng = np.random.default_rng(5)
    x = np.unique(np.abs(rng.standard_normal(30_000).astype(np.float32)))[:20_001].copy()   # distinct magnitudes
    rng.shuffle(x)
    x *= rng.choice(np.array([-1.0, 1.0], dtype=np.float32), size=x.size)
    mags = np.sort(np.abs(x))[::-1]
    assert np.unique(mags).size == mags.size == 20_001
    for k in (1, 17, 2000, 20_000):
        lam = float(mags[k])                                        # the (k+1)-th largest magnitude
        val, idx = oracle.threshold_select(x, lam)
        tv, ti = oracle.topk(x, k)
        assert np.array_equal(idx, ti) and val.tobytes() == tv.tobytes()


def test_clt_leader_cycles_and_gather_update():
    assert [oracle.clt_leader(t, 4) for t in range(9)] == [0, 1, 2, 3, 0, 1, 2, 3, 0]
    assert oracle.clt_leader(7, 1) == 0
    rng = np.random.default_rng(6)
    x = rng.standard_normal(1000).astype(np.float32)
    idx = np.sort(rng.choice(1000, size=100, replace=False)).astype(np.int64)
    y = x.copy()
    val = oracle.gather_update(y, idx)
    assert val.tobytes() == x[idx].tobytes()
    want = x.copy()
    want[idx] = 0.0
    assert y.tobytes() == want.tobytes()
    # a follower's contribution at the leader's indices: leader selects, follower gathers
    leader_vec = rng.standard_normal(1000).astype(np.float32)
    _, lidx = oracle.topk(leader_vec, 10)
    f = x.copy()
    fv = oracle.gather_update(f, lidx)
    assert np.array_equal(fv, x[lidx]) and not f[lidx].any() and np.count_nonzero(f != x) == np.count_nonzero(x[lidx])


# --------------------------------------------------------------------------
# Algorithm 1 around the sparsifier (lines 7-9) and Eq. 2
# --------------------------------------------------------------------------
def test_index_union_is_the_sorted_set():
    assert oracle.index_union([5, 3, 5, 1, 3]).tolist() == [1, 3, 5]          # by hand
    assert oracle.index_union([]).tolist() == []
    assert oracle.index_union([7]).tolist() == [7]
    rng = np.random.default_rng(21)
    for trial in range(20):
        idx = rng.integers(0, 500, size=int(rng.integers(1, 2000)))
        u = oracle.index_union(idx)
        assert set(u.tolist()) == set(idx.tolist())                          # the same set ...
        assert np.all(np.diff(u) > 0)                                        # ... strictly ascending
    # disjoint lists (DEFT's workers): nothing is lost, the size is the sum of the sizes
    parts = [np.arange(r, 400, 4) for r in range(4)]
    assert oracle.index_union(np.concatenate(parts[::-1])).tolist() == list(range(400))


def test_sum_and_average_are_single_fp32_operations():
    rng = np.random.default_rng(22)
    a = rng.standard_normal(5000).astype(np.float32)
    b = (rng.standard_normal(5000) * 1e-3).astype(np.float32)
    want = (a.astype(np.float64) + b.astype(np.float64)).astype(np.float32)   # exact sum, one rounding
    assert oracle.sum_into(a.copy(), b).tobytes() == want.tobytes()
    for n in (2, 3, 7, 32):
        q = (a.astype(np.float64) / n).astype(np.float32)                      # exact quotient of two floats, one rounding
        assert oracle.average(a.copy(), n).tobytes() == q.tobytes()
    # worked by hand: (1 + 2 + 6) / 3 = 3
    s = np.array([1.0], dtype=np.float32)
    oracle.sum_into(s, np.array([2.0], dtype=np.float32))
    oracle.sum_into(s, np.array([6.0], dtype=np.float32))
    assert oracle.average(s, 3).tolist() == [3.0]


def test_vector_norm_and_eq2():
    assert oracle.vector_norm(np.array([3.0, -4.0], dtype=np.float32)) == 5.0
    assert oracle.vector_norm(np.ones(49, dtype=np.float32)) == 7.0
    assert oracle.vector_norm(np.zeros(10, dtype=np.float32)) == 0.0
    rng = np.random.default_rng(23)
    x = rng.standard_normal(100000).astype(np.float32)
    ref = float(np.linalg.norm(x.astype(np.float64)))
    assert abs(oracle.vector_norm(x) - ref) <= 1e-12 * ref
    # the norm of the whole vector from the norms of its layers (Pythagoras)
    start = np.array([0, 10, 5000, 100000], dtype=np.int64)
    nl = oracle.layer_norms(x, start)
    assert abs(oracle.vector_norm(x) - math.sqrt(float(np.sum(nl * nl)))) <= 1e-12 * ref
    # Eq. 2 by hand: (1 + 2 + 6) / 3
    assert oracle.error_eq2([1.0, 2.0, 6.0]) == 3.0
    assert oracle.error_eq2([2.5]) == 2.5


def test_threaded_rank_selection_equals_the_plain_one():
    rng = np.random.default_rng(24)
    sizes = rng.integers(1, 3000, size=40)
    start = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    acc = rng.standard_normal(int(start[-1])).astype(np.float32)
    k_l = np.array([int(rng.integers(1, s + 1)) for s in sizes], dtype=np.int64)
    my = np.arange(0, 40, 3, dtype=np.int32)
    v0, i0 = oracle.select_rank(acc, start, k_l, my)
    for threads in (1, 2, 0):
        v1, i1, used = oracle.select_rank_threads(acc, start, k_l, my, threads)
        assert used >= 1 and i1.tolist() == i0.tolist() and v1.tobytes() == v0.tobytes()
