// DEFT gradient-selection oracle: TEST INFRASTRUCTURE, NOT THE PRODUCT.
//
// A plain, slow CPU statement of what the DEFT hot path
// computes (Yoon & Oh, "DEFT: Exploiting Gradient Norm Difference between
// Model Layers for Scalable Gradient Sparsification", ICPP 2023).  It is
// used only by the tests, the smoke check and the benchmark's CPU-baseline
// leg (one routine below runs a rank's layers on several host threads for that
// leg's all-cores figure; everything else is single-threaded).  It shares no code, header, table or helper with the CUDA library
// and neither side includes or links the other.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -fPIC -shared (no fast-math,
// no FTZ/DAZ), so every fp64 operation below is one IEEE round-to-nearest
// operation in the order written.
//
// Parity pins (all in tests/, run without a GPU): every function here is
// pinned by closed forms, invariants, library routines, exact rational
// arithmetic or brute force; none is "parity unpinned".
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <utility>
#include <vector>

extern "C" {

// ---------------------------------------------------------------------------
// Algorithm 2 (two-stage gradient vector partitioning), Section 4.1.
// A tensor whose size exceeds n_g / n_workers is cut into n_workers
// contiguous fragments; the first (size % n_workers) fragments hold one
// element more than the quotient.  Every fragment and every unsplit tensor
// is a "layer".  The comparison `size > n_g / N` is evaluated as
// `size * N > n_g` in integers, which is the same predicate for real and
// for floor division.  Fragments of size zero (only possible when a split
// tensor has fewer elements than workers) are dropped.
// Returns the number of layers L, or -1 if cap is too small / input invalid.
// layer_start has L+1 entries, layer_tensor[l] is the source tensor id.
// ---------------------------------------------------------------------------
int64_t oracle_split_layers(const int64_t* tensor_sizes, int64_t T, int64_t n_workers,
                            int64_t* layer_start, int32_t* layer_tensor, int64_t cap) {
    if (T < 1 || n_workers < 1) return -1;
    int64_t n_g = 0;
    for (int64_t t = 0; t < T; ++t) {
        if (tensor_sizes[t] < 1) return -1;
        n_g += tensor_sizes[t];
    }
    int64_t L = 0;
    int64_t alloc_pos = 0;
    for (int64_t t = 0; t < T; ++t) {
        const int64_t size = tensor_sizes[t];
        if ((__int128)size * (__int128)n_workers > (__int128)n_g) {
            const int64_t quotient = size / n_workers;
            int64_t remainder = size % n_workers;
            for (int64_t i = 0; i < n_workers; ++i) {
                int64_t size_layer = quotient;
                if (remainder > 0) {
                    size_layer = size_layer + 1;
                    remainder = remainder - 1;
                }
                if (size_layer == 0) continue;
                if (L >= cap) return -1;
                layer_start[L] = alloc_pos;
                layer_tensor[L] = (int32_t)t;
                alloc_pos = alloc_pos + size_layer;
                ++L;
            }
        } else {
            if (L >= cap) return -1;
            layer_start[L] = alloc_pos;
            layer_tensor[L] = (int32_t)t;
            alloc_pos = alloc_pos + size;
            ++L;
        }
    }
    layer_start[L] = alloc_pos;
    return L;
}

// ---------------------------------------------------------------------------
// Algorithm 1, line 5: acc = e + eta*G.  The caller passes the already
// scaled gradient, so this is one fp32 round-to-nearest add per element,
// written over e.
// ---------------------------------------------------------------------------
void oracle_accumulate(float* e, const float* g, int64_t n_g) {
    for (int64_t i = 0; i < n_g; ++i) {
        volatile float s = e[i] + g[i];  // volatile: forces the fp32 rounding
        e[i] = s;
    }
}

// ---------------------------------------------------------------------------
// Section 4.2: the gradient norm of each layer (L2, the paper's only stated
// norm, Section 2).  norm_l = sqrt(sum_i acc_i^2), summed sequentially in
// fp64 over the layer.
// ---------------------------------------------------------------------------
void oracle_layer_norms(const float* acc, const int64_t* layer_start, int64_t L, double* norms) {
    for (int64_t l = 0; l < L; ++l) {
        double s = 0.0;
        for (int64_t i = layer_start[l]; i < layer_start[l + 1]; ++i) {
            const double x = (double)acc[i];
            s = s + x * x;
        }
        norms[l] = std::sqrt(s);
    }
}

// ---------------------------------------------------------------------------
// Algorithm 3 (gradient-norm-based local k assignment), Section 4.2.
// Layers are visited in priority order (norm descending, equal norms by
// lower layer id).  Each layer receives
//     k_temp = floor(k_remain * (norm / norm_remain))   (0 if norm_remain <= 0)
//     k_l    = size        if size < k_temp
//              max(1, k_temp) otherwise
// and k_remain is reduced by k_l.  norm_remain for the layer at priority
// position p is the sum of the norms at positions p..L-1, accumulated from
// the back (the same quantity the listing maintains by subtraction, without
// its cancellation error; the last ratio is exactly 1).
//
// mode 0 (PAPER): stop there; sum k_l may differ from k.
// mode 1 (EXACT): integer-only repair so that sum k_l == k.  Shortfall is
//   handed out in priority order up to each layer's size; excess is taken
//   back one element per layer per round, in priority order, never below 1.
//   Needs L <= k <= n_g.
// Returns 0 on success, -2 if EXACT is infeasible, -3 if a norm is not
// finite or negative, -1 on other bad input.  k_l is indexed by layer id.
// ---------------------------------------------------------------------------
int64_t oracle_allocate_k(const double* norms, const int64_t* layer_size, int64_t L, int64_t k,
                          int64_t mode, int64_t* k_l, int64_t* sum_k_out) {
    if (L < 1 || k < 1) return -1;
    int64_t n_g = 0;
    for (int64_t l = 0; l < L; ++l) {
        if (layer_size[l] < 1) return -1;
        if (!std::isfinite(norms[l]) || norms[l] < 0.0) return -3;
        n_g += layer_size[l];
    }
    if (mode == 1 && (k < L || k > n_g)) return -2;

    // priority order
    std::vector<int64_t> order(L);
    for (int64_t l = 0; l < L; ++l) order[l] = l;
    std::stable_sort(order.begin(), order.end(),
                     [&](int64_t a, int64_t b) { return norms[a] > norms[b]; });

    // norm_remain at each priority position
    std::vector<double> norm_remain(L + 1);
    norm_remain[L] = 0.0;
    for (int64_t p = L - 1; p >= 0; --p) norm_remain[p] = norms[order[p]] + norm_remain[p + 1];

    int64_t k_remain = k;
    for (int64_t p = 0; p < L; ++p) {
        const int64_t l = order[p];
        double k_temp;
        if (norm_remain[p] > 0.0) {
            const double ratio = norms[l] / norm_remain[p];
            k_temp = std::floor((double)k_remain * ratio);
        } else {
            k_temp = 0.0;
        }
        int64_t kl;
        if ((double)layer_size[l] < k_temp) {
            kl = layer_size[l];
        } else {
            kl = (k_temp < 1.0) ? 1 : (int64_t)k_temp;
        }
        k_l[l] = kl;
        k_remain = k_remain - kl;
    }

    if (mode == 1) {
        int64_t sum = 0;
        for (int64_t l = 0; l < L; ++l) sum += k_l[l];
        int64_t rem = k - sum;
        if (rem > 0) {
            for (int64_t p = 0; p < L && rem > 0; ++p) {
                const int64_t l = order[p];
                int64_t add = layer_size[l] - k_l[l];
                if (add > rem) add = rem;
                k_l[l] += add;
                rem -= add;
            }
        }
        while (rem < 0) {
            for (int64_t p = 0; p < L && rem < 0; ++p) {
                const int64_t l = order[p];
                if (k_l[l] > 1) {
                    k_l[l] -= 1;
                    rem += 1;
                }
            }
        }
    }
    int64_t sum = 0;
    for (int64_t l = 0; l < L; ++l) sum += k_l[l];
    if (sum_k_out) *sum_k_out = sum;
    return 0;
}

// ---------------------------------------------------------------------------
// Algorithm 4 (bin-packing-based layer allocation), Section 4.3, Eq. 3.
// Every layer has a selection cost; the costliest layer not yet placed goes
// to the worker whose bin is lightest so far, until every layer is placed.
// Equal costs: the layer that comes first in address order.  Equal loads: the
// bin with the lowest number.  (Costs are never negative, so "not yet
// placed" is kept as a flag of its own rather than as a special cost value.)
// Layer ids are positions in address order.
// ---------------------------------------------------------------------------
static void pack_greedily(const std::vector<double>& layer_cost, int64_t n_workers, int32_t* bin_of_layer,
                          double* bin_load /* n_workers */) {
    const int64_t L = (int64_t)layer_cost.size();
    std::vector<char> placed(L, 0);
    for (int64_t b = 0; b < n_workers; ++b) bin_load[b] = 0.0;
    for (int64_t round = 0; round < L; ++round) {
        int64_t costliest = -1;
        for (int64_t l = 0; l < L; ++l) {
            if (placed[l]) continue;
            if (costliest < 0 || layer_cost[l] > layer_cost[costliest]) costliest = l;
        }
        int64_t lightest = 0;
        for (int64_t b = 1; b < n_workers; ++b)
            if (bin_load[b] < bin_load[lightest]) lightest = b;
        bin_of_layer[costliest] = (int32_t)lightest;
        bin_load[lightest] = bin_load[lightest] + layer_cost[costliest];
        placed[costliest] = 1;
    }
}

// Eq. 3: the cost of selecting k_x gradients out of the n_{g,x} of layer x is n_{g,x} * log(k_x)
// (natural logarithm; the base only scales every load).
void oracle_partition(const int64_t* layer_size, const int64_t* k_l, int64_t L, int64_t n_workers,
                      int32_t* bin_of_layer, double* size_bin /* n_workers */) {
    std::vector<double> layer_cost(L);
    for (int64_t l = 0; l < L; ++l) layer_cost[l] = (double)layer_size[l] * std::log((double)k_l[l]);
    pack_greedily(layer_cost, n_workers, bin_of_layer, size_bin);
}

// Variant of Algorithm 4 for hardware whose selection time follows the bytes a worker scans
// rather than size * ln(k) (a linear-time selection): the same greedy packing with the layer's
// size as its cost.  Not in the paper; an ablation of the load model of Eq. 3.
void oracle_partition_by_size(const int64_t* layer_size, int64_t L, int64_t n_workers,
                              int32_t* bin_of_layer, double* size_bin /* n_workers */) {
    std::vector<double> layer_cost(L);
    for (int64_t l = 0; l < L; ++l) layer_cost[l] = (double)layer_size[l];
    pack_greedily(layer_cost, n_workers, bin_of_layer, size_bin);
}

// Algorithm 4, lines 1-2: the bin a rank reads in a given iteration.
int64_t oracle_rank_bin(int64_t iteration, int64_t rank, int64_t n_workers) {
    const int64_t cycle = iteration % n_workers;
    return (cycle + rank) % n_workers;
}

// Smallest possible maximum bin load (Eq. 5 minimised over all n_workers^L
// assignments), by exhaustive enumeration.  For tiny inputs only.
double oracle_partition_optimum(const double* cost, int64_t L, int64_t n_workers) {
    std::vector<int64_t> assign(L, 0);
    std::vector<double> load(n_workers);
    double best = -1.0;
    for (;;) {
        for (int64_t b = 0; b < n_workers; ++b) load[b] = 0.0;
        for (int64_t i = 0; i < L; ++i) load[assign[i]] += cost[i];
        double mx = 0.0;
        for (int64_t b = 0; b < n_workers; ++b) mx = std::max(mx, load[b]);
        if (best < 0.0 || mx < best) best = mx;
        int64_t i = 0;
        while (i < L) {
            if (++assign[i] < n_workers) break;
            assign[i] = 0;
            ++i;
        }
        if (i == L) break;
    }
    return best;
}

// ---------------------------------------------------------------------------
// Algorithm 5 (layer-wise gradient selection), Section 4.4: topk(|acc|, k)
// on one layer [st, end).  Magnitudes are compared as the IEEE bit pattern
// with the sign bit cleared; equal magnitudes are won by the lower index.
// Output: the k selected entries in ascending index, as signed values and
// int64 global indices.  Definition written out: sort everything.
// ---------------------------------------------------------------------------
void oracle_select_layer(const float* acc, int64_t st, int64_t end, int64_t k,
                         float* val_out, int64_t* idx_out) {
    const int64_t n = end - st;
    std::vector<std::pair<uint32_t, int64_t>> items(n);
    for (int64_t i = 0; i < n; ++i) {
        uint32_t bits;
        std::memcpy(&bits, &acc[st + i], 4);
        items[i] = std::make_pair(bits & 0x7fffffffu, st + i);
    }
    std::sort(items.begin(), items.end(),
              [](const std::pair<uint32_t, int64_t>& a, const std::pair<uint32_t, int64_t>& b) {
                  if (a.first != b.first) return a.first > b.first;
                  return a.second < b.second;
              });
    std::vector<int64_t> chosen(k);
    for (int64_t j = 0; j < k; ++j) chosen[j] = items[j].second;
    std::sort(chosen.begin(), chosen.end());
    for (int64_t j = 0; j < k; ++j) {
        idx_out[j] = chosen[j];
        val_out[j] = acc[chosen[j]];
    }
}

// Algorithm 5 over a rank's allocated layers (ascending layer ids): the
// per-layer results concatenated.  Returns the rank's k (sum of k_l).
int64_t oracle_select_rank(const float* acc, const int64_t* layer_start, const int64_t* k_l,
                           const int32_t* my_layers, int64_t n_my, float* val_out,
                           int64_t* idx_out) {
    int64_t k = 0;
    for (int64_t j = 0; j < n_my; ++j) {
        const int64_t part = my_layers[j];
        oracle_select_layer(acc, layer_start[part], layer_start[part + 1], k_l[part], val_out + k,
                            idx_out + k);
        k = k + k_l[part];
    }
    return k;
}

// Algorithm 1, lines 11-12: acc[idx] = 0; the buffer then is e_{t+1}.
void oracle_residual_update(float* acc, const int64_t* idx, int64_t count) {
    for (int64_t j = 0; j < count; ++j) acc[idx[j]] = 0.0f;
}

// ---------------------------------------------------------------------------
// Comparison sparsifiers (Section 3; not part of DEFT itself).
// ---------------------------------------------------------------------------
// Hard-threshold sparsifier (Section 3.2): every entry whose magnitude is larger than a fixed
// threshold is selected, one O(n_g) check per entry.  "Larger" is read as strict, and the
// magnitudes are compared in the same order Algorithm 5's selection uses (IEEE bit pattern
// with the sign cleared), so a NaN entry counts as larger than any threshold.  Output in
// ascending index.  Returns the number of selected entries; writes at most cap of them.
int64_t oracle_threshold_select(const float* acc, int64_t n, float threshold, float* val, int64_t* idx,
                                int64_t cap) {
    uint32_t tbits;
    std::memcpy(&tbits, &threshold, 4);
    tbits &= 0x7fffffffu;
    int64_t count = 0;
    for (int64_t i = 0; i < n; ++i) {
        uint32_t b;
        std::memcpy(&b, &acc[i], 4);
        if ((b & 0x7fffffffu) > tbits) {
            if (count < cap) { val[count] = acc[i]; idx[count] = i; }
            ++count;
        }
    }
    return count;
}

// CLT-k (Sections 1 and 3.1): one worker per iteration, the leader, selects the top k of ITS
// vector (= Algorithm 5 with one layer) and broadcasts the indices; the leaders take turns
// ("cyclic").  Every worker then contributes its own values at the leader's indices and
// clears them from its residual.
int64_t oracle_clt_leader(int64_t iteration, int64_t n_workers) { return iteration % n_workers; }

void oracle_gather_update(float* acc, const int64_t* idx, int64_t count, float* val) {
    for (int64_t j = 0; j < count; ++j) {
        val[j] = acc[idx[j]];
        acc[idx[j]] = 0.0f;
    }
}

// ---------------------------------------------------------------------------
// Algorithm 1 around the sparsifier, for several workers.
// ---------------------------------------------------------------------------
// Line 7: after the all-gather every worker holds all workers' index lists; the gradients that take
// part in the update are the SET of those indices.  Returns its size; out receives it ascending.
int64_t oracle_index_union(const int64_t* idx, int64_t count, int64_t* out) {
    std::vector<int64_t> all(idx, idx + count);
    std::sort(all.begin(), all.end());
    all.erase(std::unique(all.begin(), all.end()), all.end());
    for (size_t i = 0; i < all.size(); ++i) out[i] = all[i];
    return (int64_t)all.size();
}

// Lines 8-9: the workers' values at the selected indices are summed (AllReduce, SUM) and divided by
// the number of workers; fp32, one rounded operation each, workers added in rank order.
void oracle_sum_into(float* dst, const float* src, int64_t count) {
    for (int64_t i = 0; i < count; ++i) {
        volatile float s = dst[i] + src[i];
        dst[i] = s;
    }
}
void oracle_average(float* sum, int64_t count, int64_t n_workers) {
    const float n = (float)n_workers;
    for (int64_t i = 0; i < count; ++i) {
        volatile float q = sum[i] / n;
        sum[i] = q;
    }
}

// Eq. 2: a worker's error is the L2 norm of its residual (fp64, summed sequentially); the error of
// the iteration is the mean of the workers' errors.
double oracle_vector_norm(const float* x, int64_t n) {
    double s = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        const double v = (double)x[i];
        s = s + v * v;
    }
    return std::sqrt(s);
}
double oracle_error_eq2(const double* worker_error, int64_t n_workers) {
    double s = 0.0;
    for (int64_t i = 0; i < n_workers; ++i) s = s + worker_error[i];
    return s / (double)n_workers;
}

// ---------------------------------------------------------------------------
// The per-layer selections of a rank farmed out over host threads (layers are independent: Algorithm 5
// is a loop over them).  Same result as oracle_select_rank; used only to time the oracle on all of the
// host's cores.  threads < 1: as many as the hardware reports.  Returns the threads used.
// ---------------------------------------------------------------------------
int64_t oracle_hardware_threads(void) {
    const unsigned n = std::thread::hardware_concurrency();
    return n ? (int64_t)n : 1;
}

int64_t oracle_select_rank_threads(const float* acc, const int64_t* layer_start, const int64_t* k_l,
                                   const int32_t* my_layers, int64_t n_my, float* val_out, int64_t* idx_out,
                                   int64_t threads) {
    if (threads < 1) threads = oracle_hardware_threads();
    if (threads > n_my) threads = n_my > 0 ? n_my : 1;
    std::vector<int64_t> out_off(n_my + 1, 0);
    for (int64_t j = 0; j < n_my; ++j) out_off[j + 1] = out_off[j] + k_l[my_layers[j]];
    std::atomic<int64_t> next(0);
    auto work = [&]() {
        for (;;) {
            const int64_t j = next.fetch_add(1);
            if (j >= n_my) break;
            const int64_t part = my_layers[j];
            oracle_select_layer(acc, layer_start[part], layer_start[part + 1], k_l[part], val_out + out_off[j],
                                idx_out + out_off[j]);
        }
    };
    std::vector<std::thread> pool;
    for (int64_t t = 1; t < threads; ++t) pool.emplace_back(work);
    work();
    for (auto& th : pool) th.join();
    return threads;
}

}  // extern "C"
