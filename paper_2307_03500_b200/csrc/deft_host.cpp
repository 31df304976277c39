// Host-side planners of libdeft: Algorithm 2 (layer table), Algorithm 3 (local k),
// Algorithm 4 (bin packing) of the DEFT paper.  Pure functions, no CUDA.
// Compiled with -ffp-contract=off: every fp64 operation is a single IEEE operation.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <cstdint>
#include <functional>
#include <numeric>
#include <queue>
#include <utility>
#include <vector>

#include "deft.h"

namespace {
// (key ascending, then id ascending)
struct SortKey {
    uint64_t key;
    int32_t id;
    bool operator<(const SortKey& o) const { return key != o.key ? key < o.key : id < o.id; }
};

// Sorts keys (filled by the caller, keys[i].id == i) ascending.  The order a planner needs changes little
// from one step to the next, so the keys are first laid out in the order the previous call on this thread
// ended with and finished by insertion (a handful of moves per step instead of L log L compares); when
// the moves add up (a different model, a shuffled vector) the standard sort takes over.  The order is
// total (ties by id), so the result does not depend on the starting point.  `order` is kept by the caller
// per planner (thread-local).
void sort_from_last_order(std::vector<SortKey>& keys, std::vector<int32_t>& order, std::vector<SortKey>& tmp) {
    const size_t n = keys.size();
    bool usable = order.size() == n;
    if (usable) {
        tmp.resize(n);
        for (size_t i = 0; i < n; ++i) {
            const int32_t id = order[i];
            if (id < 0 || (size_t)id >= n) { usable = false; break; }
            tmp[i] = keys[(size_t)id];
        }
    }
    if (usable) {
        size_t moves = 0;
        const size_t budget = 8 * n + 64;
        size_t i = 1;
        for (; i < n && moves <= budget; ++i) {
            const SortKey x = tmp[i];
            size_t j = i;
            while (j > 0 && x < tmp[j - 1]) {
                tmp[j] = tmp[j - 1];
                --j;
                ++moves;
            }
            tmp[j] = x;
        }
        if (i < n) std::sort(tmp.begin(), tmp.end());   // (a permutation of the keys either way)
        keys.swap(tmp);
    } else {
        std::sort(keys.begin(), keys.end());
    }
    order.resize(n);
    for (size_t i = 0; i < n; ++i) order[i] = keys[i].id;
}
}  // namespace

extern "C" {

const char* deft_status_string(deft_status s) {
    switch (s) {
        case DEFT_OK: return "DEFT_OK";
        case DEFT_WARN_K_INEXACT: return "DEFT_WARN_K_INEXACT";
        case DEFT_ERR_INVALID_ARG: return "DEFT_ERR_INVALID_ARG";
        case DEFT_ERR_INFEASIBLE_K: return "DEFT_ERR_INFEASIBLE_K";
        case DEFT_ERR_NONFINITE_NORM: return "DEFT_ERR_NONFINITE_NORM";
        case DEFT_ERR_CAPACITY: return "DEFT_ERR_CAPACITY";
        case DEFT_ERR_CUDA: return "DEFT_ERR_CUDA";
        case DEFT_ERR_TOO_LARGE: return "DEFT_ERR_TOO_LARGE";
        default: return "DEFT_UNKNOWN_STATUS";
    }
}

// Algorithm 2.
deft_status deft_split_layers(const int64_t* tensor_sizes_h, int32_t T, int32_t N,
                              int64_t* layer_start_h, int32_t* layer_tensor_h, int32_t cap,
                              int32_t* L_out) {
    if (!tensor_sizes_h || !layer_start_h || !L_out || T < 1 || N < 1 || cap < 0)
        return DEFT_ERR_INVALID_ARG;
    unsigned __int128 total = 0;
    for (int32_t t = 0; t < T; ++t) {
        if (tensor_sizes_h[t] < 1) return DEFT_ERR_INVALID_ARG;
        total += (unsigned __int128)tensor_sizes_h[t];
    }
    // First pass: count the layers so that a short buffer is reported, not overrun.
    int64_t need = 0;
    for (int32_t t = 0; t < T; ++t) {
        const int64_t sz = tensor_sizes_h[t];
        const bool split = (unsigned __int128)sz * (unsigned __int128)N > total;
        need += split ? std::min<int64_t>(sz, N) : 1;
    }
    if (need > INT32_MAX) return DEFT_ERR_INVALID_ARG;
    *L_out = (int32_t)need;
    if (need > cap) return DEFT_ERR_CAPACITY;

    int32_t l = 0;
    int64_t pos = 0;
    for (int32_t t = 0; t < T; ++t) {
        const int64_t sz = tensor_sizes_h[t];
        const bool split = (unsigned __int128)sz * (unsigned __int128)N > total;
        const int64_t pieces = split ? N : 1;
        const int64_t base = sz / pieces;
        const int64_t extra = sz % pieces;  // the first `extra` pieces are one longer
        for (int64_t i = 0; i < pieces; ++i) {
            const int64_t len = base + (i < extra ? 1 : 0);
            if (len == 0) continue;
            layer_start_h[l] = pos;
            if (layer_tensor_h) layer_tensor_h[l] = t;
            pos += len;
            ++l;
        }
    }
    layer_start_h[l] = pos;
    return DEFT_OK;
}

// Algorithm 3.
deft_status deft_allocate_k(const double* norms_h, const int64_t* layer_size_h, int32_t L,
                            int64_t k, int32_t mode, int64_t* k_l_h, int64_t* sum_k_out) {
    if (!norms_h || !layer_size_h || !k_l_h || L < 1 || k < 1 ||
        (mode != DEFT_MODE_PAPER && mode != DEFT_MODE_EXACT))
        return DEFT_ERR_INVALID_ARG;
    int64_t n_g = 0;
    for (int32_t l = 0; l < L; ++l) {
        if (layer_size_h[l] < 1) return DEFT_ERR_INVALID_ARG;
        n_g += layer_size_h[l];
    }
    for (int32_t l = 0; l < L; ++l)
        if (!(norms_h[l] >= 0.0) || std::isinf(norms_h[l])) return DEFT_ERR_NONFINITE_NORM;
    if (mode == DEFT_MODE_EXACT && (k < (int64_t)L || k > n_g)) return DEFT_ERR_INFEASIBLE_K;

    // Priority: larger norm first, equal norms by lower id.  For non-negative doubles the bit pattern
    // orders like the value (-0.0 is made +0.0 first), so one sort of (inverted bits, id) pairs does it.
    static thread_local std::vector<SortKey> keys;
    static thread_local std::vector<int32_t> prio;
    static thread_local std::vector<double> tail;
    keys.resize((size_t)L);
    prio.resize((size_t)L);
    for (int32_t l = 0; l < L; ++l) {
        const double v = norms_h[l] + 0.0;
        uint64_t bits;
        std::memcpy(&bits, &v, 8);
        keys[l] = SortKey{~bits, l};
    }
    static thread_local std::vector<int32_t> last_order;
    static thread_local std::vector<SortKey> sort_tmp;
    sort_from_last_order(keys, last_order, sort_tmp);
    for (int32_t p = 0; p < L; ++p) prio[p] = keys[p].id;

    // tail[p] = norms of priority positions p, p+1, ..., L-1 added from the back.
    tail.resize((size_t)L + 1);
    tail[L] = 0.0;
    for (int32_t p = L; p-- > 0;) tail[p] = norms_h[prio[p]] + tail[p + 1];

    // share[p] = norm / norm_remain (0 when nothing remains): independent of the running k, so all the
    // divisions are done before the sequential part (each is the same single IEEE division as before)
    static thread_local std::vector<double> share;
    share.resize((size_t)L);
    for (int32_t p = 0; p < L; ++p) share[p] = tail[p] > 0.0 ? norms_h[prio[p]] / tail[p] : -1.0;
    int64_t left = k;
    for (int32_t p = 0; p < L; ++p) {
        const int32_t l = prio[p];
        double want = 0.0;
        if (share[p] >= 0.0) {
            const double prod = (double)left * share[p];
            want = std::floor(prod);
        }
        const int64_t sz = layer_size_h[l];
        int64_t give;
        if ((double)sz < want) give = sz;
        else if (want < 1.0) give = 1;
        else give = (int64_t)want;
        k_l_h[l] = give;
        left -= give;
    }

    int64_t sum = k - left;
    if (mode == DEFT_MODE_EXACT && sum != k) {
        int64_t gap = k - sum;  // > 0: hand out more; < 0: take back
        if (gap > 0) {
            for (int32_t p = 0; p < L && gap > 0; ++p) {
                const int32_t l = prio[p];
                const int64_t room = layer_size_h[l] - k_l_h[l];
                const int64_t add = room < gap ? room : gap;
                k_l_h[l] += add;
                gap -= add;
            }
        } else {
            while (gap < 0) {
                for (int32_t p = 0; p < L && gap < 0; ++p) {
                    const int32_t l = prio[p];
                    if (k_l_h[l] > 1) {
                        --k_l_h[l];
                        ++gap;
                    }
                }
            }
        }
        sum = k;
    }
    if (sum_k_out) *sum_k_out = sum;
    return (sum == k) ? DEFT_OK : DEFT_WARN_K_INEXACT;
}

// Algorithm 4 (packing part).  cost_model: DEFT_COST_EQ3 = size * ln(k) (Eq. 3),
// DEFT_COST_SIZE = size (the bytes a worker scans).
deft_status deft_partition_model(const int64_t* layer_size_h, const int64_t* k_l_h, int32_t L, int32_t N,
                                 int32_t cost_model, int32_t* bin_of_layer_h, double* bin_load_h) {
    if (!layer_size_h || !bin_of_layer_h || L < 1 || N < 1 ||
        (cost_model != DEFT_COST_EQ3 && cost_model != DEFT_COST_SIZE) || (cost_model == DEFT_COST_EQ3 && !k_l_h))
        return DEFT_ERR_INVALID_ARG;
    for (int32_t l = 0; l < L; ++l)
        if (layer_size_h[l] < 1 || (cost_model == DEFT_COST_EQ3 && k_l_h[l] < 1)) return DEFT_ERR_INVALID_ARG;

    // ln(k) for small k comes from a table filled with std::log itself (same bits, no call)
    static const std::vector<double> log_small = [] {
        std::vector<double> t(4096);
        for (int i = 1; i < 4096; ++i) t[i] = std::log((double)i);
        return t;
    }();
    static thread_local std::vector<double> c;
    static thread_local std::vector<SortKey> keys;
    static thread_local std::vector<double> load;
    c.resize((size_t)L);
    keys.resize((size_t)L);
    for (int32_t l = 0; l < L; ++l) {
        if (cost_model == DEFT_COST_EQ3) {
            const int64_t kk = k_l_h[l];
            c[l] = (double)layer_size_h[l] * (kk < 4096 ? log_small[(size_t)kk] : std::log((double)kk));
        } else {
            c[l] = (double)layer_size_h[l];
        }
    }
    // "largest remaining cost, lowest id on ties" L times = one stable pass over the layers
    // sorted by descending cost; "smallest load, lowest id on ties" = a min-heap on (load, bin).
    // Each bin receives its costs in the same order as in the listing, so the fp64 sums are the same.
    // (costs are non-negative: their bit patterns order like the values; ties go to the lower id)
    for (int32_t l = 0; l < L; ++l) {
        const double v = c[l] + 0.0;
        uint64_t bits;
        std::memcpy(&bits, &v, 8);
        keys[l] = SortKey{~bits, l};
    }
    static thread_local std::vector<int32_t> last_order;
    static thread_local std::vector<SortKey> sort_tmp;
    sort_from_last_order(keys, last_order, sort_tmp);
    load.assign((size_t)N, 0.0);
    typedef std::pair<double, int32_t> Bin;   // (load, id): smallest load first, then lowest id
    static thread_local std::vector<Bin> heap;
    heap.clear();
    for (int32_t b = 0; b < N; ++b) heap.push_back(Bin(0.0, b));   // already a heap: equal loads, ascending ids
    const auto lighter_last = std::greater<Bin>();
    for (int32_t i = 0; i < L; ++i) {
        const int32_t pick = keys[i].id;
        std::pop_heap(heap.begin(), heap.end(), lighter_last);
        Bin& lightest = heap.back();
        bin_of_layer_h[pick] = lightest.second;
        load[lightest.second] += c[pick];
        lightest.first = load[lightest.second];
        std::push_heap(heap.begin(), heap.end(), lighter_last);
    }
    if (bin_load_h)
        for (int32_t b = 0; b < N; ++b) bin_load_h[b] = load[b];
    return DEFT_OK;
}

// Algorithm 4 (packing part) with the load model of Eq. 3.
deft_status deft_partition(const int64_t* layer_size_h, const int64_t* k_l_h, int32_t L,
                           int32_t N, int32_t* bin_of_layer_h, double* bin_load_h) {
    if (!k_l_h) return DEFT_ERR_INVALID_ARG;
    return deft_partition_model(layer_size_h, k_l_h, L, N, DEFT_COST_EQ3, bin_of_layer_h, bin_load_h);
}

// Eq. 2: the error of an iteration is the mean of the workers' errors.
deft_status deft_error_eq2(const double* worker_error_h, int32_t n_workers, double* error_out) {
    if (!worker_error_h || !error_out || n_workers < 1) return DEFT_ERR_INVALID_ARG;
    double s = 0.0;
    for (int32_t i = 0; i < n_workers; ++i) s = s + worker_error_h[i];
    *error_out = s / (double)n_workers;
    return DEFT_OK;
}

int32_t deft_rank_bin(int64_t iteration, int32_t rank, int32_t N) {
    if (N < 1 || rank < 0 || rank >= N || iteration < 0) return -1;
    return (int32_t)((iteration % N + rank) % N);
}

deft_status deft_bin_layers(const int32_t* bin_of_layer_h, int32_t L, int32_t bin,
                            int32_t* my_layers_h, int32_t cap, int32_t* n_my_out) {
    if (!bin_of_layer_h || !n_my_out || L < 1 || bin < 0 || cap < 0 || (cap > 0 && !my_layers_h))
        return DEFT_ERR_INVALID_ARG;
    int32_t n = 0;
    for (int32_t l = 0; l < L; ++l) n += (bin_of_layer_h[l] == bin);
    *n_my_out = n;
    if (n > cap) return DEFT_ERR_CAPACITY;
    n = 0;
    for (int32_t l = 0; l < L; ++l)
        if (bin_of_layer_h[l] == bin) my_layers_h[n++] = l;
    return DEFT_OK;
}

}  // extern "C"
