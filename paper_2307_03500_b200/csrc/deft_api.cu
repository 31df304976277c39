// C-ABI entry points of libdeft that touch the GPU: argument checks, the per-step plan
// (host-built tables of every rank's layers), workspace carve-up and kernel launches.
#include <algorithm>
#include <chrono>
#include <cstring>
#include <vector>

#include "deft_common.cuh"

namespace deft {

static thread_local int32_t g_last_cuda_error = 0;
static unsigned long long* g_select_timing = nullptr;
static int g_stream_kernel = -1;   // deft_debug_select_kernel: -1 by size, 0 never, 1 whenever possible
static int g_step_fused = 1;       // deft_debug_step_staging: deft_step for all workers stages during the accumulate pass
static int g_stream_ring = 1;      // deft_debug_select_ring: the single-pass kernel reads through a ring of bulk copies

// Limits of the single-pass selection kernel (see select_rank).
constexpr int64_t kStreamMaxElems = 600000000;      // elements of one call
constexpr int64_t kStreamMinElems = 48000000;       // below this the five-step kernel is the faster one (measured)
constexpr int kStreamMaxLayers = 1024;              // layers of one call (its layer map lives in shared memory)

void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = (int32_t)e; }

int sm_count() {
    static thread_local int cached_dev = -1;
    static thread_local int cached_sms = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev != cached_dev) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
            sms = 148;
        cached_dev = dev;
        cached_sms = sms;
    }
    return cached_sms;
}

namespace {

// select_rank(prestaged = true): the call's layers do not suit the single-pass kernel (internal, never returned to callers)
constexpr deft_status kNotPrestaged = 1000;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

struct LayerItem { int64_t start, end, k; int32_t layer_id; double norm = 0.0; };

// Writes the plan blob for `ranks` lists of layers (each ascending in address).
deft_status fill_plan(void* blob, size_t blob_bytes, int32_t L, int64_t iteration,
                      const std::vector<std::vector<LayerItem>>& ranks) {
    const int64_t N = (int64_t)ranks.size();
    if (blob_bytes < plan_bytes(L, N)) return DEFT_ERR_CAPACITY;
    char* base = static_cast<char*>(blob);
    PlanHeader* hdr = reinterpret_cast<PlanHeader*>(base);
    RankInfo* ri = reinterpret_cast<RankInfo*>(base + sizeof(PlanHeader));
    LayerDesc* desc = reinterpret_cast<LayerDesc*>(base + sizeof(PlanHeader) + sizeof(RankInfo) * (size_t)(N + 1));
    std::memset(blob, 0, plan_bytes(L, N));
    int64_t tiles_all = 0, elems_all = 0, k_all = 0;
    int64_t slots_all = 0;   // staging slots handed out: every layer's region starts on a 128-byte boundary
    auto slots_of = [](int64_t size) { return (size + kRegionAlign - 1) / kRegionAlign * kRegionAlign; };
    int64_t d = 0;
    for (int64_t r = 0; r < N; ++r) {
        RankInfo& R = ri[r];
        R.desc_first = (int32_t)d;
        R.n_my = (int32_t)ranks[r].size();
        R.tile_base = (int32_t)tiles_all;
        R.elem_base = slots_all;
        R.out_off = k_all;
        int64_t tiles = 0, elems = 0, slots = 0, k = 0, prev_end = -1;
        for (const LayerItem& it : ranks[r]) {
            if (it.start < 0 || it.end <= it.start || it.end - it.start > DEFT_MAX_LAYER_ELEMS)
                return DEFT_ERR_INVALID_ARG;
            if (it.start < prev_end) return DEFT_ERR_INVALID_ARG;
            if (it.k < 1 || it.k > it.end - it.start) return DEFT_ERR_INVALID_ARG;
            LayerDesc& D = desc[d++];
            D.start = it.start;
            D.end = it.end;
            D.k = it.k;
            D.out_off = k;
            D.elem_off = slots_all + slots;
            D.tile_first = (int32_t)tiles;
            D.layer_id = it.layer_id;
            D.norm = it.norm;
            tiles += (it.end - 1) / kTile - it.start / kTile + 1;
            elems += it.end - it.start;
            slots += slots_of(it.end - it.start);
            k += it.k;
            prev_end = it.end;
            if (tiles_all + tiles > INT32_MAX) return DEFT_ERR_INVALID_ARG;
        }
        LayerDesc& Z = desc[d++];   // sentinel
        Z.out_off = k;
        Z.elem_off = slots_all + slots;
        Z.tile_first = (int32_t)tiles;
        Z.layer_id = -1;
        R.tiles = (int32_t)tiles;
        R.elems = elems;
        R.k = k;
        tiles_all += tiles;
        elems_all += elems;
        slots_all += slots;
        k_all += k;
    }
    // all ranks' layers as one list in address order
    {
        RankInfo& M = ri[N];
        std::vector<LayerDesc> all;
        all.reserve((size_t)L);
        for (int64_t r = 0; r < N; ++r)
            for (int32_t j = 0; j < ri[r].n_my; ++j) {
                LayerDesc D = desc[ri[r].desc_first + j];
                D.out_off += ri[r].out_off;
                all.push_back(D);
            }
        auto by_start = [](const LayerDesc& a, const LayerDesc& b) { return a.start < b.start; };
        if ((int64_t)all.size() == (int64_t)L) {   // layer ids that are address order: place, do not sort
            std::vector<LayerDesc> placed((size_t)L);
            std::vector<char> seen((size_t)L, 0);
            bool ok = true;
            for (const LayerDesc& D : all) {
                if (D.layer_id < 0 || D.layer_id >= L || seen[D.layer_id]) { ok = false; break; }
                seen[D.layer_id] = 1;
                placed[D.layer_id] = D;
            }
            if (ok && std::is_sorted(placed.begin(), placed.end(), by_start)) all.swap(placed);
            else std::sort(all.begin(), all.end(), by_start);
        } else {
            std::sort(all.begin(), all.end(), by_start);
        }
        bool disjoint = (int64_t)all.size() <= (int64_t)L;
        for (size_t i = 1; i < all.size() && disjoint; ++i) disjoint = all[i].start >= all[i - 1].end;
        M.desc_first = (int32_t)d;
        M.n_my = 0;
        if (disjoint && !all.empty()) {
            int64_t tiles = 0, elems = 0, slots = 0;
            for (LayerDesc& D : all) {
                D.tile_first = (int32_t)tiles;
                D.elem_off = slots;
                tiles += (D.end - 1) / kTile - D.start / kTile + 1;
                elems += D.end - D.start;
                slots += slots_of(D.end - D.start);
                desc[d++] = D;
            }
            LayerDesc& Z = desc[d++];   // sentinel
            Z.out_off = k_all;
            Z.elem_off = slots;
            Z.tile_first = (int32_t)tiles;
            Z.layer_id = -1;
            M.n_my = (int32_t)all.size();
            M.tiles = (int32_t)tiles;
            M.elems = elems;
            M.k = k_all;
        }
    }
    hdr->magic = kPlanMagic;
    hdr->L = L;
    hdr->N = (int32_t)N;
    hdr->total_tiles = (int32_t)tiles_all;
    hdr->total_elems = elems_all;
    hdr->total_k = k_all;
    hdr->iteration = iteration;
    return DEFT_OK;
}

inline bool plan_ok(const void* plan_h) {
    return plan_h && static_cast<const PlanHeader*>(plan_h)->magic == kPlanMagic;
}

// clear = false: the caller has already cleared the per-layer counters on this stream.
deft_status upload_plan(const void* plan_h, void* plan_d, void* ws_d, size_t ws_bytes, cudaStream_t stream,
                        bool clear = true) {
    const PlanHeader* hdr = static_cast<const PlanHeader*>(plan_h);
    const WsLayout w = ws_layout(hdr->total_elems, hdr->L, hdr->total_tiles);
    if (w.total > ws_bytes) return DEFT_ERR_CAPACITY;
    DEFT_CUDA_TRY(cudaMemcpyAsync(plan_d, plan_h, plan_bytes(hdr->L, hdr->N), cudaMemcpyHostToDevice, stream));
    if (clear)
        DEFT_CUDA_TRY(cudaMemsetAsync(static_cast<char*>(ws_d) + w.zero_begin, 0, w.zero_end - w.zero_begin, stream));
    return DEFT_OK;
}

// Hard-threshold mode of the selection kernel (one layer, threshold given).
struct FixedThreshold {
    bool on = false;
    uint32_t key = 0;                       // magnitude key of the threshold
    unsigned long long* count_d = nullptr;  // receives the number of entries above it
};

deft_status select_rank(const float* acc_d, const void* plan_h, const void* plan_d, int32_t rank,
                        float* val_d, int64_t* idx_d, int64_t out_cap, void* ws_d, size_t ws_bytes,
                        cudaStream_t stream, bool zero_selected = false, FixedThreshold fixed = FixedThreshold(),
                        bool prestaged = false) {
    const PlanHeader* hdr = static_cast<const PlanHeader*>(plan_h);
    if (rank < 0 || rank > hdr->N) return DEFT_ERR_INVALID_ARG;   // rank N = all ranks' layers as one list
    const RankInfo& R = plan_ranks(plan_h)[rank];
    if (R.n_my == 0) return DEFT_OK;
    if (!fixed.on && out_cap < R.k) return DEFT_ERR_CAPACITY;
    const WsLayout w = ws_layout(hdr->total_elems, hdr->L, hdr->total_tiles);
    if (w.total > ws_bytes) return DEFT_ERR_CAPACITY;
    char* ws = static_cast<char*>(ws_d);
    SelParams p;
    p.acc = acc_d;
    p.desc = plan_descs(plan_d, hdr->N) + R.desc_first;
    p.n_my = R.n_my;
    p.tiles = R.tiles;
    p.acc_rw = zero_selected ? const_cast<float*>(acc_d) : nullptr;
    p.state = reinterpret_cast<LayerState*>(ws + w.state);
    p.hist1 = reinterpret_cast<uint32_t*>(ws + w.hist1);
    p.hist2 = reinterpret_cast<uint32_t*>(ws + w.hist2);
    p.hist3 = reinterpret_cast<uint32_t*>(ws + w.hist3);
    p.spec_ctl = reinterpret_cast<uint32_t*>(ws + w.hint);
    p.hint = reinterpret_cast<LayerHint*>(ws + w.hint + 256);
    p.retry = reinterpret_cast<RetryHeader*>(ws + w.retry);
    p.retry_desc = reinterpret_cast<LayerDesc*>(ws + w.retry_desc);
    p.from_retry = 0;
    p.prestaged = 0;
    p.stage_tab = reinterpret_cast<const StageTab*>(ws + w.stage_tab);
    p.retry_elem_base = R.elem_base;
    p.runge = reinterpret_cast<uint2*>(ws + w.runge) + 2 * ((size_t)R.tile_base + (size_t)rank);
    p.staging = reinterpret_cast<uint2*>(ws + w.staging);
    p.val = val_d;
    p.idx = idx_d;
    p.timing = g_select_timing;
    p.fixed_thr = fixed.on ? 1 : 0;
    p.thr_key = fixed.key;
    p.out_cap = out_cap;
    p.out_total = R.k;
    p.count_out = fixed.count_d;
    // one CTA per SM at most (co-resident by construction); fewer when the rank is small
    const int sms = sm_count();
    int want = (R.tiles + 1) / 2;
    if (want < R.n_my) want = R.n_my;
    if (want < 1) want = 1;
    p.grid = want < sms ? want : sms;
    // limits of one CTA's share: tiles, and streamed (non-direct) layers
    const LayerDesc* hd = plan_descs(plan_h, hdr->N) + R.desc_first;
    p.weighted = 0;
    p.interleave = (R.n_my == 1 && (int64_t)R.tiles >= (int64_t)kInterleaveTiles * p.grid) ? 1 : 0;
    if (p.interleave) {
        const int nsuper = (R.tiles + kSuper - 1) / kSuper;
        if ((int64_t)((nsuper + p.grid - 1) / p.grid) * kSuper > kMaxLocalTiles) return DEFT_ERR_TOO_LARGE;
        return launch_select(p, stream);
    }
    // q0[b] = first tile of CTA b, b = 0..grid
    auto within_limits = [&](const std::vector<int>& q0) {
        int j = 0;
        for (int b = 0; b < p.grid; ++b) {
            if (q0[b + 1] - q0[b] > kMaxLocalTiles) return false;
            while (j + 1 < R.n_my && hd[j + 1].tile_first <= q0[b]) ++j;
            int streamed = 0;
            for (int jj = j; jj < R.n_my && hd[jj].tile_first < q0[b + 1]; ++jj)
                streamed += (hd[jj].end - hd[jj].start > kDirectElems);
            if (streamed > kMaxLocalLayers) return false;
        }
        return true;
    };
    std::vector<int> q0((size_t)p.grid + 1);
    for (int b = 0; b <= p.grid; ++b) q0[b] = (int)((int64_t)R.tiles * b / p.grid);
    if (!within_limits(q0)) return DEFT_ERR_TOO_LARGE;
    // The single-pass kernel takes the call when at least half of what it streams can be speculated on (sparse
    // layers of moderate k; whether a cut is remembered for them only the device knows).  Its finishing CTA
    // handles a layer alone, so dense layers, layers that select very many entries and layers without a
    // remembered cut go on its retry list, which the same launch works off with the five steps behind a grid
    // barrier: those steps then split only THESE layers' tiles over the CTAs, which balances a call that
    // mixes sparse and dense layers better than one split over all of them (0.62 against 1.1 ms on a 355 M-element
    // vector at density 0.01); a call that is mostly dense is better off with the five steps alone.
    if (!fixed.on && (g_stream_kernel > 0 || (g_stream_kernel < 0 && R.elems >= kStreamMinElems))) {
        int64_t streamed = 0, sparse = 0;
        int n_streamed = 0;
        // every CTA keeps a table of all streamed layers and a map of all layers; its stripes are tiles / grid tiles
        bool ok = R.elems <= kStreamMaxElems && R.n_my <= kStreamMaxLayers &&
                  (int64_t)R.tiles / p.grid + 2 * kSuper <= kStreamLocalTiles;
        for (int j = 0; j < R.n_my && ok; ++j) {
            const int64_t size = hd[j].end - hd[j].start;
            if (size <= kDirectElems) continue;
            streamed += size;
            if (++n_streamed > kMaxLocalLayers) ok = false;
            if (hd[j].k * kSpecDensity <= size) {
                if (!prestaged && hd[j].k > kStreamMaxK) ok = false;   // (reading for itself it takes all sparse layers or none)
                if (stream_can_finish(hd[j].k, prestaged)) sparse += size;   // layers it can finish itself
            }
        }
        if (ok && (streamed == 0 || 2 * sparse >= streamed)) {
            p.prestaged = prestaged ? 1 : 0;
            return launch_select_stream(p, streamed != 0, g_stream_ring != 0, stream);
        }
    }
    if (prestaged) return kNotPrestaged;   // the caller clears what the accumulate pass staged and calls again
    if (R.n_my > 1 && R.n_my <= kMaxWeightedLayers && (int64_t)R.tiles >= (int64_t)kInterleaveTiles * p.grid) {
        const int n = R.n_my;
        std::vector<uint32_t> Wp((size_t)n + 1), wt((size_t)n);
        std::vector<int> tf((size_t)n + 1);
        uint64_t acc = 0;
        for (int j = 0; j < n; ++j) {
            wt[j] = tile_weight(hd[j].k, hd[j].end - hd[j].start);
            tf[j] = hd[j].tile_first;
            Wp[j] = (uint32_t)acc;
            acc += (uint64_t)wt[j] * (uint64_t)(hd[j + 1].tile_first - hd[j].tile_first);
            if (acc > 0xffffffffull) break;
        }
        if (acc > 0 && acc <= 0xffffffffull) {
            Wp[n] = (uint32_t)acc;
            tf[n] = R.tiles;
            for (int b = 0; b <= p.grid; ++b) q0[b] = weighted_boundary(Wp.data(), wt.data(), tf.data(), n, R.tiles, b, p.grid);
            if (within_limits(q0)) p.weighted = 1;
        }
    }
    return launch_select(p, stream);
}

// One-shot path: plan for a single rank, kept in the scratch area at the head of the workspace.
deft_status select_once(const float* acc_d, const std::vector<LayerItem>& items, float* val_d,
                        int64_t* idx_d, int64_t out_cap, void* ws_d, size_t ws_bytes, cudaStream_t stream) {
    const int32_t L = (int32_t)items.size();
    std::vector<std::vector<LayerItem>> ranks(1, items);
    std::vector<char> blob(plan_bytes(L, 1));
    deft_status s = fill_plan(blob.data(), blob.size(), L, 0, ranks);
    if (s != DEFT_OK) return s;
    const PlanHeader* hdr = reinterpret_cast<const PlanHeader*>(blob.data());
    if (out_cap < hdr->total_k) return DEFT_ERR_CAPACITY;
    const WsLayout w = ws_layout(hdr->total_elems, hdr->L, hdr->total_tiles);
    if (w.total > ws_bytes) return DEFT_ERR_CAPACITY;
    void* plan_d = static_cast<char*>(ws_d) + w.plan;
    // The blob is pageable host memory: the runtime stages it before returning, so it may
    // be released as soon as this call returns.
    s = upload_plan(blob.data(), plan_d, ws_d, ws_bytes, stream);
    if (s != DEFT_OK) return s;
    return select_rank(acc_d, blob.data(), plan_d, 0, val_d, idx_d, out_cap, ws_d, ws_bytes, stream);
}

}  // namespace
}  // namespace deft

using namespace deft;

extern "C" {

int32_t deft_last_cuda_error(void) { return g_last_cuda_error; }

void deft_debug_select_timing(void* timing_d) { g_select_timing = static_cast<unsigned long long*>(timing_d); }

int64_t deft_select_launch_max_elems(void) { return (int64_t)sm_count() * kMaxLocalTiles * kTile; }

void deft_debug_step_staging(int32_t on) { g_step_fused = on != 0 ? 1 : 0; }
void deft_debug_select_ring(int32_t on) { g_stream_ring = on != 0 ? 1 : 0; }
void deft_debug_select_kernel(int32_t single_pass) { g_stream_kernel = single_pass < 0 ? -1 : (single_pass != 0 ? 1 : 0); }

deft_status deft_workspace_init(void* ws_d, size_t ws_bytes, int32_t n_layers, void* stream) {
    if (!ws_d || n_layers < 1 || !aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    const WsLayout w = ws_layout(1, n_layers, 1);   // the kept area's place depends on the layer count only
    const size_t bytes = 256 + sizeof(LayerHint) * (size_t)n_layers;
    if (w.hint + bytes > ws_bytes) return DEFT_ERR_CAPACITY;
    DEFT_CUDA_TRY(cudaMemsetAsync(static_cast<char*>(ws_d) + w.hint, 0, bytes, static_cast<cudaStream_t>(stream)));
    return DEFT_OK;
}

deft_status deft_select_stats(const void* ws_d, size_t ws_bytes, int32_t n_layers, uint64_t* stats_h, void* stream) {
    if (!ws_d || !stats_h || n_layers < 1) return DEFT_ERR_INVALID_ARG;
    const WsLayout w = ws_layout(1, n_layers, 1);
    if (w.hint + 256 > ws_bytes) return DEFT_ERR_CAPACITY;
    uint32_t words[10];
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DEFT_CUDA_TRY(cudaMemcpyAsync(words, static_cast<const char*>(ws_d) + w.hint, sizeof(words), cudaMemcpyDeviceToHost, st));
    DEFT_CUDA_TRY(cudaStreamSynchronize(st));
    stats_h[0] = words[4];
    stats_h[1] = words[5];
    stats_h[2] = words[6];
    stats_h[3] = words[8];
    stats_h[4] = words[9];
    stats_h[5] = stats_h[6] = stats_h[7] = 0;
    return DEFT_OK;
}

size_t deft_workspace_bytes(int64_t max_elems, int32_t max_layers) {
    if (max_elems < 1 || max_layers < 1) return 0;
    return ws_layout(max_elems, max_layers, max_tiles(max_elems, max_layers)).total;
}

deft_status deft_layer_norms(float* resid_acc_d, const float* grad_d, int64_t n_g,
                             const int64_t* layer_start_d, int32_t L, double* norms_d, void* ws_d,
                             size_t ws_bytes, void* stream) {
    if (!resid_acc_d || !layer_start_d || !norms_d || !ws_d || n_g < 1 || L < 1)
        return DEFT_ERR_INVALID_ARG;
    if (!aligned16(resid_acc_d) || (grad_d && !aligned16(grad_d)) || !aligned256(ws_d))
        return DEFT_ERR_INVALID_ARG;
    const size_t part = ws_layout(n_g, L, 1).norm_partial;   // clear of everything the library keeps across calls
    if (part + norms_ws_bytes(n_g, L) > ws_bytes) return DEFT_ERR_CAPACITY;
    return launch_layer_norms(resid_acc_d, grad_d, n_g, layer_start_d, L, norms_d,
                              reinterpret_cast<double*>(static_cast<char*>(ws_d) + part),
                              static_cast<cudaStream_t>(stream));
}

size_t deft_plan_bytes(int32_t L, int32_t N) {
    if (L < 1 || N < 1 || N > kMaxRanks) return 0;
    return plan_bytes(L, N);
}

// The plan of a whole model (every layer in exactly one bin, layer ids in address order), written
// straight into the blob in two passes over the layers: the per-step path, kept free of allocations.
static deft_status plan_build_impl(const int64_t* layer_start_h, const int64_t* k_l_h,
                                   const int32_t* bin_of_layer_h, const double* norms_h, int32_t L, int32_t N,
                                   int64_t iteration, void* plan_h, size_t plan_bytes_cap) {
    if (!layer_start_h || !k_l_h || !bin_of_layer_h || !plan_h || L < 1 || N < 1 || N > kMaxRanks ||
        iteration < 0)
        return DEFT_ERR_INVALID_ARG;
    if (plan_bytes_cap < plan_bytes(L, N)) return DEFT_ERR_CAPACITY;
    char* base = static_cast<char*>(plan_h);
    PlanHeader* hdr = reinterpret_cast<PlanHeader*>(base);
    RankInfo* ri = reinterpret_cast<RankInfo*>(base + sizeof(PlanHeader));
    LayerDesc* desc = reinterpret_cast<LayerDesc*>(base + sizeof(PlanHeader) + sizeof(RankInfo) * (size_t)(N + 1));
    struct Acc { int64_t tiles, elems, slots, k; int32_t n; };
    static thread_local std::vector<Acc> acc;
    static thread_local std::vector<int32_t> rank_of;
    acc.assign((size_t)N, Acc{0, 0, 0, 0, 0});
    rank_of.resize((size_t)L);
    const int32_t cycle = (int32_t)(iteration % N);
    auto tiles_of = [](int64_t st, int64_t en) { return (en - 1) / kTile - st / kTile + 1; };
    auto slots_of = [](int64_t size) { return (size + kRegionAlign - 1) / kRegionAlign * kRegionAlign; };
    // pass 1: what every rank holds
    for (int32_t l = 0; l < L; ++l) {
        const int32_t b = bin_of_layer_h[l];
        const int64_t st = layer_start_h[l], en = layer_start_h[l + 1], size = en - st;
        if (b < 0 || b >= N || st < 0 || size < 1 || size > DEFT_MAX_LAYER_ELEMS || k_l_h[l] < 1 || k_l_h[l] > size)
            return DEFT_ERR_INVALID_ARG;
        // rank r reads bin (cycle + r) % N  <=>  bin b is read by rank (b - cycle) mod N
        const int32_t r = b - cycle < 0 ? b - cycle + N : b - cycle;
        rank_of[l] = r;
        Acc& A = acc[r];
        A.tiles += tiles_of(st, en);
        A.elems += size;
        A.slots += slots_of(size);
        A.k += k_l_h[l];
        A.n += 1;
    }
    int64_t tiles_all = 0, elems_all = 0, slots_all = 0, k_all = 0, d = 0;
    for (int32_t r = 0; r < N; ++r) {
        RankInfo& R = ri[r];
        const Acc A = acc[r];
        R.desc_first = (int32_t)d;
        R.n_my = A.n;
        R.tiles = (int32_t)A.tiles;
        R.tile_base = (int32_t)tiles_all;
        R.elems = A.elems;
        R.k = A.k;
        R.out_off = k_all;
        R.elem_base = slots_all;
        R.reserved[0] = R.reserved[1] = 0;
        LayerDesc& Z = desc[d + A.n];   // the rank's sentinel
        Z = LayerDesc{};
        Z.out_off = A.k;
        Z.elem_off = slots_all + A.slots;
        Z.tile_first = (int32_t)A.tiles;
        Z.layer_id = -1;
        d += A.n + 1;
        tiles_all += A.tiles;
        elems_all += A.elems;
        slots_all += A.slots;
        k_all += A.k;
        if (tiles_all > INT32_MAX) return DEFT_ERR_INVALID_ARG;
        acc[r] = Acc{0, 0, 0, 0, 0};   // pass 2 counts up again
    }
    // pass 2: the ranks' lists, and all layers as one list in address order behind them
    RankInfo& M = ri[N];
    LayerDesc* all = desc + d;
    int64_t m_tiles = 0, m_slots = 0;
    for (int32_t l = 0; l < L; ++l) {
        const int32_t r = rank_of[l];
        Acc& A = acc[r];
        const int64_t st = layer_start_h[l], en = layer_start_h[l + 1], size = en - st;
        LayerDesc D;
        D.start = st;
        D.end = en;
        D.k = k_l_h[l];
        D.out_off = A.k;
        D.elem_off = ri[r].elem_base + A.slots;
        D.tile_first = (int32_t)A.tiles;
        D.layer_id = l;
        D.norm = norms_h ? norms_h[l] : 0.0;
        D.reserved = 0;
        desc[ri[r].desc_first + A.n] = D;
        D.out_off += ri[r].out_off;
        D.elem_off = m_slots;
        D.tile_first = (int32_t)m_tiles;
        all[l] = D;
        const int64_t t = tiles_of(st, en);
        A.tiles += t;
        A.slots += slots_of(size);
        A.k += k_l_h[l];
        A.n += 1;
        m_tiles += t;
        m_slots += slots_of(size);
    }
    LayerDesc& Z = all[L];
    Z = LayerDesc{};
    Z.out_off = k_all;
    Z.elem_off = m_slots;
    Z.tile_first = (int32_t)m_tiles;
    Z.layer_id = -1;
    M.desc_first = (int32_t)d;
    M.n_my = L;
    M.tiles = (int32_t)m_tiles;
    M.tile_base = 0;
    M.elems = elems_all;
    M.k = k_all;
    M.out_off = 0;
    M.elem_base = 0;
    M.reserved[0] = M.reserved[1] = 0;
    hdr->magic = kPlanMagic;
    hdr->L = L;
    hdr->N = N;
    hdr->total_tiles = (int32_t)tiles_all;
    hdr->total_elems = elems_all;
    hdr->total_k = k_all;
    hdr->iteration = iteration;
    hdr->reserved[0] = hdr->reserved[1] = hdr->reserved[2] = 0;
    return DEFT_OK;
}

deft_status deft_plan_build(const int64_t* layer_start_h, const int64_t* k_l_h,
                            const int32_t* bin_of_layer_h, int32_t L, int32_t N, int64_t iteration,
                            void* plan_h, size_t plan_bytes_cap) {
    return plan_build_impl(layer_start_h, k_l_h, bin_of_layer_h, nullptr, L, N, iteration, plan_h, plan_bytes_cap);
}

static deft_status plan_step_impl(const double* norms_h, const int64_t* layer_start_h, int32_t L, int32_t N,
                                  int64_t k, int32_t mode, int32_t cost_model, int64_t iteration, int64_t* k_l_h,
                                  int64_t* sum_k_out, int32_t* bin_of_layer_h, double* bin_load_h, void* plan_h,
                                  size_t plan_bytes_cap, void* plan_d, void* ws_d, size_t ws_bytes, void* stream,
                                  bool clear) {
    if (!norms_h || !layer_start_h || !k_l_h || !bin_of_layer_h || !plan_h || !plan_d || !ws_d || L < 1)
        return DEFT_ERR_INVALID_ARG;
    static thread_local std::vector<int64_t> size;
    size.resize((size_t)L);
    for (int32_t l = 0; l < L; ++l) size[l] = layer_start_h[l + 1] - layer_start_h[l];
    const deft_status sa = deft_allocate_k(norms_h, size.data(), L, k, mode, k_l_h, sum_k_out);
    if (sa < 0) return sa;
    deft_status s = deft_partition_model(size.data(), k_l_h, L, N, cost_model, bin_of_layer_h, bin_load_h);
    if (s != DEFT_OK) return s;
    // the plan also carries the norms: the selection kernel scales its speculative cuts with them
    s = plan_build_impl(layer_start_h, k_l_h, bin_of_layer_h, norms_h, L, N, iteration, plan_h, plan_bytes_cap);
    if (s != DEFT_OK) return s;
    if (!aligned16(plan_d) || !aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    s = upload_plan(plan_h, plan_d, ws_d, ws_bytes, static_cast<cudaStream_t>(stream), clear);
    if (s != DEFT_OK) return s;
    return sa;   // DEFT_OK, or the Algorithm 3 warning
}

deft_status deft_plan_step(const double* norms_h, const int64_t* layer_start_h, int32_t L, int32_t N,
                           int64_t k, int32_t mode, int32_t cost_model, int64_t iteration, int64_t* k_l_h,
                           int64_t* sum_k_out, int32_t* bin_of_layer_h, double* bin_load_h, void* plan_h,
                           size_t plan_bytes_cap, void* plan_d, void* ws_d, size_t ws_bytes, void* stream) {
    return plan_step_impl(norms_h, layer_start_h, L, N, k, mode, cost_model, iteration, k_l_h, sum_k_out,
                          bin_of_layer_h, bin_load_h, plan_h, plan_bytes_cap, plan_d, ws_d, ws_bytes, stream, true);
}

deft_status deft_plan_rank_info(const void* plan_h, int32_t rank, int32_t* n_layers_out,
                                int64_t* elems_out, int64_t* k_out, int64_t* out_off_out) {
    if (!plan_ok(plan_h)) return DEFT_ERR_INVALID_ARG;
    const PlanHeader* hdr = static_cast<const PlanHeader*>(plan_h);
    if (rank < 0 || rank > hdr->N) return DEFT_ERR_INVALID_ARG;   // rank N = all ranks' layers as one list
    const RankInfo& R = plan_ranks(plan_h)[rank];
    if (n_layers_out) *n_layers_out = R.n_my;
    if (elems_out) *elems_out = R.elems;
    if (k_out) *k_out = R.k;
    if (out_off_out) *out_off_out = R.out_off;
    return DEFT_OK;
}

deft_status deft_plan_rank_table(const void* plan_h, int32_t N, int32_t* n_layers_h, int64_t* elems_h,
                                 int64_t* k_h, int64_t* out_off_h) {
    if (!plan_ok(plan_h)) return DEFT_ERR_INVALID_ARG;
    const PlanHeader* hdr = static_cast<const PlanHeader*>(plan_h);
    if (N != hdr->N) return DEFT_ERR_INVALID_ARG;
    const RankInfo* R = plan_ranks(plan_h);
    for (int32_t r = 0; r < N; ++r) {
        if (n_layers_h) n_layers_h[r] = R[r].n_my;
        if (elems_h) elems_h[r] = R[r].elems;
        if (k_h) k_h[r] = R[r].k;
        if (out_off_h) out_off_h[r] = R[r].out_off;
    }
    return DEFT_OK;
}

deft_status deft_plan_upload(const void* plan_h, void* plan_d, void* ws_d, size_t ws_bytes, void* stream) {
    if (!plan_ok(plan_h) || !plan_d || !ws_d || !aligned16(plan_d) || !aligned256(ws_d))
        return DEFT_ERR_INVALID_ARG;
    return upload_plan(plan_h, plan_d, ws_d, ws_bytes, static_cast<cudaStream_t>(stream));
}

deft_status deft_select_planned(const float* acc_d, const void* plan_h, const void* plan_d,
                                int32_t rank, float* val_d, int64_t* idx_d, int64_t out_cap,
                                void* ws_d, size_t ws_bytes, void* stream) {
    if (!plan_ok(plan_h) || !plan_d || !acc_d || !ws_d || out_cap < 0) return DEFT_ERR_INVALID_ARG;
    if (!aligned16(acc_d) || !aligned16(plan_d) || !aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    const PlanHeader* hdr = static_cast<const PlanHeader*>(plan_h);
    if (rank < 0 || rank >= hdr->N) return DEFT_ERR_INVALID_ARG;
    if (plan_ranks(plan_h)[rank].n_my > 0 && (!val_d || !idx_d)) return DEFT_ERR_INVALID_ARG;
    return select_rank(acc_d, plan_h, plan_d, rank, val_d, idx_d, out_cap, ws_d, ws_bytes,
                       static_cast<cudaStream_t>(stream));
}

deft_status deft_select_update_ranks(float* acc_d, int64_t n_g, const void* plan_h, const void* plan_d,
                                     int32_t rank_begin, int32_t rank_end, float* val_d, int64_t* idx_d,
                                     int64_t out_cap, void* ws_d, size_t ws_bytes, void* const* events,
                                     void* stream) {
    if (!plan_ok(plan_h) || !plan_d || !acc_d || !ws_d || !val_d || !idx_d || n_g < 1)
        return DEFT_ERR_INVALID_ARG;
    if (!aligned16(acc_d) || !aligned16(plan_d) || !aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    const PlanHeader* hdr = static_cast<const PlanHeader*>(plan_h);
    if (rank_begin < 0 || rank_end > hdr->N || rank_begin > rank_end) return DEFT_ERR_INVALID_ARG;
    if (out_cap < hdr->total_k) return DEFT_ERR_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (int32_t r = rank_begin; r < rank_end; ++r) {
        const RankInfo& R = plan_ranks(plan_h)[r];
        void* const* ev = events ? events + 3 * (size_t)(r - rank_begin) : nullptr;
        if (ev) DEFT_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(ev[0]), st));
        // the selection kernel zeroes what it selects on its way out (same result as a separate
        // deft_residual_update of the rank's indices, one launch less)
        const deft_status s = select_rank(acc_d, plan_h, plan_d, r, val_d + R.out_off, idx_d + R.out_off, R.k,
                                          ws_d, ws_bytes, st, true);
        if (s != DEFT_OK) return s;
        if (ev) DEFT_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(ev[1]), st));
        if (ev) DEFT_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(ev[2]), st));
    }
    return DEFT_OK;
}

deft_status deft_select_update_all(float* acc_d, int64_t n_g, const void* plan_h, const void* plan_d,
                                   float* val_d, int64_t* idx_d, int64_t out_cap, void* ws_d, size_t ws_bytes,
                                   void* stream) {
    if (!plan_ok(plan_h) || !plan_d || !acc_d || !ws_d || !val_d || !idx_d || n_g < 1)
        return DEFT_ERR_INVALID_ARG;
    if (!aligned16(acc_d) || !aligned16(plan_d) || !aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    const PlanHeader* hdr = static_cast<const PlanHeader*>(plan_h);
    if (out_cap < hdr->total_k) return DEFT_ERR_CAPACITY;
    const RankInfo& M = plan_ranks(plan_h)[hdr->N];
    if (M.n_my > 0) {
        const deft_status s = select_rank(acc_d, plan_h, plan_d, hdr->N, val_d, idx_d, M.k, ws_d, ws_bytes,
                                          static_cast<cudaStream_t>(stream), true);
        if (s != DEFT_ERR_TOO_LARGE) return s;   // beyond one launch's limits: one launch per rank instead
    }
    return deft_select_update_ranks(acc_d, n_g, plan_h, plan_d, 0, hdr->N, val_d, idx_d, out_cap, ws_d, ws_bytes,
                                    nullptr, stream);
}

deft_status deft_step(float* resid_acc_d, const float* grad_d, int64_t n_g, const int64_t* layer_start_h,
                      const int64_t* layer_start_d, int32_t L, int32_t N, int64_t k, int32_t mode,
                      int32_t cost_model, int64_t iteration, int32_t rank, double* norms_d, double* norms_h,
                      int64_t* k_l_h, int64_t* sum_k_out, int32_t* bin_of_layer_h, double* bin_load_h,
                      void* plan_h, size_t plan_bytes_cap, void* plan_d, float* val_d, int64_t* idx_d,
                      int64_t out_cap, void* ws_d, size_t ws_bytes, void* const* events, void* stream) {
    if (!norms_h || rank < -1 || rank >= N) return DEFT_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto mark = [&](int i) -> cudaError_t {
        return events ? cudaEventRecord(static_cast<cudaEvent_t>(events[i]), st) : cudaSuccess;
    };
    if (!resid_acc_d || !layer_start_d || !norms_d || !ws_d || n_g < 1 || L < 1) return DEFT_ERR_INVALID_ARG;
    if (!aligned16(resid_acc_d) || (grad_d && !aligned16(grad_d)) || !aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    const size_t part = ws_layout(n_g, L, 1).norm_partial;
    if (part + norms_ws_bytes(n_g, L) > ws_bytes) return DEFT_ERR_CAPACITY;
    // If norms_h is pinned memory the device can write (the usual case), the kernel that finishes
    // the norms stores them there itself and this thread polls for them: the step then needs no
    // stream synchronisation, whose wake-up costs tens of microseconds of device idle time.
    double* mapped = nullptr;
    {
        cudaPointerAttributes at;
        if (cudaPointerGetAttributes(&at, norms_h) == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer)
            mapped = static_cast<double*>(at.devicePointer);
        else
            (void)cudaGetLastError();
    }
    const uint64_t kUnset = 0x7ff8dead00000000ull;   // a NaN pattern no norm can have
    volatile uint64_t* slots = reinterpret_cast<volatile uint64_t*>(norms_h);
    if (mapped)
        for (int32_t l = 0; l < L; ++l) slots[l] = kUnset | (uint32_t)l;
    // With all workers in one launch and a vector the single-pass selection kernel takes, the accumulate pass
    // stages every entry above its layer's remembered cut on the way (the per-layer counters are cleared
    // BEFORE it then): the selection launch finds its entries staged and reads nothing.
    const WsLayout wl = ws_layout(1, L, 1);   // the cleared area's place depends on the layer count only
    if (wl.zero_end > ws_bytes) return DEFT_ERR_CAPACITY;
    bool fused = g_step_fused != 0 && g_stream_kernel != 0 && rank < 0 && L <= kStreamMaxLayers && n_g <= kStreamMaxElems &&
                 (g_stream_kernel > 0 || n_g >= kStreamMinElems);
    StageLaunch sl{};
    if (fused) {
        int64_t tiles_all = 0;
        for (int32_t l = 0; l < L; ++l) {
            const int64_t a = layer_start_h[l], b = layer_start_h[l + 1];
            if (a < 0 || b <= a) { fused = false; break; }
            tiles_all += (b - 1) / kTile - a / kTile + 1;
        }
        if (fused && layer_start_h[L] == n_g && tiles_all <= INT32_MAX) {
            const WsLayout w = ws_layout(n_g, L, tiles_all);
            if (w.total > ws_bytes) return DEFT_ERR_CAPACITY;
            char* ws = static_cast<char*>(ws_d);
            sl.hint = reinterpret_cast<const LayerHint*>(ws + w.hint + 256);
            sl.tab = reinterpret_cast<StageTab*>(ws + w.stage_tab);
            sl.state = reinterpret_cast<LayerState*>(ws + w.state);
            sl.runge = reinterpret_cast<uint2*>(ws + w.runge) + 2 * (size_t)N;   // the all-layers list's table
            sl.staging = reinterpret_cast<uint2*>(ws + w.staging);
        } else {
            fused = false;
        }
    }
    if (fused)
        DEFT_CUDA_TRY(cudaMemsetAsync(static_cast<char*>(ws_d) + wl.zero_begin, 0, wl.zero_end - wl.zero_begin, st));
    DEFT_CUDA_TRY(mark(0));
    deft_status s = launch_layer_norms(resid_acc_d, grad_d, n_g, layer_start_d, L, norms_d,
                                       reinterpret_cast<double*>(static_cast<char*>(ws_d) + part), st, mapped,
                                       fused ? &sl : nullptr);
    if (s != DEFT_OK) return s;
    DEFT_CUDA_TRY(mark(1));
    // the per-layer counters of the selection are cleared while the host plans
    if (!fused)
        DEFT_CUDA_TRY(cudaMemsetAsync(static_cast<char*>(ws_d) + wl.zero_begin, 0, wl.zero_end - wl.zero_begin, st));
    bool have = false;
    if (mapped) {
        const auto t0 = std::chrono::steady_clock::now();
        for (uint64_t spins = 0;; ++spins) {
            bool all = true;
            for (int32_t l = L - 1; l >= 0 && all; --l) all = (slots[l] >> 32) != (kUnset >> 32);
            if (all) { have = true; break; }
            if ((spins & 0x3ff) == 0x3ff &&
                std::chrono::steady_clock::now() - t0 > std::chrono::seconds(2)) break;   // bounded wait
        }
    }
    if (!have) {
        DEFT_CUDA_TRY(cudaMemcpyAsync(norms_h, norms_d, sizeof(double) * (size_t)L, cudaMemcpyDeviceToHost, st));
        DEFT_CUDA_TRY(cudaStreamSynchronize(st));   // Algorithms 3 and 4 run on the host and need this step's norms
    }
    const deft_status sp = plan_step_impl(norms_h, layer_start_h, L, N, k, mode, cost_model, iteration, k_l_h,
                                          sum_k_out, bin_of_layer_h, bin_load_h, plan_h, plan_bytes_cap, plan_d,
                                          ws_d, ws_bytes, stream, false);
    if (sp < 0) return sp;
    DEFT_CUDA_TRY(mark(2));
    if (rank < 0) {
        s = kNotPrestaged;
        if (fused) {
            const PlanHeader* hdr = static_cast<const PlanHeader*>(plan_h);
            const RankInfo& M = plan_ranks(plan_h)[hdr->N];
            if (!val_d || !idx_d) return DEFT_ERR_INVALID_ARG;
            if (out_cap < hdr->total_k) return DEFT_ERR_CAPACITY;
            if (M.n_my == L)
                s = select_rank(resid_acc_d, plan_h, plan_d, hdr->N, val_d, idx_d, M.k, ws_d, ws_bytes, st, true,
                                FixedThreshold(), true);
            if (s == kNotPrestaged || s == DEFT_ERR_TOO_LARGE) {   // not this step: forget what was staged
                DEFT_CUDA_TRY(cudaMemsetAsync(static_cast<char*>(ws_d) + wl.zero_begin, 0, wl.zero_end - wl.zero_begin, st));
                s = kNotPrestaged;
            }
        }
        if (s == kNotPrestaged)
            s = deft_select_update_all(resid_acc_d, n_g, plan_h, plan_d, val_d, idx_d, out_cap, ws_d, ws_bytes, stream);
    } else {
        const RankInfo& R = plan_ranks(plan_h)[rank];
        if (!val_d || !idx_d) return DEFT_ERR_INVALID_ARG;
        s = select_rank(resid_acc_d, plan_h, plan_d, rank, val_d, idx_d, out_cap < R.k ? out_cap : R.k, ws_d,
                        ws_bytes, st, true);
    }
    if (s != DEFT_OK) return s;
    DEFT_CUDA_TRY(mark(3));
    return sp;   // DEFT_OK, or the Algorithm 3 warning
}

deft_status deft_select(const float* acc_d, const int64_t* layer_start_h, const int64_t* k_l_h,
                        const int32_t* my_layers_h, int32_t n_my, float* val_d, int64_t* idx_d,
                        int64_t out_cap, void* ws_d, size_t ws_bytes, void* stream) {
    if (n_my < 0 || out_cap < 0) return DEFT_ERR_INVALID_ARG;
    if (n_my == 0) return DEFT_OK;
    if (!acc_d || !layer_start_h || !k_l_h || !my_layers_h || !val_d || !idx_d || !ws_d)
        return DEFT_ERR_INVALID_ARG;
    if (!aligned16(acc_d) || !aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    std::vector<LayerItem> items((size_t)n_my);
    for (int32_t j = 0; j < n_my; ++j) {
        const int32_t l = my_layers_h[j];
        if (l < 0 || (j > 0 && l <= my_layers_h[j - 1])) return DEFT_ERR_INVALID_ARG;
        items[j] = LayerItem{layer_start_h[l], layer_start_h[l + 1], k_l_h[l], j};
    }
    return select_once(acc_d, items, val_d, idx_d, out_cap, ws_d, ws_bytes,
                       static_cast<cudaStream_t>(stream));
}

deft_status deft_topk_baseline(const float* acc_d, int64_t n, int64_t k, float* val_d,
                               int64_t* idx_d, void* ws_d, size_t ws_bytes, void* stream) {
    if (!acc_d || !val_d || !idx_d || !ws_d || n < 1 || n > DEFT_MAX_LAYER_ELEMS || k < 1 || k > n)
        return DEFT_ERR_INVALID_ARG;
    if (!aligned16(acc_d) || !aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    std::vector<LayerItem> items(1, LayerItem{0, n, k, 0});
    return select_once(acc_d, items, val_d, idx_d, k, ws_d, ws_bytes, static_cast<cudaStream_t>(stream));
}

deft_status deft_threshold_select(float* acc_d, int64_t n, float threshold, int32_t zero_selected, float* val_d,
                                  int64_t* idx_d, int64_t out_cap, int64_t* count_d, void* ws_d, size_t ws_bytes,
                                  void* stream) {
    if (!acc_d || !count_d || !ws_d || n < 1 || n > DEFT_MAX_LAYER_ELEMS || out_cap < 0 ||
        (out_cap > 0 && (!val_d || !idx_d)) || threshold != threshold)
        return DEFT_ERR_INVALID_ARG;
    if (!aligned16(acc_d) || !aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    std::vector<std::vector<LayerItem>> ranks(1, std::vector<LayerItem>(1, LayerItem{0, n, 1, 0}));
    std::vector<char> blob(plan_bytes(1, 1));
    deft_status s = fill_plan(blob.data(), blob.size(), 1, 0, ranks);
    if (s != DEFT_OK) return s;
    const PlanHeader* hdr = reinterpret_cast<const PlanHeader*>(blob.data());
    const WsLayout w = ws_layout(hdr->total_elems, hdr->L, hdr->total_tiles);
    if (w.total > ws_bytes) return DEFT_ERR_CAPACITY;
    void* plan_d = static_cast<char*>(ws_d) + w.plan;
    s = upload_plan(blob.data(), plan_d, ws_d, ws_bytes, st);
    if (s != DEFT_OK) return s;
    DEFT_CUDA_TRY(cudaMemsetAsync(count_d, 0, sizeof(int64_t), st));
    FixedThreshold fixed;
    fixed.on = true;
    uint32_t bits;
    std::memcpy(&bits, &threshold, 4);
    fixed.key = bits & 0x7fffffffu;
    fixed.count_d = reinterpret_cast<unsigned long long*>(count_d);
    return select_rank(acc_d, blob.data(), plan_d, 0, val_d, idx_d, out_cap, ws_d, ws_bytes, st, zero_selected != 0,
                       fixed);
}

int32_t deft_clt_leader(int64_t iteration, int32_t N) {
    if (N < 1 || iteration < 0) return -1;
    return (int32_t)(iteration % N);
}

deft_status deft_gather_update(float* acc_d, int64_t n_g, const int64_t* idx_d, int64_t count, float* val_d,
                               void* stream) {
    if (count < 0 || n_g < 1 || count > n_g) return DEFT_ERR_INVALID_ARG;
    if (count == 0) return DEFT_OK;
    if (!acc_d || !idx_d || !val_d) return DEFT_ERR_INVALID_ARG;
    return launch_gather_update(acc_d, idx_d, count, val_d, static_cast<cudaStream_t>(stream));
}

size_t deft_union_workspace_bytes(int64_t n_g) { return n_g < 1 ? 0 : union_ws_bytes(n_g); }

deft_status deft_index_union(const int64_t* idx_d, int64_t count, int64_t n_g, int64_t* union_d, int64_t out_cap,
                             int64_t* count_d, void* ws_d, size_t ws_bytes, void* stream) {
    if (count < 0 || n_g < 1 || out_cap < 0 || !count_d || !ws_d || (count > 0 && !idx_d) || (out_cap > 0 && !union_d))
        return DEFT_ERR_INVALID_ARG;
    if (!aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    if (union_ws_bytes(n_g) > ws_bytes) return DEFT_ERR_CAPACITY;
    return launch_index_union(idx_d, count, n_g, union_d, out_cap, reinterpret_cast<long long*>(count_d), ws_d,
                              static_cast<cudaStream_t>(stream));
}

deft_status deft_sum_into(float* dst_d, const float* src_d, int64_t count, void* stream) {
    if (count < 0 || (count > 0 && (!dst_d || !src_d))) return DEFT_ERR_INVALID_ARG;
    return launch_sum_into(dst_d, src_d, count, static_cast<cudaStream_t>(stream));
}

deft_status deft_average(float* sum_d, int64_t count, int32_t n_workers, void* stream) {
    if (count < 0 || n_workers < 1 || (count > 0 && !sum_d)) return DEFT_ERR_INVALID_ARG;
    return launch_divide(sum_d, count, (float)n_workers, static_cast<cudaStream_t>(stream));
}

size_t deft_vector_norm_workspace_bytes(int64_t n) { return n < 1 ? 0 : 256 + align_up(norms_ws_bytes(n, 1), 256); }

deft_status deft_vector_norm(const float* x_d, int64_t n, double* norm_d, void* ws_d, size_t ws_bytes, void* stream) {
    if (!x_d || !norm_d || !ws_d || n < 1) return DEFT_ERR_INVALID_ARG;
    if (!aligned16(x_d) || !aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    if (deft_vector_norm_workspace_bytes(n) > ws_bytes) return DEFT_ERR_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int64_t* ls_d = static_cast<int64_t*>(ws_d);
    const deft_status s = launch_fill_start(ls_d, n, st);
    if (s != DEFT_OK) return s;
    // the accumulate + norm kernel in its norms-only form (no gradient: nothing is written to x)
    return launch_layer_norms(const_cast<float*>(x_d), nullptr, n, ls_d, 1, norm_d,
                              reinterpret_cast<double*>(static_cast<char*>(ws_d) + 256), st);
}

deft_status deft_residual_update(float* acc_d, int64_t n_g, const int64_t* idx_d, int64_t count,
                                 void* stream) {
    if (count < 0 || n_g < 1 || count > n_g) return DEFT_ERR_INVALID_ARG;
    if (count == 0) return DEFT_OK;
    if (!acc_d || !idx_d) return DEFT_ERR_INVALID_ARG;
    return launch_residual_update(acc_d, idx_d, count, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
