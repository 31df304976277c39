// C-ABI entry points of libdeft that touch the GPU: argument checks, workspace carve-up,
// the small host-built layer table of one rank, and the kernel launch sequence.
#include <vector>

#include "deft_common.cuh"

namespace deft {

static thread_local int32_t g_last_cuda_error = 0;

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

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

// Builds the rank's layer table (with sentinel) on the host.  Returns a status.
deft_status build_rank_table(const int64_t* layer_start_h, const int64_t* k_l_h,
                             const int32_t* my_layers_h, int32_t n_my, std::vector<LayerDesc>& out,
                             int64_t& tiles, int64_t& elems, int64_t& k_total) {
    out.resize((size_t)n_my + 1);
    tiles = elems = k_total = 0;
    for (int32_t j = 0; j < n_my; ++j) {
        const int32_t l = my_layers_h[j];
        if (l < 0 || (j > 0 && l <= my_layers_h[j - 1])) return DEFT_ERR_INVALID_ARG;
        const int64_t s = layer_start_h[l], e = layer_start_h[l + 1];
        if (s < 0 || e <= s || e - s > DEFT_MAX_LAYER_ELEMS) return DEFT_ERR_INVALID_ARG;
        if (j > 0 && s < out[j - 1].end) return DEFT_ERR_INVALID_ARG;
        const int64_t k = k_l_h[l];
        if (k < 1 || k > e - s) return DEFT_ERR_INVALID_ARG;
        if (tiles > INT32_MAX - (e - s) / kTile - 2) return DEFT_ERR_INVALID_ARG;
        LayerDesc& d = out[j];
        d.start = s;
        d.end = e;
        d.k = k;
        d.out_off = k_total;
        d.elem_off = elems;
        d.tile_first = (int32_t)tiles;
        d.pad = 0;
        tiles += (e - 1) / kTile - s / kTile + 1;
        elems += e - s;
        k_total += k;
    }
    LayerDesc& z = out[n_my];
    z.start = z.end = 0;
    z.k = 0;
    z.out_off = k_total;
    z.elem_off = elems;
    z.tile_first = (int32_t)tiles;
    z.pad = 0;
    return DEFT_OK;
}

deft_status select_common(const float* acc_d, const std::vector<LayerDesc>& table, int32_t n_my,
                          int64_t tiles, int64_t elems, int64_t k_total, float* val_d, int64_t* idx_d,
                          int64_t out_cap, void* ws_d, size_t ws_bytes, cudaStream_t stream) {
    if (out_cap < k_total) return DEFT_ERR_CAPACITY;
    const SelectWorkspace w = carve_select_ws(ws_d, n_my, tiles, elems);
    if (w.total_bytes > ws_bytes) return DEFT_ERR_CAPACITY;
    // The table lives in pageable host memory: the runtime stages it before returning, so
    // the vector may be released as soon as this call returns.
    DEFT_CUDA_TRY(cudaMemcpyAsync(w.desc, table.data(), sizeof(LayerDesc) * ((size_t)n_my + 1),
                                  cudaMemcpyHostToDevice, stream));
    return launch_select(acc_d, w, n_my, (int32_t)tiles, val_d, idx_d, stream);
}

}  // namespace
}  // namespace deft

using namespace deft;

extern "C" {

int32_t deft_last_cuda_error(void) { return g_last_cuda_error; }

size_t deft_workspace_bytes(int64_t max_elems, int32_t max_layers) {
    if (max_elems < 1 || max_layers < 1) return 0;
    const SelectWorkspace w =
        carve_select_ws(nullptr, max_layers, max_tiles(max_elems, max_layers), max_elems);
    const size_t a = w.total_bytes;
    const size_t b = align_up(norms_ws_bytes(max_elems, max_layers), 256);
    return a > b ? a : b;
}

deft_status deft_layer_norms(float* resid_acc_d, const float* grad_d, int64_t n_g,
                             const int64_t* layer_start_d, int32_t L, double* norms_d, void* ws_d,
                             size_t ws_bytes, void* stream) {
    if (!resid_acc_d || !layer_start_d || !norms_d || !ws_d || n_g < 1 || L < 1)
        return DEFT_ERR_INVALID_ARG;
    if (!aligned16(resid_acc_d) || (grad_d && !aligned16(grad_d)) || !aligned256(ws_d))
        return DEFT_ERR_INVALID_ARG;
    if (norms_ws_bytes(n_g, L) > ws_bytes) return DEFT_ERR_CAPACITY;
    return launch_layer_norms(resid_acc_d, grad_d, n_g, layer_start_d, L, norms_d,
                              static_cast<double*>(ws_d), static_cast<cudaStream_t>(stream));
}

deft_status deft_select(const float* acc_d, const int64_t* layer_start_h, const int64_t* k_l_h,
                        const int32_t* my_layers_h, int32_t n_my, float* val_d, int64_t* idx_d,
                        int64_t out_cap, void* ws_d, size_t ws_bytes, void* stream) {
    if (n_my < 0 || out_cap < 0) return DEFT_ERR_INVALID_ARG;
    if (n_my == 0) return DEFT_OK;
    if (!acc_d || !layer_start_h || !k_l_h || !my_layers_h || !val_d || !idx_d || !ws_d)
        return DEFT_ERR_INVALID_ARG;
    if (!aligned16(acc_d) || !aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    std::vector<LayerDesc> table;
    int64_t tiles, elems, k_total;
    const deft_status s =
        build_rank_table(layer_start_h, k_l_h, my_layers_h, n_my, table, tiles, elems, k_total);
    if (s != DEFT_OK) return s;
    return select_common(acc_d, table, n_my, tiles, elems, k_total, val_d, idx_d, out_cap, ws_d,
                         ws_bytes, static_cast<cudaStream_t>(stream));
}

deft_status deft_topk_baseline(const float* acc_d, int64_t n, int64_t k, float* val_d,
                               int64_t* idx_d, void* ws_d, size_t ws_bytes, void* stream) {
    if (!acc_d || !val_d || !idx_d || !ws_d || n < 1 || n > DEFT_MAX_LAYER_ELEMS || k < 1 || k > n)
        return DEFT_ERR_INVALID_ARG;
    if (!aligned16(acc_d) || !aligned256(ws_d)) return DEFT_ERR_INVALID_ARG;
    const int64_t layer_start[2] = {0, n};
    const int32_t only = 0;
    std::vector<LayerDesc> table;
    int64_t tiles, elems, k_total;
    const deft_status s = build_rank_table(layer_start, &k, &only, 1, table, tiles, elems, k_total);
    if (s != DEFT_OK) return s;
    return select_common(acc_d, table, 1, tiles, elems, k_total, val_d, idx_d, k, ws_d, ws_bytes,
                         static_cast<cudaStream_t>(stream));
}

deft_status deft_residual_update(float* acc_d, int64_t n_g, const int64_t* idx_d, int64_t count,
                                 void* stream) {
    if (count < 0 || n_g < 1 || count > n_g) return DEFT_ERR_INVALID_ARG;
    if (count == 0) return DEFT_OK;
    if (!acc_d || !idx_d) return DEFT_ERR_INVALID_ARG;
    return launch_residual_update(acc_d, idx_d, count, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
