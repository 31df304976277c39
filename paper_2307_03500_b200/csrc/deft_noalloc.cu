// deft_layer_norms_static: the accumulate + per-layer norm call for callers that cannot
// provide a workspace.  Its scratch (the per-tile partial sums) lives in a fixed array in
// device memory that is part of the library image, so the call needs no buffer from the
// caller and allocates nothing.
#include <mutex>

#include "deft_common.cuh"

namespace deft {
namespace {

constexpr int kStaticSlots = 16384;   // partial-sum slots: ceil(n_g / kTileA) + L + 1 must fit
constexpr int kMaxDevices = 64;

// File-scope scratch.  Every GPU that loads the library holds these 128 KB until the
// process exits.  The name below is only a host-side handle: the device address is
// obtained once per device with cudaGetSymbolAddress and that pointer goes to the kernels.
static __device__ __align__(256) double g_norm_partials[kStaticSlots];

std::mutex g_setup_mutex;
double* g_partials_ptr[kMaxDevices] = {nullptr};

// Device address of g_norm_partials on the current device (looked up on first use).
deft_status static_scratch(double** out) {
    int dev = 0;
    DEFT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return DEFT_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_partials_ptr[dev]) {
        double* ptr = nullptr;
        DEFT_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_norm_partials));
        if (!ptr) return DEFT_ERR_CUDA;
        g_partials_ptr[dev] = ptr;
    }
    *out = g_partials_ptr[dev];
    return DEFT_OK;
}

}  // namespace
}  // namespace deft

using namespace deft;

extern "C" {

int64_t deft_layer_norms_static_max_slots(void) { return kStaticSlots; }

deft_status deft_layer_norms_static(float* resid_acc_d, const float* grad_d, int64_t n_g,
                                    const int64_t* layer_start_d, int32_t L, double* norms_d,
                                    void* stream) {
    if (!resid_acc_d || !layer_start_d || !norms_d || n_g < 1 || L < 1) return DEFT_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(resid_acc_d) & 15u) || (grad_d && (reinterpret_cast<uintptr_t>(grad_d) & 15u)))
        return DEFT_ERR_INVALID_ARG;
    const int64_t need = (n_g + kTileA - 1) / kTileA + (int64_t)L + 1;
    if (need > kStaticSlots) return DEFT_ERR_CAPACITY;   // too large for the built-in scratch
    double* partials = nullptr;
    const deft_status s = static_scratch(&partials);
    if (s != DEFT_OK) return s;
    // Every slot the finalize kernel reads is written by the accumulate kernel of this same
    // call first, so nothing left over from an earlier call is ever read.
    return launch_layer_norms(resid_acc_d, grad_d, n_g, layer_start_d, L, norms_d, partials,
                              static_cast<cudaStream_t>(stream));
}

}  // extern "C"
