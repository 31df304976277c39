// Shared device/host definitions of libdeft's CUDA side (sm_100a only).
#pragma once
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>

#include "deft.h"

namespace deft {

// ---------------------------------------------------------------------------------
// Selection geometry.  A layer is cut into tiles that are aligned in ADDRESS space
// (multiples of kTile elements from the start of the vector), so that every full tile
// is read with aligned 128-bit loads whatever the layer boundaries are; the first and
// last tile of a layer may be partial and are read element-wise under a mask.
// ---------------------------------------------------------------------------------
constexpr int kTile = 4096;      // elements per tile
constexpr int kThreads = 256;    // threads per CTA in the streaming kernels
constexpr int kWarps = kThreads / 32;
constexpr int kSlabs = 4;        // float4 loads per thread per tile (kTile = kThreads*4*kSlabs)

// Radix digits over the 31-bit magnitude key (IEEE bits with the sign cleared):
// level 1 = bits 30..20 (exponent + 3 mantissa bits), level 2 = bits 19..9, level 3 = bits 8..0.
constexpr int kBins1 = 2048, kBins2 = 2048, kBins3 = 512;
constexpr int kShift1 = 20, kShift2 = 9;

// Accumulate+norm geometry.
constexpr int kTileA = 8192;     // elements per CTA iteration

struct LayerDesc {               // one per layer of the rank (+1 sentinel), 48 bytes
    int64_t start, end;          // element range in the flat vector
    int64_t k;                   // entries to select (1..size)
    int64_t out_off;             // position of the layer's first output entry
    int64_t elem_off;            // elements in the rank's earlier layers (= staging base)
    int32_t tile_first;          // rank-local id of the layer's first tile
    int32_t pad;
};
static_assert(sizeof(LayerDesc) == 48, "LayerDesc layout");

struct LayerState {              // written by the scan kernels, 32 bytes
    uint32_t b1, krem1;          // level-1 bucket of the k-th key; how many still to take inside it
    uint32_t b2, krem2;          // same for level 2 (inside bucket b1)
    uint32_t T, need;            // exact threshold key; how many entries equal to T to take
    uint32_t pad0, pad1;
};
static_assert(sizeof(LayerState) == 32, "LayerState layout");

struct SelectWorkspace {         // carve-up of the caller's workspace for one selection call
    LayerDesc* desc;             // [n_my + 1]
    LayerState* state;           // [n_my]            \  zeroed
    uint32_t* hist1;             // [n_my][kBins1]     | at the start
    uint32_t* hist2;             // [n_my][kBins2]     | of every
    uint32_t* hist3;             // [n_my][kBins3]    /  call
    size_t zero_bytes;           // bytes from `state` to the end of hist3
    uint32_t* cnt;               // [tiles] staged entries per tile
    uint2* ge;                   // [tiles] (#key > T, #key == T) per tile, then their exclusive scans
    uint2* staging;              // [n_r]   (value bits, offset in tile) of every entry with key >= bucket b1
    size_t total_bytes;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline SelectWorkspace carve_select_ws(void* base, int64_t n_my, int64_t tiles, int64_t elems) {
    SelectWorkspace w{};
    size_t off = 0;
    char* p = static_cast<char*>(base);
    w.desc = reinterpret_cast<LayerDesc*>(p + off);
    off = align_up(off + sizeof(LayerDesc) * (size_t)(n_my + 1), 256);
    const size_t z0 = off;
    w.state = reinterpret_cast<LayerState*>(p + off);
    off = align_up(off + sizeof(LayerState) * (size_t)n_my, 256);
    w.hist1 = reinterpret_cast<uint32_t*>(p + off);
    off += sizeof(uint32_t) * (size_t)n_my * kBins1;
    w.hist2 = reinterpret_cast<uint32_t*>(p + off);
    off += sizeof(uint32_t) * (size_t)n_my * kBins2;
    w.hist3 = reinterpret_cast<uint32_t*>(p + off);
    off += sizeof(uint32_t) * (size_t)n_my * kBins3;
    w.zero_bytes = off - z0;
    off = align_up(off, 256);
    w.cnt = reinterpret_cast<uint32_t*>(p + off);
    off = align_up(off + sizeof(uint32_t) * (size_t)tiles, 256);
    w.ge = reinterpret_cast<uint2*>(p + off);
    off = align_up(off + sizeof(uint2) * (size_t)tiles, 256);
    w.staging = reinterpret_cast<uint2*>(p + off);
    off = align_up(off + sizeof(uint2) * (size_t)elems, 256);
    w.total_bytes = off;
    return w;
}

// Upper bound on the tiles of `layers` layers holding `elems` elements in total.
inline int64_t max_tiles(int64_t elems, int64_t layers) { return elems / kTile + 2 * layers; }

inline size_t norms_ws_bytes(int64_t n_g, int64_t L) {
    return sizeof(double) * (size_t)((n_g + kTileA - 1) / kTileA + L + 1);
}

// Sticky per-thread CUDA error code for deft_last_cuda_error().
void set_last_cuda_error(cudaError_t e);
int sm_count();

#define DEFT_CUDA_TRY(expr)                                  \
    do {                                                     \
        cudaError_t err__ = (expr);                          \
        if (err__ != cudaSuccess) {                          \
            ::deft::set_last_cuda_error(err__);              \
            return DEFT_ERR_CUDA;                            \
        }                                                    \
    } while (0)

// Launchers (each enqueues on `stream` and returns a status).
deft_status launch_layer_norms(float* resid_acc_d, const float* grad_d, int64_t n_g,
                               const int64_t* layer_start_d, int32_t L, double* norms_d,
                               double* partial_d, cudaStream_t stream);
deft_status launch_select(const float* acc_d, const SelectWorkspace& w, int32_t n_my, int32_t tiles,
                          float* val_d, int64_t* idx_d, cudaStream_t stream);
deft_status launch_residual_update(float* acc_d, const int64_t* idx_d, int64_t count,
                                   cudaStream_t stream);

}  // namespace deft
