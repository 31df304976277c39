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
// One warp processes one tile at a time.  Every CTA owns a contiguous run of a rank's
// tiles in every phase and keeps the entries it stages for them.
// ---------------------------------------------------------------------------------
constexpr int kTile = 2048;          // elements per tile
constexpr int kSelThreads = 512;     // one persistent CTA per SM (128 registers per thread)
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSlots = 4;            // level-1 shared-memory histograms live at once per CTA

// Radix digits over the 31-bit magnitude key (IEEE bits with the sign cleared):
// level 1 = bits 30..19 (exponent + 4 mantissa bits), level 2 = bits 18..9, level 3 = bits 8..0.
constexpr int kBins1 = 4096, kBins2 = 1024, kBins3 = 512;
constexpr int kShift1 = 19, kShift2 = 9;
// Layers that one CTA loads whole ("direct") use coarser digits: bits 30..19, 18..9, 8..0.
constexpr int kDBins1 = 4096, kDBins2 = 1024, kDBins3 = 512;
constexpr int kDShift1 = 19, kDShift2 = 9;

// Layers of at most kDirectElems elements are not streamed: one CTA loads each of them whole.
constexpr int kDirectElems = 16384;
// Staged entries a CTA keeps in shared memory; the rest spills to the staging stream in HBM.
constexpr int kResident = 8192;
// Limits of one CTA's share of a rank (checked on the host before launch).
constexpr int kMaxLocalTiles = 4096;    // tiles per CTA
constexpr int kStreamLocalTiles = 2048;  // tiles per CTA in the single-pass kernel (its read keeps a smaller tile table)
constexpr int kMaxLocalLayers = 256;    // streamed layers per CTA
// A rank that is one layer of at least kInterleaveTiles tiles per CTA is split over the CTAs in
// super-tiles of kSuper tiles dealt out round-robin instead of one contiguous run per CTA.
constexpr int kSuper = 16;
constexpr int kInterleaveTiles = 64;

constexpr int kMaxRanks = 4096;      // workers per plan
constexpr int kRegionAlign = 16;     // a layer's region of the staging area starts on a multiple of this many entries (128 bytes)
constexpr int kSpecDensity = 8;      // no speculative cut for layers that select more than 1 / kSpecDensity of their entries

// Cost-weighted split of a large multi-layer rank (second read onwards).  The first read costs
// the same for every tile; from the staging pass on, a tile costs more the more of its entries
// pass the first-level cut, and what a CTA stages it also carries through the later steps.  The
// expected number of staged entries per tile is known before launch (k_l / size_l), so the
// tiles are dealt out in contiguous runs of equal estimated cost instead of equal length.
constexpr int kMaxWeightedLayers = 8192;

#if defined(__CUDACC__)
#define DEFT_HD __host__ __device__
#else
#define DEFT_HD
#endif

// Layers the single-pass kernel's finishing CTA takes (one CTA per layer: 2 to 7 us per 1000 staged entries, the
// more the fewer of them fit in shared memory).  When the kernel stages for itself (tight cuts: about two
// staged entries per selected one) those that select up to 65536 entries; when the accumulate pass has staged
// (wider margins) up to 16384: a layer that selects more is read again by the whole grid instead.
constexpr int64_t kStreamMaxK = 65536, kStreamMaxKPrestaged = 16384;
DEFT_HD inline bool stream_can_finish(int64_t k, bool prestaged) {
    return k <= (prestaged ? kStreamMaxKPrestaged : kStreamMaxK);
}

// Cost of one tile of a layer in units of 1/64 of a tile that stages nothing (constants fitted
// to step timings on B200: +50 % once most 16-byte loads of the tile hold an entry, +0.55 % per
// staged entry for the later passes).  Layers that are not streamed cost nothing.
DEFT_HD inline uint32_t tile_weight(int64_t k, int64_t size) {
    if (size <= kDirectElems) return 0u;
    int64_t rho = (k * 3072 + size - 1) / size;   // expected staged entries per tile (1.5 x k_l's share)
    if (rho > kTile) rho = kTile;
    return (uint32_t)(64 + 2 * (rho < 16 ? rho : 16) + rho * 3 / 8);
}

// First tile of CTA b of G.  Wp[j] = sum over layers before j of tiles * weight (j = 0..n),
// w[j] = weight of a tile of layer j, tf[j] = first tile of layer j (tf[n] = tiles).
DEFT_HD inline int weighted_boundary(const uint32_t* Wp, const uint32_t* w, const int* tf, int n, int tiles,
                                     int b, int G) {
    if (b <= 0) return 0;
    if (b >= G) return tiles;
    const uint64_t target = (uint64_t)Wp[n] * (uint64_t)b / (uint64_t)G;
    int lo = 0, hi = n;                           // smallest j with Wp[j + 1] > target
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (Wp[mid + 1] > target) hi = mid; else lo = mid + 1;
    }
    if (lo >= n) return tiles;
    return tf[lo] + (int)((target - Wp[lo]) / w[lo]);
}

// Accumulate+norm geometry.
constexpr int kNormThreads = 256;
constexpr int kNormWarps = kNormThreads / 32;
constexpr int kTileA = 8192;         // elements per CTA (one tile each)

// ---------------------------------------------------------------------------------
// The plan: a position-independent blob built on the host once per step, copied to the
// device as it is.  [PlanHeader][RankInfo x (N + 1)][LayerDesc x (L + N)][LayerDesc x (L + 1)]
// — each rank's layer list is followed by one sentinel entry.  RankInfo[N] and the last list
// describe all N ranks' layers as ONE list in address order, with output offsets that place
// every layer where its own rank's call would put it (for running all workers' selections on
// one device in a single launch); n_my = 0 there if the ranks' layers overlap.
// ---------------------------------------------------------------------------------
constexpr uint32_t kPlanMagic = 0x44454654u;  // "DEFT"

struct PlanHeader {                  // 64 bytes
    uint32_t magic;
    int32_t L, N;
    int32_t total_tiles;
    int64_t total_elems;             // elements over all ranks' layers
    int64_t total_k;                 // entries over all ranks
    int64_t iteration;
    int64_t reserved[3];
};
static_assert(sizeof(PlanHeader) == 64, "PlanHeader layout");

struct RankInfo {                    // 64 bytes
    int32_t desc_first;              // index of the rank's first LayerDesc
    int32_t n_my;                    // layers of the rank
    int32_t tiles;                   // tiles (= chunks) of the rank
    int32_t tile_base;               // first chunk of the rank in the chunk arrays
    int64_t elems;                   // elements the rank scans
    int64_t k;                       // entries the rank selects
    int64_t out_off;                 // sum of k over lower ranks
    int64_t elem_base;               // first staging entry of the rank
    int64_t reserved[2];
};
static_assert(sizeof(RankInfo) == 64, "RankInfo layout");

struct LayerDesc {                   // 64 bytes
    int64_t start, end;              // element range in the flat vector
    int64_t k;                       // entries to select (1..size)
    int64_t out_off;                 // position of the layer's first output entry within the rank
    int64_t elem_off;                // absolute staging index of the layer's first slot
    int32_t tile_first;              // rank-local id of the layer's first tile
    int32_t layer_id;                // id in the model's layer table (state / histogram index)
    double norm;                     // this step's L2 norm of the layer, or 0 if the plan was built without norms
    int64_t reserved;
};
static_assert(sizeof(LayerDesc) == 64, "LayerDesc layout");

inline size_t plan_bytes(int64_t L, int64_t N) {
    return sizeof(PlanHeader) + sizeof(RankInfo) * (size_t)(N + 1) + sizeof(LayerDesc) * (size_t)(L + N) +
           sizeof(LayerDesc) * (size_t)(L + 1);
}
inline const RankInfo* plan_ranks(const void* plan) {
    return reinterpret_cast<const RankInfo*>(static_cast<const char*>(plan) + sizeof(PlanHeader));
}
inline const LayerDesc* plan_descs(const void* plan, int64_t N) {
    return reinterpret_cast<const LayerDesc*>(static_cast<const char*>(plan) + sizeof(PlanHeader) +
                                              sizeof(RankInfo) * (size_t)(N + 1));
}

struct LayerState {                  // per layer, written by the kernels; 64 bytes
    uint32_t b1, above1;             // level-1 bucket of the k-th key; keys strictly above that bucket
    uint32_t b2, krem2;              // level 2 (inside b1): bucket, and how many still to take inside it
    uint32_t T, need;                // exact threshold key; entries equal to T to take (lowest indices)
    uint32_t ticket1;                // tiles whose first read is complete
    uint32_t cursor;                 // single-pass kernel: room handed out in the layer's staging region
    unsigned long long done;         // single-pass kernel: what the CTAs that are through with the layer add up to:
                                     // tiles << 41 | CTAs that stopped staging << 31 | entries staged
    uint32_t pad[5];                 // of a rank's first layer: [0] next small layer to hand out, [1] next layer to finish (single-pass kernel)
    uint32_t spec_bad;               // five steps: a CTA stopped staging for the layer (its speculative cut counts as failed)
};
static_assert(sizeof(LayerState) == 64, "LayerState layout");

// What a selection leaves behind per layer for the next call on the same workspace (the only
// per-layer data that lives across calls; it steers speed, never results).
struct LayerHint {                   // 32 bytes
    uint32_t pos_p1;                 // 1 + position (key >> 15: 1/16 first-level bucket) of the `rank`-th largest key; 0 = nothing remembered
    uint32_t norm_bits;              // that call's layer norm (float bits)
    uint32_t rank;                   // the rank the bucket belongs to (k + margin of that call)
    uint32_t err;                    // how the predictions have been doing, in the same unit: running mean of (found -
                                     // predicted) as int16 in the low half, running mean deviation in the high half
    uint32_t err_same;               // the same two numbers for the prediction "where it was last time" (no norm, no rank
                                     // known yet): what staging during the accumulate pass goes by
    uint32_t pad[3];
};
static_assert(sizeof(LayerHint) == 32, "LayerHint layout");

// Staging during the accumulate pass (before the step's plan exists): where a layer's staged entries and
// its tiles' table entries go follows from the layer table alone: the layout the plan gives the list of
// all layers in address order.  Written by a small kernel before the accumulate pass.
struct StageTab {                    // per layer, 16 bytes
    uint32_t cut;                    // entries with key >= cut are staged (0xffffffff: none for this layer)
    int32_t tile_first;              // the layer's first tile in the all-layers list
    int64_t elem_off;                // first slot of the layer's staging region
};
static_assert(sizeof(StageTab) == 16, "StageTab layout");

// Layers the single-pass kernel could not finish (no usable cut, cut too high, too dense) are
// appended here for a following launch of the five-step kernel on exactly those layers.
struct RetryHeader {                 // 64 bytes, cleared at plan upload
    unsigned long long packed;       // layers appended << 32 | their tiles; cleared again by the steps that work the list off
    uint32_t pad[14];
};
static_assert(sizeof(RetryHeader) == 64, "RetryHeader layout");

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Carve-up of the caller's workspace.  Offsets depend only on (elems, L, tiles).
struct WsLayout {
    size_t plan;                     // scratch device plan for the one-shot calls
    size_t zero_begin, zero_end;     // [retry header | state | hist1 | hist2 | hist3]: cleared at plan upload
    size_t retry, state, hist1, hist2, hist3;
    size_t retry_desc;               // (L + 1) layer descriptors of the retry list
    size_t norm_partial;             // partial sums of the accumulate + norm call (its place depends on L only)
    size_t runge, staging;
    size_t hint;                     // 256 bytes of control words, then one LayerHint per layer; kept across calls
    size_t stage_tab;                // one StageTab per layer (+ 1): rewritten by every step that stages during the accumulate pass
    size_t total;
};

inline WsLayout ws_layout(int64_t elems, int64_t L, int64_t tiles) {
    WsLayout w{};
    size_t off = 0;
    w.plan = off;     off += align_up(plan_bytes(L, 1), 256);
    w.zero_begin = off;
    w.retry = off;    off += 256;
    w.state = off;    off += align_up(sizeof(LayerState) * (size_t)L, 256);
    w.hist1 = off;    off += sizeof(uint32_t) * (size_t)kBins1 * (size_t)L;
    w.hist2 = off;    off += sizeof(uint32_t) * (size_t)kBins2 * (size_t)L;
    w.hist3 = off;    off += sizeof(uint32_t) * (size_t)kBins3 * (size_t)L;
    w.zero_end = off;
    w.hint = off;     off += 256 + align_up(sizeof(LayerHint) * (size_t)L, 256);   // control words, then one entry per layer
    w.retry_desc = off; off += align_up(sizeof(LayerDesc) * (size_t)(L + 1), 256);
    w.stage_tab = off; off += align_up(sizeof(StageTab) * (size_t)(L + 1), 256);
    w.norm_partial = off; off += align_up(sizeof(double) * (size_t)((elems + kTileA - 1) / kTileA + L + 1), 256);
    const size_t slots = 2 * (size_t)tiles + 2 * (size_t)kMaxRanks;   // rank r starts at 2*(tile_base + r)
    w.runge = off;    off += align_up(sizeof(uint2) * slots, 256);
    // + slack: the interleaved split rounds a rank up to whole super-tiles; a retry list places every
    // layer at a multiple of kTile entries (up to two tiles more than its size)
    w.staging = off;  off += align_up(sizeof(uint2) * ((size_t)elems + 4 * (size_t)kSuper * kTile + (2 * (size_t)kTile + kRegionAlign) * (size_t)L), 256);
    w.total = off;
    return w;
}

// Upper bound on the tiles of `layers` layers holding `elems` elements in total.
inline int64_t max_tiles(int64_t elems, int64_t layers) { return elems / kTile + 2 * layers; }

inline size_t norms_ws_bytes(int64_t n_g, int64_t L) {
    return sizeof(double) * (size_t)((n_g + kTileA - 1) / kTileA + L + 1);
}

// Arguments of the fused selection kernel (one rank).
struct SelParams {
    const float* acc;
    float* acc_rw;                   // NULL, or the same vector: selected entries are zeroed on the way out
    const LayerDesc* desc;           // the rank's layers + sentinel (device)
    int32_t n_my, tiles;
    int32_t grid;                    // CTAs of the launch (one per SM at most)
    int32_t interleave;              // 1: super-tiles dealt out round-robin (one large layer); 0: contiguous runs
    int32_t weighted;                // 1: contiguous runs of equal estimated cost from the second read on
    LayerState* state;               // [L]
    uint32_t* hist1;                 // [L][kBins1]
    uint32_t* hist2;                 // [L][kBins2]
    uint32_t* hist3;                 // [L][kBins3]
    uint32_t* spec_ctl;              // control words: five steps: [1] CTAs that had to read twice in this call, [2] CTAs
                                     // that have finished this call, [3] layers whose speculative cut failed in this
                                     // call, [7] calls in which some cut failed (running total); single-pass kernel,
                                     // running totals: [4] layers it finished, [5] layers whose cut failed, [6]
                                     // layers it had no usable cut for, [8] waits on its ring that gave up, [9] staged
                                     // entries of the layers it finished (modulo 2^32)
    LayerHint* hint;                 // [L] what the previous call found; read and updated
    uint2* runge;                    // five-step kernel: this rank's (CTA, layer) pairs (slot = CTA + layer position):
                                     // totals.  Single-pass kernel: per tile of the rank (first entry within the layer's
                                     // staging region, entries)
    RetryHeader* retry;              // layers left for a following launch, see RetryHeader
    LayerDesc* retry_desc;           // [L + 1]
    int32_t from_retry;              // five steps: 1 = the layer list is the retry list (no speculation, no small layers)
    int32_t prestaged;               // single-pass kernel: 1 = the accumulate pass has staged already (cuts in stage_tab): no read
    const StageTab* stage_tab;       // [L] by layer id
    int64_t retry_elem_base;         // staging index at which the retry list's layers are placed
    uint2* staging;                  // absolute base of the spill area; (value bits, offset in tile)
    float* val;                      // the rank's output
    int64_t* idx;
    // hard-threshold mode (one layer, no search): every entry whose key exceeds thr_key is selected
    int32_t fixed_thr;               // 1: hard-threshold mode
    uint32_t thr_key;                // magnitude key of the threshold
    int64_t out_cap;                 // entries val / idx can take (positions beyond it are not written)
    int64_t out_total;               // entries the call writes when nothing is cut off: the sum of its layers' k
    unsigned long long* count_out;   // hard-threshold mode: number of entries above the threshold (zeroed before launch)
    unsigned long long* timing;      // optional: 1024 words of phase stamps and per-CTA counters; NULL = off
};

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
// stage != NULL: the pass also stages every entry at or above its layer's remembered cut (see deft_norms.cu)
struct StageLaunch {
    const LayerHint* hint;           // [L] what the previous selection left behind
    StageTab* tab;                   // [L + 1] written by the call
    LayerState* state;               // [L] cleared before the call
    uint2* runge;                    // tile table of the all-layers list
    uint2* staging;
};
deft_status launch_layer_norms(float* resid_acc_d, const float* grad_d, int64_t n_g,
                               const int64_t* layer_start_d, int32_t L, double* norms_d,
                               double* partial_d, cudaStream_t stream, double* norms_host_mapped = nullptr,
                               const StageLaunch* stage = nullptr);
deft_status launch_select(const SelParams& p, cudaStream_t stream);
deft_status launch_select_stream(const SelParams& p, bool has_streamed, bool ring, cudaStream_t stream);
deft_status launch_residual_update(float* acc_d, const int64_t* idx_d, int64_t count,
                                   cudaStream_t stream);
deft_status launch_gather_update(float* acc_d, const int64_t* idx_d, int64_t count, float* val_d,
                                 cudaStream_t stream);

// Algorithm 1's pieces around the sparsifier (deft_algo1.cu).
size_t union_ws_bytes(int64_t n);
deft_status launch_index_union(const int64_t* idx_d, int64_t count, int64_t n, int64_t* out_d, int64_t out_cap,
                               long long* count_out_d, void* ws_d, cudaStream_t stream);
deft_status launch_sum_into(float* dst_d, const float* src_d, int64_t count, cudaStream_t stream);
deft_status launch_divide(float* x_d, int64_t count, float by, cudaStream_t stream);
deft_status launch_fill_start(int64_t* ls_d, int64_t n, cudaStream_t stream);

}  // namespace deft
