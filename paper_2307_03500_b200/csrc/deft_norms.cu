// Error-feedback accumulate fused with segmented per-layer sums of squares
// (Algorithm 1 line 5 + the per-layer gradient norm of Section 4.2).
//
// One streaming pass: 8 B read + 4 B written per element.  The vector is cut into
// address-aligned tiles of kTileA elements; a tile that lies inside one layer takes the
// vectorised path, a tile that crosses layer boundaries is processed piece by piece.
// Every (tile, layer) piece owns the partial-sum slot `tile + layer`, which is unique
// because both numbers only grow along the vector, so no atomics and no zero-fill are
// needed and the result is bit-identical from run to run.
#include "deft_select_dev.cuh"

namespace deft {
namespace {

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the CTA in a fixed order; the result is valid in thread 0.
__device__ __forceinline__ double block_sum(double v, double* sh) {
    v = warp_sum(v);
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();  // sh may still be read from the previous use
    if (lane == 0) sh[w] = v;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 0; i < kNormWarps; ++i) t += sh[i];
    }
    return t;
}

// Largest l in [0, L-1] with layer_start[l] <= pos.
__device__ __forceinline__ int layer_of(const int64_t* __restrict__ ls, int L, int64_t pos) {
    int lo = 0, hi = L - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (__ldg(ls + mid) <= pos) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// ---- staging during the accumulate pass ----
// With kStage the pass also puts every entry at or above its layer's cut (StageTab::cut, from what the
// previous selection left behind) into the layer's staging region and fills the tile table, exactly as the
// read of the single-pass selection kernel would: that kernel then has nothing to read.  A CTA's 8192
// elements are four of the selection's tiles and touch at most two layers that are staged at all (layers
// of up to kDirectElems elements are not), so there are at most eight (layer, tile) lists per CTA.
// Marked entries are appended to their list in shared memory in no particular order (they are few: the
// accumulate arithmetic and its order stay untouched); at the end one warp per list sorts it by offset,
// takes room in the layer's region and writes it out.  A list that overflows marks the layer as flooded
// (the selection then reads it the ordinary way).
constexpr int kStageCap = 256;                       // entries per (layer, tile) list
constexpr int kStageLists = 2 * (kTileA / kTile);    // two layers x four tiles
static_assert(kStageLists == kNormWarps && kTileA % kTile == 0, "one warp per list");

struct StageArgs {
    const StageTab* tab;     // [L]
    LayerState* state;       // [L]
    uint2* runge;            // tile table of the all-layers list
    uint2* staging;
};

struct StageShared {
    uint2 ent[kStageLists][kStageCap];   // (value bits, offset in the selection tile)
    uint32_t cnt[kStageLists];
    int layer[2];                        // the CTA's staged layers (-1: none)
    uint32_t cut[2];
};

__device__ __forceinline__ void stage_append(StageShared* ss, int slot, int64_t lo, int64_t i, uint32_t bits) {
    const int list = slot * (kTileA / kTile) + (int)((i - lo) / kTile);
    const uint32_t pos = atomicAdd(&ss->cnt[list], 1u);
    if (pos < (uint32_t)kStageCap) ss->ent[list][pos] = make_uint2(bits, (uint32_t)(i % kTile));
}

template <bool kHasGrad, bool kStage>
__global__ void __launch_bounds__(kNormThreads, kStage ? 6 : 1)
k_accum_norms(float* __restrict__ e, const float* __restrict__ g, int64_t n,
              const int64_t* __restrict__ ls, int L, double* __restrict__ partial, int64_t tiles, const StageArgs sa) {
    __shared__ double sh[kNormWarps];
    __shared__ __align__(16) unsigned char ss_raw[kStage ? sizeof(StageShared) : 16];
    StageShared* ss = reinterpret_cast<StageShared*>(ss_raw);
    for (int64_t t = blockIdx.x; t < tiles; t += gridDim.x) {
        const int64_t lo = t * kTileA;
        const int64_t hi = (lo + kTileA < n) ? lo + kTileA : n;
        int l = layer_of(ls, L, lo);
        const int l_first = l;
        const bool whole = hi - lo == kTileA && __ldg(ls + l + 1) >= hi;   // the tile lies inside layer l
        if (kStage) {
            __syncthreads();   // the lists of the previous tile have been written out
            if (threadIdx.x < kStageLists) ss->cnt[threadIdx.x] = 0u;
            if (threadIdx.x == 0) {
                // the (at most two) staged layers that overlap [lo, hi); a tile inside one layer needs no search
                int found = 0;
                ss->layer[0] = ss->layer[1] = -1;
                ss->cut[0] = ss->cut[1] = 0xffffffffu;
                if (whole) {
                    if (__ldg(ls + l + 1) - __ldg(ls + l) > kDirectElems) ss->layer[0] = l;   // (its cut: every thread reads it itself)
                } else {
                    for (int ll = l_first; ll < L && __ldg(ls + ll) < hi && found < 2; ++ll) {
                        if (__ldg(ls + ll + 1) - __ldg(ls + ll) > kDirectElems) {
                            ss->layer[found] = ll;
                            ss->cut[found] = sa.tab[ll].cut;
                            ++found;
                        }
                    }
                }
            }
            __syncthreads();
        }
        if (whole) {
            // whole tile inside layer l: 8 float4 per thread, squares in fp32 per 8 elements
            float4* e4 = reinterpret_cast<float4*>(e + lo);
            const float4* g4 = reinterpret_cast<const float4*>(g + lo);
            double acc = 0.0;
            uint32_t cut = 0xffffffffu;
            float cutf = 0.0f;
            if (kStage) {
                cut = (__ldg(ls + l + 1) - __ldg(ls + l) > kDirectElems) ? sa.tab[l].cut : 0xffffffffu;
                if (threadIdx.x == 0) ss->cut[0] = cut;   // for the warps that write the lists out (behind a barrier)
                cutf = __uint_as_float(cut < 0x7f800000u ? cut : 0x7f800000u);
            }
#pragma unroll
            for (int i = 0; i < kTileA / (kNormThreads * 4); i += 2) {
                const int a = i * kNormThreads + threadIdx.x, b = a + kNormThreads;
                float4 x = e4[a], y = e4[b];
                if (kHasGrad) {
                    const float4 gx = __ldg(g4 + a), gy = __ldg(g4 + b);
                    x.x = __fadd_rn(x.x, gx.x); x.y = __fadd_rn(x.y, gx.y);
                    x.z = __fadd_rn(x.z, gx.z); x.w = __fadd_rn(x.w, gx.w);
                    y.x = __fadd_rn(y.x, gy.x); y.y = __fadd_rn(y.y, gy.y);
                    y.z = __fadd_rn(y.z, gy.z); y.w = __fadd_rn(y.w, gy.w);
                    e4[a] = x;
                    e4[b] = y;
                }
                if (kStage && cut != 0xffffffffu) {
                    // one test of the largest magnitude per 16 bytes; the exact test per component where it passes
                    // (written so that a NaN passes)
                    const float mx = amax2(amax2(x.x, x.y), amax2(x.z, x.w));
                    const float my = amax2(amax2(y.x, y.y), amax2(y.z, y.w));
                    if (!(fabsf(mx) < cutf)) {
                        const uint32_t bx[4] = {__float_as_uint(x.x), __float_as_uint(x.y), __float_as_uint(x.z), __float_as_uint(x.w)};
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            if (key_of(bx[c]) >= cut) stage_append(ss, 0, lo, lo + (int64_t)a * 4 + c, bx[c]);
                    }
                    if (!(fabsf(my) < cutf)) {
                        const uint32_t by[4] = {__float_as_uint(y.x), __float_as_uint(y.y), __float_as_uint(y.z), __float_as_uint(y.w)};
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            if (key_of(by[c]) >= cut) stage_append(ss, 0, lo, lo + (int64_t)b * 4 + c, by[c]);
                    }
                }
                float s = x.x * x.x;
                s = fmaf(x.y, x.y, s); s = fmaf(x.z, x.z, s); s = fmaf(x.w, x.w, s);
                s = fmaf(y.x, y.x, s); s = fmaf(y.y, y.y, s); s = fmaf(y.z, y.z, s);
                s = fmaf(y.w, y.w, s);
                acc += (double)s;
            }
            const double tot = block_sum(acc, sh);
            if (threadIdx.x == 0) partial[t + l] = tot;
        } else {
            // tile crosses layer boundaries (or is the ragged tail): one piece per layer
            int64_t ps = lo;
            while (ps < hi) {
                const int64_t lend = __ldg(ls + l + 1);
                const int64_t pe = lend < hi ? lend : hi;
                double acc = 0.0;
                int slot = -1;
                uint32_t cut = 0xffffffffu;
                if (kStage) {
                    slot = ss->layer[0] == l ? 0 : (ss->layer[1] == l ? 1 : -1);
                    if (slot >= 0) cut = ss->cut[slot];
                }
                for (int64_t i = ps + threadIdx.x; i < pe; i += kNormThreads) {
                    float x = e[i];
                    if (kHasGrad) {
                        x = __fadd_rn(x, __ldg(g + i));
                        e[i] = x;
                    }
                    if (kStage && cut != 0xffffffffu && key_of(__float_as_uint(x)) >= cut)
                        stage_append(ss, slot, lo, i, __float_as_uint(x));
                    acc += (double)x * (double)x;
                }
                const double tot = block_sum(acc, sh);
                if (threadIdx.x == 0 && pe > ps) partial[t + l] = tot;
                ps = pe;
                ++l;
            }
        }
        if (kStage) {
            __syncthreads();
            // one warp per (layer, tile) list: sort by offset, take room, write; every tile of a staged layer
            // with a cut gets its table entry, empty or not
            const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
            const int slot = warp / (kTileA / kTile), blk = warp % (kTileA / kTile);
            const int ll = ss->layer[slot];
            const int64_t b0 = lo + (int64_t)blk * kTile, b1 = b0 + kTile;
            if (ll >= 0 && ss->cut[slot] != 0xffffffffu) {
                const int64_t s0 = __ldg(ls + ll), s1 = __ldg(ls + ll + 1);
                if (s0 < b1 && s1 > b0 && b0 < hi) {   // the layer has elements in this tile
                    const StageTab tb = sa.tab[ll];
                    const int64_t tile_in_layer = b0 / kTile - s0 / kTile;
                    const uint32_t n_all = ss->cnt[warp];
                    const uint32_t nn = n_all < (uint32_t)kStageCap ? n_all : (uint32_t)kStageCap;
                    uint32_t first = 0;
                    if (lane == 0) {
                        if (n_all > (uint32_t)kStageCap) atomicOr(&sa.state[ll].spec_bad, 1u);
                        first = nn ? atomicAdd(&sa.state[ll].cursor, nn) : 0u;
                        sa.runge[tb.tile_first + tile_in_layer] = make_uint2(first, nn);
                    }
                    first = __shfl_sync(0xffffffffu, first, 0);
                    uint2* dst = sa.staging + tb.elem_off + first;
                    for (uint32_t i = lane; i < nn; i += 32) {
                        const uint2 me = ss->ent[warp][i];
                        uint32_t before = 0;
                        for (uint32_t j = 0; j < nn; ++j) before += ss->ent[warp][j].y < me.y ? 1u : 0u;
                        dst[before] = make_uint2(me.x, me.y | ((uint32_t)tile_in_layer << 11));
                    }
                }
            }
        }
    }
}

// Before a staging accumulate pass: per layer the cut it stages by and where its entries and table rows go
// (the layout the plan gives the list of all layers in address order).  One CTA.
__global__ void __launch_bounds__(512) k_stage_prepare(const int64_t* __restrict__ ls, int L, const LayerHint* hint, StageTab* tab) {
    __shared__ unsigned long long warp_tot[2][16];
    __shared__ unsigned long long carry[2];
    if (threadIdx.x < 2) carry[threadIdx.x] = 0ull;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int l0 = 0; l0 < L; l0 += 512) {
        const int l = l0 + (int)threadIdx.x;
        unsigned long long tiles = 0, slots = 0;
        int64_t size = 0;
        if (l < L) {
            const int64_t s = ls[l], e = ls[l + 1];
            size = e - s;
            if (size > 0) {
                tiles = (unsigned long long)((e - 1) / kTile - s / kTile + 1);
                slots = (unsigned long long)((size + kRegionAlign - 1) / kRegionAlign * kRegionAlign);
            }
        }
        unsigned long long it = tiles, is = slots;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long a = __shfl_up_sync(0xffffffffu, it, o), b = __shfl_up_sync(0xffffffffu, is, o);
            if (lane >= o) { it += a; is += b; }
        }
        if (lane == 31) { warp_tot[0][warp] = it; warp_tot[1][warp] = is; }
        __syncthreads();
        unsigned long long bt = carry[0], bs = carry[1];
        for (int w = 0; w < warp; ++w) { bt += warp_tot[0][w]; bs += warp_tot[1][w]; }
        if (l < L) {
            StageTab tb;
            tb.cut = size > kDirectElems ? prestage_cut(hint + l, size) : 0xffffffffu;
            tb.tile_first = (int32_t)(bt + it - tiles);
            tb.elem_off = (int64_t)(bs + is - slots);
            tab[l] = tb;
        }
        __syncthreads();
        if (threadIdx.x == 511) { carry[0] = bt + it; carry[1] = bs + is; }
        __syncthreads();
    }
}

// One CTA per layer: add the layer's partial sums in a fixed order, take the root.
__global__ void __launch_bounds__(kNormThreads)
k_norm_finalize(const int64_t* __restrict__ ls, int L, const double* __restrict__ partial,
                double* __restrict__ norms, double* norms_host) {
    __shared__ double sh[kNormWarps];
    const int l = blockIdx.x;
    const int64_t s = ls[l], e = ls[l + 1];
    double acc = 0.0;
    if (e > s) {
        const int64_t t0 = s / kTileA, t1 = (e - 1) / kTileA;
        for (int64_t t = t0 + threadIdx.x; t <= t1; t += kNormThreads) acc += partial[t + l];
    }
    const double tot = block_sum(acc, sh);
    if (threadIdx.x == 0) {
        const double v = sqrt(tot);
        norms[l] = v;
        if (norms_host) {   // mapped host memory a waiting host thread polls: no stream synchronisation needed
            *reinterpret_cast<volatile double*>(norms_host + l) = v;
            __threadfence_system();
        }
    }
}

}  // namespace

deft_status launch_layer_norms(float* resid_acc_d, const float* grad_d, int64_t n_g,
                               const int64_t* layer_start_d, int32_t L, double* norms_d,
                               double* partial_d, cudaStream_t stream, double* norms_host_mapped,
                               const StageLaunch* stage) {
    const int64_t tiles = (n_g + kTileA - 1) / kTileA;
    // one CTA per tile: the hardware scheduler keeps the SMs evenly busy to the end, which a
    // resident grid-stride loop did not (0.645 -> 0.600 ms on 333.6 M elements); the loop in the
    // kernel only matters beyond 2^31 - 1 tiles
    const int64_t max_grid = 0x7fffffff;
    const int grid = (int)(tiles < max_grid ? tiles : max_grid);
    StageArgs sa{};
    if (stage) {
        k_stage_prepare<<<1, 512, 0, stream>>>(layer_start_d, L, stage->hint, stage->tab);
        sa.tab = stage->tab;
        sa.state = stage->state;
        sa.runge = stage->runge;
        sa.staging = stage->staging;
    }
    if (grad_d && stage)
        k_accum_norms<true, true><<<grid, kNormThreads, 0, stream>>>(resid_acc_d, grad_d, n_g, layer_start_d, L, partial_d, tiles, sa);
    else if (grad_d)
        k_accum_norms<true, false><<<grid, kNormThreads, 0, stream>>>(resid_acc_d, grad_d, n_g, layer_start_d, L, partial_d, tiles, sa);
    else if (stage)
        k_accum_norms<false, true><<<grid, kNormThreads, 0, stream>>>(resid_acc_d, nullptr, n_g, layer_start_d, L, partial_d, tiles, sa);
    else
        k_accum_norms<false, false><<<grid, kNormThreads, 0, stream>>>(resid_acc_d, nullptr, n_g, layer_start_d, L, partial_d, tiles, sa);
    DEFT_CUDA_TRY(cudaGetLastError());
    k_norm_finalize<<<L, kNormThreads, 0, stream>>>(layer_start_d, L, partial_d, norms_d, norms_host_mapped);
    DEFT_CUDA_TRY(cudaGetLastError());
    return DEFT_OK;
}

}  // namespace deft
