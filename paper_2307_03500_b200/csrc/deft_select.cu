// Layer-wise top-k selection for one worker (Algorithm 5) as a segmented radix select
// over magnitude bit patterns followed by an ordered compaction.
//
// The vector is read twice:
//   pass 1 (k_hist1)  per-layer histogram of key bits 30..20
//   pass 2 (k_filter) every entry whose level-1 bucket is >= the bucket b1 holding the
//                     k-th largest key is copied, in index order, to a staging stream
//                     (one chunk per tile); the level-2 histogram of bucket b1 is built
//                     on the way
// Everything after that touches only the staging stream (about k entries plus the
// candidates of bucket b1): the level-3 histogram, the exact threshold key T with the
// number of entries equal to T still needed, per-chunk counts, their per-layer exclusive
// scans, and the final ordered write of (value, int64 index).
//
// Determinism: histograms use integer atomics (order-free), every output position is a
// function of counts only, ties at T are taken in index order.
#include "deft_common.cuh"

namespace deft {
namespace {

__device__ __forceinline__ uint32_t key_of(uint32_t bits) { return bits & 0x7fffffffu; }

// Largest j in [0, n_my-1] with desc[j].tile_first <= q.
__device__ __forceinline__ int layer_of_tile(const LayerDesc* __restrict__ desc, int n_my, int q) {
    int lo = 0, hi = n_my - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (desc[mid].tile_first <= q) lo = mid; else hi = mid - 1;
    }
    return lo;
}

struct TileSpan {
    int64_t lo;   // first element of the address-aligned tile
    int s, e;     // valid offsets [s, e) inside the tile (the part that belongs to the layer)
};

__device__ __forceinline__ TileSpan tile_span(const LayerDesc& d, int q) {
    const int64_t t = d.start / kTile + (q - d.tile_first);
    TileSpan r;
    r.lo = t * kTile;
    const int64_t s = d.start > r.lo ? d.start : r.lo;
    const int64_t e = d.end < r.lo + kTile ? d.end : r.lo + kTile;
    r.s = (int)(s - r.lo);
    r.e = (int)(e - r.lo);
    return r;
}

// Thread <-> element mapping inside a tile: warp w owns 512 consecutive elements; in slab i
// lane `lane` holds the 4 elements starting at offset w*512 + (i*32 + lane)*4.  Index order
// is therefore (warp, slab, lane, component).
__device__ __forceinline__ int tile_offset(int w, int i, int lane) { return w * 512 + (i * 32 + lane) * 4; }

// Loads the tile's 16 values of this thread as raw bits; `valid` gets one bit per value.
__device__ __forceinline__ void load_tile(const float* __restrict__ acc, const TileSpan& ts,
                                          uint32_t (&bits)[kSlabs][4], uint32_t& valid) {
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (ts.s == 0 && ts.e == kTile) {
        const uint4* p = reinterpret_cast<const uint4*>(acc + ts.lo);
#pragma unroll
        for (int i = 0; i < kSlabs; ++i) {
            const uint4 v = __ldg(p + (tile_offset(w, i, lane) >> 2));
            bits[i][0] = v.x; bits[i][1] = v.y; bits[i][2] = v.z; bits[i][3] = v.w;
        }
        valid = 0xffffu;
    } else {
        valid = 0;
        const uint32_t* p = reinterpret_cast<const uint32_t*>(acc + ts.lo);
#pragma unroll
        for (int i = 0; i < kSlabs; ++i) {
            const int o = tile_offset(w, i, lane);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const bool in = (o + c >= ts.s) && (o + c < ts.e);
                bits[i][c] = in ? __ldg(p + o + c) : 0u;
                valid |= (in ? 1u : 0u) << (i * 4 + c);
            }
        }
    }
}

__device__ __forceinline__ void flush_hist(uint32_t* sh, uint32_t* __restrict__ g, int bins) {
    for (int i = threadIdx.x; i < bins; i += kThreads) {
        const uint32_t c = sh[i];
        if (c) {
            atomicAdd(g + i, c);
            sh[i] = 0;
        }
    }
}

// ---------------------------------------------------------------------------------
// pass 1: level-1 histograms.  Each CTA owns a contiguous run of tiles, keeps the
// histogram of the current layer in shared memory and flushes it when the layer changes.
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
k_hist1(const float* __restrict__ acc, const LayerDesc* __restrict__ desc, int n_my, int tiles,
        uint32_t* __restrict__ hist1) {
    __shared__ uint32_t sh[kBins1];
    const int q0 = (int)((int64_t)tiles * blockIdx.x / gridDim.x);
    const int q1 = (int)((int64_t)tiles * (blockIdx.x + 1) / gridDim.x);
    if (q0 >= q1) return;
    for (int i = threadIdx.x; i < kBins1; i += kThreads) sh[i] = 0;
    int j = layer_of_tile(desc, n_my, q0);
    LayerDesc d = desc[j];
    int next_first = desc[j + 1].tile_first;
    __syncthreads();
    for (int q = q0; q < q1; ++q) {
        if (q >= next_first) {
            __syncthreads();
            flush_hist(sh, hist1 + (size_t)j * kBins1, kBins1);
            __syncthreads();
            ++j;
            d = desc[j];
            next_first = desc[j + 1].tile_first;
        }
        const TileSpan ts = tile_span(d, q);
        uint32_t bits[kSlabs][4], valid;
        load_tile(acc, ts, bits, valid);
#pragma unroll
        for (int i = 0; i < kSlabs; ++i)
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (valid & (1u << (i * 4 + c))) atomicAdd(&sh[key_of(bits[i][c]) >> kShift1], 1u);
    }
    __syncthreads();
    flush_hist(sh, hist1 + (size_t)j * kBins1, kBins1);
}

// ---------------------------------------------------------------------------------
// Histogram scans: one CTA per layer walks the bins from the top and finds the bucket
// that holds the k-th largest key, and how many keys lie strictly above that bucket.
// ---------------------------------------------------------------------------------
template <int kLevel>
__global__ void __launch_bounds__(kThreads)
k_scan(const LayerDesc* __restrict__ desc, LayerState* __restrict__ state,
       const uint32_t* __restrict__ hist) {
    constexpr int kBins = (kLevel == 3) ? kBins3 : kBins1;
    constexpr int kPer = kBins / kThreads;
    __shared__ uint32_t warp_tot[kWarps];
    const int j = blockIdx.x;
    LayerState st = state[j];
    const uint32_t k = (kLevel == 1) ? (uint32_t)desc[j].k : (kLevel == 2) ? st.krem1 : st.krem2;
    const uint32_t* h = hist + (size_t)j * kBins;
    // thread t owns bins [kBins - kPer*(t+1), kBins - kPer*t): thread order = descending bins
    const int base = kBins - kPer * (threadIdx.x + 1);
    uint32_t c[kPer], sum = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) { c[i] = h[base + i]; sum += c[i]; }
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) warp_tot[w] = incl;
    __syncthreads();
    uint32_t before = 0;
    for (int i = 0; i < w; ++i) before += warp_tot[i];
    const uint32_t excl = before + incl - sum;   // keys in bins above this thread's bins
    if (excl < k && k <= excl + sum) {
        uint32_t run = excl;
        int bucket = base;
#pragma unroll
        for (int i = kPer - 1; i >= 0; --i) {
            if (run + c[i] >= k) { bucket = base + i; break; }
            run += c[i];
        }
        if (kLevel == 1) { st.b1 = bucket; st.krem1 = k - run; }
        if (kLevel == 2) { st.b2 = bucket; st.krem2 = k - run; }
        if (kLevel == 3) {
            st.T = (st.b1 << kShift1) | (st.b2 << kShift2) | (uint32_t)bucket;
            st.need = k - run;
        }
        state[j] = st;
    }
}

// ---------------------------------------------------------------------------------
// pass 2: staging.  Entries with key >= (b1 << 20) are written in index order to the
// tile's chunk of the staging stream; entries inside bucket b1 also feed the level-2
// histogram.
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
k_filter(const float* __restrict__ acc, const LayerDesc* __restrict__ desc, int n_my, int tiles,
         const LayerState* __restrict__ state, uint32_t* __restrict__ hist2,
         uint32_t* __restrict__ cnt, uint2* __restrict__ staging) {
    __shared__ uint32_t sh[kBins2];
    __shared__ uint32_t warp_tot[kWarps];
    const int q0 = (int)((int64_t)tiles * blockIdx.x / gridDim.x);
    const int q1 = (int)((int64_t)tiles * (blockIdx.x + 1) / gridDim.x);
    if (q0 >= q1) return;
    for (int i = threadIdx.x; i < kBins2; i += kThreads) sh[i] = 0;
    int j = layer_of_tile(desc, n_my, q0);
    LayerDesc d = desc[j];
    int next_first = desc[j + 1].tile_first;
    uint32_t b1 = state[j].b1;
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    for (int q = q0; q < q1; ++q) {
        if (q >= next_first) {
            __syncthreads();
            flush_hist(sh, hist2 + (size_t)j * kBins2, kBins2);
            __syncthreads();
            ++j;
            d = desc[j];
            next_first = desc[j + 1].tile_first;
            b1 = state[j].b1;
        }
        const TileSpan ts = tile_span(d, q);
        uint32_t bits[kSlabs][4], valid;
        load_tile(acc, ts, bits, valid);
        uint32_t keep = 0;     // one bit per value: goes to staging
        uint32_t packed = 0;   // per-slab counts, 8 bits each (a warp holds at most 128 per slab)
#pragma unroll
        for (int i = 0; i < kSlabs; ++i) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t key = key_of(bits[i][c]);
                const uint32_t bucket = key >> kShift1;
                const bool v = (valid >> (i * 4 + c)) & 1u;
                if (v && bucket >= b1) {
                    keep |= 1u << (i * 4 + c);
                    packed += 1u << (8 * i);
                    if (bucket == b1) atomicAdd(&sh[(key >> kShift2) & (kBins2 - 1)], 1u);
                }
            }
        }
        // ordered positions: (warp, slab, lane, component)
        uint32_t incl = packed;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const uint32_t tot = __shfl_sync(0xffffffffu, incl, 31);
        const uint32_t excl = incl - packed;
        const uint32_t t0 = tot & 0xff, t1 = (tot >> 8) & 0xff, t2 = (tot >> 16) & 0xff, t3 = tot >> 24;
        if (lane == 0) warp_tot[w] = t0 + t1 + t2 + t3;
        __syncthreads();
        uint32_t warp_base = 0, tile_total = 0;
#pragma unroll
        for (int i = 0; i < kWarps; ++i) {
            const uint32_t v = warp_tot[i];
            if (i < w) warp_base += v;
            tile_total += v;
        }
        if (tile_total) {
            const int64_t chunk = d.elem_off + (ts.lo + ts.s - d.start);
            const uint32_t slab_base[kSlabs] = {0u, t0, t0 + t1, t0 + t1 + t2};
#pragma unroll
            for (int i = 0; i < kSlabs; ++i) {
                uint32_t pos = warp_base + slab_base[i] + ((excl >> (8 * i)) & 0xff);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if (keep & (1u << (i * 4 + c))) {
                        staging[chunk + pos] = make_uint2(bits[i][c], (uint32_t)(tile_offset(w, i, lane) + c));
                        ++pos;
                    }
                }
            }
        }
        if (threadIdx.x == 0) cnt[q] = tile_total;
        __syncthreads();   // warp_tot is reused by the next tile
    }
    __syncthreads();
    flush_hist(sh, hist2 + (size_t)j * kBins2, kBins2);
}

// ---------------------------------------------------------------------------------
// Staging passes: one warp per chunk.
// ---------------------------------------------------------------------------------
struct ChunkRef {
    int j;
    int64_t base;   // first staging entry of the chunk
    int64_t lo;     // first element of the tile
};

__device__ __forceinline__ ChunkRef chunk_ref(const LayerDesc* __restrict__ desc, int n_my, int q) {
    ChunkRef r;
    r.j = layer_of_tile(desc, n_my, q);
    const LayerDesc d = desc[r.j];
    const TileSpan ts = tile_span(d, q);
    r.base = d.elem_off + (ts.lo + ts.s - d.start);
    r.lo = ts.lo;
    return r;
}

// level-3 histogram of the entries whose top 22 key bits equal (b1, b2)
__global__ void __launch_bounds__(kThreads)
k_hist3(const LayerDesc* __restrict__ desc, int n_my, int tiles, const LayerState* __restrict__ state,
        const uint32_t* __restrict__ cnt, const uint2* __restrict__ staging,
        uint32_t* __restrict__ hist3) {
    const int lane = threadIdx.x & 31;
    const int gw = blockIdx.x * kWarps + (threadIdx.x >> 5);
    for (int q = gw; q < tiles; q += gridDim.x * kWarps) {
        const uint32_t n = cnt[q];
        if (n == 0) continue;
        const ChunkRef cr = chunk_ref(desc, n_my, q);
        const LayerState st = state[cr.j];
        const uint32_t prefix = (st.b1 << (kShift1 - kShift2)) | st.b2;
        for (uint32_t e0 = 0; e0 < n; e0 += 32) {
            const uint32_t e = e0 + lane;
            uint32_t key = 0;
            bool is = false;
            if (e < n) {
                key = key_of(staging[cr.base + e].x);
                is = (key >> kShift2) == prefix;
            }
            const unsigned act = __ballot_sync(0xffffffffu, is);
            if (is) {
                const uint32_t bin = key & (kBins3 - 1);
                const unsigned peers = __match_any_sync(act, bin);
                if (lane == __ffs(peers) - 1)
                    atomicAdd(hist3 + (size_t)cr.j * kBins3 + bin, (uint32_t)__popc(peers));
            }
        }
    }
}

// per chunk: how many entries lie above T, how many equal T
__global__ void __launch_bounds__(kThreads)
k_count(const LayerDesc* __restrict__ desc, int n_my, int tiles, const LayerState* __restrict__ state,
        const uint32_t* __restrict__ cnt, const uint2* __restrict__ staging, uint2* __restrict__ ge) {
    const int lane = threadIdx.x & 31;
    const int gw = blockIdx.x * kWarps + (threadIdx.x >> 5);
    for (int q = gw; q < tiles; q += gridDim.x * kWarps) {
        const uint32_t n = cnt[q];
        uint32_t n_gt = 0, n_eq = 0;
        if (n) {
            const ChunkRef cr = chunk_ref(desc, n_my, q);
            const uint32_t T = state[cr.j].T;
            for (uint32_t e0 = 0; e0 < n; e0 += 32) {
                const uint32_t e = e0 + lane;
                bool gt = false, eq = false;
                if (e < n) {
                    const uint32_t key = key_of(staging[cr.base + e].x);
                    gt = key > T;
                    eq = key == T;
                }
                n_gt += __popc(__ballot_sync(0xffffffffu, gt));
                n_eq += __popc(__ballot_sync(0xffffffffu, eq));
            }
        }
        if (lane == 0) ge[q] = make_uint2(n_gt, n_eq);
    }
}

// per layer: exclusive scan of the chunk counts (one CTA per layer, 16 chunks per thread per round)
__global__ void __launch_bounds__(kThreads)
k_chunk_scan(const LayerDesc* __restrict__ desc, uint2* __restrict__ ge) {
    constexpr int kPer = 16;
    __shared__ uint2 warp_tot[kWarps];
    const int j = blockIdx.x;
    const int q0 = desc[j].tile_first, q1 = desc[j + 1].tile_first;
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t carry_gt = 0, carry_eq = 0;
    for (int r0 = q0; r0 < q1; r0 += kThreads * kPer) {
        const int first = r0 + threadIdx.x * kPer;
        uint2 v[kPer];
        uint32_t s_gt = 0, s_eq = 0;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            v[i] = (first + i < q1) ? ge[first + i] : make_uint2(0u, 0u);
            s_gt += v[i].x;
            s_eq += v[i].y;
        }
        uint32_t i_gt = s_gt, i_eq = s_eq;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t a = __shfl_up_sync(0xffffffffu, i_gt, o);
            const uint32_t b = __shfl_up_sync(0xffffffffu, i_eq, o);
            if (lane >= o) { i_gt += a; i_eq += b; }
        }
        __syncthreads();   // warp_tot from the previous round has been read
        if (lane == 31) warp_tot[w] = make_uint2(i_gt, i_eq);
        __syncthreads();
        uint32_t b_gt = carry_gt, b_eq = carry_eq, all_gt = 0, all_eq = 0;
#pragma unroll
        for (int i = 0; i < kWarps; ++i) {
            const uint2 t = warp_tot[i];
            if (i < w) { b_gt += t.x; b_eq += t.y; }
            all_gt += t.x;
            all_eq += t.y;
        }
        uint32_t run_gt = b_gt + i_gt - s_gt, run_eq = b_eq + i_eq - s_eq;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            if (first + i < q1) ge[first + i] = make_uint2(run_gt, run_eq);
            run_gt += v[i].x;
            run_eq += v[i].y;
        }
        carry_gt += all_gt;
        carry_eq += all_eq;
    }
}

// final ordered write of (value, index)
__global__ void __launch_bounds__(kThreads)
k_emit(const LayerDesc* __restrict__ desc, int n_my, int tiles, const LayerState* __restrict__ state,
       const uint32_t* __restrict__ cnt, const uint2* __restrict__ staging,
       const uint2* __restrict__ ge, float* __restrict__ val, int64_t* __restrict__ idx) {
    const int lane = threadIdx.x & 31;
    const uint32_t lt = (1u << lane) - 1u;
    const int gw = blockIdx.x * kWarps + (threadIdx.x >> 5);
    for (int q = gw; q < tiles; q += gridDim.x * kWarps) {
        const uint32_t n = cnt[q];
        if (n == 0) continue;
        const ChunkRef cr = chunk_ref(desc, n_my, q);
        const LayerState st = state[cr.j];
        const uint2 before = ge[q];
        uint32_t eq_run = before.y;
        int64_t out = desc[cr.j].out_off + before.x + (before.y < st.need ? before.y : st.need);
        for (uint32_t e0 = 0; e0 < n; e0 += 32) {
            const uint32_t e = e0 + lane;
            uint2 ent = make_uint2(0u, 0u);
            bool gt = false, eq = false;
            if (e < n) {
                ent = staging[cr.base + e];
                const uint32_t key = key_of(ent.x);
                gt = key > st.T;
                eq = key == st.T;
            }
            const unsigned eq_b = __ballot_sync(0xffffffffu, eq);
            const bool sel = gt || (eq && (eq_run + __popc(eq_b & lt) < st.need));
            const unsigned sel_b = __ballot_sync(0xffffffffu, sel);
            if (sel) {
                const int64_t pos = out + __popc(sel_b & lt);
                val[pos] = __uint_as_float(ent.x);
                idx[pos] = cr.lo + (int64_t)ent.y;
            }
            out += __popc(sel_b);
            eq_run += __popc(eq_b);
        }
    }
}

__global__ void k_zero_at(float* __restrict__ acc, const int64_t* __restrict__ idx, int64_t count) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count;
         i += (int64_t)gridDim.x * blockDim.x)
        acc[idx[i]] = 0.0f;
}

}  // namespace

deft_status launch_select(const float* acc_d, const SelectWorkspace& w, int32_t n_my, int32_t tiles,
                          float* val_d, int64_t* idx_d, cudaStream_t stream) {
    const int sms = sm_count();
    const int grid_stream = tiles < sms * 8 ? tiles : sms * 8;
    const int chunk_ctas = (tiles + kWarps - 1) / kWarps;
    const int grid_chunks = chunk_ctas < sms * 8 ? chunk_ctas : sms * 8;

    DEFT_CUDA_TRY(cudaMemsetAsync(w.state, 0, w.zero_bytes, stream));
    k_hist1<<<grid_stream, kThreads, 0, stream>>>(acc_d, w.desc, n_my, tiles, w.hist1);
    k_scan<1><<<n_my, kThreads, 0, stream>>>(w.desc, w.state, w.hist1);
    k_filter<<<grid_stream, kThreads, 0, stream>>>(acc_d, w.desc, n_my, tiles, w.state, w.hist2,
                                                   w.cnt, w.staging);
    k_scan<2><<<n_my, kThreads, 0, stream>>>(w.desc, w.state, w.hist2);
    k_hist3<<<grid_chunks, kThreads, 0, stream>>>(w.desc, n_my, tiles, w.state, w.cnt, w.staging,
                                                  w.hist3);
    k_scan<3><<<n_my, kThreads, 0, stream>>>(w.desc, w.state, w.hist3);
    k_count<<<grid_chunks, kThreads, 0, stream>>>(w.desc, n_my, tiles, w.state, w.cnt, w.staging, w.ge);
    k_chunk_scan<<<n_my, kThreads, 0, stream>>>(w.desc, w.ge);
    k_emit<<<grid_chunks, kThreads, 0, stream>>>(w.desc, n_my, tiles, w.state, w.cnt, w.staging, w.ge,
                                                 val_d, idx_d);
    DEFT_CUDA_TRY(cudaGetLastError());
    return DEFT_OK;
}

deft_status launch_residual_update(float* acc_d, const int64_t* idx_d, int64_t count,
                                   cudaStream_t stream) {
    if (count == 0) return DEFT_OK;
    const int64_t want = (count + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 16;
    k_zero_at<<<(int)(want < cap ? want : cap), 256, 0, stream>>>(acc_d, idx_d, count);
    DEFT_CUDA_TRY(cudaGetLastError());
    return DEFT_OK;
}

}  // namespace deft
