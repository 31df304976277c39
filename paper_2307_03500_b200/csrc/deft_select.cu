// Layer-wise top-k selection for one worker (Algorithm 5) as ONE persistent cooperative
// kernel: a segmented radix select over magnitude bit patterns followed by an ordered
// compaction.  One CTA of 512 threads per SM; phases are separated by grid barriers.
// Every CTA owns a contiguous run of the rank's tiles in all phases.
//
//   phase A  read 1: per-layer histogram of key bits 30..19 (shared-memory histograms,
//            flushed with integer atomics).  Layers of at most kDirectElems elements take
//            no part in phases A and B: phase C loads each of them whole.
//   phase B  read 2: every warp finds, for the layers it is about to stream, the bucket b1
//            that holds the k-th largest key, then copies every entry with bucket >= b1 to
//            the staging stream.  The entries a CTA stages for one layer form one contiguous
//            run in index order (warps buffer their tile's entries in shared memory, an
//            intra-CTA scan of the counts gives each warp its place).
//   phase C  per layer, one CTA: pulls the layer's runs (about k entries plus the candidates
//            of bucket b1) into shared memory, finishes the radix select there (bits 18..9,
//            bits 8..0, ties by lowest index) and writes (value, int64 index) in ascending
//            index with coalesced stores.
// A layer whose staged entries do not fit in shared memory (huge k, or massive ties) is
// flagged "big" in phase B and finished by the general path instead: level-2/level-3
// histograms in global memory, per-run counts, a per-layer scan of the counts and a
// run-parallel ordered write, with a grid barrier between the steps.
//
// Determinism: histograms use integer atomics (order-free), every output position is a
// function of counts only, ties at the threshold are taken in index order.
#include <cooperative_groups.h>

#include "deft_common.cuh"

namespace cg = cooperative_groups;

namespace deft {
namespace {

constexpr int kDirectElems = 16384;   // layers up to this size skip the streaming phases: one CTA loads them whole
constexpr int kBufCap = 256;       // per-warp staging buffer (entries) in phase B
constexpr int kMaxRuns = 256;      // >= CTAs in the grid

// shared-memory carve-up (bytes)
constexpr int kSmMain = 0;   // A: kSlots level-1 histograms | B: warp buffers + level-2 slots | C: entries
constexpr int kSmMainA = kSlots * kBins1 * 4;
constexpr int kSmMainB = kSelWarps * kBufCap * 8 + kSlots * kBins2 * 4;
constexpr int kSmMainC = 2 * kSmallEntries * 4;
constexpr int kSmMainBytes = kSmMainA > kSmMainC ? (kSmMainA > kSmMainB ? kSmMainA : kSmMainB)
                                                 : (kSmMainC > kSmMainB ? kSmMainC : kSmMainB);
constexpr int kSmH1 = kSmMain + kSmMainBytes;              // one level-1 histogram (direct layers)
constexpr int kSmH1Bytes = kBins1 * 4;
constexpr int kSmH = kSmH1 + kSmH1Bytes;                   // one level-2 / level-3 histogram
constexpr int kSmHBytes = kBins2 * 4;
constexpr int kSmMisc = kSmH + kSmHBytes;                  // small tables, see MiscOff
constexpr int kSmMiscBytes = 8192;
constexpr int kSmemBytes = kSmMisc + kSmMiscBytes;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
static_assert(kBins2 >= kBins3, "the level-3 histogram reuses the level-2 buffer");
static_assert(kDirectElems <= kSmallEntries, "a direct layer must fit the phase C buffers");

enum MiscOff : int {   // word offsets inside the misc area
    kMScratch = 0,     // 64: block scan scratch
    kMOut3 = 64,       // 4: result of block_scan_select
    kMTab = 72,        // 2*kSlots: (b1, kind) per slot of the current group
    kMRunTotal = 96,   // kSlots: entries staged so far per slot
    kMCnt = 112,       // 2*32: per-warp counts of a round (double buffered)
    kMLay = 176,       // 2*32: per-warp slot of a round
    kMWarpCnt = 240,   // 32: per-warp packed counts in phase C
    kMRoff = 288,      // kMaxRuns + 1: run offsets of one layer
    kMBsum = 560,      // kSlots * 32: block sums of the group's level-1 histograms
    kMRrel = 832,      // kMaxRuns: element offset (relative to the layer) entry offsets of a run count from
    kMRbase = 1088,    // 2 * kMaxRuns: first staging entry of a run (int64)
};
static_assert(kMRbase + 2 * kMaxRuns <= kSmMiscBytes / 4, "misc area");
static_assert(kMBsum + kSlots * 32 <= kSmMiscBytes / 4, "misc area");
static_assert((kSlots * 32) % kSelWarps == 0 && kSelWarps >= kSlots, "prologue work split");
static_assert(kMRoff + kMaxRuns + 1 <= kSmMiscBytes / 4, "misc area");

enum LayerKind : uint32_t { kKindSmall = 0, kKindBig = 1, kKindDirect = 2 };

__device__ __forceinline__ uint32_t key_of(uint32_t bits) { return bits & 0x7fffffffu; }

__device__ __forceinline__ void stamp(const SelParams& p, int slot) {
    if (p.timing && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        atomicMax(p.timing + slot, t);
    }
}

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
    int s, e;     // offsets [s, e) inside the tile that belong to the layer
};

__device__ __forceinline__ TileSpan tile_span(int64_t start, int64_t end, int tile_first, int q) {
    const int64_t t = start / kTile + (q - tile_first);
    TileSpan r;
    r.lo = t * kTile;
    const int64_t s = start > r.lo ? start : r.lo;
    const int64_t e = end < r.lo + kTile ? end : r.lo + kTile;
    r.s = (int)(s - r.lo);
    r.e = (int)(e - r.lo);
    return r;
}

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t x = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += x;
    }
    return v;
}

// Sum over lanes >= mine (lane 31 is the top).
__device__ __forceinline__ uint32_t warp_suffix_sum(uint32_t v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t x = __shfl_down_sync(0xffffffffu, v, o);
        if (lane + o < 32) v += x;
    }
    return v;
}

// Exclusive prefix of v over the CTA in thread order; `total` = sum over the CTA.
// scratch: 33 words of shared memory.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* scratch, uint32_t& total) {
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t incl = warp_incl_scan(v, lane);
    __syncthreads();   // scratch may still be in use
    if (lane == 31) scratch[w] = incl;
    __syncthreads();
    if (w == 0) {
        const uint32_t x = lane < kSelWarps ? scratch[lane] : 0u;
        const uint32_t xi = warp_incl_scan(x, lane);
        scratch[lane] = xi - x;
        if (lane == 31) scratch[32] = xi;
    }
    __syncthreads();
    total = scratch[32];
    return scratch[w] + incl - v;
}

// CTA-wide: walks a histogram (at most 8 * kSelThreads bins) from its top bin down and finds
// the bucket that holds the k-th largest key.  out[0] = bucket, out[1] = keys strictly above it.
template <bool kGlobal>
__device__ __forceinline__ void block_scan_select(const uint32_t* h, int nbins, uint32_t k,
                                                  uint32_t* scratch, uint32_t* out) {
    const int per = (nbins + kSelThreads - 1) / kSelThreads;
    const int base = nbins - per * ((int)threadIdx.x + 1);   // thread order = descending bins
    uint32_t c[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
    uint32_t sum = 0;
    for (int i = 0; i < per; ++i)
        if (base + i >= 0) { c[i] = kGlobal ? __ldcg(h + base + i) : h[base + i]; sum += c[i]; }
    if (threadIdx.x == 0) { out[0] = 0; out[1] = 0; }
    uint32_t total;
    const uint32_t excl = block_excl_scan(sum, scratch, total);   // keys in bins above mine
    if (sum != 0 && excl < k && k <= excl + sum) {
        uint32_t run = excl;
        for (int i = per - 1; i >= 0; --i) {
            if (run + c[i] >= k) { out[0] = (uint32_t)(base + i); out[1] = run; break; }
            run += c[i];
        }
    }
    __syncthreads();
}
static_assert(kBins1 <= 8 * kSelThreads, "at most 8 bins per thread");

// The same search on a level-1 histogram (kBins1 bins) in global memory, in two steps.
// Step 1 (any warp, any order): the sum of one 128-bin block, read with one coalesced request.
__device__ __forceinline__ uint32_t hist1_block_sum(const uint32_t* __restrict__ h, int block, int lane) {
    const uint4 v = __ldcg(reinterpret_cast<const uint4*>(h + 128 * block) + lane);
    return __reduce_add_sync(0xffffffffu, v.x + v.y + v.z + v.w);
}
// Step 2 (one warp): `mine` = the sum of block `lane` (lane 31 holds the top bins).
__device__ __forceinline__ void warp_scan_select(const uint32_t* __restrict__ h, uint32_t mine, uint32_t k,
                                                 int lane, uint32_t& bucket, uint32_t& above,
                                                 uint32_t& inbucket) {
    static_assert(kBins1 == 4096, "32 blocks of 128 bins");
    const uint32_t suf = warp_suffix_sum(mine, lane);
    const uint32_t ab = suf - mine;   // keys in blocks above mine
    const unsigned hit = __ballot_sync(0xffffffffu, mine != 0 && ab < k && k <= ab + mine);
    bucket = 0; above = 0; inbucket = 0;
    if (hit == 0) return;            // k exceeds the histogram total: cannot happen for a valid plan
    const int owner = __ffs(hit) - 1;
    const uint32_t ab_owner = __shfl_sync(0xffffffffu, ab, owner);
    // the owner block's 128 bins, four per lane
    const uint4 c = __ldcg(reinterpret_cast<const uint4*>(h + 128 * owner) + lane);
    const uint32_t s2 = c.x + c.y + c.z + c.w;
    const uint32_t ab2 = ab_owner + warp_suffix_sum(s2, lane) - s2;
    const unsigned hit2 = __ballot_sync(0xffffffffu, s2 != 0 && ab2 < k && k <= ab2 + s2);
    if (hit2 == 0) return;
    const int l2 = __ffs(hit2) - 1;
    const uint32_t cc[4] = {c.x, c.y, c.z, c.w};
    uint32_t b = 0, a = ab2, n = 0;
#pragma unroll
    for (int i = 3; i >= 0; --i) {   // descending bins inside the lane
        if (n == 0) {
            if (a + cc[i] >= k) { b = 128 * owner + 4 * lane + i; n = cc[i]; }
            else a += cc[i];
        }
    }
    bucket = __shfl_sync(0xffffffffu, b, l2);
    above = __shfl_sync(0xffffffffu, a, l2);
    inbucket = __shfl_sync(0xffffffffu, n, l2);
}

// ---------------------------------------------------------------------------------
// tile workers (one warp per tile)
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void hist_tile(const float* __restrict__ acc, const TileSpan& ts,
                                          uint32_t* h, int lane) {
    if (ts.s == 0 && ts.e == kTile) {
        const uint4* p = reinterpret_cast<const uint4*>(acc + ts.lo) + lane;
#pragma unroll 1
        for (int it = 0; it < kTile / 1024; ++it) {
            uint4 v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = __ldg(p + it * 256 + i * 32);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                atomicAdd(&h[key_of(v[i].x) >> kShift1], 1u);
                atomicAdd(&h[key_of(v[i].y) >> kShift1], 1u);
                atomicAdd(&h[key_of(v[i].z) >> kShift1], 1u);
                atomicAdd(&h[key_of(v[i].w) >> kShift1], 1u);
            }
        }
    } else {
        // partial tile: ragged head and tail (< 4 elements each) by scalar loads, the 16-byte
        // aligned middle by guarded vector loads, 8 in flight per lane
        const uint32_t* p = reinterpret_cast<const uint32_t*>(acc + ts.lo);
        const int s4 = (ts.s + 3) & ~3, e4 = ts.e & ~3;
        if (s4 >= e4) {
            for (int o = ts.s + lane; o < ts.e; o += 32) atomicAdd(&h[key_of(__ldg(p + o)) >> kShift1], 1u);
            return;
        }
        if (lane < s4 - ts.s) atomicAdd(&h[key_of(__ldg(p + ts.s + lane)) >> kShift1], 1u);
        if (lane >= 4 && lane - 4 < ts.e - e4) atomicAdd(&h[key_of(__ldg(p + e4 + lane - 4)) >> kShift1], 1u);
        const uint4* p4 = reinterpret_cast<const uint4*>(p);
        const int g1 = e4 >> 2;
        for (int g0 = (s4 >> 2); g0 < g1; g0 += 256) {
            uint4 v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int g = g0 + i * 32 + lane;
                v[i] = g < g1 ? __ldg(p4 + g) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (g0 + i * 32 + lane < g1) {
                    atomicAdd(&h[key_of(v[i].x) >> kShift1], 1u);
                    atomicAdd(&h[key_of(v[i].y) >> kShift1], 1u);
                    atomicAdd(&h[key_of(v[i].z) >> kShift1], 1u);
                    atomicAdd(&h[key_of(v[i].w) >> kShift1], 1u);
                }
            }
        }
    }
}

// Destination of the ordered copy: entries beyond `cap` are counted but not stored.
struct FilterOut {
    uint2* dst;      // shared or global memory
    uint32_t cap;
    uint32_t yorg;   // added to the offset inside the tile: offset from the run's first tile
};

// One step of the ordered copy over at most 32 consecutive elements [o0, o1), one per lane.
__device__ __forceinline__ void filter_scalar(const uint32_t* __restrict__ p, int o0, int o1, uint32_t b1,
                                              bool big, uint32_t* h2, const FilterOut& out, int lane,
                                              uint32_t& run) {
    const uint32_t lt = (1u << lane) - 1u;
    const int o = o0 + lane;
    uint32_t bits = 0;
    bool keep = false;
    if (o < o1) {
        bits = __ldg(p + o);
        const uint32_t key = key_of(bits);
        const uint32_t bucket = key >> kShift1;
        keep = bucket >= b1;
        if (big && bucket == b1) atomicAdd(&h2[(key >> kShift2) & (kBins2 - 1)], 1u);
    }
    const unsigned m = __ballot_sync(0xffffffffu, keep);
    const uint32_t pos = run + __popc(m & lt);
    if (keep && pos < out.cap) out.dst[pos] = make_uint2(bits, out.yorg + (uint32_t)o);
    run += __popc(m);
}

// The ordered copy over the 16-byte groups [g0, g1) of a tile, 8 vector loads per lane per
// step (1024 elements).  Element order inside a step: (load, lane, component) = ascending
// offset.
template <bool kFull>
__device__ __forceinline__ void filter_groups(const uint32_t* __restrict__ p, int g0, int g1, uint32_t b1,
                                              bool big, uint32_t* h2, const FilterOut& out, int lane,
                                              uint32_t& run) {
    const uint4* p4 = reinterpret_cast<const uint4*>(p);
#pragma unroll 1
    for (int gb = g0; gb < g1; gb += 256) {
        uint4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int g = gb + i * 32 + lane;
            v[i] = (kFull || g < g1) ? __ldg(p4 + g) : make_uint4(0u, 0u, 0u, 0u);
        }
        uint32_t keep = 0;                 // bit (4*i + c): component c of load i goes to staging
        uint32_t packed[2] = {0u, 0u};     // per-load counts, 8 bits each (a warp holds <= 128 per load)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (kFull || gb + i * 32 + lane < g1) {
                const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t key = key_of(w[c]);
                    const uint32_t bucket = key >> kShift1;
                    if (bucket >= b1) {
                        keep |= 1u << (i * 4 + c);
                        packed[i >> 2] += 1u << (8 * (i & 3));
                        if (big && bucket == b1) atomicAdd(&h2[(key >> kShift2) & (kBins2 - 1)], 1u);
                    }
                }
            }
        }
        if (__any_sync(0xffffffffu, keep != 0)) {
            const uint32_t incl0 = warp_incl_scan(packed[0], lane), incl1 = warp_incl_scan(packed[1], lane);
            const uint32_t tot0 = __shfl_sync(0xffffffffu, incl0, 31), tot1 = __shfl_sync(0xffffffffu, incl1, 31);
            const uint32_t excl[2] = {incl0 - packed[0], incl1 - packed[1]};
            uint32_t load_base = run;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t tot_i = ((i < 4 ? tot0 : tot1) >> (8 * (i & 3))) & 0xff;
                if ((keep >> (4 * i)) & 0xfu) {
                    const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
                    uint32_t pos = load_base + ((excl[i >> 2] >> (8 * (i & 3))) & 0xff);
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if (keep & (1u << (i * 4 + c))) {
                            if (pos < out.cap)
                                out.dst[pos] = make_uint2(w[c], out.yorg + (uint32_t)((gb + i * 32 + lane) * 4 + c));
                            ++pos;
                        }
                }
                load_base += tot_i;
            }
            run = load_base;
        }
    }
}

// Copies the tile's entries with bucket >= b1 to `out` in index order; returns how many
// there are (which may exceed out.cap).
__device__ __forceinline__ uint32_t filter_tile(const float* __restrict__ acc, const TileSpan& ts,
                                                uint32_t b1, bool big, uint32_t* h2,
                                                const FilterOut& out, int lane) {
    uint32_t run = 0;
    const uint32_t* p = reinterpret_cast<const uint32_t*>(acc + ts.lo);
    if (ts.s == 0 && ts.e == kTile) {
        filter_groups<true>(p, 0, kTile / 4, b1, big, h2, out, lane, run);
        return run;
    }
    // partial tile: ragged head (< 4), 16-byte aligned middle, ragged tail (< 4)
    const int s4 = (ts.s + 3) & ~3, e4 = ts.e & ~3;
    if (s4 >= e4) {
        for (int o0 = ts.s; o0 < ts.e; o0 += 32)
            filter_scalar(p, o0, (o0 + 32 < ts.e) ? o0 + 32 : ts.e, b1, big, h2, out, lane, run);
        return run;
    }
    if (ts.s < s4) filter_scalar(p, ts.s, s4, b1, big, h2, out, lane, run);
    filter_groups<false>(p, s4 >> 2, e4 >> 2, b1, big, h2, out, lane, run);
    if (e4 < ts.e) filter_scalar(p, e4, ts.e, b1, big, h2, out, lane, run);
    return run;
}

struct CtaRange { int q0, q1, jA, jB; };

__device__ __forceinline__ int cta_q0(const SelParams& p, int b) { return (int)((int64_t)p.tiles * b / gridDim.x); }

__device__ __forceinline__ CtaRange cta_range(const SelParams& p) {
    CtaRange r;
    r.q0 = cta_q0(p, blockIdx.x);
    r.q1 = cta_q0(p, blockIdx.x + 1);
    r.jA = r.jB = 0;
    if (r.q0 < r.q1) {
        r.jA = layer_of_tile(p.desc, p.n_my, r.q0);
        r.jB = layer_of_tile(p.desc, p.n_my, r.q1 - 1);
    }
    return r;
}

// The CTA whose run of tiles contains tile q.
__device__ __forceinline__ int cta_of_tile(const SelParams& p, int q) {
    return (int)((((int64_t)q + 1) * gridDim.x + p.tiles - 1) / p.tiles) - 1;
}

__device__ __forceinline__ bool is_direct(const SelParams& p, int j) {
    return p.desc[j].end - p.desc[j].start <= kDirectElems;
}

// Where CTA b's run of layer j lives: first staging entry and the element offset (relative
// to the layer start, possibly negative) that entry offsets are counted from.
struct RunRef { int64_t base; int64_t rel; };

__device__ __forceinline__ RunRef run_ref(const SelParams& p, int j, int b) {
    const int64_t start = p.desc[j].start;
    const int tf = p.desc[j].tile_first;
    const int q0 = cta_q0(p, b);
    const int qf = q0 > tf ? q0 : tf;   // the run's first tile
    RunRef r;
    r.rel = (start / kTile + (qf - tf)) * kTile - start;
    r.base = p.desc[j].elem_off + (r.rel > 0 ? r.rel : 0);
    return r;
}

// ---------------------------------------------------------------------------------
// phase A: level-1 histograms of the CTA's run of tiles, kSlots layers at a time
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void phase_hist1(const SelParams& p, unsigned char* smem) {
    const CtaRange r = cta_range(p);
    if (r.q0 >= r.q1) return;
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem + kSmMain);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int jg = r.jA; jg <= r.jB; jg += kSlots) {
        const int je = (jg + kSlots - 1 < r.jB) ? jg + kSlots - 1 : r.jB;
        const int ns = je - jg + 1;
        for (int i = threadIdx.x; i < ns * kBins1; i += kSelThreads) hist[i] = 0;
        __syncthreads();
        const int qa = r.q0 > p.desc[jg].tile_first ? r.q0 : p.desc[jg].tile_first;
        const int qb = r.q1 < p.desc[je + 1].tile_first ? r.q1 : p.desc[je + 1].tile_first;
        int jj = jg;
        for (int q = qa + warp; q < qb; q += kSelWarps) {
            while (q >= p.desc[jj + 1].tile_first) ++jj;
            if (is_direct(p, jj)) continue;   // loaded whole by one CTA in phase C
            const TileSpan ts = tile_span(p.desc[jj].start, p.desc[jj].end, p.desc[jj].tile_first, q);
            hist_tile(p.acc, ts, hist + (jj - jg) * kBins1, lane);
        }
        __syncthreads();
        for (int i = threadIdx.x; i < ns * kBins1; i += kSelThreads) {
            const uint32_t c = hist[i];   // slots of direct layers stay zero
            if (c) atomicAdd(p.hist1 + (size_t)p.desc[jg + i / kBins1].layer_id * kBins1 + (i % kBins1), c);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------
// phase B: bucket search for the CTA's layers (one warp each), then the staging pass in
// rounds of one tile per warp
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void phase_filter(const SelParams& p, unsigned char* smem) {
    const CtaRange r = cta_range(p);
    if (r.q0 >= r.q1) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint2* wbuf = reinterpret_cast<uint2*>(smem + kSmMain) + warp * kBufCap;
    uint32_t* hist2s = reinterpret_cast<uint32_t*>(smem + kSmMain + kSelWarps * kBufCap * 8);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* tab = misc + kMTab;
    uint32_t* run_total = misc + kMRunTotal;
    uint32_t* cnt_s = misc + kMCnt;
    int* lay_s = reinterpret_cast<int*>(misc + kMLay);
    uint32_t* bsum = misc + kMBsum;

    for (int jg = r.jA; jg <= r.jB; jg += kSlots) {
        const int je = (jg + kSlots - 1 < r.jB) ? jg + kSlots - 1 : r.jB;
        const int ns = je - jg + 1;
        // block sums of the group's level-1 histograms: every warp takes its share of the
        // ns * 32 blocks, all requests in flight at once
        {
            uint32_t sums[kSlots * 32 / kSelWarps];
#pragma unroll
            for (int u = 0; u < kSlots * 32 / kSelWarps; ++u) {
                const int item = u * kSelWarps + warp;   // (slot, block)
                const int s_ = item >> 5;
                sums[u] = 0;
                if (s_ < ns && !is_direct(p, jg + s_))
                    sums[u] = hist1_block_sum(p.hist1 + (size_t)p.desc[jg + s_].layer_id * kBins1, item & 31, lane);
            }
            if (lane == 0) {
#pragma unroll
                for (int u = 0; u < kSlots * 32 / kSelWarps; ++u) bsum[u * kSelWarps + warp] = sums[u];
            }
        }
        __syncthreads();
        if (warp < ns) {
            const int j = jg + warp;
            uint32_t b1 = 0, kind = kKindDirect;
            if (!is_direct(p, j)) {
                const int lid = p.desc[j].layer_id;
                uint32_t above, cand;
                warp_scan_select(p.hist1 + (size_t)lid * kBins1, bsum[warp * 32 + lane], (uint32_t)p.desc[j].k, lane,
                                 b1, above, cand);
                const int ntiles = p.desc[j + 1].tile_first - p.desc[j].tile_first;
                kind = (ntiles > kSmallTiles || above + cand > (uint32_t)kSmallEntries) ? kKindBig : kKindSmall;
                if (lane == 0) {
                    LayerState st;
                    st.b1 = b1; st.above1 = above; st.cand1 = cand; st.big = kind;
                    st.b2 = 0; st.krem2 = 0; st.T = 0; st.need = 0;
                    p.state[lid] = st;   // every CTA that streams this layer writes the same values
                    if (kind == kKindBig) atomicOr(&p.flags->any_big, 1u);
                }
            }
            if (lane == 0) {
                tab[2 * warp] = b1;
                tab[2 * warp + 1] = kind;
                run_total[warp] = 0;
            }
        }
        __syncthreads();
        stamp(p, 11);
        bool any_big = false;
        for (int s = 0; s < ns; ++s) any_big |= (tab[2 * s + 1] == kKindBig);
        if (any_big) {
            for (int i = threadIdx.x; i < ns * kBins2; i += kSelThreads) hist2s[i] = 0;
            __syncthreads();
        }
        const int qa = r.q0 > p.desc[jg].tile_first ? r.q0 : p.desc[jg].tile_first;
        const int qb = r.q1 < p.desc[je + 1].tile_first ? r.q1 : p.desc[je + 1].tile_first;
        int jj = jg;
        int par = 0;
        for (int qr = qa; qr < qb; qr += kSelWarps, par ^= 32) {
            const int q = qr + warp;
            uint32_t n = 0, b1 = 0;
            int slot = -1;
            TileSpan ts{0, 0, 0};
            int64_t run_base = 0;
            uint32_t yorg = 0;
            if (q < qb) {
                while (q >= p.desc[jj + 1].tile_first) ++jj;
                const uint32_t kind = tab[2 * (jj - jg) + 1];
                if (kind != kKindDirect) {
                    slot = jj - jg;
                    const int64_t start = p.desc[jj].start;
                    const int tf = p.desc[jj].tile_first;
                    ts = tile_span(start, p.desc[jj].end, tf, q);
                    const int qf = r.q0 > tf ? r.q0 : tf;   // first tile of this CTA's run of the layer
                    const int64_t rel = (start / kTile + (qf - tf)) * kTile - start;
                    run_base = p.desc[jj].elem_off + (rel > 0 ? rel : 0);
                    yorg = (uint32_t)((q - qf) * kTile);
                    b1 = tab[2 * slot];
                    const FilterOut fo{wbuf, (uint32_t)kBufCap, yorg};
                    n = filter_tile(p.acc, ts, b1, kind == kKindBig, hist2s + slot * kBins2, fo, lane);
                }
            }
            if (lane == 0) { cnt_s[par + warp] = n; lay_s[par + warp] = slot; }
            __syncthreads();
            if (n > 0) {   // uniform over the warp
                const uint32_t c = (lane < warp && lay_s[par + lane] == slot) ? cnt_s[par + lane] : 0u;   // warp < kSelWarps
                const uint32_t excl = __reduce_add_sync(0xffffffffu, c);   // entries of lower warps, same layer
                uint2* dst = p.staging + run_base + run_total[slot] + excl;
                if (n <= (uint32_t)kBufCap) {
                    for (uint32_t e = lane; e < n; e += 32) dst[e] = wbuf[e];
                } else {   // the buffer overflowed: stream the tile again (L1/L2), straight to its place
                    const FilterOut fo{dst, 0xffffffffu, yorg};
                    filter_tile(p.acc, ts, b1, false, nullptr, fo, lane);
                }
            }
            __syncthreads();
            if (threadIdx.x < ns) {
                uint32_t tot = 0;
                for (int w = 0; w < kSelWarps; ++w)
                    if (lay_s[par + w] == (int)threadIdx.x) tot += cnt_s[par + w];
                run_total[threadIdx.x] += tot;   // read by the next round after its barrier
            }
        }
        stamp(p, 12);
        __syncthreads();
        if (threadIdx.x < ns && tab[2 * threadIdx.x + 1] != kKindDirect)
            p.runcnt[blockIdx.x + jg + threadIdx.x] = run_total[threadIdx.x];
        if (any_big) {
            for (int i = threadIdx.x; i < ns * kBins2; i += kSelThreads) {
                const int s = i / kBins2;
                const uint32_t c = hist2s[i];
                if (c && tab[2 * s + 1] == kKindBig)
                    atomicAdd(p.hist2 + (size_t)p.desc[jg + s].layer_id * kBins2 + (i % kBins2), c);
            }
        }
        __syncthreads();
    }
}

// Ordered write of one batch of 32 consecutive staged entries (one per lane).  gt_before /
// eq_before: entries above / equal to the threshold that precede the batch in the layer.
__device__ __forceinline__ void emit_batch(const SelParams& p, int64_t out_off, int64_t elem0, bool valid,
                                           uint32_t bits, int64_t off, uint32_t T, uint32_t need,
                                           uint32_t& gt_before, uint32_t& eq_before, int lane) {
    const uint32_t lt = (1u << lane) - 1u;
    const uint32_t key = key_of(bits);
    const bool gt = valid && key > T, eq = valid && key == T;
    const unsigned gt_b = __ballot_sync(0xffffffffu, gt), eq_b = __ballot_sync(0xffffffffu, eq);
    const uint32_t my_gt = gt_before + __popc(gt_b & lt), my_eq = eq_before + __popc(eq_b & lt);
    if (gt || (eq && my_eq < need)) {
        // selected entries before me: every larger key, and the first `need` equal ones
        const int64_t pos = out_off + my_gt + (my_eq < need ? my_eq : need);
        p.val[pos] = __uint_as_float(bits);
        p.idx[pos] = elem0 + off;
    }
    gt_before += __popc(gt_b);
    eq_before += __popc(eq_b);
}

// ---------------------------------------------------------------------------------
// phase C: one CTA finishes one layer from shared memory
// ---------------------------------------------------------------------------------
// Back end: skey[0..E) / soff[0..E) hold, in index order, every entry of the layer whose
// level-1 bucket is >= b1.  Finishes the radix select (level 2 inside b1, level 3 inside
// (b1, b2), ties by lowest index) and writes the k selected entries.
__device__ __forceinline__ void finish_layer(const SelParams& p, int j, uint32_t E, uint32_t b1,
                                             uint32_t above1, unsigned char* smem) {
    uint32_t* skey = reinterpret_cast<uint32_t*>(smem + kSmMain);
    uint32_t* soff = skey + kSmallEntries;
    uint32_t* h = reinterpret_cast<uint32_t*>(smem + kSmH);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* scratch = misc + kMScratch;
    uint32_t* out3 = misc + kMOut3;
    uint32_t* wcnt = misc + kMWarpCnt;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t start = p.desc[j].start;
    const uint32_t k = (uint32_t)p.desc[j].k;
    const int64_t out_off = p.desc[j].out_off;

    // level 2 inside bucket b1 (h is zero on entry)
    for (uint32_t f = tid; f < E; f += kSelThreads) {
        const uint32_t key = key_of(skey[f]);
        if ((key >> kShift1) == b1) atomicAdd(&h[(key >> kShift2) & (kBins2 - 1)], 1u);
    }
    __syncthreads();
    block_scan_select<false>(h, kBins2, k - above1, scratch, out3);
    const uint32_t b2 = out3[0];
    const uint32_t krem2 = k - above1 - out3[1];
    __syncthreads();
    for (int i = tid; i < kBins3; i += kSelThreads) h[i] = 0;
    __syncthreads();

    // level 3 inside (b1, b2)
    const uint32_t prefix = (b1 << (kShift1 - kShift2)) | b2;
    for (uint32_t f = tid; f < E; f += kSelThreads) {
        const uint32_t key = key_of(skey[f]);
        if ((key >> kShift2) == prefix) atomicAdd(&h[key & (kBins3 - 1)], 1u);
    }
    __syncthreads();
    block_scan_select<false>(h, kBins3, krem2, scratch, out3);
    const uint32_t T = (prefix << kShift2) | out3[0];
    const uint32_t need = krem2 - out3[1];
    __syncthreads();
    stamp(p, 10);

    // every warp counts its contiguous share of the entries
    const uint32_t wper = ((E + kSelWarps - 1) / kSelWarps + 31) & ~31u;   // multiple of 32
    const uint32_t f0 = (uint32_t)warp * wper < E ? (uint32_t)warp * wper : E;
    const uint32_t f1 = f0 + wper < E ? f0 + wper : E;
    uint32_t n_gt = 0, n_eq = 0;
    for (uint32_t f = f0 + lane; f < f1; f += 32) {
        const uint32_t key = key_of(skey[f]);
        n_gt += key > T;
        n_eq += key == T;
    }
    n_gt = __reduce_add_sync(0xffffffffu, n_gt);
    n_eq = __reduce_add_sync(0xffffffffu, n_eq);
    if (lane == 0) wcnt[warp] = n_gt | (n_eq << 16);   // both totals <= kSmallEntries < 65536
    __syncthreads();
    const uint32_t mine = lane < kSelWarps ? wcnt[lane] : 0u;
    const uint32_t before = __shfl_sync(0xffffffffu, warp_incl_scan(mine, lane) - mine, warp);
    uint32_t gt_before = before & 0xffff, eq_before = before >> 16;
    stamp(p, 13);

    // ordered, coalesced write
    for (uint32_t fb = f0; fb < f1; fb += 32) {
        const uint32_t f = fb + lane;
        const bool valid = f < f1;
        emit_batch(p, out_off, start, valid, valid ? skey[f] : 0u, valid ? (int64_t)soff[f] : 0, T, need,
                   gt_before, eq_before, lane);
    }
    __syncthreads();   // shared memory is reused by the next layer
}

// Front end for a streamed small layer: pull its runs into shared memory.
__device__ __forceinline__ void resolve_small(const SelParams& p, int j, const LayerState& st,
                                              unsigned char* smem) {
    uint32_t* skey = reinterpret_cast<uint32_t*>(smem + kSmMain);   // value bits of the staged entries
    uint32_t* soff = skey + kSmallEntries;                          // their offsets inside the layer
    uint32_t* h = reinterpret_cast<uint32_t*>(smem + kSmH);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* scratch = misc + kMScratch;
    uint32_t* roff = misc + kMRoff;
    int* rrel = reinterpret_cast<int*>(misc + kMRrel);
    int64_t* rbase = reinterpret_cast<int64_t*>(misc + kMRbase);
    const int tid = threadIdx.x;
    const int tf = p.desc[j].tile_first, tfe = p.desc[j + 1].tile_first;

    // (a) the layer's runs: one per CTA that streamed some of its tiles
    const int b0 = cta_of_tile(p, tf), b1c = cta_of_tile(p, tfe - 1);
    const int nr = b1c - b0 + 1;
    uint32_t c = 0;
    if (tid < nr) {
        const int b = b0 + tid;
        if (cta_q0(p, b) < cta_q0(p, b + 1)) c = __ldcg(p.runcnt + b + j);
    }
    uint32_t E;
    const uint32_t ex = block_excl_scan(c, scratch, E);
    if (tid <= nr) roff[tid] = tid < nr ? ex : E;
    if (tid < nr) {
        const RunRef ref = run_ref(p, j, b0 + tid);
        rrel[tid] = (int)ref.rel;
        rbase[tid] = ref.base;
    }
    for (int i = tid; i < kBins2; i += kSelThreads) h[i] = 0;
    __syncthreads();
    stamp(p, 8);
    if (p.timing && tid == 0) atomicMax(p.timing + 14, (unsigned long long)E);

    // (b) pull the runs into shared memory in stream (= index) order: flat over the
    //     entries, 8 loads per thread in flight, the run found by bisection of roff
    for (uint32_t fb = 0; fb < E; fb += 8 * kSelThreads) {
        uint2 ent[8];
        int rel[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t f = fb + u * kSelThreads + tid;
            ent[u] = make_uint2(0u, 0u);
            rel[u] = 0;
            if (f < E) {
                int lo = 0;   // last run whose offset is <= f (empty runs share offsets); fixed trip count
#pragma unroll
                for (int step = kMaxRuns / 2; step >= 1; step >>= 1)
                    if (lo + step < nr && roff[lo + step] <= f) lo += step;
                rel[u] = rrel[lo];
                ent[u] = __ldcg(p.staging + rbase[lo] + (f - roff[lo]));
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t f = fb + u * kSelThreads + tid;
            if (f < E) {
                skey[f] = ent[u].x;
                soff[f] = (uint32_t)(rel[u] + (int)ent[u].y);
            }
        }
    }
    __syncthreads();
    stamp(p, 9);
    finish_layer(p, j, E, st.b1, st.above1, smem);
}

// Front end for a direct layer (at most kDirectElems elements): load it whole, find the
// level-1 bucket from a shared-memory histogram.  Phases A and B never touch these layers.
__device__ __forceinline__ void resolve_direct(const SelParams& p, int j, unsigned char* smem) {
    uint32_t* skey = reinterpret_cast<uint32_t*>(smem + kSmMain);
    uint32_t* soff = skey + kSmallEntries;
    uint32_t* h1 = reinterpret_cast<uint32_t*>(smem + kSmH1);
    uint32_t* h = reinterpret_cast<uint32_t*>(smem + kSmH);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* scratch = misc + kMScratch;
    uint32_t* out3 = misc + kMOut3;
    const int tid = threadIdx.x;
    const int64_t start = p.desc[j].start;
    const uint32_t n = (uint32_t)(p.desc[j].end - start);
    const uint32_t* x = reinterpret_cast<const uint32_t*>(p.acc + start);
    for (int i = tid; i < kBins1; i += kSelThreads) h1[i] = 0;
    for (int i = tid; i < kBins2; i += kSelThreads) h[i] = 0;
    __syncthreads();
    for (uint32_t fb = 0; fb < n; fb += 8 * kSelThreads) {
        uint32_t v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t f = fb + u * kSelThreads + tid;
            v[u] = f < n ? __ldg(x + f) : 0u;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t f = fb + u * kSelThreads + tid;
            if (f < n) {
                skey[f] = v[u];
                soff[f] = f;
                atomicAdd(&h1[key_of(v[u]) >> kShift1], 1u);
            }
        }
    }
    __syncthreads();
    block_scan_select<false>(h1, kBins1, (uint32_t)p.desc[j].k, scratch, out3);
    const uint32_t b1 = out3[0], above1 = out3[1];
    __syncthreads();
    finish_layer(p, j, n, b1, above1, smem);
}

// ---------------------------------------------------------------------------------
// general path for big layers (grid-wide steps; every CTA works on its own runs)
// ---------------------------------------------------------------------------------
template <int kLevel>
__device__ __forceinline__ void big_scan(const SelParams& p, unsigned char* smem) {
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* scratch = misc + kMScratch;
    uint32_t* out3 = misc + kMOut3;
    for (int j = blockIdx.x; j < p.n_my; j += gridDim.x) {
        const int lid = p.desc[j].layer_id;
        if (__ldcg(&p.state[lid].big) != kKindBig) continue;   // uniform over the CTA
        const uint32_t k = (uint32_t)p.desc[j].k;
        if (kLevel == 2) {
            const uint32_t above1 = __ldcg(&p.state[lid].above1);
            block_scan_select<true>(p.hist2 + (size_t)lid * kBins2, kBins2, k - above1, scratch, out3);
            if (threadIdx.x == 0) {
                p.state[lid].b2 = out3[0];
                p.state[lid].krem2 = k - above1 - out3[1];
            }
        } else {
            const uint32_t krem2 = __ldcg(&p.state[lid].krem2);
            block_scan_select<true>(p.hist3 + (size_t)lid * kBins3, kBins3, krem2, scratch, out3);
            if (threadIdx.x == 0) {
                const uint32_t b1 = __ldcg(&p.state[lid].b1), b2 = __ldcg(&p.state[lid].b2);
                p.state[lid].T = (b1 << kShift1) | (b2 << kShift2) | out3[0];
                p.state[lid].need = krem2 - out3[1];
            }
        }
        __syncthreads();
    }
}

// level-3 histogram of the entries whose top 22 key bits equal (b1, b2)
__device__ __forceinline__ void big_hist3(const SelParams& p, unsigned char* smem) {
    const CtaRange r = cta_range(p);
    if (r.q0 >= r.q1) return;
    uint32_t* h = reinterpret_cast<uint32_t*>(smem + kSmH);
    for (int j = r.jA; j <= r.jB; ++j) {
        const int lid = p.desc[j].layer_id;
        if (is_direct(p, j) || __ldcg(&p.state[lid].big) != kKindBig) continue;   // uniform
        const uint32_t prefix = (__ldcg(&p.state[lid].b1) << (kShift1 - kShift2)) | __ldcg(&p.state[lid].b2);
        const uint32_t n = __ldcg(p.runcnt + blockIdx.x + j);
        const uint2* src = p.staging + run_ref(p, j, blockIdx.x).base;
        for (int i = threadIdx.x; i < kBins3; i += kSelThreads) h[i] = 0;
        __syncthreads();
        for (uint32_t e = threadIdx.x; e < n; e += kSelThreads) {
            const uint32_t key = key_of(__ldcg(src + e).x);
            if ((key >> kShift2) == prefix) atomicAdd(&h[key & (kBins3 - 1)], 1u);
        }
        __syncthreads();
        for (int i = threadIdx.x; i < kBins3; i += kSelThreads)
            if (h[i]) atomicAdd(p.hist3 + (size_t)lid * kBins3 + i, h[i]);
        __syncthreads();
    }
}

// per run: how many entries lie above T, how many equal T
__device__ __forceinline__ void big_count(const SelParams& p, unsigned char* smem) {
    const CtaRange r = cta_range(p);
    if (r.q0 >= r.q1) return;
    uint32_t* scratch = reinterpret_cast<uint32_t*>(smem + kSmMisc) + kMScratch;
    for (int j = r.jA; j <= r.jB; ++j) {
        const int lid = p.desc[j].layer_id;
        if (is_direct(p, j) || __ldcg(&p.state[lid].big) != kKindBig) continue;   // uniform
        const uint32_t T = __ldcg(&p.state[lid].T);
        const uint32_t n = __ldcg(p.runcnt + blockIdx.x + j);
        const uint2* src = p.staging + run_ref(p, j, blockIdx.x).base;
        uint32_t n_gt = 0, n_eq = 0;
        for (uint32_t e = threadIdx.x; e < n; e += kSelThreads) {
            const uint32_t key = key_of(__ldcg(src + e).x);
            n_gt += key > T;
            n_eq += key == T;
        }
        uint32_t tot_gt, tot_eq;
        block_excl_scan(n_gt, scratch, tot_gt);
        block_excl_scan(n_eq, scratch, tot_eq);
        if (threadIdx.x == 0) p.runge[blockIdx.x + j] = make_uint2(tot_gt, tot_eq);
        __syncthreads();
    }
}

// per big layer: exclusive scan of its runs' counts (one CTA per layer)
__device__ __forceinline__ void big_run_scan(const SelParams& p, unsigned char* smem) {
    uint32_t* scratch = reinterpret_cast<uint32_t*>(smem + kSmMisc) + kMScratch;
    for (int j = blockIdx.x; j < p.n_my; j += gridDim.x) {
        if (__ldcg(&p.state[p.desc[j].layer_id].big) != kKindBig) continue;   // uniform
        const int b0 = cta_of_tile(p, p.desc[j].tile_first), b1c = cta_of_tile(p, p.desc[j + 1].tile_first - 1);
        const int nr = b1c - b0 + 1;
        uint2 v = make_uint2(0u, 0u);
        const int b = b0 + (int)threadIdx.x;
        const bool live = (int)threadIdx.x < nr && cta_q0(p, b) < cta_q0(p, b + 1);
        if (live) v = __ldcg(p.runge + b + j);
        uint32_t tot;
        const uint32_t e_gt = block_excl_scan(v.x, scratch, tot);
        const uint32_t e_eq = block_excl_scan(v.y, scratch, tot);
        if (live) p.runge[b + j] = make_uint2(e_gt, e_eq);
        __syncthreads();
    }
}

// final ordered write of (value, index) for this CTA's runs of big layers
__device__ __forceinline__ void big_emit(const SelParams& p, unsigned char* smem) {
    const CtaRange r = cta_range(p);
    if (r.q0 >= r.q1) return;
    uint32_t* wcnt = reinterpret_cast<uint32_t*>(smem + kSmMisc) + kMWarpCnt;   // 2 x 32 words follow
    uint32_t* wcnt_eq = reinterpret_cast<uint32_t*>(smem + kSmMisc) + kMCnt;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int j = r.jA; j <= r.jB; ++j) {
        const int lid = p.desc[j].layer_id;
        if (is_direct(p, j) || __ldcg(&p.state[lid].big) != kKindBig) continue;   // uniform
        const uint32_t T = __ldcg(&p.state[lid].T), need = __ldcg(&p.state[lid].need);
        const uint32_t n = __ldcg(p.runcnt + blockIdx.x + j);
        const RunRef ref = run_ref(p, j, blockIdx.x);
        const uint2* src = p.staging + ref.base;
        const uint2 before = __ldcg(p.runge + blockIdx.x + j);
        uint32_t gt_base = before.x, eq_base = before.y;
        const int64_t start = p.desc[j].start, out_off = p.desc[j].out_off;
        for (uint32_t e0 = 0; e0 < n; e0 += kSelThreads) {
            const uint32_t e = e0 + threadIdx.x;
            const bool valid = e < n;
            uint2 ent = make_uint2(0u, 0u);
            if (valid) ent = __ldcg(src + e);
            const uint32_t key = key_of(ent.x);
            const unsigned gt_b = __ballot_sync(0xffffffffu, valid && key > T);
            const unsigned eq_b = __ballot_sync(0xffffffffu, valid && key == T);
            __syncthreads();   // the count tables may still be read by the previous batch
            if (lane == 0) { wcnt[warp] = __popc(gt_b); wcnt_eq[warp] = __popc(eq_b); }
            __syncthreads();
            const uint32_t cg_ = lane < kSelWarps ? wcnt[lane] : 0u, ce_ = lane < kSelWarps ? wcnt_eq[lane] : 0u;
            const uint32_t ig = warp_incl_scan(cg_, lane), ie = warp_incl_scan(ce_, lane);
            uint32_t gt_before = gt_base + __shfl_sync(0xffffffffu, ig - cg_, warp);
            uint32_t eq_before = eq_base + __shfl_sync(0xffffffffu, ie - ce_, warp);
            emit_batch(p, out_off, start, valid, ent.x, ref.rel + (int64_t)ent.y, T, need, gt_before, eq_before, lane);
            gt_base += __shfl_sync(0xffffffffu, ig, 31);
            eq_base += __shfl_sync(0xffffffffu, ie, 31);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSelThreads, 1) k_select_fused(const SelParams p) {
    extern __shared__ __align__(16) unsigned char smem[];
    cg::grid_group grid = cg::this_grid();

    if (p.timing && threadIdx.x == 0 && blockIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        p.timing[0] = t;
    }
    phase_hist1(p, smem);
    stamp(p, 1);
    grid.sync();
    stamp(p, 2);
    phase_filter(p, smem);
    stamp(p, 3);
    grid.sync();
    stamp(p, 4);

    for (int j = blockIdx.x; j < p.n_my; j += gridDim.x) {
        if (is_direct(p, j)) {   // uniform over the CTA
            resolve_direct(p, j, smem);
            continue;
        }
        const int lid = p.desc[j].layer_id;
        LayerState st;
        st.b1 = __ldcg(&p.state[lid].b1);
        st.above1 = __ldcg(&p.state[lid].above1);
        st.cand1 = __ldcg(&p.state[lid].cand1);
        st.big = __ldcg(&p.state[lid].big);
        if (st.big != kKindSmall) continue;   // uniform over the CTA
        resolve_small(p, j, st, smem);
    }
    stamp(p, 5);
    if (__ldcg(&p.flags->any_big) == 0) return;   // same value in every CTA: written before the barrier

    big_scan<2>(p, smem);
    grid.sync();
    big_hist3(p, smem);
    grid.sync();
    big_scan<3>(p, smem);
    grid.sync();
    big_count(p, smem);
    grid.sync();
    big_run_scan(p, smem);
    grid.sync();
    big_emit(p, smem);
    stamp(p, 6);
}

__global__ void k_zero_at(float* __restrict__ acc, const int64_t* __restrict__ idx, int64_t count) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count;
         i += (int64_t)gridDim.x * blockDim.x)
        acc[idx[i]] = 0.0f;
}

}  // namespace

deft_status launch_select(const SelParams& p, cudaStream_t stream) {
    static thread_local int attr_dev = -1;
    int dev = 0;
    DEFT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != attr_dev) {
        DEFT_CUDA_TRY(cudaFuncSetAttribute(k_select_fused, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kSmemBytes));
        attr_dev = dev;
    }
    // one CTA per SM at most (co-resident by construction); fewer when the rank is tiny
    int sms = sm_count();
    if (sms > kMaxRuns) sms = kMaxRuns;
    int want = (p.tiles + 3) / 4;
    if (want < p.n_my) want = p.n_my;
    if (want < 1) want = 1;
    const int grid = want < sms ? want : sms;
    SelParams args = p;
    void* kargs[] = {&args};
    DEFT_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(k_select_fused), dim3(grid),
                                              dim3(kSelThreads), kargs, kSmemBytes, stream));
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
