// Layer-wise top-k selection for one worker (Algorithm 5) as ONE persistent cooperative
// kernel: a segmented radix select over magnitude bit patterns followed by an ordered
// compaction.  One CTA of 512 threads per SM; five steps separated by grid barriers.  Every
// CTA owns the same contiguous run of the rank's tiles in every step, and keeps what it
// stages for them (in shared memory; overflow spills to HBM), so after the second read of the
// vector all work is local to the CTA that staged the data.
//
//   A   read 1: per-layer histogram of key bits 30..19 in shared memory, flushed with integer
//       atomics; the CTA that flushes a layer's last tiles finds the bucket b1 holding the
//       k-th largest key
//   B   read 2: one warp per tile keeps the whole tile in registers, and moves every entry
//       with bucket >= b1, in index order, behind the CTA's staging cursor; bucket-b1 entries
//       feed the level-2 histogram (bits 18..9); last flusher finds bucket b2
//   S2  level-3 histogram (bits 8..0) over the staged entries of bucket (b1, b2); last
//       flusher fixes the exact threshold key T and how many entries equal to T are needed
//   S3  per tile: staged entries above T / equal to T; per (CTA, layer) totals
//   S4  every CTA adds up the totals of the CTAs before it, scans its own tiles, and writes
//       (value, int64 index) in ascending index (equal keys: lowest indices first);
//       optionally zeroes the selected entries of the vector (residual update)
// Layers of at most kDirectElems elements take no part in this: at the end one CTA loads
// each of them whole and finishes it from shared memory.
//
// Determinism: histograms use integer atomics (order-free); the staging order inside a CTA
// depends on warp timing but every output position is a function of counts and of the tile
// an entry came from, so the result is bit-identical from run to run.
#include <cooperative_groups.h>

#include "deft_common.cuh"

namespace cg = cooperative_groups;

namespace deft {
namespace {

// shared-memory carve-up (bytes)
constexpr int kSmMain = 0;   // A: kSlots level-1 histograms | B..S4: resident entries | direct: keys
constexpr int kSmMainBytes = 128 * 1024;
static_assert(kSlots * kBins1 * 4 <= kSmMainBytes && kResident * 8 <= kSmMainBytes &&
              kDirectElems * 4 <= kSmMainBytes, "main region");
constexpr int kSmAux = kSmMain + kSmMainBytes;   // B: level-2 slots | S2: level-3 slots | direct: level-1 + level-2/3
constexpr int kSmAuxBytes = 32 * 1024;
static_assert(kSlots * kBins2 * 4 <= kSmAuxBytes && kBins1 * 4 + kBins2 * 4 <= kSmAuxBytes, "aux region");
constexpr int kSmMisc = kSmAux + kSmAuxBytes;
constexpr int kSmMiscBytes = 2048;
constexpr int kSmGroup = kSmMisc + kSmMiscBytes;   // GroupShared
constexpr int kSmGroupBytes = 512;
constexpr int kSmemBytes = kSmGroup + kSmGroupBytes;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
static_assert(kBins2 >= kBins3, "the level-3 histogram reuses the level-2 buffer");

enum MiscOff : int {   // word offsets inside the misc area
    kMScratch = 0,     // 64: block scan scratch
    kMOut3 = 64,       // 4: result of block_scan_select
    kMTabA = 72,       // kSlots: per-slot value of the current step (b1 | prefix | T)
    kMTabB = 80,       // kSlots: second per-slot value (need)
    kMLast = 88,       // kSlots: this CTA flushed the layer's last tiles
    kMTotGt = 96,      // kSlots
    kMTotEq = 104,     // kSlots
    kMCursor = 112,    // 1: staged entries of this CTA so far
    kMWarpCnt = 128,   // 32: per-warp packed counts (direct layers)
};
static_assert(kMWarpCnt + 32 <= kSmMiscBytes / 4, "misc area");
static_assert(kSlots <= 8, "misc tables are 8 wide");

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

// ---------------------------------------------------------------------------------
// tile workers: one warp holds a whole tile (kTile = 2048 elements) in registers
// ---------------------------------------------------------------------------------
// 16-byte group g of the tile (0..511) is read by lane g % 32 as load g / 32.  Groups that
// do not touch [s, e) are not read; a group that straddles s or e is read whole (the bytes
// outside the layer are inside the same 16-byte aligned group, hence readable) and masked.
struct TileRegs {
    uint4 v[16];
};
static_assert(kTile == 16 * 32 * 4, "16 vector loads per lane");

__device__ __forceinline__ void load_tile(const float* __restrict__ acc, const TileSpan& ts, int lane,
                                          TileRegs& t) {
    const uint4* p4 = reinterpret_cast<const uint4*>(acc + ts.lo) + lane;
    if (ts.s == 0 && ts.e == kTile) {
#pragma unroll
        for (int i = 0; i < 16; ++i) t.v[i] = __ldg(p4 + i * 32);
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int o = (i * 32 + lane) * 4;
            t.v[i] = (o + 4 > ts.s && o < ts.e) ? __ldg(p4 + i * 32) : make_uint4(0u, 0u, 0u, 0u);
        }
    }
}

__device__ __forceinline__ void hist_tile(const float* __restrict__ acc, const TileSpan& ts,
                                          uint32_t* h, int lane) {
    TileRegs t;
    load_tile(acc, ts, lane, t);
    if (ts.s == 0 && ts.e == kTile) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            atomicAdd(&h[key_of(t.v[i].x) >> kShift1], 1u);
            atomicAdd(&h[key_of(t.v[i].y) >> kShift1], 1u);
            atomicAdd(&h[key_of(t.v[i].z) >> kShift1], 1u);
            atomicAdd(&h[key_of(t.v[i].w) >> kShift1], 1u);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int o = (i * 32 + lane) * 4;
            const uint32_t w[4] = {t.v[i].x, t.v[i].y, t.v[i].z, t.v[i].w};
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (o + c >= ts.s && o + c < ts.e) atomicAdd(&h[key_of(w[c]) >> kShift1], 1u);
        }
    }
}

// Where a CTA's staged entry number `pos` lives.
struct Stage {
    uint2* res;      // shared memory, kResident entries
    uint2* spill;    // HBM, this CTA's part of the staging area
};
__device__ __forceinline__ void stage_put(const Stage& st, uint32_t pos, uint2 v) {
    if (pos < (uint32_t)kResident) st.res[pos] = v; else st.spill[pos - kResident] = v;
}
__device__ __forceinline__ uint2 stage_get(const Stage& st, uint32_t pos) {
    return pos < (uint32_t)kResident ? st.res[pos] : __ldcg(st.spill + (pos - kResident));
}
// Entry `pos` of a tile whose entries [first, first + n) are known to be all resident
// (`all_res`, uniform over the warp): a plain shared-memory access, no address-space test.
__device__ __forceinline__ uint2 stage_get_tile(const Stage& st, const uint2* res_sh, bool all_res, uint32_t pos) {
    if (all_res) return res_sh[pos];
    return stage_get(st, pos);
}

// Bit c of the result: component c of v has key >= thr.
__device__ __forceinline__ uint32_t keep4(const uint4& v, uint32_t thr) {
    return (key_of(v.x) >= thr ? 1u : 0u) | (key_of(v.y) >= thr ? 2u : 0u) |
           (key_of(v.z) >= thr ? 4u : 0u) | (key_of(v.w) >= thr ? 8u : 0u);
}

// Bit c of the result: offset o + c lies in [s, e).
__device__ __forceinline__ uint32_t valid4(int o, int s, int e) {
    const int lo = s - o > 0 ? s - o : 0, hi = e - o < 4 ? e - o : 4;
    return hi > lo ? ((1u << hi) - 1u) & ~((1u << lo) - 1u) : 0u;
}

// Moves the tile's entries with bucket >= b1 behind the CTA's cursor, in index order
// (load, lane, component = ascending offset).  Returns (first entry, entries).
// The common case (a handful of entries per tile) costs about 3 instructions per element.
__device__ __forceinline__ uint2 filter_tile(const float* __restrict__ acc, const TileSpan& ts, uint32_t b1,
                                             uint32_t* h2, const Stage& st, uint2* res_sh, uint32_t* cursor,
                                             int lane) {
    TileRegs t;
    load_tile(acc, ts, lane, t);
    const uint32_t thr = b1 << kShift1;          // key >= thr  <=>  bucket >= b1
    uint32_t keep[2] = {0u, 0u};                 // bit (4*(i%8) + c) of keep[i/8]
#pragma unroll
    for (int i = 0; i < 16; ++i) keep[i >> 3] |= keep4(t.v[i], thr) << (4 * (i & 7));
    if (!(ts.s == 0 && ts.e == kTile)) {
        uint32_t vm[2] = {0u, 0u};
#pragma unroll
        for (int i = 0; i < 16; ++i) vm[i >> 3] |= valid4((i * 32 + lane) * 4, ts.s, ts.e) << (4 * (i & 7));
        keep[0] &= vm[0];
        keep[1] &= vm[1];
    }
    if (!__any_sync(0xffffffffu, (keep[0] | keep[1]) != 0)) return make_uint2(0u, 0u);
    // per-load counts, 8 bits each (a warp holds <= 128 per load), four loads per word
    uint32_t packed[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const uint32_t kw = keep[g >> 1] >> (16 * (g & 1));
        packed[g] = __popc(kw & 0xfu) | (__popc(kw & 0xf0u) << 8) | (__popc(kw & 0xf00u) << 16) |
                    (__popc(kw & 0xf000u) << 24);
    }
    uint32_t excl[4], tot[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const uint32_t incl = warp_incl_scan(packed[g], lane);
        tot[g] = __shfl_sync(0xffffffffu, incl, 31);
        excl[g] = incl - packed[g];
    }
    uint32_t n = 0;
#pragma unroll
    for (int g = 0; g < 4; ++g) n += (tot[g] & 0xff) + ((tot[g] >> 8) & 0xff) + ((tot[g] >> 16) & 0xff) + (tot[g] >> 24);
    uint32_t first = 0;
    if (lane == 0) first = atomicAdd(cursor, n);
    first = __shfl_sync(0xffffffffu, first, 0);
    const bool all_res = first + n <= (uint32_t)kResident;   // uniform over the warp
    uint32_t load_base = first;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const uint32_t tot_i = (tot[i >> 2] >> (8 * (i & 3))) & 0xff;
        const uint32_t k4 = (keep[i >> 3] >> (4 * (i & 7))) & 0xfu;
        if (k4) {
            const uint32_t w[4] = {t.v[i].x, t.v[i].y, t.v[i].z, t.v[i].w};
            uint32_t pos = load_base + ((excl[i >> 2] >> (8 * (i & 3))) & 0xff);
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (k4 & (1u << c)) {
                    const uint32_t key = key_of(w[c]);
                    if ((key >> kShift1) == b1) atomicAdd(&h2[(key >> kShift2) & (kBins2 - 1)], 1u);
                    const uint2 ent = make_uint2(w[c], (uint32_t)((i * 32 + lane) * 4 + c));
                    if (all_res) res_sh[pos] = ent; else stage_put(st, pos, ent);
                    ++pos;
                }
        }
        load_base += tot_i;
    }
    return make_uint2(first, n);
}

// The tile-table records of a warp's next 32 tiles (tile q0 + i * kSelWarps is held by lane i),
// fetched with one request so that the walk over the tiles does not wait for memory per tile.
struct TtBatch {
    uint4 rec;
    int q0;
};
__device__ __forceinline__ void tt_fetch(const SelParams& p, int q0, int qb, int lane, TtBatch& b) {
    const int q = q0 + lane * kSelWarps;
    b.q0 = q0;
    b.rec = q < qb ? __ldcg(p.tt + q) : make_uint4(0u, 0u, 0u, 0u);
}
__device__ __forceinline__ uint4 tt_get(const TtBatch& b, int q) {
    const int i = (q - b.q0) / kSelWarps;
    uint4 r;
    r.x = __shfl_sync(0xffffffffu, b.rec.x, i);
    r.y = __shfl_sync(0xffffffffu, b.rec.y, i);
    r.z = __shfl_sync(0xffffffffu, b.rec.z, i);
    r.w = __shfl_sync(0xffffffffu, b.rec.w, i);
    return r;
}

// ---------------------------------------------------------------------------------
// work split
// ---------------------------------------------------------------------------------
struct CtaRange { int q0, q1, jA, jB; };

__device__ __forceinline__ int cta_q0(const SelParams& p, int b) { return (int)((int64_t)p.tiles * b / gridDim.x); }

__device__ __forceinline__ CtaRange cta_range(const SelParams& p) {
    CtaRange r;
    r.q0 = cta_q0(p, blockIdx.x);
    r.q1 = cta_q0(p, blockIdx.x + 1);
    r.jA = 0; r.jB = -1;
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

// The streamed (non-direct) layers of the CTA's range, kSlots at a time.  The per-slot facts
// the tile loops need live in shared memory so that walking the tiles touches no global or
// local memory.
struct GroupShared {
    int lay[kSlots];        // layer position in the rank's list
    int lid[kSlots];        // layer id in the model (state / histogram index)
    int tf[kSlots];         // first tile of the layer
    int tfe[kSlots];        // one past its last tile
    int64_t start[kSlots];
    int64_t end[kSlots];
    int64_t out_off[kSlots];
};
struct Group {
    int ns;
    int qa, qb;   // the CTA's tiles from the first to the last layer of the group
};

// Every thread computes the same group; threads < ns publish the per-slot facts.  The caller
// must __syncthreads() before the facts are read.
__device__ __forceinline__ bool next_group(const SelParams& p, const CtaRange& r, int& jn, Group& g,
                                           GroupShared* gs) {
    g.ns = 0;
    int j = jn, first = -1, last = -1;
    for (; j <= r.jB && g.ns < kSlots; ++j) {
        if (is_direct(p, j)) continue;
        if (g.ns == (int)threadIdx.x) {
            gs->lay[g.ns] = j;
            gs->lid[g.ns] = p.desc[j].layer_id;
            gs->tf[g.ns] = p.desc[j].tile_first;
            gs->tfe[g.ns] = p.desc[j + 1].tile_first;
            gs->start[g.ns] = p.desc[j].start;
            gs->end[g.ns] = p.desc[j].end;
            gs->out_off[g.ns] = p.desc[j].out_off;
        }
        if (first < 0) first = j;
        last = j;
        ++g.ns;
    }
    jn = j;
    if (g.ns == 0) return false;
    const int tf = p.desc[first].tile_first, tfe = p.desc[last + 1].tile_first;
    g.qa = r.q0 > tf ? r.q0 : tf;
    g.qb = r.q1 < tfe ? r.q1 : tfe;
    return true;
}

// Per-warp walk over the group's tiles: tile q belongs to slot s (or to a direct layer that
// lies between two slots: result < 0).  `s` is a cursor that only moves forward.
__device__ __forceinline__ int tile_slot(const Group& g, const GroupShared* gs, int q, int& s) {
    while (s < g.ns - 1 && q >= gs->tfe[s]) ++s;
    return (q >= gs->tf[s] && q < gs->tfe[s]) ? s : -1;
}

// After the CTA has flushed its counts of the group's layers (a __syncthreads() lies between
// the flush and this call): take a ticket per layer; last[s] = this CTA flushed the layer's
// last tiles, so the layer's histogram is complete.
template <int kTicket>
__device__ __forceinline__ void take_tickets(const SelParams& p, const CtaRange& r, const Group& g,
                                             const GroupShared* gs, uint32_t* last) {
    if ((int)threadIdx.x < g.ns) {
        const int sl = threadIdx.x;
        LayerState* st = p.state + gs->lid[sl];
        uint32_t* t = kTicket == 1 ? &st->ticket1 : kTicket == 2 ? &st->ticket2 : &st->ticket3;
        const int a = r.q0 > gs->tf[sl] ? r.q0 : gs->tf[sl], b = r.q1 < gs->tfe[sl] ? r.q1 : gs->tfe[sl];
        const uint32_t mine = b > a ? (uint32_t)(b - a) : 0u;   // this CTA's tiles of the layer
        __threadfence();
        const uint32_t old = atomicAdd(t, mine);
        last[sl] = (old + mine == (uint32_t)(gs->tfe[sl] - gs->tf[sl])) ? 1u : 0u;
    }
    __syncthreads();
}

// ---------------------------------------------------------------------------------
// step A: level-1 histograms
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void step_hist1(const SelParams& p, const CtaRange& r, unsigned char* smem) {
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem + kSmMain);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    Group g;
    GroupShared* gs = reinterpret_cast<GroupShared*>(smem + kSmGroup);
    for (int jn = r.jA; next_group(p, r, jn, g, gs);) {
        __syncthreads();   // the group's facts are published
        for (int i = threadIdx.x; i < g.ns * kBins1; i += kSelThreads) hist[i] = 0;
        __syncthreads();
        int s = 0;
        for (int q = g.qa + warp; q < g.qb; q += kSelWarps) {
            const int slot = tile_slot(g, gs, q, s);
            if (slot < 0) continue;
            const TileSpan ts = tile_span(gs->start[slot], gs->end[slot], gs->tf[slot], q);
            hist_tile(p.acc, ts, hist + slot * kBins1, lane);
        }
        __syncthreads();
        for (int i = threadIdx.x; i < g.ns * kBins1; i += kSelThreads) {
            const uint32_t c = hist[i];
            if (c) atomicAdd(p.hist1 + (size_t)gs->lid[i / kBins1] * kBins1 + (i % kBins1), c);
        }
        __syncthreads();
        take_tickets<1>(p, r, g, gs, misc + kMLast);
        for (int s2 = 0; s2 < g.ns; ++s2) {
            if (!misc[kMLast + s2]) continue;   // uniform over the CTA
            const int j = gs->lay[s2];
            const int lid = p.desc[j].layer_id;
            __threadfence();
            block_scan_select<true>(p.hist1 + (size_t)lid * kBins1, kBins1, (uint32_t)p.desc[j].k,
                                    misc + kMScratch, misc + kMOut3);
            if (threadIdx.x == 0) {
                p.state[lid].b1 = misc[kMOut3];
                p.state[lid].above1 = misc[kMOut3 + 1];
            }
            __syncthreads();
        }
        __syncthreads();   // the group's facts are no longer read
    }
}

// ---------------------------------------------------------------------------------
// step B: staging pass + level-2 histograms
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void step_filter(const SelParams& p, const CtaRange& r, const Stage& st,
                                            unsigned char* smem) {
    uint32_t* hist2s = reinterpret_cast<uint32_t*>(smem + kSmAux);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) misc[kMCursor] = 0;
    Group g;
    GroupShared* gs = reinterpret_cast<GroupShared*>(smem + kSmGroup);
    for (int jn = r.jA; next_group(p, r, jn, g, gs);) {
        __syncthreads();   // the group's facts are published
        if ((int)threadIdx.x < g.ns) misc[kMTabA + threadIdx.x] = __ldcg(&p.state[gs->lid[threadIdx.x]].b1);
        for (int i = threadIdx.x; i < g.ns * kBins2; i += kSelThreads) hist2s[i] = 0;
        __syncthreads();
        int s = 0;
        for (int q = g.qa + warp; q < g.qb; q += kSelWarps) {
            const int slot = tile_slot(g, gs, q, s);
            if (slot < 0) continue;
            const TileSpan ts = tile_span(gs->start[slot], gs->end[slot], gs->tf[slot], q);
            const uint2 fn = filter_tile(p.acc, ts, misc[kMTabA + slot], hist2s + slot * kBins2, st,
                                         reinterpret_cast<uint2*>(smem + kSmMain), misc + kMCursor, lane);
            if (lane == 0) p.tt[q] = make_uint4(fn.x, fn.y, 0u, 0u);
        }
        __syncthreads();
        for (int i = threadIdx.x; i < g.ns * kBins2; i += kSelThreads) {
            const uint32_t c = hist2s[i];
            if (c) atomicAdd(p.hist2 + (size_t)gs->lid[i / kBins2] * kBins2 + (i % kBins2), c);
        }
        __syncthreads();
        take_tickets<2>(p, r, g, gs, misc + kMLast);
        for (int s2 = 0; s2 < g.ns; ++s2) {
            if (!misc[kMLast + s2]) continue;   // uniform over the CTA
            const int j = gs->lay[s2];
            const int lid = p.desc[j].layer_id;
            __threadfence();
            const uint32_t krem1 = (uint32_t)p.desc[j].k - __ldcg(&p.state[lid].above1);
            block_scan_select<true>(p.hist2 + (size_t)lid * kBins2, kBins2, krem1, misc + kMScratch, misc + kMOut3);
            if (threadIdx.x == 0) {
                p.state[lid].b2 = misc[kMOut3];
                p.state[lid].krem2 = krem1 - misc[kMOut3 + 1];
            }
            __syncthreads();
        }
        __syncthreads();   // the group's facts are no longer read
    }
}

// ---------------------------------------------------------------------------------
// step S2: level-3 histograms over the staged entries of bucket (b1, b2)
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void step_hist3(const SelParams& p, const CtaRange& r, const Stage& st,
                                           unsigned char* smem) {
    uint32_t* h3 = reinterpret_cast<uint32_t*>(smem + kSmAux);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint2* res_sh = reinterpret_cast<const uint2*>(smem + kSmMain);
    Group g;
    GroupShared* gs = reinterpret_cast<GroupShared*>(smem + kSmGroup);
    for (int jn = r.jA; next_group(p, r, jn, g, gs);) {
        __syncthreads();   // the group's facts are published
        if ((int)threadIdx.x < g.ns) {
            const LayerState* ls = p.state + gs->lid[threadIdx.x];
            misc[kMTabA + threadIdx.x] = (__ldcg(&ls->b1) << (kShift1 - kShift2)) | __ldcg(&ls->b2);
        }
        for (int i = threadIdx.x; i < g.ns * kBins3; i += kSelThreads) h3[i] = 0;
        __syncthreads();
        stamp(p, 8);
        int s = 0;
        TtBatch tb;
        for (int q = g.qa + warp; q < g.qb; q += kSelWarps) {
            if ((q - g.qa - warp) % (32 * kSelWarps) == 0) tt_fetch(p, q, g.qb, lane, tb);
            const int slot = tile_slot(g, gs, q, s);
            if (slot < 0) continue;
            const uint4 t = tt_get(tb, q);
            const uint32_t prefix = misc[kMTabA + slot];
            const bool all_res = t.x + t.y <= (uint32_t)kResident;
            for (uint32_t e = lane; e < t.y; e += 32) {
                const uint32_t key = key_of(stage_get_tile(st, res_sh, all_res, t.x + e).x);
                if ((key >> kShift2) == prefix) atomicAdd(&h3[slot * kBins3 + (key & (kBins3 - 1))], 1u);
            }
        }
        stamp(p, 9);
        __syncthreads();
        for (int i = threadIdx.x; i < g.ns * kBins3; i += kSelThreads) {
            const uint32_t c = h3[i];
            if (c) atomicAdd(p.hist3 + (size_t)gs->lid[i / kBins3] * kBins3 + (i % kBins3), c);
        }
        __syncthreads();
        stamp(p, 10);
        take_tickets<3>(p, r, g, gs, misc + kMLast);
        stamp(p, 11);
        for (int s2 = 0; s2 < g.ns; ++s2) {
            if (!misc[kMLast + s2]) continue;   // uniform over the CTA
            const int lid = gs->lid[s2];
            __threadfence();
            const uint32_t krem2 = __ldcg(&p.state[lid].krem2);
            block_scan_select<true>(p.hist3 + (size_t)lid * kBins3, kBins3, krem2, misc + kMScratch, misc + kMOut3);
            if (threadIdx.x == 0) {
                const uint32_t b1 = __ldcg(&p.state[lid].b1), b2 = __ldcg(&p.state[lid].b2);
                p.state[lid].T = (b1 << kShift1) | (b2 << kShift2) | misc[kMOut3];
                p.state[lid].need = krem2 - misc[kMOut3 + 1];
            }
            __syncthreads();
        }
        __syncthreads();   // the group's facts are no longer read
    }
}

// ---------------------------------------------------------------------------------
// step S3: per tile and per (CTA, layer): staged entries above T / equal to T
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void step_count(const SelParams& p, const CtaRange& r, const Stage& st,
                                           unsigned char* smem) {
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint2* res_sh = reinterpret_cast<const uint2*>(smem + kSmMain);
    Group g;
    GroupShared* gs = reinterpret_cast<GroupShared*>(smem + kSmGroup);
    for (int jn = r.jA; next_group(p, r, jn, g, gs);) {
        __syncthreads();   // the group's facts are published
        if ((int)threadIdx.x < g.ns) {
            misc[kMTabA + threadIdx.x] = __ldcg(&p.state[gs->lid[threadIdx.x]].T);
            misc[kMTotGt + threadIdx.x] = 0;
            misc[kMTotEq + threadIdx.x] = 0;
        }
        __syncthreads();
        int s = 0;
        TtBatch tb;
        for (int q = g.qa + warp; q < g.qb; q += kSelWarps) {
            if ((q - g.qa - warp) % (32 * kSelWarps) == 0) tt_fetch(p, q, g.qb, lane, tb);
            const int slot = tile_slot(g, gs, q, s);
            if (slot < 0) continue;
            const uint4 t = tt_get(tb, q);
            const uint32_t T = misc[kMTabA + slot];
            uint32_t n_gt = 0, n_eq = 0;
            const bool all_res = t.x + t.y <= (uint32_t)kResident;
            for (uint32_t e = lane; e < t.y; e += 32) {
                const uint32_t key = key_of(stage_get_tile(st, res_sh, all_res, t.x + e).x);
                n_gt += key > T;
                n_eq += key == T;
            }
            n_gt = __reduce_add_sync(0xffffffffu, n_gt);
            n_eq = __reduce_add_sync(0xffffffffu, n_eq);
            if (lane == 0) {
                p.tt[q] = make_uint4(t.x, t.y, n_gt, n_eq);
                atomicAdd(&misc[kMTotGt + slot], n_gt);
                atomicAdd(&misc[kMTotEq + slot], n_eq);
            }
        }
        __syncthreads();
        if ((int)threadIdx.x < g.ns)
            p.runge[blockIdx.x + gs->lay[threadIdx.x]] = make_uint2(misc[kMTotGt + threadIdx.x], misc[kMTotEq + threadIdx.x]);
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
        if (p.acc_rw) p.acc_rw[elem0 + off] = 0.0f;
    }
    gt_before += __popc(gt_b);
    eq_before += __popc(eq_b);
}

// ---------------------------------------------------------------------------------
// step S4: prefix over the CTAs before this one, scan of the own tiles, ordered write
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void step_emit(const SelParams& p, const CtaRange& r, const Stage& st,
                                          unsigned char* smem) {
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* scratch = misc + kMScratch;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint2* res_sh = reinterpret_cast<const uint2*>(smem + kSmMain);
    Group g;
    GroupShared* gs = reinterpret_cast<GroupShared*>(smem + kSmGroup);
    for (int jn = r.jA; next_group(p, r, jn, g, gs);) {
        __syncthreads();   // the group's facts are published
        for (int s2 = 0; s2 < g.ns; ++s2) {
            const int j = gs->lay[s2];
            const int tf = p.desc[j].tile_first, tfe = p.desc[j + 1].tile_first;
            // totals of the CTAs that hold earlier tiles of the layer
            const int b0 = cta_of_tile(p, tf);
            uint32_t v_gt = 0, v_eq = 0;
            for (int b = b0 + (int)threadIdx.x; b < (int)blockIdx.x; b += kSelThreads) {
                if (cta_q0(p, b) < cta_q0(p, b + 1)) {
                    const uint2 c = __ldcg(p.runge + b + j);
                    v_gt += c.x;
                    v_eq += c.y;
                }
            }
            uint32_t base_gt, base_eq;
            block_excl_scan(v_gt, scratch, base_gt);
            block_excl_scan(v_eq, scratch, base_eq);
            // exclusive scan over this CTA's tiles of the layer, written back over the counts
            const int ta = r.q0 > tf ? r.q0 : tf, tb = r.q1 < tfe ? r.q1 : tfe;
            for (int t0 = ta; t0 < tb; t0 += kSelThreads) {
                const int q = t0 + (int)threadIdx.x;
                uint4 t = make_uint4(0u, 0u, 0u, 0u);
                if (q < tb) t = __ldcg(p.tt + q);
                uint32_t tot_gt, tot_eq;
                const uint32_t e_gt = block_excl_scan(t.z, scratch, tot_gt);
                const uint32_t e_eq = block_excl_scan(t.w, scratch, tot_eq);
                if (q < tb) p.tt[q] = make_uint4(t.x, t.y, base_gt + e_gt, base_eq + e_eq);
                base_gt += tot_gt;
                base_eq += tot_eq;
            }
            if (threadIdx.x == 0) {
                const LayerState* ls = p.state + p.desc[j].layer_id;
                misc[kMTabA + s2] = __ldcg(&ls->T);
                misc[kMTabB + s2] = __ldcg(&ls->need);
            }
        }
        __syncthreads();
        int s = 0;
        TtBatch tb;
        for (int q = g.qa + warp; q < g.qb; q += kSelWarps) {
            if ((q - g.qa - warp) % (32 * kSelWarps) == 0) tt_fetch(p, q, g.qb, lane, tb);
            const int slot = tile_slot(g, gs, q, s);
            if (slot < 0) continue;
            const uint4 t = tt_get(tb, q);
            if (t.y == 0) continue;
            const uint32_t T = misc[kMTabA + slot], need = misc[kMTabB + slot];
            const int64_t lo = (gs->start[slot] / kTile + (q - gs->tf[slot])) * kTile;
            const int64_t out_off = gs->out_off[slot];
            uint32_t gt_before = t.z, eq_before = t.w;
            const bool all_res = t.x + t.y <= (uint32_t)kResident;
            for (uint32_t e0 = 0; e0 < t.y; e0 += 32) {
                const uint32_t e = e0 + lane;
                const bool valid = e < t.y;
                uint2 ent = make_uint2(0u, 0u);
                if (valid) ent = stage_get_tile(st, res_sh, all_res, t.x + e);
                emit_batch(p, out_off, lo, valid, ent.x, (int64_t)ent.y, T, need, gt_before, eq_before, lane);
            }
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------
// direct layers: one CTA loads the layer whole and finishes it from shared memory
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void resolve_direct(const SelParams& p, int j, unsigned char* smem) {
    uint32_t* skey = reinterpret_cast<uint32_t*>(smem + kSmMain);
    uint32_t* h1 = reinterpret_cast<uint32_t*>(smem + kSmAux);
    uint32_t* h = h1 + kBins1;
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kSmMisc);
    uint32_t* scratch = misc + kMScratch;
    uint32_t* out3 = misc + kMOut3;
    uint32_t* wcnt = misc + kMWarpCnt;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t start = p.desc[j].start;
    const uint32_t n = (uint32_t)(p.desc[j].end - start);
    const uint32_t k = (uint32_t)p.desc[j].k;
    const int64_t out_off = p.desc[j].out_off;
    const uint32_t* x = reinterpret_cast<const uint32_t*>(p.acc + start);
    for (int i = tid; i < kBins1; i += kSelThreads) h1[i] = 0;
    for (int i = tid; i < kBins2; i += kSelThreads) h[i] = 0;
    __syncthreads();
    // level 1 over the whole layer
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
                atomicAdd(&h1[key_of(v[u]) >> kShift1], 1u);
            }
        }
    }
    __syncthreads();
    block_scan_select<false>(h1, kBins1, k, scratch, out3);
    const uint32_t b1 = out3[0], above1 = out3[1];
    __syncthreads();
    // level 2 inside bucket b1
    for (uint32_t f = tid; f < n; f += kSelThreads) {
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
    for (uint32_t f = tid; f < n; f += kSelThreads) {
        const uint32_t key = key_of(skey[f]);
        if ((key >> kShift2) == prefix) atomicAdd(&h[key & (kBins3 - 1)], 1u);
    }
    __syncthreads();
    block_scan_select<false>(h, kBins3, krem2, scratch, out3);
    const uint32_t T = (prefix << kShift2) | out3[0];
    const uint32_t need = krem2 - out3[1];
    __syncthreads();
    // every warp counts its contiguous share, then the ordered, coalesced write
    const uint32_t wper = ((n + kSelWarps - 1) / kSelWarps + 31) & ~31u;   // multiple of 32
    const uint32_t f0 = (uint32_t)warp * wper < n ? (uint32_t)warp * wper : n;
    const uint32_t f1 = f0 + wper < n ? f0 + wper : n;
    uint32_t n_gt = 0, n_eq = 0;
    for (uint32_t f = f0 + lane; f < f1; f += 32) {
        const uint32_t key = key_of(skey[f]);
        n_gt += key > T;
        n_eq += key == T;
    }
    n_gt = __reduce_add_sync(0xffffffffu, n_gt);
    n_eq = __reduce_add_sync(0xffffffffu, n_eq);
    if (lane == 0) wcnt[warp] = n_gt | (n_eq << 16);   // both totals <= kDirectElems < 65536
    __syncthreads();
    const uint32_t mine = lane < kSelWarps ? wcnt[lane] : 0u;
    const uint32_t before = __shfl_sync(0xffffffffu, warp_incl_scan(mine, lane) - mine, warp);
    uint32_t gt_before = before & 0xffff, eq_before = before >> 16;
    for (uint32_t fb = f0; fb < f1; fb += 32) {
        const uint32_t f = fb + lane;
        const bool valid = f < f1;
        emit_batch(p, out_off, start, valid, valid ? skey[f] : 0u, (int64_t)f, T, need, gt_before, eq_before, lane);
    }
    __syncthreads();   // shared memory is reused by the next layer
}
static_assert(kDirectElems < 65536, "packed per-warp counts");

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
    const CtaRange r = cta_range(p);
    Stage st;
    st.res = reinterpret_cast<uint2*>(smem + kSmMain);
    st.spill = p.staging;
    if (r.q0 < r.q1) {
        // the CTA's part of the staging area starts where its first tile's elements would go
        const TileSpan ts = tile_span(p.desc[r.jA].start, p.desc[r.jA].end, p.desc[r.jA].tile_first, r.q0);
        st.spill = p.staging + p.desc[r.jA].elem_off + (ts.lo + ts.s - p.desc[r.jA].start);
    }

    step_hist1(p, r, smem);
    stamp(p, 1);
    grid.sync();
    step_filter(p, r, st, smem);
    stamp(p, 2);
    grid.sync();
    step_hist3(p, r, st, smem);
    stamp(p, 3);
    grid.sync();
    step_count(p, r, st, smem);
    stamp(p, 4);
    grid.sync();
    step_emit(p, r, st, smem);
    stamp(p, 5);
    for (int j = blockIdx.x; j < p.n_my; j += gridDim.x)
        if (is_direct(p, j)) resolve_direct(p, j, smem);   // uniform over the CTA
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
    // one CTA per SM at most (co-resident by construction); fewer when the rank is small
    const int sms = sm_count();
    int want = (p.tiles + 1) / 2;
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
